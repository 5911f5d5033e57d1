"""ctypes binding of libmuon_b200.so: argument marshalling only.

Every function mirrors one entry point of include/muon_b200.h under the same name.  Tensors
are torch CUDA tensors used purely as device memory; no arithmetic happens here.  If the
shared library is missing the import of this module fails loudly -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmuon_b200.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_21594_b200.build` "
                      "(there is no CPU or PyTorch fallback)")

lib = C.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_BAD_LAYOUT, ERR_UNSUPPORTED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_DEVICE_TIMEOUT = 0, -1, -2, -3, -4, -5, -6
ERR_TOO_LARGE = -7
STATIC_SCRATCH_BYTES = 16 * 1024 * 1024 + 16384
DTYPE_BF16, DTYPE_FP32 = 0, 1
NS_BF16, NS_FP32 = 0, 1
ENGINE_TENSOR, ENGINE_CUDA_CORE, ENGINE_TENSOR_1CTA = 0, 1, 2
ORTHO_NO_NORMALIZE = 1
PHASE_MOMENTUM, PHASE_NS, PHASE_UPDATE, PHASE_GATHER, PHASE_SCATTER = range(5)
PHASE_NAMES = ("momentum", "ns", "update", "gather", "scatter")


class Shape(C.Structure):
    _fields_ = [("rows", C.c_int32), ("cols", C.c_int32)]


class View(C.Structure):
    _fields_ = [("rows", C.c_int32), ("cols", C.c_int32), ("ld", C.c_int64)]


class Segment(C.Structure):
    _fields_ = [("matrix", C.c_int32), ("reserved", C.c_int32), ("elem_begin", C.c_int64),
                ("elem_count", C.c_int64), ("flat_offset", C.c_int64)]


class LayoutDesc(C.Structure):
    _fields_ = [("elem_size", C.c_int32), ("align_elems", C.c_int32), ("num_shards", C.c_int32),
                ("num_matrices", C.c_int32), ("shard_len", C.c_int64), ("shapes", C.POINTER(Shape)),
                ("num_segments", C.c_int64), ("segments", C.POINTER(Segment))]


class Options(C.Structure):
    _fields_ = [("grad_dtype", C.c_int32), ("ns_precision", C.c_int32), ("nesterov", C.c_int32),
                ("coeffs_per_step", C.c_int32), ("eps", C.c_float), ("engine", C.c_int32),
                ("chunk_elems", C.c_int64), ("coeffs_per_matrix", C.c_int32), ("launch_per_product", C.c_int32)]


_vp = C.c_void_p
_sig = {
    "muon_default_options": (C.c_int, [C.POINTER(Options)]),
    "muon_create": (C.c_int, [C.POINTER(_vp), C.POINTER(Options)]),
    "muon_destroy": (None, [_vp]),
    "muon_workspace_bytes": (C.c_int, [C.POINTER(Options), C.POINTER(Shape), C.c_int32, C.POINTER(C.c_size_t)]),
    "muon_set_workspace": (C.c_int, [_vp, _vp, C.c_size_t]),
    "muon_plan_describe": (C.c_int, [C.POINTER(Options), C.POINTER(Shape), C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]),
    "muon_plan_launch_sets": (C.c_int, [C.POINTER(Options), C.POINTER(Shape), C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]),
    "muon_plan_pipeline": (C.c_int, [C.POINTER(Options), C.POINTER(Shape), C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                     C.POINTER(C.c_int32), C.c_int32]),
    "muon_symmetric_tiles": (C.c_int, [C.c_int32, C.POINTER(C.c_uint16), C.c_int32, C.POINTER(C.c_int32)]),
    "muon_layout_validate": (C.c_int, [C.POINTER(LayoutDesc)]),
    "muon_layout_create": (C.c_int, [_vp, C.POINTER(LayoutDesc), C.POINTER(_vp)]),
    "muon_layout_destroy": (None, [_vp]),
    "muon_materialize": (C.c_int, [_vp, _vp, _vp, C.POINTER(_vp), _vp]),
    "muon_scatter": (C.c_int, [_vp, _vp, _vp, C.POINTER(_vp), _vp]),
    "muon_owner_plan": (C.c_int, [C.POINTER(Shape), C.c_int32, C.c_int32, C.c_int64, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                  C.POINTER(C.c_int32)]),
    "muon_shard_momentum": (C.c_int, [_vp, _vp, C.c_int32, _vp, _vp, _vp, C.c_float, _vp]),
    "muon_materialize_owned": (C.c_int, [_vp, _vp, _vp, C.POINTER(_vp), _vp]),
    "muon_scatter_owned": (C.c_int, [_vp, _vp, _vp, C.POINTER(_vp), _vp]),
    "muon_shard_apply": (C.c_int, [_vp, _vp, C.c_int32, _vp, C.POINTER(_vp), C.c_float, C.c_float, _vp]),
    "muon_step_batched": (C.c_int, [_vp, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.POINTER(Shape), C.c_int32,
                                    C.c_float, C.c_float, C.c_float, C.c_int32, C.POINTER(C.c_float), _vp]),
    "muon_step_batched_out": (C.c_int, [_vp, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.POINTER(Shape),
                                        C.c_int32, C.c_float, C.c_float, C.c_float, C.c_int32, C.POINTER(C.c_float), _vp]),
    "muon_views_overlap": (C.c_int, [C.POINTER(_vp), C.POINTER(View), C.c_int32, C.c_int32, C.POINTER(C.c_int32)]),
    "muon_step_batched_views": (C.c_int, [_vp, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.POINTER(View),
                                          C.c_int32, C.c_float, C.c_float, C.c_float, C.c_int32, C.POINTER(C.c_float), _vp]),
    "muon_step_flat": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, C.c_float, C.c_float, C.c_float, C.c_int32, C.POINTER(C.c_float), _vp]),
    "muon_step_flat_host": (C.c_int, [_vp, _vp, _vp, _vp, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp), C.POINTER(_vp),
                                      C.c_float, C.c_float, C.c_float, C.c_int32, C.POINTER(C.c_float), _vp]),
    "muon_orthogonalize_batched": (C.c_int, [_vp, C.POINTER(_vp), C.POINTER(_vp), C.POINTER(Shape), C.c_int32,
                                             C.c_int32, C.POINTER(C.c_float), C.c_uint32, _vp]),
    "muon_ns_product": (C.c_int, [_vp, _vp, _vp, _vp, _vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                  C.c_int64, C.c_int64, C.c_int64, C.c_int32, C.c_int32, C.c_float, C.c_float, _vp,
                                  C.c_int32, _vp]),
    "muon_orthogonalize_static": (C.c_int, [_vp, _vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_float),
                                            C.c_float, C.c_uint32, _vp, _vp]),
    "muon_last_device_status": (C.c_int, [_vp, _vp, C.POINTER(C.c_int32)]),
    "muon_clear_device_status": (C.c_int, [_vp, _vp]),
    "muon_synchronize_and_check": (C.c_int, [_vp, _vp]),
    "muon_tensor_map_encodes": (C.c_int64, [_vp]),
    "muon_self_test_bounded_wait": (C.c_int, [_vp, _vp]),
    "muon_profile_enable": (C.c_int, [_vp, C.c_int32]),
    "muon_profile_reset": (C.c_int, [_vp]),
    "muon_profile_read": (C.c_int, [_vp, C.c_int32, C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "muon_launch_count": (C.c_int64, [_vp]),
    "muon_status_string": (C.c_char_p, [C.c_int]),
}
EXPORTED = tuple(_sig)
for _name, (_res, _args) in _sig.items():
    _f = getattr(lib, _name)
    _f.restype = _res
    _f.argtypes = _args


class MuonError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lib.muon_status_string(code).decode()} ({code})")


def _check(code: int, where: str) -> None:
    if code != OK:
        raise MuonError(code, where)


def _shapes(shapes: Sequence[Tuple[int, int]]):
    arr = (Shape * max(1, len(shapes)))()
    for i, (r, c) in enumerate(shapes):
        arr[i].rows, arr[i].cols = int(r), int(c)
    return arr


def _ptrs(tensors) -> "C.Array":
    arr = (_vp * max(1, len(tensors)))()
    for i, t in enumerate(tensors):
        arr[i] = None if t is None else (t if isinstance(t, int) else t.data_ptr())
    return arr


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


def muon_default_options(**over) -> Options:
    o = Options()
    _check(lib.muon_default_options(C.byref(o)), "muon_default_options")
    for k, v in over.items():
        setattr(o, k, v)
    return o


def muon_workspace_bytes(opt: Options, shapes) -> int:
    out = C.c_size_t(0)
    _check(lib.muon_workspace_bytes(C.byref(opt), _shapes(shapes), len(shapes), C.byref(out)), "muon_workspace_bytes")
    return int(out.value)


def muon_plan_pipeline(opt: Options, shapes) -> Tuple[List[int], List[int]]:
    """(launch set of every matrix, order in which the host-buffer pipeline runs the sets)."""
    n = C.c_int32(0)
    set_of = (C.c_int32 * max(1, len(shapes)))()
    cap = len(shapes) + 2
    order = (C.c_int32 * cap)()
    _check(lib.muon_plan_pipeline(C.byref(opt), _shapes(shapes), len(shapes), C.byref(n), set_of, order, cap), "muon_plan_pipeline")
    return [int(set_of[i]) for i in range(len(shapes))], [int(order[k]) for k in range(int(n.value))]


def muon_views_overlap(bases, views, elem_size: int) -> bool:
    """bases: addresses (ints) of element (0,0) of each view; views: list of (rows, cols, ld).  Host arithmetic only."""
    va = (View * max(1, len(views)))()
    for i, (r, c, ld) in enumerate(views):
        va[i].rows, va[i].cols, va[i].ld = int(r), int(c), int(ld)
    out = C.c_int32(0)
    _check(lib.muon_views_overlap(_ptrs(bases), va, len(views), int(elem_size), C.byref(out)), "muon_views_overlap")
    return bool(out.value)


def muon_plan_describe(opt: Options, shapes) -> Tuple[int, List[int]]:
    n = C.c_int32(0)
    chunk_of = (C.c_int32 * max(1, len(shapes)))()
    _check(lib.muon_plan_describe(C.byref(opt), _shapes(shapes), len(shapes), C.byref(n), chunk_of), "muon_plan_describe")
    return int(n.value), [int(chunk_of[i]) for i in range(len(shapes))]


def muon_plan_launch_sets(opt: Options, shapes) -> Tuple[int, List[int]]:
    n = C.c_int32(0)
    set_of = (C.c_int32 * max(1, len(shapes)))()
    _check(lib.muon_plan_launch_sets(C.byref(opt), _shapes(shapes), len(shapes), C.byref(n), set_of), "muon_plan_launch_sets")
    return int(n.value), [int(set_of[i]) for i in range(len(shapes))]


def muon_symmetric_tiles(blocks: int) -> List[Tuple[int, int, int, int]]:
    """The tile list of a symmetric product over blocks x blocks blocks of 128: [(ra, rb, cc, cd)], 0xFFFF = none."""
    n = C.c_int32(0)
    _check(lib.muon_symmetric_tiles(blocks, None, 0, C.byref(n)), "muon_symmetric_tiles")
    buf = (C.c_uint16 * max(1, 4 * n.value))()
    _check(lib.muon_symmetric_tiles(blocks, buf, n.value, C.byref(n)), "muon_symmetric_tiles")
    return [(buf[4 * i], buf[4 * i + 1], buf[4 * i + 2], buf[4 * i + 3]) for i in range(n.value)]


def muon_owner_plan(shapes, ranks: int, batch_elems: int = 0) -> Tuple[List[int], List[int], int]:
    """(owner_of, batch_of, num_batches): compute owners and batches of the owner-sharded step (host only)."""
    n = len(shapes)
    owner = (C.c_int32 * max(1, n))()
    batch = (C.c_int32 * max(1, n))()
    nb = C.c_int32(0)
    _check(lib.muon_owner_plan(_shapes(shapes), n, ranks, batch_elems, owner, batch, C.byref(nb)), "muon_owner_plan")
    return [int(owner[i]) for i in range(n)], [int(batch[i]) for i in range(n)], int(nb.value)


def make_layout_desc(layout, elem_size: int):
    """Builds a LayoutDesc (plus the arrays it points to) from a workloads.Layout."""
    shapes = _shapes(layout.shapes)
    segs = (Segment * max(1, len(layout.segments)))()
    for i, s in enumerate(layout.segments):
        segs[i].matrix, segs[i].reserved = s.matrix, 0
        segs[i].elem_begin, segs[i].elem_count, segs[i].flat_offset = s.elem_begin, s.elem_count, s.flat_offset
    d = LayoutDesc(elem_size, layout.align, layout.num_shards, len(layout.shapes), layout.shard_len,
                   shapes, len(layout.segments), segs)
    d._keep = (shapes, segs)
    return d


def muon_layout_validate(desc: LayoutDesc) -> int:
    return int(lib.muon_layout_validate(C.byref(desc)))


def muon_orthogonalize_static(inp, out, rows, cols, ns_precision, ns_steps, coeffs, eps=1e-7, flags=0, status=None,
                              stream=None) -> None:
    """One-matrix Newton-Schulz with the library's built-in scratch: needs no Context and allocates nothing.
    `inp`, `out` (and the optional zeroed int32 `status`) are CUDA tensors the caller owns."""
    co = (C.c_float * 3)(*[float(c) for c in coeffs[:3]])
    _check(lib.muon_orthogonalize_static(inp.data_ptr(), out.data_ptr(), rows, cols, ns_precision, ns_steps, co, eps, flags,
                                         None if status is None else status.data_ptr(), _stream(stream)),
           "muon_orthogonalize_static")


# ---- logical-matrix views: pure address arithmetic on tensors that share one physical layout
def views_of_rows(tensor, row_counts):
    """Row blocks of a 2-D tensor (fused QKV projections, gate/up halves stacked along rows).
    Returns [(element offset, (rows, cols, ld))]."""
    assert tensor.dim() == 2 and tensor.stride(1) == 1 and sum(row_counts) == tensor.shape[0]
    ld, out, r0 = tensor.stride(0), [], 0
    for n in row_counts:
        out.append((r0 * ld, (n, tensor.shape[1], ld)))
        r0 += n
    return out


def views_of_cols(tensor, col_counts):
    """Column blocks of a 2-D tensor (factors packed side by side, e.g. the two parts of an MLA projection)."""
    assert tensor.dim() == 2 and tensor.stride(1) == 1 and sum(col_counts) == tensor.shape[1]
    ld, out, c0 = tensor.stride(0), [], 0
    for n in col_counts:
        out.append((c0, (tensor.shape[0], n, ld)))
        c0 += n
    return out


def views_of_interleaved_rows(tensor, ways: int):
    """`ways` logical matrices stored row-interleaved in one 2-D tensor (gate and up projections kept as rows
    g0, u0, g1, u1, ...): logical matrix w owns physical rows w, w + ways, ...; its row stride is ways * ld."""
    assert tensor.dim() == 2 and tensor.stride(1) == 1 and tensor.shape[0] % ways == 0
    ld = tensor.stride(0)
    return [(w * ld, (tensor.shape[0] // ways, tensor.shape[1], ways * ld)) for w in range(ways)]


def views_of_planes(tensor):
    """The E matrix planes of an [E, M, N] tensor: E independent M x N matrices, never one E x MN matrix."""
    assert tensor.dim() == 3 and tensor.stride(2) == 1
    return [(e * tensor.stride(0), (tensor.shape[1], tensor.shape[2], tensor.stride(1))) for e in range(tensor.shape[0])]


def view_addresses(tensor, views):
    """Device addresses of element (0,0) of each view of `tensor`."""
    return [tensor.data_ptr() + off * tensor.element_size() for off, _ in views]


class Layout:
    """Owner of a muon_layout_t handle."""

    def __init__(self, ctx: "Context", layout, elem_size: int):
        self.desc = make_layout_desc(layout, elem_size)
        self.handle = _vp()
        _check(lib.muon_layout_create(ctx.handle, C.byref(self.desc), C.byref(self.handle)), "muon_layout_create")

    def close(self):
        if self.handle:
            lib.muon_layout_destroy(self.handle)
            self.handle = _vp()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _coeffs(coeffs):
    """Host coefficient table: one row, or one row per matrix (2-D input), flattened row-major."""
    flat = np.asarray(coeffs, dtype=np.float32).reshape(-1)
    return (C.c_float * flat.size)(*flat.tolist())


class Context:
    """Owner of a muon_ctx_t handle and (optionally) of a torch-allocated workspace."""

    def __init__(self, opt: Optional[Options] = None):
        self.opt = opt if opt is not None else muon_default_options()
        self.handle = _vp()
        _check(lib.muon_create(C.byref(self.handle), C.byref(self.opt)), "muon_create")
        self._ws = None

    def close(self):
        if self.handle:
            lib.muon_destroy(self.handle)
            self.handle = _vp()
            self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- workspace
    def muon_set_workspace(self, tensor) -> None:
        self._ws = tensor
        _check(lib.muon_set_workspace(self.handle, tensor.data_ptr(), tensor.numel() * tensor.element_size()),
               "muon_set_workspace")

    def ensure_workspace(self, shapes) -> int:
        """Allocates (through torch) a workspace large enough for `shapes`; returns its size."""
        import torch

        need = muon_workspace_bytes(self.opt, shapes)
        if self._ws is None or self._ws.numel() < need:
            self._ws = None
            self.muon_set_workspace(torch.empty(max(need, 256), dtype=torch.uint8, device="cuda"))
        return need

    # -- layout path
    def muon_materialize(self, flat, layout: Layout, matrices, stream=None) -> None:
        _check(lib.muon_materialize(self.handle, flat.data_ptr(), layout.handle, _ptrs(matrices), _stream(stream)),
               "muon_materialize")

    def muon_scatter(self, flat, layout: Layout, matrices, stream=None) -> None:
        _check(lib.muon_scatter(self.handle, flat.data_ptr(), layout.handle, _ptrs(matrices), _stream(stream)),
               "muon_scatter")

    # -- owner-sharded step: the shard-local halves and the subset copies
    def muon_shard_momentum(self, layout: Layout, shard: int, local_grads, local_momenta, local_staged, mu, stream=None) -> None:
        _check(lib.muon_shard_momentum(self.handle, layout.handle, shard, local_grads.data_ptr(), local_momenta.data_ptr(),
                                       local_staged.data_ptr(), mu, _stream(stream)), "muon_shard_momentum")

    def muon_materialize_owned(self, flat, layout: Layout, matrices, stream=None) -> None:
        _check(lib.muon_materialize_owned(self.handle, flat.data_ptr(), layout.handle, _ptrs(matrices), _stream(stream)),
               "muon_materialize_owned")

    def muon_scatter_owned(self, flat, layout: Layout, matrices, stream=None) -> None:
        _check(lib.muon_scatter_owned(self.handle, flat.data_ptr(), layout.handle, _ptrs(matrices), _stream(stream)),
               "muon_scatter_owned")

    def muon_shard_apply(self, layout: Layout, shard: int, local_params, updates, lr, wd, stream=None) -> None:
        _check(lib.muon_shard_apply(self.handle, layout.handle, shard, local_params.data_ptr(), _ptrs(updates), lr, wd,
                                    _stream(stream)), "muon_shard_apply")

    # -- compute
    def muon_step_batched(self, params, grads, momenta, shapes, lr, mu, wd, ns_steps, coeffs, stream=None) -> None:
        co = _coeffs(coeffs)
        _check(lib.muon_step_batched(self.handle, _ptrs(params), _ptrs(grads), _ptrs(momenta), _shapes(shapes),
                                     len(shapes), lr, mu, wd, ns_steps, co, _stream(stream)), "muon_step_batched")

    def muon_step_batched_out(self, params, grads, momenta, updates, shapes, lr, mu, wd, ns_steps, coeffs, stream=None) -> None:
        co = _coeffs(coeffs)
        _check(lib.muon_step_batched_out(self.handle, _ptrs(params), _ptrs(grads), _ptrs(momenta),
                                         None if updates is None else _ptrs(updates), _shapes(shapes), len(shapes),
                                         lr, mu, wd, ns_steps, co, _stream(stream)), "muon_step_batched_out")

    def muon_step_batched_views(self, params, grads, momenta, updates, views, lr, mu, wd, ns_steps, coeffs, stream=None) -> None:
        """params/grads/momenta/updates: lists of device addresses (ints) of element (0,0) of each view;
        views: list of (rows, cols, ld)."""
        co = _coeffs(coeffs)
        va = (View * max(1, len(views)))()
        for i, (r, c, ld) in enumerate(views):
            va[i].rows, va[i].cols, va[i].ld = int(r), int(c), int(ld)
        _check(lib.muon_step_batched_views(self.handle, _ptrs(params), _ptrs(grads), _ptrs(momenta),
                                           None if updates is None else _ptrs(updates), va, len(views), lr, mu, wd, ns_steps,
                                           co, _stream(stream)), "muon_step_batched_views")

    def muon_step_flat(self, layout: Layout, flat_params, flat_grads, flat_momenta, flat_updates, lr, mu, wd, ns_steps, coeffs,
                       stream=None) -> None:
        co = _coeffs(coeffs)
        _check(lib.muon_step_flat(self.handle, layout.handle, flat_params.data_ptr(), flat_grads.data_ptr(),
                                  flat_momenta.data_ptr(), None if flat_updates is None else flat_updates.data_ptr(),
                                  lr, mu, wd, ns_steps, co, _stream(stream)), "muon_step_flat")

    def muon_step_flat_host(self, host_flat_grads, host_flat_updates, layout: Layout, params, grads, momenta,
                            updates, lr, mu, wd, ns_steps, coeffs, stream=None) -> None:
        """host_flat_*: CPU tensors (pinned for asynchronous copies)."""
        co = _coeffs(coeffs)
        _check(lib.muon_step_flat_host(self.handle, host_flat_grads.data_ptr(), host_flat_updates.data_ptr(),
                                       layout.handle, _ptrs(params), _ptrs(grads), _ptrs(momenta),
                                       _ptrs(updates), lr, mu, wd, ns_steps, co, _stream(stream)), "muon_step_flat_host")

    def muon_orthogonalize_batched(self, inputs, outputs, shapes, ns_steps, coeffs, flags=0, stream=None) -> None:
        co = _coeffs(coeffs)
        _check(lib.muon_orthogonalize_batched(self.handle, _ptrs(inputs), _ptrs(outputs), _shapes(shapes), len(shapes),
                                              ns_steps, co, flags, _stream(stream)), "muon_orthogonalize_batched")

    def muon_ns_product(self, p, q, d, c, m, n, k, ldp, ldq, ldc, stride_p, stride_q, stride_c, batch, nn,
                        alpha=1.0, beta=0.0, gamma=None, gamma_mode=0, stream=None) -> None:
        _check(lib.muon_ns_product(self.handle, p.data_ptr(), q.data_ptr(), None if d is None else d.data_ptr(),
                                   c.data_ptr(), m, n, k, ldp, ldq, ldc, stride_p, stride_q, stride_c, batch, nn,
                                   alpha, beta, None if gamma is None else gamma.data_ptr(), gamma_mode,
                                   _stream(stream)), "muon_ns_product")

    def muon_last_device_status(self, stream=None) -> int:
        v = C.c_int32(0)
        _check(lib.muon_last_device_status(self.handle, _stream(stream), C.byref(v)), "muon_last_device_status")
        return int(v.value)

    def muon_clear_device_status(self, stream=None) -> None:
        _check(lib.muon_clear_device_status(self.handle, _stream(stream)), "muon_clear_device_status")

    def muon_synchronize_and_check(self, stream=None) -> int:
        """Returns OK or ERR_DEVICE_TIMEOUT (does not raise for the latter: it is the answer, not a failure of the call)."""
        rc = int(lib.muon_synchronize_and_check(self.handle, _stream(stream)))
        if rc not in (OK, ERR_DEVICE_TIMEOUT):
            _check(rc, "muon_synchronize_and_check")
        return rc

    def muon_tensor_map_encodes(self) -> int:
        return int(lib.muon_tensor_map_encodes(self.handle))

    def muon_self_test_bounded_wait(self, stream=None) -> None:
        _check(lib.muon_self_test_bounded_wait(self.handle, _stream(stream)), "muon_self_test_bounded_wait")

    # -- profiling
    def muon_profile_enable(self, on: bool) -> None:
        _check(lib.muon_profile_enable(self.handle, 1 if on else 0), "muon_profile_enable")

    def muon_profile_reset(self) -> None:
        _check(lib.muon_profile_reset(self.handle), "muon_profile_reset")

    def muon_profile_read(self):
        out = {}
        for ph, name in enumerate(PHASE_NAMES):
            ms, n = C.c_double(0), C.c_int64(0)
            _check(lib.muon_profile_read(self.handle, ph, C.byref(ms), C.byref(n)), "muon_profile_read")
            out[name] = (float(ms.value), int(n.value))
        return out

    def muon_launch_count(self) -> int:
        return int(lib.muon_launch_count(self.handle))
