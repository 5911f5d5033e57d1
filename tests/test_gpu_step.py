"""GPU parity of the Muon step against the CPU oracle, element by element, through the C ABI.

Tolerances (relative Frobenius error per matrix): bf16 Newton-Schulz vs the bf16-emulating oracle
<= 1e-2; fp32 mode vs the fp64 oracle <= 1e-4; a single teacher-forced NS step <= 2e-3; momentum
and the update are compared in fp32 precision (1e-6).  Parity is measured on O (the NS output),
on the stored momentum M' and on dW = W' - W, never only on W'.
"""
import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import workloads as wl
from gpu_util import QUINTIC, bf16_input, dev_f32, host_f64, rel

pytestmark = pytest.mark.gpu

TOL_BF16 = 1e-2
TOL_FP32 = 1e-4
TOL_SINGLE_STEP = 2e-3
ENGINES = ["tensor", "tensor_1cta", "cuda_core"]


def _ctx(mb, precision="bf16", engine="tensor", grad="bf16", **kw):
    opt = mb.muon_default_options(
        ns_precision=mb.NS_BF16 if precision == "bf16" else mb.NS_FP32,
        engine={"tensor": mb.ENGINE_TENSOR, "tensor_1cta": mb.ENGINE_TENSOR_1CTA, "cuda_core": mb.ENGINE_CUDA_CORE}[engine],
        grad_dtype=mb.DTYPE_BF16 if grad == "bf16" else mb.DTYPE_FP32, **kw)
    return mb.Context(opt)


def _ortho(mb, ctx, mats_np, steps=5, coeffs=QUINTIC, flags=0):
    """Runs muon_orthogonalize_batched; returns (outputs as float64, inputs as float64 of the device values)."""
    bf = ctx.opt.ns_precision == mb.NS_BF16
    ins, vals = [], []
    for x in mats_np:
        if bf:
            t, v = bf16_input(x.astype(np.float32))
        else:
            t, v = dev_f32(x), x.astype(np.float32).astype(np.float64)
        ins.append(t)
        vals.append(v)
    outs = [torch.full_like(t, float("nan")) for t in ins]
    shapes = [tuple(x.shape) for x in mats_np]
    ctx.ensure_workspace(shapes)
    ctx.muon_orthogonalize_batched(ins, outs, shapes, steps, coeffs, flags)
    torch.cuda.synchronize()
    assert ctx.muon_last_device_status() == 0
    return [host_f64(o) for o in outs], vals


# ----------------------------------------------------------------------------- Newton-Schulz alone
@pytest.mark.parametrize("engine", ENGINES)
def test_ns_bf16_tiny_config_vs_oracle(engine):
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", engine)
    shapes = wl.shapes_tiny()
    mats = [wl.grad_np("tiny", 0, i, s) for i, s in enumerate(shapes)]
    outs, vals = _ortho(mb, ctx, mats)
    for i, (o, v) in enumerate(zip(outs, vals)):
        ref = orc.newton_schulz(v, 5, QUINTIC, 1e-7, "bf16")
        assert rel(o, ref) <= TOL_BF16, (i, shapes[i], rel(o, ref))
        hi = orc.newton_schulz(v, 5, QUINTIC, 1e-7, "fp64")
        assert rel(o, hi) <= 1.5 * rel(ref, hi)       # the device is as far from the exact result as the bf16 oracle is
    ctx.close()


@pytest.mark.parametrize("engine", ENGINES)
def test_ns_bf16_ragged_shapes_vs_oracle(engine):
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", engine)
    shapes = [(37, 53), (130, 7), (5, 1000), (1, 1), (300, 129), (129, 300), (200, 264), (8, 8), (1, 77), (77, 1)]
    mats = [wl.grad_np("ragged", 0, i, s) for i, s in enumerate(shapes)]
    outs, vals = _ortho(mb, ctx, mats)
    for i, (o, v) in enumerate(zip(outs, vals)):
        assert np.isfinite(o).all()
        ref = orc.newton_schulz(v, 5, QUINTIC, 1e-7, "bf16")
        assert rel(o, ref) <= TOL_BF16, (i, shapes[i], rel(o, ref))
    ctx.close()


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("shape", [(256, 256), (256, 1024), (1024, 256), (384, 640), (200, 264)])
def test_ns_single_step_teacher_forced(engine, shape):
    """Feed the oracle's bf16 X_k to one device NS step and compare with the oracle's X_{k+1}: the sharp,
    chaos-free check of every product and epilogue."""
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", engine)
    G = orc.bf16_rne(wl.grad_np("teacher", 0, shape[0], shape).astype(np.float64))
    trace = []
    orc.newton_schulz(G, 3, QUINTIC, 1e-7, "bf16", trace=trace)
    for k in (0, 2):
        Xk = trace[k][2]                       # working orientation (wide)
        Xk = Xk.T if shape[0] > shape[1] else Xk
        outs, vals = _ortho(mb, ctx, [Xk.astype(np.float32)], steps=1, flags=mb.ORTHO_NO_NORMALIZE)
        assert np.array_equal(vals[0], Xk)
        wide = vals[0].T if shape[0] > shape[1] else vals[0]
        ref = orc.ns_single_step(wide, *QUINTIC, mode="bf16")
        ref = ref.T if shape[0] > shape[1] else ref
        e = rel(outs[0], ref)
        assert e <= TOL_SINGLE_STEP, (k, e)
        assert np.mean(outs[0] != ref) < 0.10
    ctx.close()


def test_ns_fp32_mode_vs_fp64_oracle():
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "fp32")
    shapes = wl.shapes_tiny() + [(37, 53), (130, 7), (300, 129)]
    mats = [wl.grad_np("fp32", 0, i, s) for i, s in enumerate(shapes)]
    outs, vals = _ortho(mb, ctx, mats)
    for i, (o, v) in enumerate(zip(outs, vals)):
        ref = orc.newton_schulz(v, 5, QUINTIC, 1e-7, "fp64")
        assert rel(o, ref) <= TOL_FP32, (i, shapes[i], rel(o, ref))
    ctx.close()


def test_ns_fp32_cubic_converges_to_polar_factor_on_device():
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "fp32")
    rng = np.random.default_rng(4)
    U, _ = np.linalg.qr(rng.standard_normal((48, 48)))
    V, _ = np.linalg.qr(rng.standard_normal((80, 48)))
    G = (U * np.linspace(1, 3, 48)) @ V.T
    outs, _ = _ortho(mb, ctx, [G.astype(np.float32)], steps=40, coeffs=(1.5, -0.5, 0.0))
    assert rel(outs[0], U @ V.T) < 1e-4
    ctx.close()


def test_ns_per_step_coefficients():
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "fp32", coeffs_per_step=1)
    co = [3.0, -3.2, 1.2, 3.4445, -4.7750, 2.0315, 2.0, -1.5, 0.5]
    G = wl.grad_np("perstep", 0, 0, (40, 72))
    outs, vals = _ortho(mb, ctx, [G], steps=3, coeffs=co)
    assert rel(outs[0], orc.newton_schulz(vals[0], 3, co, 1e-7, "fp64")) <= TOL_FP32
    ctx.close()


@pytest.mark.parametrize("engine", ENGINES)
def test_zero_gradient_and_scaling(engine):
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", engine)
    Z = np.zeros((64, 96), dtype=np.float32)
    G = wl.grad_np("scale", 0, 0, (64, 96), std=1.0)
    outs, vals = _ortho(mb, ctx, [Z, G, G * np.float32(2.0 ** 40), G * np.float32(2.0 ** 20)])
    assert np.array_equal(outs[0], np.zeros((64, 96)))
    assert np.isfinite(outs[1]).all()
    # powers of two commute with every rounding and eps is negligible at these norms
    assert rel(outs[2], outs[1]) < 1e-3 and rel(outs[3], outs[1]) < 1e-3
    ctx.close()


@pytest.mark.parametrize("engine", ENGINES)
def test_batched_equals_alone_and_rerun_bit_exact(engine):
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", engine)
    shapes = [(256, 256)] * 3 + [(1024, 256), (256, 1024), (130, 200)]
    mats = [wl.grad_np("batch", 0, i, s) for i, s in enumerate(shapes)]
    together, _ = _ortho(mb, ctx, mats)
    again, _ = _ortho(mb, ctx, mats)
    for a, b in zip(together, again):
        assert np.array_equal(a, b)
    for i, m in enumerate(mats):
        alone, _ = _ortho(mb, ctx, [m])
        assert np.array_equal(alone[0], together[i]), i
    # a matrix whose row pitch rules out the 16-byte kernels must not change how its neighbours are summed
    mixed_shapes = [(256, 256), (37, 53), (384, 640)]
    mixed = [mats[0], wl.grad_np("batch", 0, 7, (37, 53)), wl.grad_np("batch", 0, 8, (384, 640))]
    mixed_out, _ = _ortho(mb, ctx, mixed)
    assert np.array_equal(mixed_out[0], together[0])
    for i in (1, 2):
        alone, _ = _ortho(mb, ctx, [mixed[i]])
        assert np.array_equal(alone[0], mixed_out[i]), mixed_shapes[i]
    # a small chunk cap changes the batching but not the numbers
    ctx2 = _ctx(mb, "bf16", engine, chunk_elems=70000)
    capped, _ = _ortho(mb, ctx2, mats)
    for a, b in zip(together, capped):
        assert np.array_equal(a, b)
    ctx.close()
    ctx2.close()


def test_batched_equals_alone_at_full_size_shapes():
    """Bit-exact "batched == alone" where a persistent CTA pair walks many tiles of several matrices:
    two 4096 x 4096 and two 1408 x 2048 matrices (and the tall orientation of the latter)."""
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", "tensor")
    shapes = [(4096, 4096), (1408, 2048), (4096, 4096), (2048, 1408), (1408, 2048)]
    mats = [wl.grad_np("batchbig", 0, i, s, row_scaled=(s[0] == 4096)) for i, s in enumerate(shapes)]
    together, vals = _ortho(mb, ctx, mats)
    for i in (0, 1, 3):
        alone, _ = _ortho(mb, ctx, [mats[i]])
        assert np.array_equal(alone[0], together[i]), i
    # and one of them against the oracle, so that "identical" is also "right"
    ref = orc.newton_schulz(vals[1], 5, QUINTIC, 1e-7, "bf16")
    assert rel(together[1], ref) <= TOL_BF16
    ctx.close()


# ----------------------------------------------------------------------------- the full step
def _run_steps(mb, ctx, config, shapes, n_steps, grad_bf16, row_scaled=False, lr=0.02, mu=0.95, wd=0.01):
    Ws = [wl.param_np(config, i, s) for i, s in enumerate(shapes)]
    dW, dM = [dev_f32(w) for w in Ws], [torch.zeros(s, dtype=torch.float32, device="cuda") for s in shapes]
    ctx.ensure_workspace(shapes)
    Gs_all, hist = [], []
    for t in range(n_steps):
        Gs_dev, Gs_val = [], []
        for i, s in enumerate(shapes):
            g = wl.grad_np(config, t, i, s, row_scaled=row_scaled)
            if grad_bf16:
                d, v = bf16_input(g)
            else:
                d, v = dev_f32(g), g.astype(np.float64)
            Gs_dev.append(d)
            Gs_val.append(v)
        Gs_all.append(Gs_val)
        ctx.muon_step_batched(dW, Gs_dev, dM, shapes, lr, mu, wd, 5, QUINTIC)
        torch.cuda.synchronize()
        hist.append(([host_f64(w) for w in dW], [host_f64(m) for m in dM]))
    assert ctx.muon_last_device_status() == 0
    return Ws, Gs_all, hist


@pytest.mark.parametrize("precision,engine,grad", [("fp32", "tensor", "fp32"), ("bf16", "tensor", "fp32"),
                                                   ("bf16", "cuda_core", "fp32"), ("bf16", "tensor", "bf16")])
def test_tiny_config_three_steps(precision, engine, grad):
    """d=256 one-layer matrix set, 3 consecutive optimizer steps from seed 0 (mu 0.95 Nesterov, lr 0.02, wd 0.01)."""
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, precision, engine, grad)
    shapes = wl.shapes_tiny()
    lr, mu, wd = 0.02, 0.95, 0.01
    Ws, Gs_all, hist = _run_steps(mb, ctx, "tiny", shapes, 3, grad == "bf16")
    mode = "bf16" if precision == "bf16" else "fp64"
    tol = TOL_BF16 if precision == "bf16" else TOL_FP32
    W = [w.astype(np.float64) for w in Ws]
    M = [np.zeros(s) for s in shapes]
    for t in range(3):
        gotW, gotM = hist[t]
        for i in range(len(shapes)):
            # teacher-forced per optimizer step: the oracle continues from the device's own state
            Wprev = W[i]
            Wn, Mn, O = orc.muon_step(Wprev, Gs_all[t][i], M[i], lr, mu, wd, 5, QUINTIC, 1e-7, True, mode)
            assert rel(gotM[i], Mn) <= 1e-6, (t, i)
            e = rel(gotW[i] - Wprev, Wn - Wprev)
            assert e <= tol, (t, i, shapes[i], e)
            O_dev = (Wprev * (1 - lr * wd) - gotW[i]) / (lr * orc.update_scale(*shapes[i]))
            assert rel(O_dev, O) <= tol + 1e-4, (t, i)
            W[i], M[i] = gotW[i], gotM[i]
    ctx.close()


def test_update_limits_and_snapshot_resume():
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", "tensor", "bf16")
    shapes = [(256, 256), (320, 192)]
    ctx.ensure_workspace(shapes)
    Ws = [dev_f32(wl.param_np("lim", i, s)) for i, s in enumerate(shapes)]
    Ms = [torch.zeros(s, dtype=torch.float32, device="cuda") for s in shapes]
    Gs = [bf16_input(wl.grad_np("lim", 0, i, s))[0] for i, s in enumerate(shapes)]
    W0 = [w.clone() for w in Ws]
    ctx.muon_step_batched(Ws, Gs, Ms, shapes, 0.0, 0.95, 0.3, 5, QUINTIC)     # lr = 0: weights untouched, momentum moves
    torch.cuda.synchronize()
    for w, w0, m, g in zip(Ws, W0, Ms, Gs):
        assert torch.equal(w, w0)
        assert torch.equal(m, g.float())                                     # M0 = 0: M' = G exactly
    # 3 steps == 2 steps + snapshot/restore + 1 step, bit for bit (all state is caller-owned)
    def run(n, Wi, Mi):
        for t in range(n[0], n[1]):
            G = [bf16_input(wl.grad_np("lim", t, i, s))[0] for i, s in enumerate(shapes)]
            ctx.muon_step_batched(Wi, G, Mi, shapes, 0.02, 0.95, 0.01, 5, QUINTIC)
        torch.cuda.synchronize()
    Wa, Ma = [w.clone() for w in W0], [torch.zeros_like(m) for m in Ms]
    run((0, 3), Wa, Ma)
    Wb, Mb = [w.clone() for w in W0], [torch.zeros_like(m) for m in Ms]
    run((0, 2), Wb, Mb)
    Wc, Mc = [w.cpu().cuda() for w in Wb], [m.cpu().cuda() for m in Mb]
    run((2, 3), Wc, Mc)
    for a, c in zip(Wa + Ma, Wc + Mc):
        assert torch.equal(a, c)
    ctx.close()


@pytest.mark.parametrize("engine", ["tensor", "cuda_core"])
def test_zero_gradient_through_the_full_step(engine):
    """G = 0 with M = 0: r = 1/eps = 1e7 is folded into the first epilogues and must multiply exact zeros.
    The step then reduces to W' = W (1 - lr wd), M' = mu M = 0, with no NaN or Inf anywhere; with a non-zero
    momentum and G = 0 the update follows the oracle like any other input."""
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", engine, "bf16")
    shapes = [(256, 256), (384, 128), (64, 200)]
    ctx.ensure_workspace(shapes)
    lr, mu, wd = 0.02, 0.95, 0.01
    W_np = [wl.param_np("zerog", i, s) for i, s in enumerate(shapes)]
    Ws = [dev_f32(w) for w in W_np]
    Ms = [torch.zeros(s, dtype=torch.float32, device="cuda") for s in shapes]
    Gs = [torch.zeros(s, dtype=torch.bfloat16, device="cuda") for s in shapes]
    Os = [torch.full(s, float("nan"), dtype=torch.bfloat16, device="cuda") for s in shapes]
    ctx.muon_step_batched_out(Ws, Gs, Ms, Os, shapes, lr, mu, wd, 5, QUINTIC)
    torch.cuda.synchronize()
    assert ctx.muon_last_device_status() == 0
    decay = np.float32(1.0) - np.float32(lr) * np.float32(wd)
    for w, w0, m, o in zip(Ws, W_np, Ms, Os):
        assert torch.count_nonzero(m).item() == 0 and torch.count_nonzero(o.float()).item() == 0
        assert np.array_equal(w.cpu().numpy(), w0 * decay)       # one fp32 product per element, nothing else
    # zero gradient on top of a live momentum: u = mu * M' is not zero, the oracle decides
    M_np = [wl.grad_np("zerog", 1, i, s) for i, s in enumerate(shapes)]
    Ms = [dev_f32(m) for m in M_np]
    Ws = [dev_f32(w) for w in W_np]
    ctx.muon_step_batched(Ws, Gs, Ms, shapes, lr, mu, wd, 5, QUINTIC)
    torch.cuda.synchronize()
    for i, s in enumerate(shapes):
        Wn, Mn, _ = orc.muon_step(W_np[i].astype(np.float64), np.zeros(s), M_np[i].astype(np.float64), lr, mu, wd, 5,
                                  QUINTIC, 1e-7, True, "bf16")
        assert rel(host_f64(Ms[i]), Mn) <= 1e-6
        assert rel(host_f64(Ws[i]) - W_np[i], Wn - W_np[i]) <= TOL_BF16, i
    ctx.close()


def test_step_argument_errors_launch_nothing():
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", "tensor", "bf16")
    shapes = [(64, 64)]
    W = [torch.zeros(64, 64, device="cuda")]
    M = [torch.zeros(64, 64, device="cuda")]
    G = [torch.zeros(64, 64, device="cuda", dtype=torch.bfloat16)]
    before = ctx.muon_launch_count()
    with pytest.raises(mb.MuonError) as e:
        ctx.muon_step_batched(W, G, M, shapes, 0.02, 0.95, 0.01, 5, QUINTIC)
    assert e.value.code == mb.ERR_WORKSPACE_TOO_SMALL
    ctx.ensure_workspace(shapes)
    for bad in ([None], [W[0].view(-1)[1:]]):
        with pytest.raises(mb.MuonError) as e:
            ctx.muon_step_batched(bad, G, M, shapes, 0.02, 0.95, 0.01, 5, QUINTIC)
        assert e.value.code == mb.ERR_INVALID_ARG
    with pytest.raises(mb.MuonError):
        ctx.muon_step_batched(W, G, M, shapes, 0.02, 0.95, 0.01, 0, QUINTIC)
    with pytest.raises(mb.MuonError):
        ctx.muon_step_batched(W, G, M, shapes, float("nan"), 0.95, 0.01, 5, QUINTIC)
    with pytest.raises(mb.MuonError):
        ctx.muon_step_batched(W, G, M, [(-1, 4)], 0.02, 0.95, 0.01, 5, QUINTIC)
    assert ctx.muon_launch_count() == before
    ctx.muon_step_batched([], [], [], [], 0.02, 0.95, 0.01, 5, QUINTIC)       # count == 0: a no-op
    ctx.muon_step_batched([None], [None], [None], [(0, 7)], 0.02, 0.95, 0.01, 5, QUINTIC)
    assert ctx.muon_launch_count() == before
    ctx.close()


def test_step_out_and_flat_host_path_match_the_plain_step():
    """muon_step_batched_out emits exactly the O the update applied; muon_step_flat_host (host flat shards in,
    host flat updates out) reproduces the device-resident sequence bit for bit."""
    from paper_2609_21594_b200 import binding as mb

    shapes = wl.shapes_tiny() + [(130, 200), (200, 130)]
    lay = wl.layout_per_param(shapes, 8)
    segs = [(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in lay.segments]
    ctx = _ctx(mb, "bf16", "tensor", "bf16")
    ctx.ensure_workspace(shapes)
    L = mb.Layout(ctx, lay, 2)
    g_bits = [wl.to_bf16_bits(wl.grad_np("flat", 0, i, s)) for i, s in enumerate(shapes)]
    flat_np = orc.scatter(np.zeros(lay.flat_len, dtype=np.uint16), shapes, segs, g_bits)
    W0 = [dev_f32(wl.param_np("flat", i, s)) for i, s in enumerate(shapes)]
    # (a) device-resident reference sequence
    Wa = [w.clone() for w in W0]
    Ma = [torch.zeros(s, dtype=torch.float32, device="cuda") for s in shapes]
    Ga = [torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16).reshape(s) for b, s in zip(g_bits, shapes)]
    Oa = [torch.full(s, float("nan"), dtype=torch.bfloat16, device="cuda") for s in shapes]
    ctx.muon_step_batched_out(Wa, Ga, Ma, Oa, shapes, 0.02, 0.95, 0.01, 5, QUINTIC)
    Wp = [w.clone() for w in W0]
    Mp = [torch.zeros_like(m) for m in Ma]
    ctx.muon_step_batched(Wp, Ga, Mp, shapes, 0.02, 0.95, 0.01, 5, QUINTIC)
    torch.cuda.synchronize()
    for i, s in enumerate(shapes):
        assert torch.equal(Wa[i], Wp[i]) and torch.equal(Ma[i], Mp[i])
        O_from_W = (host_f64(W0[i]) * (1 - 0.02 * 0.01) - host_f64(Wa[i])) / (0.02 * orc.update_scale(*s))
        assert rel(host_f64(Oa[i]), O_from_W) < 2e-4            # the emitted O is the O that was applied
        ref = orc.muon_step(host_f64(W0[i]), wl.bf16_bits_to_f32(g_bits[i]).astype(np.float64).reshape(s), np.zeros(s),
                            0.02, 0.95, 0.01, 5, QUINTIC, 1e-7, True, "bf16")[2]
        assert rel(host_f64(Oa[i]), ref) <= TOL_BF16
    # (b) the same step from host flat buffers
    host_in = torch.from_numpy(flat_np.view(np.int16)).view(torch.bfloat16).pin_memory()
    host_out = torch.zeros(lay.flat_len, dtype=torch.bfloat16).pin_memory()
    Wb = [w.clone() for w in W0]
    Mb = [torch.zeros_like(m) for m in Ma]
    Gb = [torch.zeros(s, dtype=torch.bfloat16, device="cuda") for s in shapes]
    Ob = [torch.zeros(s, dtype=torch.bfloat16, device="cuda") for s in shapes]
    ctx.muon_step_flat_host(host_in, host_out, L, Wb, Gb, Mb, Ob, 0.02, 0.95, 0.01, 5, QUINTIC)
    torch.cuda.synchronize()
    for i in range(len(shapes)):
        assert torch.equal(Wb[i], Wa[i]) and torch.equal(Mb[i], Ma[i]) and torch.equal(Ob[i].view(torch.int16), Oa[i].view(torch.int16))
    back = orc.materialize(host_out.view(torch.int16).numpy().view(np.uint16), shapes, segs)
    for i in range(len(shapes)):
        assert np.array_equal(back[i], Oa[i].view(torch.int16).cpu().numpy().view(np.uint16))
    L.close()
    ctx.close()


@pytest.mark.parametrize("engine", ENGINES)
def test_per_step_coefficient_sets_on_the_bf16_engines(engine):
    """A different (a_k, b_k, c_k) at every step -- the form the paper's default (asymmetric, five-step) variant
    takes (its values are not printed, so arbitrary per-step triples stand in; they are chosen so that the iteration stays
    bounded on all three shapes -- an earlier set drove one singular value of the 130 x 200 case to 166 in float64, where
    no rounding schedule can be compared with another)."""
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", engine, coeffs_per_step=1)
    co = [3.2, -4.2, 1.7, 3.0, -3.6, 1.4, 3.4445, -4.7750, 2.0315, 2.6, -2.8, 1.0, 2.0, -1.5, 0.5]
    shapes = [(256, 384), (384, 256), (130, 200)]
    mats = [wl.grad_np("perstep16", 0, i, s) for i, s in enumerate(shapes)]
    outs, vals = _ortho(mb, ctx, mats, steps=5, coeffs=co)
    for o, v in zip(outs, vals):
        assert rel(o, orc.newton_schulz(v, 5, co, 1e-7, "bf16")) <= TOL_BF16
    ctx.close()


@pytest.mark.parametrize("engine,precision", [("tensor", "bf16"), ("tensor_1cta", "bf16"), ("cuda_core", "bf16"), ("tensor", "fp32")])
@pytest.mark.parametrize("per_step", [0, 1])
def test_per_matrix_coefficient_rows(engine, precision, per_step):
    """coeffs_per_matrix: every matrix of one call iterates with its own polynomial while sharing the launches of its
    shape group.  Two coefficient sets are mixed inside one shape group and across groups; each result must match the
    oracle run with that matrix's row and must be far from the oracle run with the other row."""
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, precision, engine, coeffs_per_step=per_step, coeffs_per_matrix=1)
    set_a = [3.4445, -4.7750, 2.0315]
    set_b = [1.5, -0.5, 0.0]
    if per_step:
        row_a = [3.2, -4.2, 1.7, 3.0, -3.6, 1.4, 3.4445, -4.7750, 2.0315, 2.6, -2.8, 1.0, 2.0, -1.5, 0.5]
        row_b = [1.5, -0.5, 0.0, 2.0, -1.5, 0.5, 1.5, -0.5, 0.0, 3.0, -3.2, 1.2, 1.5, -0.5, 0.0]
    else:
        row_a, row_b = set_a, set_b
    shapes = [(256, 384), (384, 256), (256, 384), (130, 200), (256, 384), (130, 200)]
    pick = [0, 1, 1, 0, 0, 1]
    rows = [row_a if p == 0 else row_b for p in pick]
    mats = [wl.grad_np("permat", 0, i, s) for i, s in enumerate(shapes)]
    outs, vals = _ortho(mb, ctx, mats, steps=5, coeffs=rows)
    mode, tol = ("bf16", TOL_BF16) if precision == "bf16" else ("fp64", TOL_FP32)
    for i, (o, v) in enumerate(zip(outs, vals)):
        assert rel(o, orc.newton_schulz(v, 5, rows[i], 1e-7, mode)) <= tol, i
        other = row_b if pick[i] == 0 else row_a
        assert rel(o, orc.newton_schulz(v, 5, other, 1e-7, mode)) > 5e-2, i
    ctx.close()


def test_per_matrix_coefficient_rows_one_launch_per_product():
    """The same on a set large enough for one launch per product (not the whole-iteration launch), through the full step:
    alternating rows inside one shape group; bit-identical to running each coefficient class in a call of its own."""
    from paper_2609_21594_b200 import binding as mb

    shapes = [(512, 1024)] * 20 + [(1024, 512)] * 4
    rows = [[3.4445, -4.7750, 2.0315] if i % 3 else [3.0, -3.2, 1.2] for i in range(len(shapes))]
    ctx = _ctx(mb, "bf16", "tensor", "bf16", coeffs_per_matrix=1)
    ctx.ensure_workspace(shapes)
    gen = torch.Generator(device="cuda").manual_seed(77)
    Wn = [torch.randn(s, device="cuda", generator=gen) * 0.02 for s in shapes]
    Gn = [(torch.randn(s, device="cuda", generator=gen) * 1e-3).to(torch.bfloat16) for s in shapes]
    W, M = [w.clone() for w in Wn], [torch.zeros_like(w) for w in Wn]
    O = [torch.empty(s, dtype=torch.bfloat16, device="cuda") for s in shapes]
    n0 = ctx.muon_launch_count()
    ctx.muon_step_batched_out(W, Gn, M, O, shapes, 0.02, 0.95, 0.01, 5, rows)
    torch.cuda.synchronize()
    assert ctx.muon_launch_count() - n0 == 15 + 3          # 15 product launches, stage, norm, apply
    assert ctx.muon_last_device_status() == 0
    ctx.close()
    ref = _ctx(mb, "bf16", "tensor", "bf16")
    ref.ensure_workspace(shapes)
    for cls in ([3.4445, -4.7750, 2.0315], [3.0, -3.2, 1.2]):
        idx = [i for i in range(len(shapes)) if rows[i] == cls]
        W2, M2 = [Wn[i].clone() for i in idx], [torch.zeros_like(Wn[i]) for i in idx]
        O2 = [torch.empty(shapes[i], dtype=torch.bfloat16, device="cuda") for i in idx]
        ref.muon_step_batched_out(W2, [Gn[i] for i in idx], M2, O2, [shapes[i] for i in idx], 0.02, 0.95, 0.01, 5, cls)
        torch.cuda.synchronize()
        for j, i in enumerate(idx):
            assert torch.equal(O2[j].view(torch.int16), O[i].view(torch.int16)), i
            assert torch.equal(W2[j], W[i]), i
    # one sample against the oracle
    for i in (0, 1):
        v = Gn[i].to(torch.float64).cpu().numpy()
        assert rel(host_f64(O[i]), orc.newton_schulz(v, 5, rows[i], 1e-7, "bf16")) <= TOL_BF16
    ref.close()


def test_per_matrix_coefficient_rows_across_launch_sets():
    """Rows follow their matrices through the plan's reordering: a small cap forces several launch sets, two core shapes
    share some of them, and the caller's order interleaves shapes and coefficient classes."""
    from paper_2609_21594_b200 import binding as mb

    shapes = [(256, 512), (384, 256), (512, 256), (256, 384)] * 5
    classes = ([3.4445, -4.7750, 2.0315], [3.0, -3.2, 1.2], [1.5, -0.5, 0.0])
    rows = [classes[(i * 7 + i // 3) % 3] for i in range(len(shapes))]
    ctx = _ctx(mb, "bf16", "tensor", "bf16", coeffs_per_matrix=1, chunk_elems=1 << 18)
    nsets, _ = mb.muon_plan_launch_sets(ctx.opt, shapes)
    assert nsets >= 4
    ctx.ensure_workspace(shapes)
    gen = torch.Generator(device="cuda").manual_seed(78)
    G = [(torch.randn(s, device="cuda", generator=gen) * 1e-3).to(torch.bfloat16) for s in shapes]
    O = [torch.empty(s, dtype=torch.bfloat16, device="cuda") for s in shapes]
    ctx.muon_orthogonalize_batched(G, O, shapes, 5, rows)
    torch.cuda.synchronize()
    assert ctx.muon_last_device_status() == 0
    ctx.close()
    ref = _ctx(mb, "bf16", "tensor", "bf16", chunk_elems=1 << 18)
    ref.ensure_workspace(shapes)
    for cls in classes:
        idx = [i for i in range(len(shapes)) if rows[i] == cls]
        O2 = [torch.empty(shapes[i], dtype=torch.bfloat16, device="cuda") for i in idx]
        ref.muon_orthogonalize_batched([G[i] for i in idx], O2, [shapes[i] for i in idx], 5, cls)
        torch.cuda.synchronize()
        for j, i in enumerate(idx):
            assert torch.equal(O2[j].view(torch.int16), O[i].view(torch.int16)), (i, shapes[i])
    ref.close()


@pytest.mark.parametrize("shapes", [
    [(256, 256)] * 3,
    [(1408, 2048)] * 2,
    [(2048, 2048)] * 2 + [(1408, 2048)] * 2,
    wl.shapes_1b(1),
    [(4096, 4096)] * 2 + [(1024, 4096)] * 3,
], ids=["tiny3", "moe2", "two_shapes", "1b_layer", "llama_shapes"])
def test_whole_iteration_launch_equals_one_launch_per_product_on_a_poisoned_workspace(shapes):
    """The whole-iteration launch (small sets: grid barriers between the products) against the same tiles run as fifteen
    launches: bit-identical, three times in a row, with every byte of the workspace set to 0xFF before each call -- a tile that
    read an operand before its producer had written it would read NaNs, not the (identical) values a previous call left behind.
    The larger sets run one launch per product either way; for them the test checks run-to-run identity on a poisoned workspace."""
    from paper_2609_21594_b200 import binding as mb

    def run(launch_per_product, reps):
        ctx = _ctx(mb, "bf16", "tensor", launch_per_product=launch_per_product)
        ws = torch.empty(mb.muon_workspace_bytes(ctx.opt, shapes) + 4096, dtype=torch.uint8, device="cuda")
        ctx.muon_set_workspace(ws)
        gen = torch.Generator(device="cuda").manual_seed(5)
        ins = [(torch.randn(s, device="cuda", generator=gen) * 1e-3).to(torch.bfloat16) for s in shapes]
        outs = [torch.empty_like(t) for t in ins]
        res = []
        for _ in range(reps):
            ws.fill_(0xFF)
            ctx.muon_orthogonalize_batched(ins, outs, shapes, 5, QUINTIC)
            torch.cuda.synchronize()
            res.append([o.clone() for o in outs])
        assert ctx.muon_last_device_status() == 0
        ctx.close()
        return res

    flow = run(0, 3)
    ref = run(1, 1)[0]
    for rep in flow:
        for i, (a, b) in enumerate(zip(rep, ref)):
            assert bool(torch.isfinite(a.float()).all()), i
            assert torch.equal(a.view(torch.int16), b.view(torch.int16)), i


@pytest.mark.parametrize("steps", [1, 2, 16, 17])
def test_step_counts_at_the_edges_of_the_whole_iteration_launch(steps):
    """One step, two steps, the largest count the whole-iteration launch takes (16) and one more (17: one launch per product):
    bit-identical to one launch per product, and the singular values end where the quintic's fixed band says (the map is
    chaotic inside the band, so after many steps only properties can be compared, not elements)."""
    from paper_2609_21594_b200 import binding as mb

    shapes = wl.shapes_tiny()
    mats = [wl.grad_np("edges", 0, i, s) for i, s in enumerate(shapes)]
    ctx = _ctx(mb, "bf16", "tensor")
    n0 = ctx.muon_launch_count()
    outs, vals = _ortho(mb, ctx, mats, steps=steps)
    launches = ctx.muon_launch_count() - n0
    assert launches == (1 if steps <= 16 else 3 * steps) + 3
    ctx.close()
    ref_ctx = _ctx(mb, "bf16", "tensor", launch_per_product=1)
    ref, _ = _ortho(mb, ref_ctx, mats, steps=steps)
    ref_ctx.close()
    for o, r in zip(outs, ref):
        assert np.array_equal(o, r)
    if steps <= 2:
        for o, v in zip(outs, vals):
            assert rel(o, orc.newton_schulz(v, steps, QUINTIC, 1e-7, "bf16")) <= TOL_SINGLE_STEP * steps
    else:
        for o in outs:
            sv = np.linalg.svd(o, compute_uv=False)
            assert 0.6 < sv.min() and sv.max() < 1.25, (sv.min(), sv.max())


def test_plain_momentum_rule_and_eps_option():
    """nesterov = 0 (u = M') and a non-default epsilon are options of the context, not compile-time choices."""
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "fp32", "tensor", "fp32", nesterov=0, eps=5e-2)
    shapes = [(96, 160), (160, 96)]
    ctx.ensure_workspace(shapes)
    Wn = [wl.param_np("plain", i, s) for i, s in enumerate(shapes)]
    Mn = [wl.grad_np("plain", 7, i, s) for i, s in enumerate(shapes)]
    Gn = [wl.grad_np("plain", 0, i, s) for i, s in enumerate(shapes)]
    W, M, G = [dev_f32(x) for x in Wn], [dev_f32(x) for x in Mn], [dev_f32(x) for x in Gn]
    ctx.muon_step_batched(W, G, M, shapes, 0.02, 0.9, 0.05, 5, QUINTIC)
    torch.cuda.synchronize()
    for i in range(len(shapes)):
        Wr, Mr, _ = orc.muon_step(Wn[i].astype(np.float64), Gn[i].astype(np.float64), Mn[i].astype(np.float64), 0.02, 0.9, 0.05, 5,
                                  QUINTIC, 5e-2, False, "fp64")
        assert rel(host_f64(M[i]), Mr) <= 1e-6
        assert rel(host_f64(W[i]) - Wn[i], Wr - Wn[i]) <= TOL_FP32
        # eps = 5e-2 is comparable to ||u||_F here, so a wrong epsilon or a Nesterov look-ahead would be far outside 1e-4
        Wbad = orc.muon_step(Wn[i].astype(np.float64), Gn[i].astype(np.float64), Mn[i].astype(np.float64), 0.02, 0.9, 0.05, 5,
                             QUINTIC, 1e-7, False, "fp64")[0]
        assert rel(Wbad - Wn[i], Wr - Wn[i]) > 1e-2
    ctx.close()


@pytest.mark.parametrize("engine", ["tensor", "tensor_1cta"])
def test_ns_ragged_multi_tile_shapes(engine):
    """Shapes that are no multiple of any tile size and span several 256-wide tiles: the last CTA pair owns a
    partly (1300 = 5*256 + 20) or a half-empty (1408 = 5*256 + 128) row block, columns end inside a TMA box."""
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", engine)
    shapes = [(1300, 2100), (2100, 1300), (1408, 2048), (520, 520), (385, 1031)]
    mats = [wl.grad_np("ragged_big", 0, i, s) for i, s in enumerate(shapes)]
    outs, vals = _ortho(mb, ctx, mats)
    for i, (o, v) in enumerate(zip(outs, vals)):
        assert np.isfinite(o).all()
        ref = orc.newton_schulz(v, 5, QUINTIC, 1e-7, "bf16")
        assert rel(o, ref) <= TOL_BF16, (i, shapes[i], rel(o, ref))
    ctx.close()


def test_one_launch_per_product_for_all_shape_groups_and_no_encoding_in_steady_state():
    """The tensor engine runs each Newton-Schulz product as one kernel over every shape group that is resident
    together (3 * 5 product launches for the 1B-class layer with four core shapes, not 60), a set of a few tiles per
    product runs the whole iteration in ONE launch, and after the first step on a workspace no tensor map is
    encoded again."""
    from paper_2609_21594_b200 import binding as mb

    def run(shapes, name, **opt):
        ctx = _ctx(mb, "bf16", "tensor", **opt)
        ctx.ensure_workspace(shapes)
        ins = [bf16_input(wl.grad_np(name, 0, i, s))[0] for i, s in enumerate(shapes)]
        outs = [torch.empty_like(t) for t in ins]
        ctx.muon_orthogonalize_batched(ins, outs, shapes, 5, QUINTIC)          # binds the plan: encodes once
        torch.cuda.synchronize()
        first = [o.clone() for o in outs]
        enc0 = ctx.muon_tensor_map_encodes()
        assert enc0 > 0
        ctx.muon_profile_enable(True)
        ctx.muon_profile_reset()
        n0 = ctx.muon_launch_count()
        for _ in range(3):
            ctx.muon_orthogonalize_batched(ins, outs, shapes, 5, QUINTIC)
        torch.cuda.synchronize()
        ph = ctx.muon_profile_read()
        ctx.muon_profile_enable(False)
        assert ctx.muon_tensor_map_encodes() == enc0                           # steady state: nothing encoded
        assert all(torch.equal(a, b) for a, b in zip(first, outs))
        launches = (ph["ns"][1] // 3, (ctx.muon_launch_count() - n0) // 3)
        # a new workspace address re-binds once
        ctx.muon_set_workspace(torch.empty(mb.muon_workspace_bytes(ctx.opt, shapes) + 4096, dtype=torch.uint8, device="cuda"))
        ctx.muon_orthogonalize_batched(ins, outs, shapes, 5, QUINTIC)
        torch.cuda.synchronize()
        assert ctx.muon_tensor_map_encodes() == 2 * enc0
        assert all(torch.equal(a, b) for a, b in zip(first, outs))
        assert ctx.muon_last_device_status() == 0
        ctx.close()
        return launches, [host_f64(o) for o in outs], ins

    # d=256 layer, two core shapes, a handful of tiles per product: one launch for the whole iteration
    (ns, total), outs, ins = run(wl.shapes_tiny(), "grouped")
    assert ns == 1 and total == 1 + 2 + 1                                      # + stage, norm, apply
    (ns15, total15), outs15, _ = run(wl.shapes_tiny(), "grouped", launch_per_product=1)
    assert ns15 == 15 and total15 == 15 + 2 + 1
    assert all(np.array_equal(a, b) for a, b in zip(outs, outs15))
    ref = orc.newton_schulz(host_f64(ins[4]), 5, QUINTIC, 1e-7, "bf16")
    assert rel(outs[4], ref) <= TOL_BF16
    # one layer of the 1B-class stack: four core shapes in one launch set, too many tiles for the single launch
    (ns, total), _, _ = run(wl.shapes_1b(1), "grouped1b")
    assert ns == 15 and total == 15 + 2 + 1


def test_many_small_heterogeneous_matrices():
    """1500 small matrices of a dozen interleaved shapes (several shape groups, tall and wide mixed in one group,
    batches far larger than the SM count): every 50th one is checked against the oracle, all must be finite and
    batched == alone for a few."""
    from paper_2609_21594_b200 import binding as mb

    ctx = _ctx(mb, "bf16", "tensor")
    base = [(16, 16), (32, 48), (48, 32), (64, 64), (8, 120), (120, 8), (96, 160), (160, 96), (130, 40), (24, 24), (1, 64), (100, 100)]
    shapes = [base[i % len(base)] for i in range(1500)]
    mats = [wl.grad_np("swarm", 0, i, s) for i, s in enumerate(shapes)]
    outs, vals = _ortho(mb, ctx, mats)
    for o in outs:
        assert np.isfinite(o).all()
    for i in range(0, len(shapes), 50):
        ref = orc.newton_schulz(vals[i], 5, QUINTIC, 1e-7, "bf16")
        assert rel(outs[i], ref) <= TOL_BF16, (i, shapes[i], rel(outs[i], ref))
    for i in (3, 700, 1499):
        alone, _ = _ortho(mb, ctx, [mats[i]])
        assert np.array_equal(alone[0], outs[i])
    ctx.close()


def test_torch_optimizer_front_end_matches_the_oracle():
    """The torch.optim wrapper only marshals: two optimizer steps on three parameters equal the oracle's."""
    from paper_2609_21594_b200.optim import Muon

    shapes = [(256, 384), (384, 256), (128, 128)]
    params = [torch.nn.Parameter(dev_f32(wl.param_np("optim", i, s))) for i, s in enumerate(shapes)]
    opt = Muon(params, lr=0.02, momentum=0.95, weight_decay=0.01, ns_precision="fp32")
    W = [host_f64(p) for p in params]
    M = [np.zeros(s) for s in shapes]
    for t in range(2):
        for i, p in enumerate(params):
            p.grad = dev_f32(wl.grad_np("optim", t, i, shapes[i]))
        opt.step()
        torch.cuda.synchronize()
        for i, p in enumerate(params):
            g = wl.grad_np("optim", t, i, shapes[i]).astype(np.float64)
            Wn, Mn, _ = orc.muon_step(W[i], g, M[i], 0.02, 0.95, 0.01, 5, QUINTIC, 1e-7, True, "fp64")
            assert rel(host_f64(p) - W[i], Wn - W[i]) <= TOL_FP32
            assert rel(host_f64(opt.state[p]["momentum_buffer"]), Mn) <= 1e-6
            W[i], M[i] = host_f64(p), host_f64(opt.state[p]["momentum_buffer"])
