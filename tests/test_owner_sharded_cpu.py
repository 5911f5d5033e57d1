"""The owner-sharded step on a CPU: the host planner against brute force, and the exchange bookkeeping of
paper_2609_21594_b200.owner_sharded with two gloo ranks.  Compute is stubbed by the oracle (the CUDA library is
not involved), so what is tested is exactly the host logic: who owns what, which shard and which update sits
where in the exchange buffers, in which order collectives are issued and settled, and that the step assembled
from shard-local pieces equals the oracle's whole-matrix step."""
import itertools
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import binding as mb
from paper_2609_21594_b200 import owner_sharded as osd
from paper_2609_21594_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
LR, MU, WD = 0.02, 0.95, 0.01


def _cost(shape):
    s, l = min(shape), max(shape)
    return 3.0 * s * s * l + s ** 3


# ----------------------------------------------------------------------------- the planner
def test_owner_plan_owns_every_matrix_once_and_is_deterministic():
    shapes = wl.shapes_llama8b(2) + [(0, 7), (5, 0)]
    owner, batch, nb = mb.muon_owner_plan(shapes, 8, 1 << 29)
    again = mb.muon_owner_plan(shapes, 8, 1 << 29)
    assert (owner, batch, nb) == again
    for (m, n), o, b in zip(shapes, owner, batch):
        if m == 0 or n == 0:
            assert o == -1 and b == -1
        else:
            assert 0 <= o < 8 and 0 <= b < nb
    # batches in descending size: no matrix of a later batch is larger than one of an earlier batch
    sizes = [[m * n for (m, n), b in zip(shapes, batch) if b == k] for k in range(nb)]
    assert all(sizes[k] for k in range(nb))
    for k in range(nb - 1):
        assert min(sizes[k]) >= max(sizes[k + 1])
    # the cap closes a batch (a single matrix may exceed it on its own)
    assert all(sum(s) <= (1 << 29) or len(s) == 1 for s in sizes)
    # one batch when no cap is given
    assert mb.muon_owner_plan(shapes, 8, 0)[2] == 1


@pytest.mark.parametrize("seed", range(12))
def test_owner_plan_is_within_four_thirds_of_the_best_assignment(seed):
    """Brute force over all owner assignments of up to 9 matrices on 2-3 ranks."""
    rng = np.random.default_rng(seed)
    n, ranks = int(rng.integers(3, 10)), int(rng.integers(2, 4))
    shapes = [(int(rng.integers(1, 40)) * 8, int(rng.integers(1, 40)) * 8) for _ in range(n)]
    owner, batch, nb = mb.muon_owner_plan(shapes, ranks, 0)
    assert nb == 1
    load = [0.0] * ranks
    for s, o in zip(shapes, owner):
        load[o] += _cost(s)
    best = min(max(sum(_cost(s) for s, o in zip(shapes, assign) if o == r) for r in range(ranks))
               for assign in itertools.product(range(ranks), repeat=n))
    assert max(load) <= (4.0 / 3.0 - 1.0 / (3.0 * ranks)) * best * (1 + 1e-12)
    assert max(load) >= best * (1 - 1e-12)


def test_owner_plan_balances_the_llama_set():
    shapes = wl.shapes_llama8b()
    owner, batch, nb = mb.muon_owner_plan(shapes, 8, 0)
    load = np.zeros(8)
    for s, o in zip(shapes, owner):
        load[o] += _cost(s)
    assert load.max() / load.mean() < 1.02


def test_build_batches_offsets_are_disjoint_and_aligned():
    shapes = wl.shapes_tiny() + wl.shapes_odd()
    owner, batch, nb = mb.muon_owner_plan(shapes, 3, 300000)
    plans = osd.build_batches(shapes, 3, owner, batch, nb)
    assert sorted(i for p in plans for i in p.matrices) == list(range(len(shapes)))
    for p in plans:
        assert p.layout.num_shards == 3
        spans = {}
        for (m, n), o, off in zip(p.shapes, p.owners, p.region_off):
            assert off % osd.REGION_ALIGN == 0 and off + m * n <= p.region_len[o]
            spans.setdefault(o, []).append((off, off + m * n))
        for o, sp in spans.items():
            sp.sort()
            assert all(a[1] <= b[0] for a, b in zip(sp, sp[1:]))


# ----------------------------------------------------------------------------- two gloo ranks, oracle compute
class OracleOps:
    """Stand-in for the CUDA library: the same shard-local operations on CPU tensors, arithmetic by the oracle."""
    grad_dtype, ns_dtype = torch.float32, torch.float32

    def owner_plan(self, shapes, world, batch_elems):
        return mb.muon_owner_plan(shapes, world, batch_elems)          # host-only entry point of the library

    def new_batch(self, plan):
        return [(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in plan.layout.segments]

    def empty(self, n, dtype):
        return torch.zeros(max(n, 1), dtype=dtype)

    def _local_segments(self, plan, rank):
        n = plan.layout.shard_len
        return [(mat, eb, ec, off - rank * n) for (mat, eb, ec, off) in plan.handle if rank * n <= off < (rank + 1) * n]

    def shard_momentum(self, plan, rank, g, m, u, mu):
        for (_, _, ec, off) in self._local_segments(plan, rank):
            m_new, uu = orc.momentum_nesterov(g[off:off + ec].numpy(), m[off:off + ec].numpy(), mu, True)
            m[off:off + ec] = torch.from_numpy(m_new.astype(np.float32))
            u[off:off + ec] = torch.from_numpy(uu.astype(np.float32))

    def materialize_owned(self, plan, flat, mats):
        whole = orc.materialize(flat.numpy(), plan.shapes, plan.handle)
        for k, t in enumerate(mats):
            if t is not None:
                t.copy_(torch.from_numpy(whole[k]))

    def orthogonalize(self, shapes, ins, outs, ns_steps, coeffs):
        for x, o in zip(ins, outs):
            o.copy_(torch.from_numpy(orc.newton_schulz(x.numpy().astype(np.float64), ns_steps, coeffs, 1e-7, "fp64").astype(np.float32)))

    def shard_apply(self, plan, rank, w, updates, lr, wd):
        for (mat, eb, ec, off) in self._local_segments(plan, rank):
            m, n = plan.shapes[mat]
            o = updates[mat].reshape(-1)[eb:eb + ec].numpy().astype(np.float64)
            w_old = w[off:off + ec].numpy().astype(np.float64)
            w[off:off + ec] = torch.from_numpy((w_old * (1.0 - lr * wd) - lr * orc.update_scale(m, n) * o).astype(np.float32))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


SHAPES = [(40, 24), (16, 16), (24, 40), (8, 64), (33, 7), (16, 16), (5, 5)]


def _whole(role, step, i):
    shape = SHAPES[i]
    return wl.param_np("owner", i, shape) if role == "param" else wl.grad_np("owner", step, i, shape)


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import torch.distributed as dist

    dist.init_process_group("gloo", rank=rank, world_size=world)
    ops = OracleOps()
    st = osd.OwnerShardedStep(SHAPES, ops, osd.TorchComm(), batch_elems=1500, align=4)
    assert len(st.batches) >= 2
    n_steps = 2

    def fill(buf_list, role, step):
        for b, plan in enumerate(st.batches):
            whole = [_whole(role, step, i) for i in plan.matrices]
            flat = orc.scatter(np.zeros(plan.layout.flat_len, dtype=np.float32), plan.shapes, plan.handle, whole)
            n = plan.layout.shard_len
            buf_list[b][:n] = torch.from_numpy(flat[rank * n:(rank + 1) * n])

    fill(st.params, "param", 0)
    for step in range(n_steps):
        fill(st.grads, "grad", step)
        st.step(LR, MU, WD, 5, wl.QUINTIC)
    # collect the shards of every batch and rebuild the whole matrices
    comm = osd.TorchComm()
    result = {}
    for b, plan in enumerate(st.batches):
        n = plan.layout.shard_len
        for name, bufs in (("W", st.params), ("M", st.momenta)):
            full = comm.all_gather(bufs[b][:n].contiguous())
            whole = orc.materialize(full.numpy(), plan.shapes, plan.handle)
            for k, i in enumerate(plan.matrices):
                result[(name, i)] = whole[k]
    out[rank] = (result, list(st.events), list(st.owner_of), [p.matrices for p in st.batches])
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_whole_matrix_step():
    if torch.cuda.is_available():
        pytest.skip("the CPU/gloo variant of the check")
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    res0, ev0, owner0, batches0 = out[0]
    res1, ev1, owner1, batches1 = out[1]
    # both ranks built the same plan and issued the same sequence of collectives
    assert owner0 == owner1 and batches0 == batches1 and ev0 == ev1
    assert sorted(i for b in batches0 for i in b) == list(range(len(SHAPES)))
    assert set(owner0) == {0, 1}                                # both ranks own something
    # order of collectives: gather b, (settle b-1), broadcasts of b ...; never two batches' broadcasts in flight
    nb = len(batches0)
    per_step = len(ev0) // 2
    ev = ev0[:per_step]
    assert ev[-1] == ("drained",)
    in_flight = set()
    for e in ev:
        if e[0] == "broadcast":
            in_flight.add(e[1])
        elif e[0] == "apply":
            in_flight.discard(e[1])
        assert len(in_flight) <= 1, ev
    assert [e[1] for e in ev if e[0] == "gather"] == list(range(nb))
    assert [e[1] for e in ev if e[0] == "apply"] == list(range(nb))
    for b in range(1, nb):                                       # admitting batch b settles batch b-1 first
        assert ev.index(("apply", b - 1)) < min(i for i, e in enumerate(ev) if e[0] == "broadcast" and e[1] == b)
    # every broadcast comes from the owner of the matrices it carries
    for e in ev:
        if e[0] == "broadcast":
            assert any(owner0[i] == e[2] for i in batches0[e[1]])
    # the assembled result equals the oracle's whole-matrix steps (same float32 storage points, fp64 arithmetic)
    for i, shape in enumerate(SHAPES):
        W = _whole("param", 0, i).astype(np.float64)
        M = np.zeros(shape)
        for step in range(2):
            W, M, _ = orc.muon_step(W, _whole("grad", step, i).astype(np.float64), M, LR, MU, WD, 5, wl.QUINTIC, 1e-7, True, "fp64")
        for res in (res0, res1):
            assert np.abs(res[("M", i)] - M).max() <= 1e-7 * max(1.0, np.abs(M).max()), i
            assert np.linalg.norm(res[("W", i)] - W) <= 1e-5 * np.linalg.norm(W), i
