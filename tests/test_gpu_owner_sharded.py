"""GPU parity of the owner-sharded step (muon_shard_momentum, muon_materialize_owned, muon_orthogonalize_batched,
muon_shard_apply, orchestrated by paper_2609_21594_b200.owner_sharded): assembled from shard-local pieces it must
reproduce muon_step_batched on the whole matrices bit for bit -- with one rank, and with four ranks that run as
threads of this process on the one GPU (their kernels never wait on one another; the exchange is emulated by
device copies between the ranks' buffers), and through that match the oracle."""
import threading

import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import owner_sharded as osd
from paper_2609_21594_b200 import workloads as wl
from gpu_util import QUINTIC, bf16_input, dev_f32, host_f64, rel

pytestmark = pytest.mark.gpu

LR, MU, WD = 0.02, 0.95, 0.01
SHAPES = [(256, 256), (512, 128), (128, 512), (256, 256), (384, 640), (37, 53), (130, 8), (64, 64), (1, 1)]


class LocalHub:
    """Exchange between ranks that are threads of one process: every collective is a rendezvous plus device copies."""

    def __init__(self, world):
        self.world = world
        self.barrier = threading.Barrier(world)
        self.slots = {}

    def comm(self, rank):
        return LocalComm(self, rank)


class LocalComm:
    def __init__(self, hub, rank):
        self.hub, self.world, self.rank = hub, hub.world, rank
        self.seq = 0

    def all_gather(self, local):
        torch.cuda.synchronize()
        key = ("g", self.seq)
        self.seq += 1
        self.hub.slots[(key, self.rank)] = local
        self.hub.barrier.wait()
        full = torch.cat([self.hub.slots[(key, r)] for r in range(self.world)])
        torch.cuda.synchronize()
        self.hub.barrier.wait()
        return full

    def broadcast(self, t, src):
        key = ("b", self.seq)
        self.seq += 1
        if self.rank == src:
            torch.cuda.synchronize()
            self.hub.slots[key] = t
        return (key, t, src)

    def wait(self, handle):
        key, t, src = handle
        self.hub.barrier.wait()
        if self.rank != src:
            t.copy_(self.hub.slots[key])
        torch.cuda.synchronize()
        self.hub.barrier.wait()


def _whole(role, step, i):
    return wl.param_np("ownergpu", i, SHAPES[i]) if role == "param" else wl.grad_np("ownergpu", step, i, SHAPES[i])


def _reference(mb, n_steps):
    ctx = mb.Context()
    ctx.ensure_workspace(SHAPES)
    W = [dev_f32(_whole("param", 0, i)) for i in range(len(SHAPES))]
    M = [torch.zeros(s, dtype=torch.float32, device="cuda") for s in SHAPES]
    for step in range(n_steps):
        G = [bf16_input(_whole("grad", step, i))[0] for i in range(len(SHAPES))]
        ctx.muon_step_batched(W, G, M, SHAPES, LR, MU, WD, 5, QUINTIC)
    torch.cuda.synchronize()
    assert ctx.muon_last_device_status() == 0
    ctx.close()
    return W, M


def _rank_main(mb, hub, rank, n_steps, batch_elems, out, errors):
    try:
        torch.cuda.set_device(0)
        ctx = mb.Context()
        comm = hub.comm(rank) if hub.world > 1 else osd.SingleComm()
        st = osd.OwnerShardedStep(SHAPES, osd.CudaOps(ctx), comm, batch_elems=batch_elems)

        def fill(bufs, role, step, bits):
            for b, plan in enumerate(st.batches):
                segs = [(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in plan.layout.segments]
                whole = [_whole(role, step, i) for i in plan.matrices]
                if bits:
                    whole = [wl.to_bf16_bits(w) for w in whole]
                flat = orc.scatter(np.zeros(plan.layout.flat_len, dtype=np.uint16 if bits else np.float32), plan.shapes, segs, whole)
                n = plan.layout.shard_len
                piece = flat[rank * n:(rank + 1) * n]
                t = torch.from_numpy(piece.view(np.int16).copy()).cuda().view(torch.bfloat16) if bits else torch.from_numpy(piece.copy()).cuda()
                bufs[b][:n].copy_(t)

        fill(st.params, "param", 0, False)
        for b in range(len(st.batches)):
            st.momenta[b].zero_()
        for step in range(n_steps):
            fill(st.grads, "grad", step, True)
            st.step(LR, MU, WD, 5, QUINTIC)
        torch.cuda.synchronize()
        assert ctx.muon_last_device_status() == 0
        res = {}
        for b, plan in enumerate(st.batches):
            n = plan.layout.shard_len
            res[b] = (st.params[b][:n].cpu().numpy(), st.momenta[b][:n].cpu().numpy())
        out[rank] = (res, [(p.matrices, p.shapes, [(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in p.layout.segments],
                            p.layout.shard_len) for p in st.batches], list(st.owner_of))
        ctx.close()
    except BaseException as e:      # noqa: BLE001 -- reported by the main thread
        errors.append((rank, repr(e)))
        try:
            hub.barrier.abort()
        except Exception:
            pass


@pytest.mark.parametrize("world,batch_elems", [(1, 0), (1, 200000), (4, 0), (4, 150000)])
def test_owner_sharded_step_is_bit_identical_to_the_whole_matrix_step(world, batch_elems):
    from paper_2609_21594_b200 import binding as mb

    n_steps = 2
    Wref, Mref = _reference(mb, n_steps)
    hub = LocalHub(world)
    out, errors = {}, []
    threads = [threading.Thread(target=_rank_main, args=(mb, hub, r, n_steps, batch_elems, out, errors)) for r in range(world)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    assert len(out) == world
    plans = out[0][1]
    if world > 1:
        assert len(set(o for o in out[0][2] if o >= 0)) > 1          # more than one rank owns matrices
    if batch_elems:
        assert len(plans) > 1
    for b, (mats, shapes, segs, shard_len) in enumerate(plans):
        for name, idx, ref in (("W", 0, Wref), ("M", 1, Mref)):
            flat = np.concatenate([out[r][0][b][idx] for r in range(world)])
            whole = orc.materialize(flat, shapes, segs)
            for k, i in enumerate(mats):
                assert np.array_equal(whole[k], ref[i].cpu().numpy()), (name, world, b, i)
    # ... and the whole-matrix step itself is the oracle's (one matrix, first step, as an anchor)
    i = 4
    g = wl.bf16_bits_to_f32(wl.to_bf16_bits(_whole("grad", 0, i))).astype(np.float64)
    W0 = _whole("param", 0, i).astype(np.float64)
    Wn, Mn, _ = orc.muon_step(W0, g, np.zeros(SHAPES[i]), LR, MU, WD, 5, QUINTIC, 1e-7, True, "bf16")
    ctx = mb.Context()
    ctx.ensure_workspace([SHAPES[i]])
    W = [dev_f32(_whole("param", 0, i))]
    M = [torch.zeros(SHAPES[i], dtype=torch.float32, device="cuda")]
    ctx.muon_step_batched(W, [bf16_input(_whole("grad", 0, i))[0]], M, [SHAPES[i]], LR, MU, WD, 5, QUINTIC)
    torch.cuda.synchronize()
    assert rel(host_f64(W[0]) - W0, Wn - W0) <= 1e-2 and rel(host_f64(M[0]), Mn) <= 1e-6
    ctx.close()


def test_shard_calls_reject_bad_arguments_and_skip_absent_updates():
    from paper_2609_21594_b200 import binding as mb

    ctx = mb.Context()
    shapes = [(64, 64), (32, 16)]
    lay = wl.layout_per_param(shapes, 2)
    L = mb.Layout(ctx, lay, 2)
    n = lay.shard_len
    w = torch.ones(n, device="cuda")
    g = torch.zeros(n, device="cuda", dtype=torch.bfloat16)
    before = ctx.muon_launch_count()
    with pytest.raises(mb.MuonError) as e:
        ctx.muon_shard_momentum(L, 2, g, w, g.clone(), MU)           # shard index out of range
    assert e.value.code == mb.ERR_INVALID_ARG
    with pytest.raises(mb.MuonError) as e:
        ctx.muon_shard_apply(L, -1, w, [None, None], LR, WD)
    assert e.value.code == mb.ERR_INVALID_ARG and ctx.muon_launch_count() == before
    # an update that is absent leaves its slice alone; the other one is applied
    o = torch.ones(32, 16, device="cuda", dtype=torch.bfloat16)
    ctx.muon_shard_apply(L, 0, w, [None, o], 0.5, 0.0)
    torch.cuda.synchronize()
    got = w.cpu().numpy()
    seg = {s.matrix: s for s in lay.segments if s.flat_offset < n}
    a = seg[0]
    assert (got[a.flat_offset:a.flat_offset + a.elem_count] == 1.0).all()
    b = seg[1]
    want = np.float32(1.0) - np.float32(0.5) * np.float32(0.2 * np.sqrt(32.0))
    assert np.allclose(got[b.flat_offset:b.flat_offset + b.elem_count], want, rtol=1e-6)
    L.close()
    ctx.close()
