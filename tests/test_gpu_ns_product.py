"""GPU parity of the batched Newton-Schulz product primitive (the three products of one step of
Eq. 1) against its plain definition: a float64 matrix product of the same bf16 values, one bf16
rounding of the result.  Exercises both engines, K-major and MN-major second operands, ragged
edges, several tiles per matrix and several matrices per launch."""
import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import workloads as wl
from gpu_util import bf16_input, host_f64, rel

pytestmark = pytest.mark.gpu


def _padded(vals_list, ld):
    """Stack same-shape matrices into a [batch, rows, ld] bf16 device tensor (pad columns hold NaN)."""
    b, (r, c) = len(vals_list), vals_list[0].shape
    t = torch.full((b, r, ld), float("nan"), dtype=torch.bfloat16, device="cuda")
    host = []
    for i, v in enumerate(vals_list):
        d, hv = bf16_input(v.astype(np.float32))
        t[i, :, :c] = d
        host.append(hv)
    return t, host


def _run(mb, engine, m, n, k, batch, nn, with_d, gamma_mode, seed):
    opt = mb.muon_default_options(engine={"tensor": mb.ENGINE_TENSOR, "tensor_1cta": mb.ENGINE_TENSOR_1CTA, "cuda_core": mb.ENGINE_CUDA_CORE}[engine])
    ctx = mb.Context(opt)
    rng = np.random.default_rng(seed)
    up8 = lambda x: (x + 7) // 8 * 8
    sym = nn == 2
    P = [rng.standard_normal((m, k)) for _ in range(batch)]
    Q = [rng.standard_normal((k, n) if nn == 1 else (n, k)) for _ in range(batch)]
    D = [rng.standard_normal((m, n)) for _ in range(batch)]
    if sym:
        assert m == n
        D = [(d + d.T) / 2 for d in D]
    ldp, ldq, ldc = up8(k), up8(n if nn == 1 else k), up8(n)
    tP, hP = _padded(P, ldp)
    tQ, hQ = (tP, hP) if sym else _padded(Q, ldq)
    tD, hD = _padded(D, ldc)
    tC = torch.full((batch, m, ldc), -7.0, dtype=torch.bfloat16, device="cuda")
    gam = rng.uniform(0.5, 2.0, size=batch).astype(np.float32)
    tG = torch.from_numpy(gam).cuda()
    alpha, beta = 2.0315, -4.775
    ctx.muon_ns_product(tP, tQ, tD if with_d else None, tC, m, n, k, ldp, ldq, ldc, m * ldp, tQ.shape[1] * ldq, m * ldc,
                        batch, nn, alpha, beta, tG if gamma_mode else None, gamma_mode)
    torch.cuda.synchronize()
    assert ctx.muon_last_device_status() == 0
    got = host_f64(tC)
    a32, b32 = float(np.float32(alpha)), float(np.float32(beta))
    worst = 0.0
    for i in range(batch):
        acc = hP[i] @ (hQ[i] if nn == 1 else hQ[i].T)
        v = a32 * acc + (b32 * hD[i] if with_d else 0.0)
        g = 1.0 if not gamma_mode else (float(gam[i]) if gamma_mode == 1 else float(gam[i]) ** 2)
        ref = orc.bf16_rne(g * v)
        out = got[i, :, :n]
        assert np.isfinite(out).all()
        worst = max(worst, rel(out, ref))
        # at most one bf16 ulp apart anywhere (fp32 vs fp64 accumulation can flip a rounding), plus the
        # absolute fp32 accumulation error where the sum cancels
        mag = np.abs(hP[i]) @ np.abs(hQ[i] if nn == 1 else hQ[i].T)
        slack = abs(g) * (abs(a32) * mag + (abs(b32) * np.abs(hD[i]) if with_d else 0.0)) * 2.0 ** -20
        assert np.all(np.abs(out - ref) <= np.abs(ref) * 2.0 ** -7 + slack)
        # pad columns: the bulk store works in 16-byte pieces, so the tensor engine may overwrite the padding of a
        # row up to the next multiple of 8 elements (never beyond ldc); anything else must be untouched
        assert np.all((got[i, :, n:] == -7.0) | np.isfinite(got[i, :, n:]))
        assert np.all(got[i, :, (n + 7) // 8 * 8:] == -7.0)
        if sym:
            assert np.array_equal(out, out.T)         # mirrored stores make the result exactly symmetric
    ctx.close()
    return worst


CASES = [
    # m, n, k, batch
    (128, 256, 64, 1),
    (128, 256, 256, 1),
    (256, 512, 320, 2),
    (200, 264, 136, 3),
    (37, 53, 1000, 2),
    (384, 640, 384, 1),
    (1, 1, 8, 1),
    (130, 7, 24, 2),
]


@pytest.mark.parametrize("engine", ["tensor", "tensor_1cta", "cuda_core"])
@pytest.mark.parametrize("nn", [0, 1])
@pytest.mark.parametrize("case", CASES)
def test_product_plain(engine, nn, case):
    from paper_2609_21594_b200 import binding as mb

    m, n, k, batch = case
    assert _run(mb, engine, m, n, k, batch, nn, False, 0, seed=m * 7 + n) < 3e-3


@pytest.mark.parametrize("engine", ["tensor", "tensor_1cta", "cuda_core"])
@pytest.mark.parametrize("nn", [0, 1])
@pytest.mark.parametrize("gamma_mode", [0, 1, 2])
def test_product_fused_epilogue(engine, nn, gamma_mode):
    from paper_2609_21594_b200 import binding as mb

    assert _run(mb, engine, 256, 320, 192, 3, nn, True, gamma_mode, seed=11 + gamma_mode) < 3e-3
    assert _run(mb, engine, 200, 264, 136, 2, nn, True, gamma_mode, seed=12 + gamma_mode) < 3e-3


def test_product_many_tiles_persistent_loop():
    """More tiles than SMs: every CTA walks several tiles, both TMEM accumulators and all stages wrap."""
    from paper_2609_21594_b200 import binding as mb

    assert _run(mb, "tensor", 1024, 1024, 512, 6, 0, True, 1, seed=3) < 3e-3
    assert _run(mb, "tensor", 1024, 2048, 1024, 3, 1, True, 2, seed=4) < 3e-3


SYM_CASES = [(128, 64, 1), (256, 320, 2), (384, 136, 3), (200, 1000, 2), (1024, 512, 2), (1408, 256, 1), (37, 53, 2)]


@pytest.mark.parametrize("engine", ["tensor", "tensor_1cta", "cuda_core"])
@pytest.mark.parametrize("case", SYM_CASES)
def test_symmetric_product(engine, case):
    """C = gamma (beta D + alpha P P^T): triangular tile schedule with mirrored stores on the tensor engine."""
    from paper_2609_21594_b200 import binding as mb

    s, k, batch = case
    assert _run(mb, engine, s, s, k, batch, 2, False, 0, seed=s + k) < 3e-3
    assert _run(mb, engine, s, s, k, batch, 2, True, 2, seed=s + k + 1) < 3e-3
