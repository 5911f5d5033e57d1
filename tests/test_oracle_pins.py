"""Pins for the CPU oracle: each test checks it against something other than itself --
an SVD closed form, a scalar recurrence, a brute-force index map, an invariant, a
hand-computed case or an independent library's rounding."""
import os

import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2609_21594_b200 import workloads as wl

QUINTIC = (3.4445, -4.7750, 2.0315)
CUBIC = (1.5, -0.5, 0.0)


def rel(a, b):
    return float(np.linalg.norm(np.asarray(a) - np.asarray(b)) / max(np.linalg.norm(np.asarray(b)), 1e-300))


def p_scalar(x, co=QUINTIC):
    a, b, c = co
    return a * x + b * x ** 3 + c * x ** 5


def g_formula(m, n, k=0):
    i = np.arange(m)[:, None]
    j = np.arange(n)[None, :]
    return (((3 * i + 5 * j + k) % 7) - 3 + 0.25 * i).astype(np.float64)


def svd_closed_form(G, steps, co, eps):
    """NS(G) = U diag(p^steps(sigma_i / (||G||_F + eps))) V^T  (Eq. 1 acts on singular values only)."""
    U, s, Vt = np.linalg.svd(G, full_matrices=False)
    x = s / (np.sqrt((G * G).sum()) + eps)
    for _ in range(steps):
        x = p_scalar(x, co)
    return (U * x) @ Vt


# ----------------------------------------------------------------------------- bf16 rounding
def test_bf16_rne_all_bf16_values_are_fixed_points():
    bits = np.arange(1 << 16, dtype=np.uint16)
    vals = wl.bf16_bits_to_f32(bits).astype(np.float64)
    finite = np.isfinite(vals)
    out = orc.bf16_rne(vals[finite])
    assert np.array_equal(out, vals[finite])
    assert np.array_equal(np.signbit(out), np.signbit(vals[finite]))


def test_bf16_rne_matches_independent_cast_on_fp32_inputs():
    rng = np.random.default_rng(0)
    raw = rng.integers(0, 1 << 32, size=400000, dtype=np.uint64).astype(np.uint32)
    x = raw.view(np.float32)
    x = x[np.isfinite(x)]
    # add exact ties and near-ties around every exponent, and the subnormal range
    bits = np.arange(0, 1 << 16, 7, dtype=np.uint32) << 16
    ties = (bits | 0x8000).view(np.float32)
    near = np.concatenate([(bits | 0x7FFF).view(np.float32), (bits | 0x8001).view(np.float32)])
    x = np.concatenate([x, ties[np.isfinite(ties)], near[np.isfinite(near)]])
    ref = torch.from_numpy(x.copy()).to(torch.bfloat16).to(torch.float64).numpy()
    got = orc.bf16_rne(x.astype(np.float64))
    assert np.array_equal(got, ref)


def test_bf16_rne_ties_from_float64():
    assert orc.bf16_rne(np.array([1.0 + 2.0 ** -8]))[0] == 1.0                      # tie -> even (1.0)
    assert orc.bf16_rne(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6      # tie -> even (mantissa 2)
    assert orc.bf16_rne(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 1.0 + 2.0 ** -7  # just above a tie
    assert orc.bf16_rne(np.array([-(1.0 + 2.0 ** -8 + 2.0 ** -40)]))[0] == -(1.0 + 2.0 ** -7)
    assert np.isinf(orc.bf16_rne(np.array([3.4e38]))[0])
    assert orc.bf16_rne(np.array([0.0]))[0] == 0.0


# ----------------------------------------------------------------------------- layout gather / scatter
@pytest.mark.parametrize("gen", [wl.layout_per_param, wl.layout_flat_concat])
@pytest.mark.parametrize("shards", [1, 3, 8])
def test_layout_roundtrip_bruteforce(gen, shards):
    shapes = wl.shapes_odd()
    lay = gen(shapes, shards)
    segs = [(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in lay.segments]
    assert orc.layout_is_valid(lay.flat_len, shapes, segs, lay.align, lay.num_shards, lay.shard_len)
    # brute-force per-element index map: flat position -> (matrix, linear element)
    owner = {}
    for (mat, eb, ec, off) in segs:
        for t in range(ec):
            assert off + t not in owner
            owner[off + t] = (mat, eb + t)
    assert len(owner) == sum(m * n for m, n in shapes)
    rng = np.random.default_rng(1)
    flat = rng.integers(1, 1 << 16, size=lay.flat_len, dtype=np.uint16)
    mats = orc.materialize(flat, shapes, segs)
    for pos, (mat, e) in owner.items():
        assert mats[mat].reshape(-1)[e] == flat[pos]
    # scatter into a canary-filled buffer: payload restored, padding untouched
    canary = np.full(lay.flat_len, 0xABCD, dtype=np.uint16)
    back = orc.scatter(canary, shapes, segs, mats)
    for pos in range(lay.flat_len):
        if pos in owner:
            assert back[pos] == flat[pos]
        else:
            assert back[pos] == 0xABCD
    # materialize(scatter(Ms)) == Ms
    mats2 = orc.materialize(back, shapes, segs)
    for a, b in zip(mats, mats2):
        assert np.array_equal(a, b)


def test_layout_numbers_of_the_llama_set():
    shapes = wl.shapes_llama8b()
    lay = wl.layout_per_param(shapes, 8)
    assert len(lay.segments) == 1792
    assert lay.shard_len == 872415232
    assert lay.flat_len == lay.payload            # all dims are multiples of 8*128: no padding
    odd = wl.layout_per_param(wl.shapes_odd(), 8)
    assert len(odd.segments) == 38
    assert odd.flat_len - odd.payload == 6676


def test_layout_validity_rejects_broken_tables():
    shapes = [(4, 6), (3, 3)]
    lay = wl.layout_per_param(shapes, 2, align=8)
    segs = [(s.matrix, s.elem_begin, s.elem_count, s.flat_offset) for s in lay.segments]
    args = (lay.flat_len, shapes, segs, 8, 2, lay.shard_len)
    assert orc.layout_is_valid(*args)
    assert not orc.layout_is_valid(lay.flat_len, shapes, segs[:-1], 8, 2, lay.shard_len)        # gap
    assert not orc.layout_is_valid(lay.flat_len, shapes, segs + [segs[0]], 8, 2, lay.shard_len)  # overlap
    bad = list(segs)
    m, eb, ec, off = bad[0]
    bad[0] = (m, eb, ec, off + 1)
    assert not orc.layout_is_valid(lay.flat_len, shapes, bad, 8, 2, lay.shard_len)               # misaligned


def test_layout_validity_shard_straddle_rule_by_hand():
    """A segment must lie inside one shard.  Hand-built table: one 1 x 12 matrix in a flat buffer of two shards
    of 8 elements.  Stored as one piece at offset 4 it covers flat[4:16] and crosses the boundary at 8: invalid.
    Cut at the boundary (4 elements in shard 0, 8 in shard 1) the same bytes are a valid layout, and the gather
    of the split table returns exactly the elements the straddling table would have named."""
    shapes = [(1, 12)]
    whole = [(0, 0, 12, 4)]
    split = [(0, 0, 4, 4), (0, 4, 8, 8)]
    assert not orc.layout_is_valid(16, shapes, whole, 4, 2, 8)
    assert orc.layout_is_valid(16, shapes, split, 4, 2, 8)
    # with a single shard of 16 nothing is crossed, so the one-piece table is fine: the rule is about shards only
    assert orc.layout_is_valid(16, shapes, whole, 4, 1, 16)
    # a piece that ends exactly at the boundary does not straddle; one element more does
    assert orc.layout_is_valid(16, [(1, 8)], [(0, 0, 8, 0)], 4, 2, 8)
    assert not orc.layout_is_valid(16, [(1, 9)], [(0, 0, 9, 0)], 4, 2, 8)
    flat = np.arange(100, 116)
    assert np.array_equal(orc.materialize(flat, shapes, split)[0].ravel(), flat[4:16])


# ----------------------------------------------------------------------------- momentum / update
def test_momentum_hand_case_and_limits():
    G = np.array([[1.0, -2.0], [0.5, 4.0]])
    M = np.array([[2.0, 2.0], [-1.0, 0.0]])
    M1, u = orc.momentum_nesterov(G, M, 0.5, True)
    assert np.array_equal(M1, np.array([[2.0, -1.0], [0.0, 4.0]]))
    assert np.array_equal(u, np.array([[2.0, -2.5], [0.5, 6.0]]))
    M1, u = orc.momentum_nesterov(G, M, 0.5, False)
    assert np.array_equal(u, M1)
    M1, u = orc.momentum_nesterov(G, M, 0.0, True)
    assert np.array_equal(u, G) and np.array_equal(M1, G)


def test_momentum_geometric_series():
    rng = np.random.default_rng(3)
    Gs = [rng.standard_normal((3, 4)) for _ in range(6)]
    mu = 0.95
    M = np.zeros((3, 4))
    for G in Gs:
        M, u = orc.momentum_nesterov(G, M, mu, True)
    closed = sum(mu ** (len(Gs) - 1 - i) * Gs[i] for i in range(len(Gs)))
    assert rel(M, closed) < 1e-14
    assert rel(u, Gs[-1] + mu * closed) < 1e-14


def test_update_hand_case_and_identities():
    W = np.array([[1.0, -1.0, 2.0], [0.0, 3.0, 0.5]])
    O = np.array([[1.0, 0.0, -1.0], [0.5, 0.5, 0.0]])
    out = orc.apply_update(W, O, lr=0.1, wd=0.5)
    sc = 0.2 * np.sqrt(3.0)
    hand = np.array([[0.95 - 0.1 * sc, -0.95, 1.9 + 0.1 * sc], [-0.05 * sc, 2.85 - 0.05 * sc, 0.475]])
    assert rel(out, hand) < 1e-15
    assert np.array_equal(orc.apply_update(W, O, lr=0.0, wd=0.3), W)
    # decay acts on the OLD weights, not on the already-updated ones
    assert abs(orc.apply_update(W, O, 0.1, 0.5)[0, 0] - (W[0, 0] - 0.1 * sc * O[0, 0]) * (1 - 0.05)) > 1e-4
    assert orc.update_scale(7, 100) == pytest.approx(2.0)
    assert orc.update_scale(100, 7) == pytest.approx(2.0)


# ----------------------------------------------------------------------------- Newton-Schulz, fp64
@pytest.mark.parametrize("shape", [(48, 80), (80, 48), (33, 33), (1, 9), (9, 1), (64, 64)])
def test_ns_matches_svd_closed_form(shape):
    rng = np.random.default_rng(shape[0] * 1000 + shape[1])
    G = rng.standard_normal(shape)
    got = orc.newton_schulz(G, 5, QUINTIC, 1e-7, "fp64")
    assert got.shape == shape
    assert rel(got, svd_closed_form(G, 5, QUINTIC, 1e-7)) < 1e-12


def test_ns_per_step_coefficients_closed_form():
    rng = np.random.default_rng(11)
    G = rng.standard_normal((12, 20))
    co = [3.0, -3.2, 1.2, 3.4445, -4.7750, 2.0315, 2.0, -1.5, 0.5]
    U, s, Vt = np.linalg.svd(G, full_matrices=False)
    x = s / (np.linalg.norm(G) + 1e-7)
    for k in range(3):
        x = p_scalar(x, co[3 * k:3 * k + 3])
    assert rel(orc.newton_schulz(G, 3, co, 1e-7), (U * x) @ Vt) < 1e-12


def test_ns_rank_one_scalar_recurrence():
    rng = np.random.default_rng(5)
    x = rng.standard_normal(7)
    y = rng.standard_normal(19)
    G = np.outer(x, y)
    t = 1.0
    seq = [t]
    for _ in range(5):
        t = p_scalar(t)
        seq.append(t)
    assert seq[1] == pytest.approx(0.7010, abs=1e-12)
    O = orc.newton_schulz(G, 5, QUINTIC, 0.0)
    assert rel(O, seq[5] * np.outer(x / np.linalg.norm(x), y / np.linalg.norm(y))) < 1e-12


def test_ns_orthonormal_rows_scalar_recurrence():
    rng = np.random.default_rng(6)
    Q, _ = np.linalg.qr(rng.standard_normal((24, 4)))
    Q = Q.T                       # 4 orthonormal rows, so X0 = Q / 2
    t = 0.5
    for _ in range(5):
        t = p_scalar(t)
    O = orc.newton_schulz(3.7 * Q, 5, QUINTIC, 0.0)
    assert rel(O, t * Q) < 1e-12


def test_ns_rectangular_diagonal():
    d = np.array([3.0, 1.0, 0.25, 0.05])
    G = np.zeros((4, 9))
    G[np.arange(4), np.arange(4)] = d
    x = d / np.linalg.norm(d)
    for _ in range(5):
        x = p_scalar(x)
    O = orc.newton_schulz(G, 5, QUINTIC, 0.0)
    expect = np.zeros((4, 9))
    expect[np.arange(4), np.arange(4)] = x
    assert rel(O, expect) < 1e-13
    assert np.count_nonzero(O) == 4


def test_ns_singular_value_band():
    rng = np.random.default_rng(7)
    G = rng.standard_normal((40, 160)) * np.exp(rng.uniform(np.log(1e-4), np.log(1e-2), size=(40, 1)))
    s0 = np.linalg.svd(G, compute_uv=False) / np.linalg.norm(G)
    assert s0.min() >= 0.003
    s5 = np.linalg.svd(orc.newton_schulz(G, 5, QUINTIC, 1e-7), compute_uv=False)
    assert s5.min() >= 0.6818 - 1e-4 and s5.max() <= 1.2024 + 1e-4


def test_ns_band_constants_of_the_quintic():
    x = np.linspace(0.0, 1.3, 1300001)
    y = p_scalar(x)
    dy = np.diff(y)
    imax = np.where((dy[:-1] > 0) & (dy[1:] <= 0))[0][0] + 1
    imin = np.where((dy[:-1] < 0) & (dy[1:] >= 0))[0][0] + 1
    assert x[imax] == pytest.approx(0.5545, abs=2e-4) and y[imax] == pytest.approx(1.2024, abs=1e-4)
    assert x[imin] == pytest.approx(1.0501, abs=2e-4) and y[imin] == pytest.approx(0.6818, abs=1e-4)


@pytest.mark.parametrize("shape", [(8, 8), (16, 48), (64, 24), (64, 64)])
def test_cubic_iteration_converges_to_polar_factor(shape):
    rng = np.random.default_rng(shape[0] + 7 * shape[1])
    k = min(shape)
    U, _ = np.linalg.qr(rng.standard_normal((shape[0], k)))
    V, _ = np.linalg.qr(rng.standard_normal((shape[1], k)))
    s = np.linspace(1.0, 3.0, k)                    # condition number 3
    G = (U * s) @ V.T
    # the iteration needs sigma(X0) < sqrt(3); Frobenius normalisation guarantees <= 1
    O = orc.newton_schulz(G, 40, CUBIC, 0.0)
    assert rel(O, U @ V.T) < 1e-13


def test_ns_invariants():
    rng = np.random.default_rng(9)
    G = rng.standard_normal((10, 17))
    O = orc.newton_schulz(G, 5, QUINTIC, 1e-7)
    assert rel(orc.newton_schulz(G.T, 5, QUINTIC, 1e-7), O.T) < 1e-13
    assert rel(orc.newton_schulz(1234.5 * G, 5, QUINTIC, 0.0), orc.newton_schulz(G, 5, QUINTIC, 0.0)) < 1e-12
    d1 = np.where(rng.random(10) < 0.5, -1.0, 1.0)
    d2 = np.where(rng.random(17) < 0.5, -1.0, 1.0)
    flipped = orc.newton_schulz(d1[:, None] * G * d2[None, :], 5, QUINTIC, 1e-7)
    assert rel(flipped, d1[:, None] * O * d2[None, :]) < 1e-13
    perm = rng.permutation(10)
    assert rel(orc.newton_schulz(G[perm], 5, QUINTIC, 1e-7), O[perm]) < 1e-12
    trace = []
    orc.newton_schulz(G, 2, QUINTIC, 1e-7, trace=trace)
    for (A, B, _) in trace:
        assert rel(A, A.T) < 1e-15 and rel(B, B.T) < 1e-15


def test_ns_zero_gradient_gives_zero_without_nan():
    O = orc.newton_schulz(np.zeros((4, 6)), 5, QUINTIC, 1e-7)
    assert np.array_equal(O, np.zeros((4, 6)))
    O = orc.newton_schulz(np.zeros((6, 4)), 5, QUINTIC, 1e-7, "bf16")
    assert np.array_equal(O, np.zeros((6, 4)))


def test_ns_dynamic_range_of_the_folded_schedule():
    rng = np.random.default_rng(10)
    G = rng.standard_normal((6, 11))
    base = orc.newton_schulz(G, 5, QUINTIC, 0.0)
    for sc in (2.0 ** 40, 2.0 ** -40):
        assert rel(orc.newton_schulz(G * sc, 5, QUINTIC, 0.0), base) < 1e-12


# ----------------------------------------------------------------------------- worked example (fixture + closed form)
def _read_golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "worked_example.txt")
    out = {}
    with open(path) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, r, c, *vals = line.split()
            out[name] = np.array([float(v) for v in vals]).reshape(int(r), int(c))
    return out


def test_worked_example_fixture():
    gold = _read_golden()
    G = g_formula(3, 5, 0)
    assert np.linalg.norm(G) == pytest.approx(8.31038506929733, rel=1e-14)
    assert rel(orc.newton_schulz(G, 5, QUINTIC, 1e-7), gold["NS5_g350"]) < 1e-14
    assert rel(gold["NS5_g350"], svd_closed_form(G, 5, QUINTIC, 1e-7)) < 1e-13
    assert rel(gold["NS5_g530"], svd_closed_form(g_formula(5, 3, 0), 5, QUINTIC, 1e-7)) < 1e-13
    sv = np.linalg.svd(gold["NS5_g350"], compute_uv=False)
    assert sv == pytest.approx([1.052390727889, 1.048037664965, 0.682175837565], abs=1e-11)
    # two full optimizer steps, re-derived with the closed form for the NS part
    lr, mu, wd = 0.02, 0.95, 0.01
    W = 0.01 * g_formula(3, 5, 2)
    M = np.zeros((3, 5))
    Wo, Mo = W.copy(), M.copy()
    for t in (1, 2):
        Gt = 1e-3 * g_formula(3, 5, 3 + t)
        M = mu * M + Gt
        O = svd_closed_form(Gt + mu * M, 5, QUINTIC, 1e-7)
        W = W * (1 - lr * wd) - lr * 0.2 * np.sqrt(5.0) * O
        Wo, Mo, _ = orc.muon_step(Wo, Gt, Mo, lr, mu, wd, 5, QUINTIC, 1e-7, True, "fp64")
        assert rel(Wo, gold[f"W_after_step{t}"]) < 1e-14
        assert rel(Mo, gold[f"M_after_step{t}"]) < 1e-14
        assert rel(gold[f"W_after_step{t}"], W) < 1e-6      # fp32 storage of the state
        assert rel(gold[f"M_after_step{t}"], M) < 1e-6


# ----------------------------------------------------------------------------- bf16 mode
def _bf(x):
    """Independent bf16 rounding of a python float through torch (float32 first, like the hardware cast)."""
    return float(torch.tensor(x, dtype=torch.float64).to(torch.bfloat16).to(torch.float64))


def test_bf16_mode_rounding_points_on_scalars():
    # 1x1 matrix: every rounding point of the schedule can be followed by hand.
    u = 0.3203125                       # exactly representable in bf16
    eps = 1e-7
    r = 1.0 / (abs(u) + eps)
    x = u
    a, b, c = QUINTIC
    A = _bf(r * r * u * u)
    P = _bf(a + b * A + c * A * A)      # the polynomial a I + b A + c A^2 is one produced matrix, rounded once
    x = _bf(r * (P * u))
    for _ in range(4):
        A = _bf(x * x)
        P = _bf(a + b * A + c * A * A)
        x = _bf(P * x)
    got = orc.newton_schulz(np.array([[u]]), 5, QUINTIC, eps, "bf16")
    assert got[0, 0] == x
    # and it is NOT what un-rounded arithmetic gives (the roundings are really applied)
    assert orc.newton_schulz(np.array([[u]]), 5, QUINTIC, eps, "fp64")[0, 0] != x


def test_bf16_mode_diagonal_matrix_follows_scalar_schedule():
    d = np.array([0.75, 0.5, 0.125])
    eps = 1e-7
    r = 1.0 / (np.sqrt((d * d).sum()) + eps)
    a, b, c = QUINTIC
    xs = []
    for u in d:
        A = _bf(r * r * u * u)
        P = _bf(a + b * A + c * A * A)
        x = _bf(r * (P * u))
        for _ in range(4):
            A = _bf(x * x)
            P = _bf(a + b * A + c * A * A)
            x = _bf(P * x)
        xs.append(x)
    got = orc.newton_schulz(np.diag(d), 5, QUINTIC, eps, "bf16")
    assert np.array_equal(got, np.diag(xs))


@pytest.mark.parametrize("shape", [(64, 64), (32, 96), (96, 32), (128, 256)])
def test_bf16_mode_within_noise_floor_of_fp64(shape):
    rng = np.random.default_rng(shape[0] * 3 + shape[1])
    G = orc.bf16_rne(rng.standard_normal(shape) * 1e-3)
    lo = orc.newton_schulz(G, 5, QUINTIC, 1e-7, "bf16")
    hi = orc.newton_schulz(G, 5, QUINTIC, 1e-7, "fp64")
    assert np.array_equal(lo, orc.bf16_rne(lo))          # output is bf16-valued
    assert rel(lo, hi) < 3e-2
    assert rel(lo, hi) > 1e-4                            # and genuinely rounded
    trace = []
    orc.newton_schulz(G, 2, QUINTIC, 1e-7, "bf16", trace=trace)
    for (A, B, X) in trace:
        for Z in (A, B, X):
            assert np.array_equal(Z, orc.bf16_rne(Z))


def test_single_step_equals_one_iteration():
    rng = np.random.default_rng(21)
    G = rng.standard_normal((5, 8))
    X0 = G / np.linalg.norm(G)
    one = orc.ns_single_step(X0, *QUINTIC)
    assert rel(one, orc.newton_schulz(G, 1, QUINTIC, 0.0)) < 1e-14
    U, s, Vt = np.linalg.svd(X0, full_matrices=False)
    assert rel(one, (U * p_scalar(s)) @ Vt) < 1e-13


def test_muon_step_bf16_stages_u_as_bf16():
    rng = np.random.default_rng(22)
    W = rng.standard_normal((6, 4)) * 0.02
    G = rng.standard_normal((6, 4)) * 1e-3
    M = rng.standard_normal((6, 4)) * 1e-3
    W1, M1, O = orc.muon_step(W, G, M, 0.02, 0.95, 0.01, 5, QUINTIC, 1e-7, True, "bf16")
    Mn = 0.95 * M + G
    U = torch.from_numpy((G + 0.95 * Mn).astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O, orc.newton_schulz(U, 5, QUINTIC, 1e-7, "bf16"))
    assert np.array_equal(M1, Mn.astype(np.float32).astype(np.float64))
    expect = W * (1 - 0.02 * 0.01) - 0.02 * 0.2 * np.sqrt(6.0) * O
    assert rel(W1, expect) < 1e-7
