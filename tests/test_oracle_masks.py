"""Pins for the mask-learning part of the CPU oracle (soft masks of Eq. 1-4, the regularisers of
Eq. 5, the hard masks of Algorithm 1 and packing with a given 2:4 mask).  Every expected value
comes from somewhere other than the function under test: a hand-worked fixture, closed forms,
scipy's softmax / numpy's argmax, distribution facts about Gumbel noise, and limits that tie the
soft masks to the hard ones."""
import itertools
import math
import os

import numpy as np
import pytest
from scipy.special import expit, softmax

from paper_2509_23410_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

# the six candidates, typed by hand: kept positions in lexicographic order
KEPT = [(0, 1), (0, 2), (0, 3), (1, 2), (1, 3), (2, 3)]
S = np.zeros((6, 4))
for _c, (_a, _b) in enumerate(KEPT):
    S[_c, _a] = S[_c, _b] = 1.0


def bf(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, np.float32))


def f32(b):
    return inputs.bf16_bits_to_f32(b)


def _read(name):
    rows = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            tag, *vals = line.split()
            rows.setdefault(tag, []).append(vals)
    return rows


# ---------------------------------------------------------------------------------------------
# hard masks


def test_hand_worked_hard_mask(oracle):
    h = _read("hard_mask_2x8.txt")
    PT = np.array(h["PT"], np.float32).reshape(1, 2)
    P6 = np.array(h["P6"], np.float32)
    W = bf(np.array(h["W"], np.float32))
    flags, patterns = oracle.hard_mask(PT, P6, 2, 8, 2, 4)
    assert flags.tolist() == [1, 0]
    assert patterns.tolist() == [int(v) for v in h["C"][0]]
    m = oracle.mask_patterns(2, 8, flags, patterns, 2, 4)
    assert (m == np.array(h["M"], np.uint8)).all()
    blob, L = oracle.pack_patterns(W, flags, patterns, 2, 4)
    assert (L.n_dense, L.n_sparse) == (1, 1)
    table = blob[L.table_off:L.table_off + 32].view(np.uint32).reshape(2, 4)
    vals = blob[table[0, 1] * 16:][:8].view(np.uint16).reshape(2, 2)
    assert (f32(vals) == np.array(h["V"], np.float32)).all()
    meta = blob[table[0, 2] * 16:][:8].view(np.uint32)
    assert meta.tolist() == [int(v[0], 16) for v in h["NIB"]]
    assert (f32(oracle.unpack(blob)) == np.array(h["H"], np.float32)).all()


def test_candidates_are_the_six_two_of_four_masks(oracle):
    # one group per candidate; the masks must be the C(4,2) distinct ways of keeping two of four
    flags = np.ones(1, np.uint8)
    m = oracle.mask_patterns(6, 4, flags, np.arange(6, dtype=np.uint8), 6, 4)
    assert (m == S.astype(np.uint8)).all()
    assert sorted(map(tuple, m.tolist())) == sorted(
        tuple(1 if j in c else 0 for j in range(4)) for c in itertools.combinations(range(4), 2))
    with pytest.raises(ValueError):
        oracle.mask_patterns(1, 4, flags, np.array([6], np.uint8), 1, 4)


def test_hard_mask_is_sign_and_argmax(oracle):
    N, K = 256, 384
    PT = inputs.tile_logits(2, 3, 0.5, 5, "hm")
    PT[0, 1] = 0.0          # a zero logit is not "> 0": the tile is 2:4
    P6 = inputs.pattern_logits(N, K, 5, "hm")
    P6[:, 7] = 0.25         # all equal -> first candidate
    P6[[2, 4], 9] = 1.0     # two-way tie between candidates 2 and 4 -> 2
    flags, patterns = oracle.hard_mask(PT, P6, N, K)
    assert (flags.reshape(2, 3) == (PT <= 0)).all() and flags[1] == 1
    assert (patterns == np.argmax(P6, axis=0)).all()      # numpy's argmax also takes the first of equals
    assert patterns[7] == 0 and patterns[9] == 2
    assert set(np.unique(patterns)) == set(range(6))


def _top2_patterns_numpy(W):
    """Candidate index of the magnitude top-2 selection (ties to the lower index), by sorting."""
    N, K = W.shape
    mag = (W & 0x7FFF).astype(np.int64).reshape(N, K // 4, 4)
    order = np.argsort(-mag, axis=2, kind="stable")[:, :, :2]
    a, b = order.min(axis=2), order.max(axis=2)
    lut = {p: c for c, p in enumerate(KEPT)}
    return np.vectorize(lambda x, y: lut[(x, y)])(a, b).astype(np.uint8)


def test_pack_patterns_against_magnitude_pack_and_numpy_mask(oracle):
    N, K = 256, 384
    W = inputs.weight(N, K, 6, "pp")
    flags = inputs.tile_flags(N, K, 0.6, 6, "pp")
    # (a) the magnitude rule expressed as patterns reproduces the magnitude pack byte for byte
    blob_a, _ = oracle.pack_patterns(W, flags, _top2_patterns_numpy(W))
    blob_b, _ = oracle.pack(W, flags)
    assert (blob_a == blob_b).all()
    # (b) arbitrary patterns: unpack(pack) == W (.) M* with M* built here from the hand-typed S
    g = inputs.generator(6, "pp", "patterns")
    patterns = g.integers(0, 6, N * K // 4).astype(np.uint8)
    dense = np.repeat(np.repeat(flags.reshape(2, 3) == 0, 128, 0), 128, 1)
    M = np.where(dense, 1, S[patterns].reshape(N, K).astype(np.uint8))
    assert (oracle.mask_patterns(N, K, flags, patterns) == M).all()
    blob, L = oracle.pack_patterns(W, flags, patterns)
    assert L.payload_bytes == 32768 * L.n_dense + 18432 * L.n_sparse
    assert (oracle.unpack(blob) == np.where(M == 1, W, 0)).all()
    # patterns of groups inside dense tiles are ignored
    p2 = patterns.reshape(N, K // 4).copy()
    p2[np.repeat(np.repeat(flags.reshape(2, 3) == 0, 128, 0), 32, 1)] = 5
    assert (oracle.pack_patterns(W, flags, p2)[0] == blob).all()
    with pytest.raises(ValueError):
        bad = patterns.copy()
        bad[np.flatnonzero(~dense.reshape(N, K // 4, 4)[:, :, 0].reshape(-1))[0]] = 7
        oracle.pack_patterns(W, flags, bad)


# ---------------------------------------------------------------------------------------------
# noise


def test_uniform_and_gumbel_distribution(oracle):
    n = 40000
    u = np.array([oracle.uniform(11, 1, i) for i in range(n)])
    assert u.min() > 0.0 and u.max() < 1.0
    assert (u * 2 ** 23 - 0.5 == np.round(u * 2 ** 23 - 0.5)).all()       # 23-bit cell centres: exact in fp32
    assert abs(u.mean() - 0.5) < 4 * math.sqrt(1 / 12 / n)
    assert abs(u.var() - 1 / 12) < 0.002
    hist = np.histogram(u, bins=16, range=(0, 1))[0]
    assert np.abs(hist - n / 16).max() < 5 * math.sqrt(n / 16)
    # streams, seeds and neighbouring counters are unrelated
    v = np.array([oracle.uniform(11, 0, i) for i in range(n)])
    w = np.array([oracle.uniform(12, 1, i) for i in range(n)])
    for other in (v, w, u[1:]):
        assert abs(np.corrcoef(u[:len(other)], other)[0, 1]) < 0.02
    z = np.array([oracle.gumbel(11, 1, i) for i in range(n)])
    assert np.allclose(z, -np.log(-np.log(u)), rtol=1e-12)
    assert abs(z.mean() - 0.5772156649) < 0.03                            # Euler-Mascheroni
    assert abs(z.var() - math.pi ** 2 / 6) < 0.08


# ---------------------------------------------------------------------------------------------
# soft masks


def test_soft_mask_closed_forms(oracle):
    N, K = 8, 16
    W = bf(np.arange(1, N * K + 1, dtype=np.float32).reshape(N, K) / 64)
    W[0, 0] = 0
    # equal candidate logits, zero tile logit, no noise: GS is uniform, every position is kept by three of
    # the six candidates -> Mt_2:4 = 1/2, Mt_tile = 1/2, Mt = 1/2 + 1/2 * 1/2 = 3/4
    Mt, Wt, sums = oracle.soft_mask(W, np.zeros((2, 2)), np.full((6, N * K // 4), 0.3), 0.7, 9.0,
                                    noise=False, tile_n=4, tile_k=8)
    assert np.allclose(Mt, 0.75, rtol=0, atol=1e-15)
    w = f32(W).astype(np.float64)
    assert np.allclose(sums, [0.75 * N * K, N * K - 1, (0.5625 * w * w).sum(), (w * w).sum()], rtol=1e-13)
    assert (Wt == bf((0.75 * w).astype(np.float32))).all()
    # tile part alone: Mt_tile = 1 / (1 + exp(-kappa p / tau)) -- a two-class softmax against a zero logit
    PT = np.array([[0.4, -0.2], [0.0, 3.0]], np.float32)
    tau, kappa = 0.5, 2.0
    Mt, _, _ = oracle.soft_mask(W, PT, np.full((6, N * K // 4), 0.3), tau, kappa, noise=False, tile_n=4, tile_k=8)
    for (i, j) in itertools.product(range(2), range(2)):
        mt = 1.0 / (1.0 + math.exp(-kappa * float(PT[i, j]) / tau))
        assert np.allclose(Mt[4 * i:4 * i + 4, 8 * j:8 * j + 8], mt + (1 - mt) * 0.5, rtol=1e-14)


def _soft_mask_scipy(oracle, W, PT, P6, tau, kappa, seed, noise, tile_n, tile_k):
    """Eq. 2-4 with scipy's softmax and numpy broadcasting (noise values are inputs)."""
    N, K = W.shape
    G = N * K // 4
    z6 = np.zeros((6, G))
    z2 = np.zeros((PT.size, 2))
    if noise:
        z6 = np.array([[oracle.gumbel(seed, 1, c * G + g) for g in range(G)] for c in range(6)])
        z2 = np.array([[oracle.gumbel(seed, 0, 2 * t + c) for c in range(2)] for t in range(PT.size)])
    gs6 = softmax((kappa * P6.astype(np.float64) + z6) / tau, axis=0)             # [6 x G]
    m24 = (gs6.T @ S).reshape(N, K)
    logits2 = np.stack([kappa * PT.astype(np.float64).reshape(-1), np.zeros(PT.size)], axis=1)
    mt = softmax((logits2 + z2) / tau, axis=1)[:, 0].reshape(PT.shape)
    mt = np.kron(mt, np.ones((tile_n, tile_k)))
    return mt + (1 - mt) * m24, mt, m24


@pytest.mark.parametrize("tau,kappa", [(2.0, 25.0), (0.05, 350.0), (0.6, 100.0)])
@pytest.mark.parametrize("noise", [False, True])
def test_soft_mask_against_scipy(oracle, tau, kappa, noise):
    N, K, tn, tk = 16, 32, 8, 16
    W = inputs.weight(N, K, 7, "sm")
    PT = inputs.tile_logits(N // tn, K // tk, 0.5, 7, "sm") * np.float32(0.01)    # soft values, not saturated
    P6 = inputs.pattern_logits(N, K, 7, "sm")
    Mt, Wt, sums = oracle.soft_mask(W, PT, P6, tau, kappa, seed=99, noise=noise, tile_n=tn, tile_k=tk)
    ref, mt, m24 = _soft_mask_scipy(oracle, W, PT, P6, tau, kappa, 99, noise, tn, tk)
    assert np.allclose(Mt, ref, rtol=1e-12, atol=1e-15)
    w = f32(W).astype(np.float64)
    assert np.allclose(sums, [ref.sum(), (w != 0).sum(), ((ref * w) ** 2).sum(), (w * w).sum()], rtol=1e-12)
    # the masked weight is the product rounded once to bf16 (a rounding-boundary case may differ by one ulp
    # between two double evaluations; none should on these inputs)
    assert (Wt == bf((ref * w).astype(np.float32))).mean() > 0.999
    # invariants of Eq. 2-4: values in [0, 1]; a group's 2:4 part sums to 2; merging never lowers either mask
    assert Mt.min() >= 0 and Mt.max() <= 1 + 4e-16          # up to double rounding of the sums
    gsum = Mt.reshape(N, K // 4, 4).sum(axis=2)
    mt_g = mt.reshape(N, K // 4, 4)[:, :, 0]
    assert np.allclose(gsum, 4 * mt_g + (1 - mt_g) * 2, rtol=1e-12)
    assert (Mt >= m24 - 1e-15).all() and (Mt >= mt - 1e-15).all()


def test_soft_mask_hardens_to_the_hard_mask(oracle):
    # tau -> 0 without noise: GS becomes the one-hot of the largest logit, so Mt -> M* of Algorithm 1
    N, K = 128, 256
    W = inputs.weight(N, K, 8, "lim")
    PT = inputs.tile_logits(1, 2, 0.5, 8, "lim")
    PT[0, 0], PT[0, 1] = 2.5, -2.5
    P6 = inputs.pattern_logits(N, K, 8, "lim", std=1.0)
    gap = np.sort(P6, axis=0)
    keep = (gap[-1] - gap[-2]) > 1e-3            # groups whose best candidate is clearly separated
    Mt, Wt, _ = oracle.soft_mask(W, PT, P6, 1e-5, 1.0, noise=False)
    flags, patterns = oracle.hard_mask(PT, P6, N, K)
    M = oracle.mask_patterns(N, K, flags, patterns)
    sel = np.repeat(keep.reshape(N, K // 4), 4, axis=1)
    assert sel.mean() > 0.99
    assert np.abs(Mt - M)[sel].max() < 1e-12
    # and the masked weight equals the pruned weight there
    blob, _ = oracle.pack_patterns(W, flags, patterns)
    What = oracle.unpack(blob)
    assert ((Wt == What) | ((Wt & 0x7FFF) == 0) & ((What & 0x7FFF) == 0))[sel].all()


def test_gumbel_max_frequencies_follow_softmax_of_scaled_logits(oracle):
    # Many groups share the same six logits.  As tau -> 0 each group picks argmax(kappa p + z), and by the
    # Gumbel-max property candidate c is picked with probability softmax(kappa p)_c: this fails if kappa also
    # scaled the noise, if the noise were not Gumbel, or if groups shared their noise.
    N, K = 64, 2048
    G = N * K // 4
    p = np.array([0.3, -0.2, 0.1, 0.0, 0.45, -0.4], np.float32)
    kappa = 3.0
    P6 = np.repeat(p[:, None], G, axis=1)
    W = bf(np.ones((N, K), np.float32))
    Mt, _, _ = oracle.soft_mask(W, np.full((1, 16), -50.0, np.float32), P6, 1e-4, kappa, seed=5, noise=True,
                                tile_n=64, tile_k=128)
    onehot = np.round(Mt.reshape(G, 4))
    sharp = np.abs(Mt.reshape(G, 4) - onehot).max(axis=1) < 1e-6     # all but the rare near-ties of the top two
    assert sharp.mean() > 0.995 and (onehot[sharp].sum(axis=1) == 2).all()
    lut = {tuple(S[c].tolist()): c for c in range(6)}
    picks = np.array([lut[tuple(r)] for r in onehot[sharp].tolist()])
    freq = np.bincount(picks, minlength=6) / sharp.sum()
    expect = softmax(kappa * p.astype(np.float64))
    assert np.abs(freq - expect).max() < 5 * math.sqrt(0.25 / G) + 0.005
    # the tile noise behaves the same way: P(dense) = sigmoid(kappa p_tile)
    T = 4096
    Mt, _, _ = oracle.soft_mask(bf(np.ones((T, 4), np.float32)), np.full((T, 1), 0.2, np.float32),
                                np.tile(np.array([[50.0], [0], [0], [0], [0], [-50.0]], np.float32), (1, T)),
                                1e-4, kappa, seed=6, noise=True, tile_n=1, tile_k=4)
    dense = (Mt[:, 3] > 0.5)              # position 3 is kept only if the tile went dense (candidate 0 keeps 0, 1)
    assert abs(dense.mean() - expit(kappa * 0.2)) < 5 * math.sqrt(0.25 / T)


def test_regularizers_closed_form(oracle):
    # one matrix: 7 * |75/100 - 0.5| - 10 * 30/60 = 1.75 - 5
    assert oracle.regularizers([[75, 100, 30, 60]], 0.5, 7, 10) == pytest.approx(-3.25, abs=1e-15)
    # sums are pooled over matrices before the quotients (a global, not a per-layer, sparsity target)
    two = [[10, 40, 1, 4], [50, 60, 5, 6]]
    assert oracle.regularizers(two, 0.9, 3, 0.1) == pytest.approx(3 * abs(60 / 100 - 0.9) - 0.1 * 6 / 10, abs=1e-15)
    assert oracle.regularizers(two, 0.9, 3, 0.1) != pytest.approx(
        3 * abs((10 / 40 + 50 / 60) / 2 - 0.9) - 0.1 * (1 / 4 + 5 / 6) / 2)


# ---------------------------------------------------------------------------------------------
# backward


def _objective(oracle, W, PT, P6, tau, kappa, seed, noise, Gw, c1, c2, tn, tk):
    Mt, _, _ = oracle.soft_mask(W, PT, P6, tau, kappa, seed=seed, noise=noise, tile_n=tn, tile_k=tk)
    w = f32(W).astype(np.float64)
    return (Gw.astype(np.float64) * Mt * w).sum() + c1 * Mt.sum() - 0.5 * c2 * ((Mt * w) ** 2).sum()


@pytest.mark.parametrize("noise", [False, True])
def test_backward_against_finite_differences(oracle, noise):
    """The analytic gradient against central differences of the (separately pinned) forward."""
    N, K, tn, tk = 8, 16, 4, 8
    W = inputs.weight(N, K, 9, "bw")
    g = inputs.generator(9, "bw", "gw")
    Gw = g.standard_normal((N, K)).astype(np.float32)
    PT = (g.standard_normal((2, 2)) * 0.05).astype(np.float32)
    P6 = (g.standard_normal((6, N * K // 4)) * 0.05).astype(np.float32)
    tau, kappa, c1, c2 = 0.8, 12.0, 0.3, 40.0
    gt, g6 = oracle.soft_mask_backward(W, PT, P6, tau, kappa, Gw, c1, c2, seed=3, noise=noise, tile_n=tn, tile_k=tk)
    F = lambda pt, p6: _objective(oracle, W, pt, p6, tau, kappa, 3, noise, Gw, c1, c2, tn, tk)
    d = np.float32(2.0 ** -12)
    for (i, j) in [(0, 0), (0, 1), (1, 0), (1, 1)]:
        a, b = PT.copy(), PT.copy()
        a[i, j] += d
        b[i, j] -= d
        fd = (F(a, P6) - F(b, P6)) / (float(a[i, j]) - float(b[i, j]))
        assert fd == pytest.approx(gt[i, j], rel=2e-4, abs=1e-7)
    for (c, grp) in [(0, 0), (5, 0), (2, 7), (3, 13), (1, 31), (4, 18)]:
        a, b = P6.copy(), P6.copy()
        a[c, grp] += d
        b[c, grp] -= d
        fd = (F(PT, a) - F(PT, b)) / (float(a[c, grp]) - float(b[c, grp]))
        assert fd == pytest.approx(g6[c, grp], rel=2e-4, abs=1e-7)
    # a softmax gradient sums to zero over the classes of a group
    assert np.abs(g6.sum(axis=0)).max() < 1e-12 * max(1.0, np.abs(g6).max())


def test_regularizer_coefficients_are_the_derivative_of_the_regularizers(oracle):
    sums = np.array([[60.0, 100, 30, 60], [20.0, 50, 8, 20]])
    rho, l1, l2 = 0.4, 7.0, 10.0
    c1, c2 = oracle.regularizer_coefficients(sums, rho, l1, l2)
    assert c1 == pytest.approx(7.0 / 150) and c2 == pytest.approx(2 * 10.0 / 80)
    # raising one element's Mt by e raises sum Mt by e and sum (Mt W)^2 by 2 e Mt W^2: compare with the regularisers
    e, mt, w = 1e-6, 0.7, 1.3
    s2 = sums.copy()
    s2[0, 0] += e
    s2[0, 2] += 2 * e * mt * w * w
    fd = (oracle.regularizers(s2, rho, l1, l2) - oracle.regularizers(sums, rho, l1, l2)) / e
    assert fd == pytest.approx(c1 - c2 * mt * w * w, rel=1e-5)
    assert oracle.regularizer_coefficients(sums, 0.9, l1, l2)[0] == pytest.approx(-7.0 / 150)   # below the target
