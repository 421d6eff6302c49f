"""Pins for the CPU oracle: each test checks the oracle against something other than itself
(hand-worked fixtures, brute force over the six 2:4 patterns, closed-form byte counts, the
paper's printed compression ratios, numpy's matmul, round trips and invariants)."""
import itertools
import os

import numpy as np
import pytest

from paper_2509_23410_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf(x):
    return inputs.f32_to_bf16_bits(np.asarray(x, np.float32))


def f32(b):
    return inputs.bf16_bits_to_f32(b)


# ---------------------------------------------------------------------------------------------
# hand-worked fixture


def _read_hand():
    rows = {"W": [], "M": [], "NIB": [], "V": [], "Y": [], "Y16": []}
    with open(os.path.join(GOLDEN, "hand_worked_4x8.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            tag, *vals = line.split()
            rows[tag].append([float(v) for v in vals])
    return {k: np.array(v) for k, v in rows.items()}


def test_hand_worked_example(oracle):
    h = _read_hand()
    W = bf(h["W"])
    flags = np.array([[1, 0]], np.uint8)
    m = oracle.mask(W, flags, 4, 4)
    assert (m == h["M"].astype(np.uint8)).all()
    What = oracle.prune(W, flags, 4, 4)
    assert (f32(What) == (h["W"] * h["M"]).astype(np.float32)).all()
    blob, L = oracle.pack(W, flags, 4, 4)
    assert (L.n_dense, L.n_sparse) == (1, 1)
    table = blob[L.table_off:L.table_off + 32].view(np.uint32).reshape(2, 4)
    assert table[0, 0] == 1 and table[1, 0] == 0 and table[1, 2] == 0xFFFFFFFF
    vals = blob[table[0, 1] * 16:][:16].view(np.uint16).reshape(4, 2)
    assert (f32(vals) == h["V"].astype(np.float32)).all()
    meta = blob[table[0, 2] * 16:][:16].view(np.uint32)
    assert (meta == h["NIB"][0].astype(np.uint32)).all()
    dense = blob[table[1, 1] * 16:][:32].view(np.uint16).reshape(4, 4)
    assert (dense == W[:, 4:]).all()
    X = bf(np.array([[1] * 8, list(range(1, 9))], np.float32))
    Y32, Y16 = oracle.gemm_f64(X, What)
    assert (Y32 == h["Y"].astype(np.float32)).all()
    assert (f32(Y16) == h["Y16"].astype(np.float32)).all()
    assert (oracle.gemm_f32(X, What) == h["Y"].astype(np.float32)).all()
    assert (oracle.unpack(blob) == What).all()


# ---------------------------------------------------------------------------------------------
# P1: all tiles dense -> plain GEMM


def test_all_dense_is_plain_gemm(oracle):
    W = inputs.weight(256, 384, 1, "p1")
    X = inputs.activation(9, 384, 1, "p1")
    flags = np.zeros((2, 3), np.uint8)
    What = oracle.prune(W, flags)
    assert (What == W).all()
    assert oracle.mask(W, flags).all()
    Y32, Y16 = oracle.gemm_f64(X, What)
    ref = f32(X).astype(np.float64) @ f32(W).astype(np.float64).T
    assert np.allclose(Y32, ref, rtol=1e-6, atol=1e-9)
    assert (Y32 == ref.astype(np.float32)).mean() > 0.99  # same value up to double summation order
    # a transposed operand or swapped index would fail this asymmetric case
    assert Y32.shape == (9, 256)


# ---------------------------------------------------------------------------------------------
# P2 / P7: at most two non-zeros per group in 2:4 tiles, dense tiles untouched, s = f/2


def test_two_of_four_and_sparsity(oracle):
    N, K = 512, 640
    W = inputs.weight(N, K, 2, "p2")
    W[W == 0] = bf(0.02)  # no exact zeros, so zeros counted below are the ones pruning introduced
    W[(W & 0x7FFF) == 0] = bf(0.02)
    flags = inputs.tile_flags(N, K, 0.5, 2, "p2")
    assert 0 < flags.sum() < flags.size
    What = oracle.prune(W, flags)
    m = oracle.mask(W, flags)
    g = m.reshape(N, K // 4, 4).sum(-1)
    tile_of_group = np.repeat(np.repeat(flags, 128, 0), 32, 1)
    assert (g[tile_of_group == 1] == 2).all()
    assert (g[tile_of_group == 0] == 4).all()
    nz = ((What & 0x7FFF) != 0).reshape(N, K // 4, 4).sum(-1)
    assert (nz[tile_of_group == 1] <= 2).all()
    dense_elems = np.repeat(np.repeat(flags, 128, 0), 128, 1) == 0
    assert (What[dense_elems] == W[dense_elems]).all()
    f = flags.mean()
    assert ((What & 0x7FFF) == 0).sum() == int(N * K * f / 2)


# ---------------------------------------------------------------------------------------------
# P3: brute force over the six candidate patterns on tiny matrices

PATTERNS = list(itertools.combinations(range(4), 2))  # lexicographic: (0,1),(0,2),...,(2,3)


def brute_force_mask(Wf, flags, tn, tk):
    N, K = Wf.shape
    m = np.ones((N, K), np.uint8)
    for n in range(N):
        for g in range(K // 4):
            if flags[n // tn, (4 * g) // tk] == 0:
                continue
            grp = np.abs(Wf[n, 4 * g:4 * g + 4].astype(np.float64))
            best, best_sum = None, -1.0
            for pat in PATTERNS:  # strict > keeps the lexicographically smallest among ties
                s = grp[pat[0]] + grp[pat[1]]
                if s > best_sum:
                    best, best_sum = pat, s
            m[n, 4 * g:4 * g + 4] = 0
            m[n, 4 * g + best[0]] = m[n, 4 * g + best[1]] = 1
    return m


@pytest.mark.parametrize("tile", [(4, 4), (8, 8), (2, 4), (8, 4)])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_brute_force_8x8(oracle, tile, seed):
    tn, tk = tile
    rng = np.random.default_rng(seed)
    # few distinct magnitudes -> many ties, zeros and +-0 included
    vals = np.array([0.0, -0.0, 0.5, -0.5, 1.0, -1.0, 2.0, 3.0], np.float32)
    Wf = vals[rng.integers(0, len(vals), (8, 8))]
    W = bf(Wf)
    flags = rng.integers(0, 2, (8 // tn, 8 // tk)).astype(np.uint8)
    flags.flat[0] = 1
    m = oracle.mask(W, flags, tn, tk)
    assert (m == brute_force_mask(Wf, flags, tn, tk)).all()
    What = oracle.prune(W, flags, tn, tk)
    X = bf(rng.integers(-3, 4, (5, 8)).astype(np.float32))
    Y32, _ = oracle.gemm_f64(X, What)
    Xf, Whf = f32(X), Wf * m
    for mm in range(5):
        for n in range(8):
            assert Y32[mm, n] == sum(float(Xf[mm, k]) * float(Whf[n, k]) for k in range(8))
    blob, _ = oracle.pack(W, flags, tn, tk)
    assert (oracle.unpack(blob) == What).all()


# ---------------------------------------------------------------------------------------------
# P4: round trip and idempotence; P5: six nibbles; P6: byte counts; P11: locality of a flag flip


def _tiles(blob, L):
    T = (L.N // L.tile_n) * (L.K // L.tile_k)
    return blob[L.table_off:L.table_off + 16 * T].view(np.uint32).reshape(T, 4)


def test_round_trip_and_idempotence(oracle):
    N, K = 384, 512
    W = inputs.weight(N, K, 3, "p4")
    flags = inputs.tile_flags(N, K, 0.6, 3, "p4")
    blob, L = oracle.pack(W, flags)
    What = oracle.prune(W, flags)
    assert (oracle.unpack(blob) == What).all()
    blob2, _ = oracle.pack(What, flags)  # packing an already pruned matrix is lossless
    assert (blob2 == blob).all()


def test_six_nibbles_and_byte_count(oracle):
    N, K = 512, 512
    W = inputs.weight(N, K, 4, "p5")
    flags = inputs.tile_flags(N, K, 0.5, 4, "p5")
    blob, L = oracle.pack(W, flags)
    nd, ns = int((flags == 0).sum()), int((flags == 1).sum())
    assert (L.n_dense, L.n_sparse) == (nd, ns)
    assert L.payload_bytes == 32768 * nd + 18432 * ns
    assert L.payload_off % 1024 == 0 and L.total_bytes == L.payload_off + L.payload_bytes
    assert L.total_bytes == blob.nbytes
    f = ns / (nd + ns)
    assert L.payload_bytes / (N * K * 2) == pytest.approx(1 - 0.4375 * f, abs=1e-12)
    hist = np.zeros(16, np.int64)
    for kind, poff, moff, _ in _tiles(blob, L):
        assert poff * 16 % 1024 == 0
        if kind == 1:
            assert moff == poff + 16384 // 16
            meta = blob[moff * 16:moff * 16 + 2048].view(np.uint32)
            for s in range(0, 32, 4):
                hist += np.bincount((meta >> s) & 0xF, minlength=16)
        else:
            assert moff == 0xFFFFFFFF
    legal = [0x4, 0x8, 0xC, 0x9, 0xD, 0xE]  # (0,1) (0,2) (0,3) (1,2) (1,3) (2,3)
    assert hist.sum() == ns * 128 * 32
    assert hist[[i for i in range(16) if i not in legal]].sum() == 0
    assert (hist[legal] > 0.14 * hist.sum()).all() and (hist[legal] < 0.19 * hist.sum()).all()


def test_table4_compression_ratio(oracle):
    """Two metadata bits per kept value reproduce the paper's printed compression ratios."""
    W = inputs.weight(128, 128, 5, "p6")
    _, Ls = oracle.pack(W, np.ones((1, 1), np.uint8))
    _, Ld = oracle.pack(W, np.zeros((1, 1), np.uint8))
    elems = 128 * 128
    kept_frac = (16384 / 2) / elems                       # kept values per element in a 2:4 tile
    meta_bits = (Ls.payload_bytes - 16384) * 8 / elems    # metadata bits per element
    assert kept_frac == 0.5 and meta_bits == 1.0 and Ld.payload_bytes == elems * 2
    with open(os.path.join(GOLDEN, "table4_compression_ratio.txt")) as fh:
        rows = [l.split() for l in fh if not l.startswith("#") and l.strip()]
    for s, printed in rows:
        f = 2 * float(s)   # global sparsity s = f / 2
        bits_per_elem = 4 * (1 - f) + f * (4 * kept_frac + meta_bits)
        assert round(16 / bits_per_elem, 2) == float(printed)


def test_flag_flip_is_local(oracle):
    N, K = 256, 384
    W = inputs.weight(N, K, 6, "p11")
    flags = np.zeros((2, 3), np.uint8)
    blob0, L0 = oracle.pack(W, flags)
    flags2 = flags.copy()
    flags2[0, 1] = 1
    blob1, L1 = oracle.pack(W, flags2)
    t0, t1 = _tiles(blob0, L0), _tiles(blob1, L1)
    assert (t0[0] == t1[0]).all()
    assert (blob0[t0[0, 1] * 16:][:32768] == blob1[t1[0, 1] * 16:][:32768]).all()
    for t in range(2, 6):  # later tiles: same bytes, shifted down by 32768 - 18432
        assert t0[t, 1] * 16 - t1[t, 1] * 16 == 32768 - 18432
        assert (blob0[t0[t, 1] * 16:][:32768] == blob1[t1[t, 1] * 16:][:32768]).all()
    assert L0.total_bytes - L1.total_bytes == 32768 - 18432


# ---------------------------------------------------------------------------------------------
# P8: with every tile 2:4 the compression does not depend on the tiling


def whole_matrix_2to4(W):
    """2:4 compression of a whole matrix with no notion of tiles (numpy sort based)."""
    N, K = W.shape
    mag = (W & 0x7FFF).astype(np.int32).reshape(N, K // 4, 4)
    order = np.argsort(-mag, axis=-1, kind="stable")      # stable: equal magnitudes by index
    pos = np.sort(order[..., :2], axis=-1)
    vals = np.take_along_axis(W.reshape(N, K // 4, 4), pos, -1)
    nib = pos[..., 0] | (pos[..., 1] << 2)
    return vals.reshape(N, K // 2), nib.astype(np.uint8)


@pytest.mark.parametrize("tile", [(128, 128), (64, 32), (16, 8)])
def test_full_2to4_is_tile_independent(oracle, tile):
    tn, tk = tile
    N, K = 256, 256
    W = inputs.weight(N, K, 7, "p8")
    W[::7, ::5] = 0
    flags = np.ones((N // tn, K // tk), np.uint8)
    blob, L = oracle.pack(W, flags, tn, tk)
    vals_ref, nib_ref = whole_matrix_2to4(W)
    vals = np.zeros_like(vals_ref)
    nib = np.zeros_like(nib_ref)
    words = (tk + 31) // 32
    for t, (kind, poff, moff, _) in enumerate(_tiles(blob, L)):
        r0, c0 = (t // (K // tk)) * tn, (t % (K // tk)) * tk
        v = blob[poff * 16:poff * 16 + tn * tk].view(np.uint16).reshape(tn, tk // 2)
        vals[r0:r0 + tn, c0 // 2:(c0 + tk) // 2] = v
        meta = blob[moff * 16:moff * 16 + tn * words * 4].view(np.uint32).reshape(tn, words)
        for g in range(tk // 4):
            nib[r0:r0 + tn, c0 // 4 + g] = (meta[:, g // 8] >> (4 * (g % 8))) & 0xF
    assert (vals == vals_ref).all() and (nib == nib_ref).all()


# ---------------------------------------------------------------------------------------------
# P10 / P12: GEMM linearity, zero, and fp32-vs-double accumulation


def test_gemm_linearity_zero_and_precision(oracle):
    N, K, M = 256, 1024, 7
    W = inputs.weight(N, K, 8, "p10")
    X = inputs.activation(M, K, 8, "p10")
    flags = inputs.tile_flags(N, K, 0.5, 8, "p10")
    What = oracle.prune(W, flags)
    Y32, Y16 = oracle.gemm_f64(X, What)
    X2 = bf(2.0 * f32(X))
    Y2, _ = oracle.gemm_f64(X2, What)
    assert (Y2 == 2.0 * Y32).all()
    Z, _ = oracle.gemm_f64(np.zeros_like(X), What)
    assert (Z == 0).all()
    Yf = oracle.gemm_f32(X, What)
    relF, maxrel = oracle.parity_metrics(Yf, Y32)
    assert relF < 1e-5 and maxrel < 1e-5
    # against numpy on the pruned weight, built without the oracle's mask: top-2 by sort
    vals, nib = whole_matrix_2to4(W)
    keep = np.zeros((N, K // 4, 4), bool)
    np.put_along_axis(keep, (nib & 3)[..., None].astype(np.int64), True, -1)
    np.put_along_axis(keep, (nib >> 2)[..., None].astype(np.int64), True, -1)
    sparse_elem = np.repeat(np.repeat(flags, 128, 0), 128, 1) == 1
    Wp = np.where(sparse_elem & ~keep.reshape(N, K), 0.0, f32(W)).astype(np.float64)
    ref = f32(X).astype(np.float64) @ Wp.T
    assert np.allclose(Y32, ref, rtol=1e-6, atol=1e-8)
    # bf16 output is the RNE rounding of the fp32 result
    assert (Y16 == bf(Y32)).all()
    # rows entry point agrees with the full one
    rows = np.array([6, 0, 3])
    assert (oracle.gemm_f64_rows(X, rows, What) == Y32[rows]).all()


def test_bf16_rounding_ties_to_even(oracle):
    # 1 + 2^-8 is exactly half way between bf16(1.0) and the next bf16: ties go to even mantissa
    X = bf(np.array([[1.0]], np.float32))
    for w, expect in [(1.0 + 2.0 ** -8, 0x3F80), (1.0 + 3 * 2.0 ** -8, 0x3F82)]:
        # build the fp32 value as a sum of two exactly representable bf16 products
        a, b = bf(np.array([[1.0, w - 1.0]], np.float32)), bf(np.array([[1.0, 1.0]], np.float32))
        _, Y16 = oracle.gemm_f64(b, a)
        assert Y16[0, 0] == expect


# ---------------------------------------------------------------------------------------------
# device image: a per-tile byte permutation with the documented structure


def test_device_image_structure(oracle):
    N, K = 256, 256
    # element value encodes (row, col) inside the tile so positions can be read back
    r, c = np.meshgrid(np.arange(N), np.arange(K), indexing="ij")
    W = ((r % 128) * 128 + (c % 128)).astype(np.uint16)   # raw bit patterns, all distinct per tile
    flags = np.array([[0, 1], [1, 0]], np.uint8)
    canon, L = oracle.pack(W, flags)
    img = oracle.device_image(canon)
    assert (img[:L.payload_off] == canon[:L.payload_off]).all()
    for kind, poff, moff, _ in _tiles(canon, L):
        nbytes = 32768 if kind == 0 else 18432
        a, b = canon[poff * 16:poff * 16 + nbytes], img[poff * 16:poff * 16 + nbytes]
        if kind == 0:
            assert (np.sort(a.view(np.uint16)) == np.sort(b.view(np.uint16))).all()
            atoms = b.view(np.uint16).reshape(2, 16, 8, 8, 8)   # half, row group, row, chunk, elem
            for half in range(2):
                for rr in (0, 1, 7, 8, 77, 127):
                    row = atoms[half, rr // 8, rr % 8]
                    for chunk in range(8):
                        first = int(row[chunk, 0])
                        assert first // 128 == rr                 # same tile row
                        col = first % 128
                        assert col % 8 == 0 and (row[chunk] == first + np.arange(8)).all()
                        assert (col - 64 * half) // 8 == chunk ^ (rr % 8)   # 16-B chunk XOR row
        else:
            va, vb = a[:16384].view(np.uint16), b[:16384].view(np.uint16)
            assert (np.sort(va) == np.sort(vb)).all()
            cm = a[16384:].view(np.uint32).reshape(128, 4)
            dm = b[16384:].view(np.uint32).reshape(128, 4)
            # every 16-bit half-word of the canonical metadata appears exactly once, at the
            # documented place: row L = 16q + 8h + i holds rows 16q+i (low) and 16q+8+i (high)
            for Lr in (0, 5, 8, 13, 16, 127):
                q, h, i = Lr // 16, (Lr // 8) % 2, Lr % 8
                for j in range(4):
                    lo = (int(cm[16 * q + i, j]) >> (16 * h)) & 0xFFFF
                    hi = (int(cm[16 * q + 8 + i, j]) >> (16 * h)) & 0xFFFF
                    assert int(dm[Lr, j]) == lo | (hi << 16)
            assert sorted(cm.view(np.uint16).tolist()) == sorted(dm.view(np.uint16).tolist())


# ---------------------------------------------------------------------------------------------
# validation


def test_rejects_bad_arguments(oracle):
    W = inputs.weight(128, 128, 9, "bad")
    with pytest.raises(ValueError):
        oracle.pack(W, np.array([[4]], np.uint8))
    with pytest.raises(ValueError):
        oracle.packed_size(100, 128, np.zeros(1, np.uint8))
    with pytest.raises(ValueError):
        oracle.packed_size(128, 128, np.zeros(1, np.uint8), 128, 6)


def test_swiglu_against_library_sigmoid_and_closed_forms(oracle):
    """silu(x) u with x sigmoid(x) from scipy (a different evaluation), the odd-part identity
    silu(x) - silu(-x) = x, a value with a closed form, and the gate/up pairing of the interleaved layout."""
    from scipy.special import expit
    rng = np.random.default_rng(7)
    M, blocks, b = 5, 3, 128
    Y = (rng.standard_normal((M, 2 * b * blocks)) * 4).astype(np.float32)
    Y[0, 0], Y[0, b] = np.float32(np.log(3.0)), np.float32(2.0)       # silu(ln 3) = 0.75 ln 3
    Y[1, 1], Y[1, b + 1] = np.float32(0.0), np.float32(123.0)          # silu(0) = 0
    Y[2, 2], Y[2, b + 2] = np.float32(-200.0), np.float32(1.0)         # exp overflows: the limit is -0
    out = oracle.swiglu(Y)
    assert out.shape == (M, b * blocks) and out.dtype == np.float32
    y = Y.astype(np.float64).reshape(M, blocks, 2, b)
    ref = (y[:, :, 0] * expit(y[:, :, 0]) * y[:, :, 1]).reshape(M, b * blocks)
    assert np.allclose(out, ref, rtol=1e-6, atol=1e-30)
    assert abs(out[0, 0] - 0.75 * np.log(3.0) * 2.0) < 1e-6
    assert out[1, 1] == 0.0 and out[2, 2] == 0.0
    # pairing: column block j of the output takes gate block 2j and up block 2j + 1, element by element
    G = np.zeros((1, 2 * b * blocks), np.float32)
    for j in range(blocks):
        G[0, 2 * b * j:2 * b * j + b] = 50.0                            # silu(50) = 50 to fp32 precision
        G[0, 2 * b * j + b:2 * b * (j + 1)] = np.arange(b) + 1000.0 * j
    got = oracle.swiglu(G)
    want = np.concatenate([50.0 * (np.arange(b) + 1000.0 * j) for j in range(blocks)])
    assert np.allclose(got[0], want, rtol=1e-6)
    # odd part of silu is x / 2 + x / 2: silu(x) - silu(-x) = x
    x = np.linspace(-30, 30, 2 * b).astype(np.float32)
    one = np.ones_like(x)
    pos = oracle.swiglu(np.stack([x[:b], one[:b], x[b:], one[b:]]).reshape(1, -1))
    neg = oracle.swiglu(np.stack([-x[:b], one[:b], -x[b:], one[b:]]).reshape(1, -1))
    assert np.allclose(pos - neg, x.reshape(1, -1), atol=1e-5)
