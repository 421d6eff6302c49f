"""Pins of the oracle's 4-bit payload kinds (tile kinds 2 and 3: dense / 2:4 with 4-bit stored values).

The paper fixes one thing about them -- the compression-ratio column of its 4-bit weight-only quantisation table,
16 / (4 - f): four bits per stored value, two metadata bits per kept value -- and no quantiser.  The reading the
oracle takes (symmetric, round to nearest even, one bf16 scale per tile row, s = bf16(max|v| / 7),
q = clamp(rint(v / s), -7, 7), v^ = bf16(q s)) is pinned here by exact rational arithmetic on the bf16 values
(no floating point on the checking side), by a hand-worked group, by its error bound and by round trips."""
from fractions import Fraction

import numpy as np
import pytest

from paper_2509_23410_b200 import inputs

f32 = inputs.bf16_bits_to_f32


def frac(bits: int) -> Fraction:
    """Exact value of a finite bf16 bit pattern."""
    sign = -1 if bits & 0x8000 else 1
    e, m = (bits >> 7) & 0xFF, bits & 0x7F
    if e == 0:
        return sign * Fraction(m, 1 << 7) * Fraction(1, 1 << 126)
    return sign * (1 + Fraction(m, 1 << 7)) * (Fraction(2) ** (e - 127))


def nearest_bf16(x: Fraction) -> int:
    """Bit pattern of the bf16 value nearest to the exact rational x, ties to even (normal range)."""
    if x == 0:
        return 0
    sign, a = (0x8000 if x < 0 else 0), abs(x)
    e = 0
    while a >= 2:
        a /= 2; e += 1
    while a < 1:
        a *= 2; e -= 1
    scaled = a * 128                      # significand in units of 2^-7, in [128, 256)
    lo = int(scaled)                      # floor
    rem = scaled - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    if lo == 256:
        lo, e = 128, e + 1
    return sign | ((e + 127) << 7) | (lo - 128)


def exact_group(bits):
    """Scale, codes and dequantised values of a group from the definition, in exact arithmetic."""
    vals = [frac(int(b)) for b in bits]
    m = max(abs(v) for v in vals)
    s_bits = nearest_bf16(m / 7)
    s = frac(s_bits)
    codes, deq = [], []
    for v in vals:
        if s == 0:
            q = 0
        else:
            r = v / s
            fl = r.numerator // r.denominator             # floor
            rem = r - fl
            q = fl + 1 if (rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1)) else fl
            q = max(-7, min(7, q))
        codes.append(q + 8)
        deq.append(nearest_bf16(q * s))
    return s_bits, np.array(codes, np.uint8), np.array(deq, np.uint16)


def test_hand_worked_group(oracle):
    """max|v| = 1: s = bf16(1/7).  1/7 = 1.001001001..b x 2^-3, eight significant bits 1.0010010 -> 146/1024 = 0.142578125.
    v/s = 7.01, -3.51, 1.75, 5.26, 0.88, -7.01, 0.44, 3.07 -> q = 7, -4, 2, 5, 1, -7, 0, 3.
    q s in units of 1/1024: 1022 (a tie between 1020 and 1024 at bf16 precision: to even = 1024 -> 1.0), -584 (exact),
    292 (exact), 730 (a tie between 728 and 732: 728 -> 0.7109375), 146, -1022 -> -1.0, 0, 438 (exact)."""
    v = inputs.f32_to_bf16_bits(np.array([1.0, -0.5, 0.25, 0.75, 0.125, -1.0, 0.0625, 0.4375], np.float32))
    s, codes, deq = oracle.q4_group(v)
    assert s == 0x3E12 and f32(np.array([s], np.uint16))[0] == 0.142578125
    assert list(codes.astype(int) - 8) == [7, -4, 2, 5, 1, -7, 0, 3]
    assert list(f32(deq)) == [1.0, -0.5703125, 0.28515625, 0.7109375, 0.142578125, -1.0, 0.0, 0.427734375]


def test_quantiser_against_exact_arithmetic(oracle):
    rng = inputs.generator(5, "q4-exact")
    for trial in range(300):
        n = int(rng.integers(1, 130))
        scale = [0.02, 1.0, 37.0, 1e-3][trial % 4]
        v = inputs.f32_to_bf16_bits((rng.standard_normal(n) * scale).astype(np.float32))
        if trial % 7 == 0:                        # many exact ties: values that are half-integer multiples of a power of two
            v = inputs.f32_to_bf16_bits((rng.integers(-15, 16, n) * 0.5).astype(np.float32))
        if trial % 11 == 0:
            v[:] = 0                              # an all-zero group: scale 0, codes 8, values +0
        s, codes, deq = oracle.q4_group(v)
        es, ecodes, edeq = exact_group(v)
        assert s == es
        assert (codes == ecodes).all()
        assert (deq == edeq).all()
        assert codes.min() >= 1 and codes.max() <= 15


def test_quantiser_error_bound_and_extremes(oracle):
    rng = inputs.generator(6, "q4-bound")
    for _ in range(200):
        v = inputs.f32_to_bf16_bits((rng.standard_normal(128) * 0.02).astype(np.float32))
        s_bits, codes, deq = oracle.q4_group(v)
        s = float(f32(np.array([s_bits], np.uint16))[0])
        x, xq = f32(v).astype(np.float64), f32(deq).astype(np.float64)
        # s is max|v| / 7 up to one bf16 rounding (relative 2^-9), so |v / s| <= 7.03 and nothing is clamped by more
        # than 0.03 s; otherwise a value is off by at most half a step plus the bf16 rounding of q s (<= 7 s 2^-9)
        assert np.abs(x - xq).max() <= 0.5 * s + 7 * s * 2.0 ** -9
        i = int(np.abs(x).argmax())
        assert abs(int(codes[i]) - 8) == 7 and np.sign(x[i]) == np.sign(int(codes[i]) - 8)
        assert (np.sign(xq) * np.sign(x) >= 0).all()             # never flips a sign


def test_compression_ratio_column_of_the_4bit_table(oracle):
    """Four bits per stored value and two metadata bits per kept value give the printed column exactly; the scales
    (two bytes per tile row) are this format's own addition, counted separately."""
    golden = [tuple(float(x) for x in line.split()) for line in
              open(inputs.__file__.replace("paper_2509_23410_b200/inputs.py", "tests/golden/table4_compression_ratio.txt"))
              if line.strip() and not line.startswith("#")]
    TN = TK = 10
    for sparsity, printed in golden:
        n_sparse = round(2 * sparsity * TN * TK)
        flags = np.full(TN * TK, 2, np.uint8)
        flags[:n_sparse] = 3
        L = oracle.packed_size(TN * 128, TK * 128, flags)
        assert (L.n_dense_q4, L.n_sparse_q4, L.n_dense, L.n_sparse) == (TN * TK - n_sparse, n_sparse, 0, 0)
        assert L.payload_bytes == 8448 * L.n_dense_q4 + 6400 * L.n_sparse_q4
        without_scales = L.payload_bytes - 256 * TN * TK
        assert round(TN * TK * 128 * 128 * 2 / without_scales, 2) == printed


def test_pack_unpack_round_trip_all_four_kinds(oracle):
    N, K = 384, 512
    W = inputs.weight(N, K, 7, "q4-rt")
    rng = inputs.generator(7, "q4-rt-flags")
    flags = rng.integers(0, 4, (N // 128, K // 128)).astype(np.uint8)
    flags.flat[:4] = [0, 1, 2, 3]
    blob, L = oracle.pack(W, flags)
    What = oracle.unpack(blob)
    assert (What == oracle.prune(W, flags)).all()
    # tiles stored in bf16 are what they were without the new kinds
    plain = oracle.prune(W, flags & 1)
    for tn in range(N // 128):
        for tk in range(K // 128):
            tile = (slice(tn * 128, tn * 128 + 128), slice(tk * 128, tk * 128 + 128))
            if flags[tn, tk] < 2:
                assert (What[tile] == plain[tile]).all()
            else:
                # same zeros as the unquantised kind (the 2:4 choice is made on the unquantised weights) ...
                assert ((f32(plain[tile]) == 0) <= (f32(What[tile]) == 0)).all()
                # ... and every row is that row's stored values through the group quantiser
                for r in (0, 77, 127):
                    row = plain[tile][r]
                    kept = row if flags[tn, tk] == 2 else row[oracle.mask(W, flags & 1)[tile][r] == 1]
                    _, _, deq = oracle.q4_group(kept)
                    got = What[tile][r] if flags[tn, tk] == 2 else What[tile][r][oracle.mask(W, flags & 1)[tile][r] == 1]
                    assert (got == deq).all()
    # 2:4 structure survives quantisation: at most two non-zeros per group of four
    nz = (f32(What).reshape(N, K // 4, 4) != 0).sum(-1).reshape(N, K // 128, 32)
    for tn in range(N // 128):
        for tk in range(K // 128):
            if flags[tn, tk] & 1:
                assert nz[tn * 128:(tn + 1) * 128, tk].max() <= 2


def test_table_entries_and_device_image_of_the_4bit_kinds(oracle):
    N, K = 256, 256
    W = inputs.weight(N, K, 8, "q4-img")
    flags = np.array([[2, 3], [3, 1]], np.uint8)
    blob, L = oracle.pack(W, flags)
    table = blob[L.table_off:L.table_off + 16 * 4].view(np.uint32).reshape(4, 4)
    off = L.payload_off
    for t, kind in enumerate(flags.reshape(-1)):
        assert table[t, 0] == kind and table[t, 1] * 16 == off and off % 256 == 0
        if kind == 2:
            assert table[t, 2] == 0xFFFFFFFF and table[t, 3] * 16 == off + 8192
            off += 8448
        elif kind == 3:
            assert table[t, 2] * 16 == off + 4096 and table[t, 3] * 16 == off + 4096 + 2048
            off += 6400
        else:
            assert table[t, 2] * 16 == off + 16384 and table[t, 3] == 0
            off += 18432
    assert off == L.total_bytes
    image = oracle.device_image(blob)
    # (by hand below: codes 1..8 of one group, canonical bytes 21 43 65 87 -> the word 0x86427531: the odd values
    # 2,4,6,8 in nibbles 4..7 above the even values 1,3,5,7 in nibbles 0..3)
    # scales as they are; the metadata of a 4-bit 2:4 tile in the order of the bf16 2:4 kind; codes: value i of
    # each group of eight in nibble (i % 2) * 4 + i // 2 of the group's 32-bit word, and the 16-byte unit j (four
    # words) of tile row r at byte (128 j + r) * 16
    def image_codes(raw, vals=None):
        nib = np.stack([raw & 0xF, raw >> 4], axis=1).reshape(-1, 8).astype(np.uint32)     # canonical value order
        slot = np.array([(i % 2) * 4 + i // 2 for i in range(8)], np.uint32)
        words = (nib << (4 * slot)).sum(axis=1, dtype=np.uint32)
        if vals is None:
            return words.view(np.uint8)
        units = words.reshape(128, vals // 32, 4)                    # [row][unit][word]
        return np.ascontiguousarray(units.transpose(1, 0, 2)).view(np.uint8).reshape(-1)
    assert image_codes(np.array([0x21, 0x43, 0x65, 0x87], np.uint8)).view(np.uint32)[0] == 0x86427531
    plain_img = oracle.device_image(oracle.pack(W, flags & 1)[0])
    plain_L = oracle.packed_size(N, K, flags & 1)
    ptable = oracle.pack(W, flags & 1)[0][plain_L.table_off:plain_L.table_off + 64].view(np.uint32).reshape(4, 4)
    for t, kind in enumerate(flags.reshape(-1)):
        o = int(table[t, 1]) * 16
        if kind == 2:
            assert (image[o:o + 8192] == image_codes(blob[o:o + 8192], 128)).all()
            assert (image[o + 8192:o + 8448] == blob[o + 8192:o + 8448]).all()
        elif kind == 3:
            assert (image[o:o + 4096] == image_codes(blob[o:o + 4096], 64)).all()
            assert (image[o + 6144:o + 6400] == blob[o + 6144:o + 6400]).all()
            pm = int(ptable[t, 2]) * 16
            assert (image[o + 4096:o + 6144] == plain_img[pm:pm + 2048]).all()
    # nibbles: every code lies in 1..15
    o = int(table[0, 1]) * 16
    codes = blob[o:o + 8192]
    assert ((codes & 0xF) >= 1).all() and ((codes >> 4) >= 1).all()


def test_gemm_on_quantised_weights_is_the_gemm_of_the_dequantised_matrix(oracle):
    """What the layer computes with 4-bit tiles is X times the dequantised, pruned weight: a different matrix from
    the bf16 one by at most half a quantisation step per element."""
    N, K, M = 256, 384, 5
    W = inputs.weight(N, K, 9, "q4-gemm")
    X = inputs.activation(M, K, 9, "q4-gemm", M)
    flags = np.array([[2, 3, 2], [3, 3, 2]], np.uint8)
    Wq = oracle.prune(W, flags)
    Y, _ = oracle.gemm_f64(X, Wq)
    ref = f32(X).astype(np.float64) @ f32(Wq).astype(np.float64).T
    assert np.allclose(Y, ref, rtol=1e-6, atol=1e-9)
    Wp = oracle.prune(W, flags & 1)
    step = np.abs(f32(Wp)).reshape(N, K // 128, 128).max(-1) / 7.0
    err = np.abs(f32(Wq) - f32(Wp)).reshape(N, K // 128, 128).max(-1)
    assert (err <= 0.52 * step).all()          # 0.5 s + 7 s 2^-9 with s within 2^-9 of max|v| / 7


def test_given_patterns_with_4bit_tiles(oracle):
    """The learned 2:4 mask (one candidate per group) is applied first, then the kept values are quantised: the
    dequantised matrix is the quantisation, row by row, of exactly the values the candidates keep."""
    N, K = 256, 256
    W = inputs.weight(N, K, 10, "q4-patterns")
    rng = inputs.generator(10, "q4-patterns-c")
    patterns = rng.integers(0, 6, (N, K // 4)).astype(np.uint8)
    flags = np.array([[3, 2], [1, 3]], np.uint8)
    blob, L = oracle.pack_patterns(W, flags, patterns)
    What = oracle.unpack(blob)
    S = np.array([[1, 1, 0, 0], [1, 0, 1, 0], [1, 0, 0, 1], [0, 1, 1, 0], [0, 1, 0, 1], [0, 0, 1, 1]], bool)   # typed by hand
    keep = S[patterns].reshape(N, K)
    for tn in range(2):
        for tk in range(2):
            kind = flags[tn, tk]
            rows, cols = slice(tn * 128, tn * 128 + 128), slice(tk * 128, tk * 128 + 128)
            Wt, Kt, got = W[rows, cols], keep[rows, cols], What[rows, cols]
            for r in range(0, 128, 17):
                if kind == 1:
                    assert (got[r] == np.where(Kt[r], Wt[r], 0)).all()
                elif kind == 2:
                    assert (got[r] == oracle.q4_group(Wt[r])[2]).all()
                else:
                    deq = oracle.q4_group(Wt[r][Kt[r]])[2]
                    expect = np.zeros(128, np.uint16)
                    expect[Kt[r]] = deq
                    assert (got[r] == expect).all()
    # and it differs from the magnitude rule's result wherever the candidates do
    assert (oracle.unpack(oracle.pack(W, flags)[0]) != What).any()
