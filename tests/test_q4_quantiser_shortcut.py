"""The 4-bit pack kernel quantises without dividing: q = rint(v / s) is computed as v * (1 / s), snapped to a grid of
2^-10 and rounded to the nearest-even integer by adding 1.5 * 2^23; the scale as bf16(m * fp32(1/7)) instead of
bf16(m / 7).  Its comments argue that for bf16 inputs this gives the bits of the divisions.  Here the argument is
checked by exhaustion on the CPU, in numpy float32 arithmetic: every pair of 8-bit significands, every exponent
difference that leaves the quotient below 8, both signs, and a reciprocal that is off by one unit in the last place
in either direction (the hardware's approximate reciprocal is good to one)."""
import numpy as np

f32 = np.float32


def _bf16_values(exponents):
    """All positive normal bf16 values with the given unbiased exponents, as float32."""
    sig = np.arange(128, 256, dtype=np.float32) / f32(128.0)               # 1.0000000 .. 1.1111111
    return (sig[None, :] * np.exp2(np.asarray(exponents, dtype=np.float32))[:, None]).astype(np.float32).ravel()


def _round_nearest_even_magic(t):
    snapped = (t + f32(12288.0)) - f32(12288.0)                            # grid of 2^-10 for |t| < 8
    return (snapped + f32(12582912.0)).view(np.int32) - np.int32(0x4B400000)


def test_codes_equal_the_quotients_rounding():
    s = _bf16_values([0])                                                  # the scale's exponent cancels: fix it
    v = _bf16_values(range(-12, 3))                                        # quotients from 2^-13 up to just below 8
    V, S = np.meshgrid(v, s, indexing="ij")
    keep = V / S <= f32(7.02)                                              # s = bf16(max / 7) bounds every quotient of a row
    V, S = V[keep], S[keep]
    want = np.rint(V / S).astype(np.int32)                                 # fp32 IEEE division, ties to even
    inv = f32(1.0) / S
    for rcp in (inv, np.nextafter(inv, f32(0)), np.nextafter(inv, f32(np.inf))):
        for sign in (f32(1.0), f32(-1.0)):
            got = _round_nearest_even_magic((sign * V) * rcp)
            assert (got == (sign * want).astype(np.int32)).all()
    # the ties themselves are in the sample: quotients that are exactly k + 1/2
    q = V / S
    assert ((q * 2 == np.rint(q * 2)) & (q != np.rint(q))).sum() >= 200


def test_scale_equals_the_divisions_rounding():
    from paper_2509_23410_b200 import inputs
    m = _bf16_values(range(-90, 128))
    want = inputs.f32_to_bf16_bits((m / f32(7.0)).astype(np.float32))
    got = inputs.f32_to_bf16_bits((m * f32(1.0 / 7.0)).astype(np.float32))
    assert (want == got).all()
