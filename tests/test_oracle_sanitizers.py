"""The oracle's C under AddressSanitizer and UndefinedBehaviorSanitizer: a tour of every exported function on small
inputs (all four tile kinds, ragged tile grids, given patterns, the mask-learning functions) in a child process
that loads the sanitised build.  Any out-of-bounds access, misaligned access, signed overflow or invalid shift ends
the child with a non-zero status."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

TOUR = r"""
import numpy as np
import oracle
from paper_2509_23410_b200 import inputs

assert oracle.build().endswith("libpatch_oracle_san.so")
g = np.random.default_rng(7)
N, K = 256, 384
W = inputs.f32_to_bf16_bits((g.standard_normal((N, K)) * 0.02).astype(np.float32))
W[3, :] = 0
W[::5, ::3] = 0
T = (N // 128) * (K // 128)
for flags in (np.zeros(T, np.uint8), np.ones(T, np.uint8), np.arange(T, dtype=np.uint8) % 4,
              np.full(T, 2, np.uint8), np.full(T, 3, np.uint8)):
    M = oracle.mask(W, flags)
    What = oracle.prune(W, flags)
    blob, L = oracle.pack(W, flags)
    assert L.total_bytes == blob.size and oracle.packed_size(N, K, flags).total_bytes == blob.size
    assert (oracle.unpack(blob) == What).all()
    assert oracle.device_image(blob).size == blob.size
    pats = g.integers(0, 6, N * K // 4).astype(np.uint8)
    blob_p, _ = oracle.pack_patterns(W, flags, pats)
    Mp = oracle.mask_patterns(N, K, flags & 1, pats)
    assert Mp.shape == M.shape and oracle.unpack(blob_p).shape == W.shape
    X = inputs.f32_to_bf16_bits(g.standard_normal((5, K)).astype(np.float32))
    Y32, Y16 = oracle.gemm_f64(X, What)
    assert oracle.gemm_f32(X, What).shape == Y32.shape == (5, N)
    rows = np.array([0, 4], np.int64)
    assert oracle.gemm_f64_rows(X, rows, What).shape == (2, N)
# small tiles, as the oracle's own pins use them
Ws = inputs.f32_to_bf16_bits(g.standard_normal((8, 16)).astype(np.float32))
fs = np.array([0, 1, 1, 0], np.uint8)
bs, _ = oracle.pack(Ws, fs, tile_n=4, tile_k=8)
assert (oracle.unpack(bs) == oracle.prune(Ws, fs, tile_n=4, tile_k=8)).all()
s, c, d = oracle.q4_group(Ws[0])
assert c.min() >= 1 and c.max() <= 15
assert oracle.swiglu(oracle.gemm_f64(X, What)[0][:, :256].astype(np.float32)).shape == (5, 128)
# mask learning
Pt = g.standard_normal(T).astype(np.float32)
P24 = g.standard_normal((6, N * K // 4)).astype(np.float32)
for noise in (False, True):
    Mt, Wt, sums = oracle.soft_mask(W, Pt, P24, 2.0, 3.0, seed=11, noise=noise)
    assert np.isfinite(Mt).all() and sums.shape == (4,)
    c1, c2 = oracle.regularizer_coefficients(sums, 0.5, 1e-3, 1e-4)
    assert np.isfinite(oracle.regularizers(sums, 0.5, 1e-3, 1e-4))
    Gw = g.standard_normal((N, K)).astype(np.float32)
    gt, g6 = oracle.soft_mask_backward(W, Pt, P24, 2.0, 3.0, Gw, c1, c2, seed=11, noise=noise)
    assert np.isfinite(gt).all() and np.isfinite(g6).all()
fl, pa = oracle.hard_mask(Pt, P24, N, K)
assert fl.max() <= 1 and pa.max() <= 5
assert np.isfinite(oracle.uniform(1, 2, 3)) and np.isfinite(oracle.gumbel(1, 2, 3))
print("tour ok")
"""


def _runtime(name):
    out = subprocess.run(["gcc", f"-print-file-name={name}"], capture_output=True, text=True).stdout.strip()
    return out if os.path.isabs(out) and os.path.exists(out) else None


def test_oracle_under_asan_and_ubsan():
    asan = _runtime("libasan.so")
    if asan is None:
        pytest.skip("no AddressSanitizer runtime beside gcc")
    env = dict(os.environ, PATCH_ORACLE_SANITIZE="1", LD_PRELOAD=asan, PYTHONPATH=ROOT,
               ASAN_OPTIONS="detect_leaks=0:abort_on_error=0", UBSAN_OPTIONS="print_stacktrace=1:halt_on_error=1")
    r = subprocess.run([sys.executable, "-c", TOUR], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "tour ok" in r.stdout, (r.stdout[-2000:], r.stderr[-4000:])
