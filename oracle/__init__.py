"""numpy-facing wrapper around the CPU oracle (``patch_oracle.c``).

TEST INFRASTRUCTURE ONLY: importable from ``tests/``, from the smoke check and from the
benchmark's CPU-baseline legs.  The product package never imports this module, and this
module never imports the product package's CUDA binding.

All matrices are numpy ``uint16`` arrays of bf16 bit patterns, C-contiguous.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "patch_oracle.c")
_LIB = os.path.join(_HERE, "libpatch_oracle.so")

KIND_DENSE, KIND_SPARSE, KIND_DENSE_Q4, KIND_SPARSE_Q4 = 0, 1, 2, 3
MAGIC = 0x48435450


class Layout(ctypes.Structure):
    _fields_ = [("magic", ctypes.c_uint32), ("version", ctypes.c_uint32),
                ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("tile_n", ctypes.c_int32), ("tile_k", ctypes.c_int32),
                ("n_dense", ctypes.c_int64), ("n_sparse", ctypes.c_int64),
                ("table_off", ctypes.c_uint64), ("payload_off", ctypes.c_uint64),
                ("payload_bytes", ctypes.c_uint64), ("total_bytes", ctypes.c_uint64),
                ("n_dense_q4", ctypes.c_int64), ("n_sparse_q4", ctypes.c_int64)]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, OpenMP over outputs, no fast-math).

    With PATCH_ORACLE_SANITIZE=1 in the environment: a serial build with AddressSanitizer and
    UndefinedBehaviorSanitizer, every finding fatal (the process must then be started with the
    sanitizer's runtime preloaded; ``tests/test_oracle_sanitizers.py`` does that)."""
    if os.environ.get("PATCH_ORACLE_SANITIZE") == "1":
        out = os.path.join(_HERE, "libpatch_oracle_san.so")
        if force or not os.path.exists(out) or os.path.getmtime(out) < os.path.getmtime(_SRC):
            subprocess.run(["gcc", "-O1", "-g", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared", "-Wall", "-Wextra",
                            "-Wno-unknown-pragmas", "-fsanitize=address,undefined", "-fno-sanitize-recover=all",
                            "-fno-omit-frame-pointer", "-o", out, _SRC, "-lm"], check=True)
        return out
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               "-Wall", "-Wextra", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_uniform.restype = ctypes.c_double
        _lib.oracle_gumbel.restype = ctypes.c_double
        _lib.oracle_regularizers.restype = ctypes.c_double
    return _lib


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def _flags(f):
    return np.ascontiguousarray(f, dtype=np.uint8).reshape(-1)


def _check(rc, what):
    if rc != 0:
        raise ValueError(f"oracle {what} failed with status {rc}")


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def q4_group(values):
    """4-bit quantiser of one group of stored values (bf16 bits): (scale bits, codes q + 8, dequantised bits)."""
    v = _u16(values).reshape(-1)
    scale = np.zeros(1, np.uint16)
    codes = np.empty(v.size, np.uint8)
    deq = np.empty(v.size, np.uint16)
    _check(lib().oracle_q4_group(_p(v), int(v.size), _p(scale), _p(codes), _p(deq)), "q4_group")
    return int(scale[0]), codes, deq


def mask(W, flags, tile_n=128, tile_k=128) -> np.ndarray:
    """Hard mask M* (uint8, 1 = keep), Algorithm 1's merged tile / 2:4 mask."""
    W = _u16(W)
    N, K = W.shape
    out = np.empty((N, K), np.uint8)
    _check(lib().oracle_mask(_p(W), ctypes.c_int64(N), ctypes.c_int64(K), _p(_flags(flags)),
                             tile_n, tile_k, _p(out)), "mask")
    return out


def prune(W, flags, tile_n=128, tile_k=128) -> np.ndarray:
    """Pruned weight What = W (.) M* (bf16 bits; pruned entries are +0)."""
    W = _u16(W)
    N, K = W.shape
    out = np.empty((N, K), np.uint16)
    _check(lib().oracle_prune(_p(W), ctypes.c_int64(N), ctypes.c_int64(K), _p(_flags(flags)),
                              tile_n, tile_k, _p(out)), "prune")
    return out


def packed_size(N, K, flags, tile_n=128, tile_k=128) -> Layout:
    L = Layout()
    _check(lib().oracle_packed_size(ctypes.c_int64(N), ctypes.c_int64(K), tile_n, tile_k,
                                    _p(_flags(flags)), ctypes.byref(L)), "packed_size")
    return L


def pack(W, flags, tile_n=128, tile_k=128):
    """Canonical packed blob (uint8 array) and its layout."""
    W = _u16(W)
    N, K = W.shape
    L = packed_size(N, K, flags, tile_n, tile_k)
    blob = np.empty(L.total_bytes, np.uint8)
    _check(lib().oracle_pack(_p(W), _p(_flags(flags)), ctypes.byref(L), _p(blob),
                             ctypes.c_uint64(blob.nbytes)), "pack")
    return blob, L


def pack_patterns(W, flags, patterns, tile_n=128, tile_k=128):
    """Canonical packed blob with the 2:4 mask given as one candidate index (row of S) per group."""
    W = _u16(W)
    N, K = W.shape
    patterns = np.ascontiguousarray(patterns, dtype=np.uint8).reshape(-1)
    assert patterns.size == N * K // 4
    L = packed_size(N, K, flags, tile_n, tile_k)
    blob = np.empty(L.total_bytes, np.uint8)
    _check(lib().oracle_pack_patterns(_p(W), _p(_flags(flags)), _p(patterns), ctypes.byref(L), _p(blob),
                                      ctypes.c_uint64(blob.nbytes)), "pack_patterns")
    return blob, L


def unpack(blob) -> np.ndarray:
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    L = Layout.from_buffer_copy(blob[:ctypes.sizeof(Layout)].tobytes())
    out = np.empty((L.N, L.K), np.uint16)
    _check(lib().oracle_unpack(_p(blob), ctypes.c_uint64(blob.nbytes), _p(out)), "unpack")
    return out


def device_image(canon_blob) -> np.ndarray:
    """Canonical blob -> device image (per-tile byte bijection; 128x128 tiles only)."""
    canon_blob = np.ascontiguousarray(canon_blob, dtype=np.uint8)
    out = np.zeros_like(canon_blob)
    _check(lib().oracle_device_image(_p(canon_blob), ctypes.c_uint64(canon_blob.nbytes), _p(out)),
           "device_image")
    return out


def gemm_f64(X, What, want_bf16=True):
    """Y = X What^T, double accumulation -> (fp32 [M x N], bf16 bits [M x N] or None)."""
    X, What = _u16(X), _u16(What)
    M, K = X.shape
    N, K2 = What.shape
    assert K == K2
    Y32 = np.empty((M, N), np.float32)
    Y16 = np.empty((M, N), np.uint16) if want_bf16 else None
    _check(lib().oracle_gemm_f64(_p(X), ctypes.c_int64(M), ctypes.c_int64(K), _p(What),
                                 ctypes.c_int64(N), _p(Y32),
                                 _p(Y16) if want_bf16 else ctypes.c_void_p(0)), "gemm_f64")
    return Y32, Y16


def gemm_f32(X, What) -> np.ndarray:
    X, What = _u16(X), _u16(What)
    M, K = X.shape
    N, _ = What.shape
    Y32 = np.empty((M, N), np.float32)
    _check(lib().oracle_gemm_f32(_p(X), ctypes.c_int64(M), ctypes.c_int64(K), _p(What),
                                 ctypes.c_int64(N), _p(Y32)), "gemm_f32")
    return Y32


def gemm_f64_rows(X, rows, What) -> np.ndarray:
    """Rows ``rows`` of Y only (sampled parity at large M)."""
    X, What = _u16(X), _u16(What)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    _, K = X.shape
    N, _ = What.shape
    Y32 = np.empty((len(rows), N), np.float32)
    _check(lib().oracle_gemm_f64_rows(_p(X), ctypes.c_int64(K), _p(rows), ctypes.c_int64(len(rows)),
                                      _p(What), ctypes.c_int64(N), _p(Y32)), "gemm_f64_rows")
    return Y32


def swiglu(Y_gu, block: int = 128) -> np.ndarray:
    """Gated product of the MLP's gate and up projections (the "up, gate and down matrices of the MLP"
    of the paper's per-layer allocation study; in the LLaMA models it measures, the MLP is
    down(silu(gate x) * up x)), for a weight that stacks the two matrices with their row-blocks
    interleaved: columns [2*block*j, 2*block*j + block) of ``Y_gu`` are gate outputs, the next
    ``block`` columns the matching up outputs.  out[m, block*j + r] = silu(g) * u with
    silu(x) = x / (1 + exp(-x)), evaluated in double on the GEMM result, returned as fp32."""
    Y = np.asarray(Y_gu)
    M, N = Y.shape
    assert N % (2 * block) == 0
    y = Y.astype(np.float64).reshape(M, N // (2 * block), 2, block)
    g, u = y[:, :, 0, :], y[:, :, 1, :]
    with np.errstate(over="ignore"):
        out = g / (1.0 + np.exp(-g)) * u
    return out.reshape(M, N // 2).astype(np.float32)


def uniform(seed, stream, idx) -> float:
    return float(lib().oracle_uniform(ctypes.c_uint64(seed), ctypes.c_uint64(stream), ctypes.c_uint64(idx)))


def gumbel(seed, stream, idx) -> float:
    return float(lib().oracle_gumbel(ctypes.c_uint64(seed), ctypes.c_uint64(stream), ctypes.c_uint64(idx)))


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def soft_mask(W, P_tile, P24, tau, kappa, seed=0, noise=True, tile_n=128, tile_k=128):
    """Soft mask of Eq. 2-4 -> (Mt float64 [N x K], Mt (.) W as bf16 bits, sums[4] for Eq. 5)."""
    W = _u16(W)
    N, K = W.shape
    P_tile, P24 = _f32(P_tile), _f32(P24)
    assert P_tile.size == (N // tile_n) * (K // tile_k) and P24.shape == (6, N * K // 4)
    Mt = np.empty((N, K), np.float64)
    Wt = np.empty((N, K), np.uint16)
    sums = np.empty(4, np.float64)
    _check(lib().oracle_soft_mask(_p(W), ctypes.c_int64(N), ctypes.c_int64(K), _p(P_tile), _p(P24), tile_n, tile_k,
                                  ctypes.c_double(tau), ctypes.c_double(kappa), ctypes.c_uint64(seed), int(bool(noise)),
                                  _p(Mt), _p(Wt), _p(sums)), "soft_mask")
    return Mt, Wt, sums


def regularizers(sums, rho, lambda1, lambda2) -> float:
    """The sparsity and weight regularisers of Eq. 5 from the per-matrix sums ([n x 4])."""
    sums = np.ascontiguousarray(sums, dtype=np.float64).reshape(-1, 4)
    return float(lib().oracle_regularizers(_p(sums), int(sums.shape[0]), ctypes.c_double(rho),
                                           ctypes.c_double(lambda1), ctypes.c_double(lambda2)))


def regularizer_coefficients(sums, rho, lambda1, lambda2):
    """(c1, c2): how one element's soft-mask value enters the gradient of Eq. 5's two regularisers."""
    sums = np.ascontiguousarray(sums, dtype=np.float64).reshape(-1, 4)
    c1, c2 = ctypes.c_double(0), ctypes.c_double(0)
    lib().oracle_regularizer_coefficients(_p(sums), int(sums.shape[0]), ctypes.c_double(rho), ctypes.c_double(lambda1),
                                          ctypes.c_double(lambda2), ctypes.byref(c1), ctypes.byref(c2))
    return float(c1.value), float(c2.value)


def soft_mask_backward(W, P_tile, P24, tau, kappa, Gw, c1, c2, seed=0, noise=True, tile_n=128, tile_k=128):
    """Gradient of sum(Gw * Mt * W) + c1 sum(Mt) - c2/2 sum((Mt W)^2) w.r.t. the logits -> (gP_tile, gP24), float64."""
    W = _u16(W)
    N, K = W.shape
    P_tile, P24, Gw = _f32(P_tile), _f32(P24), _f32(Gw)
    assert Gw.shape == (N, K) and P24.shape == (6, N * K // 4)
    gt = np.empty(P_tile.size, np.float64)
    g6 = np.empty((6, N * K // 4), np.float64)
    _check(lib().oracle_soft_mask_backward(_p(W), ctypes.c_int64(N), ctypes.c_int64(K), _p(P_tile), _p(P24), tile_n,
                                           tile_k, ctypes.c_double(tau), ctypes.c_double(kappa), ctypes.c_uint64(seed),
                                           int(bool(noise)), _p(Gw), ctypes.c_double(c1), ctypes.c_double(c2), _p(gt),
                                           _p(g6)), "soft_mask_backward")
    return gt.reshape(np.asarray(P_tile).shape), g6


def hard_mask(P_tile, P24, N, K, tile_n=128, tile_k=128):
    """Algorithm 1's hard masks -> (tile flags uint8 [TN*TK], candidate index per group uint8 [N*K/4])."""
    P_tile, P24 = _f32(P_tile), _f32(P24)
    assert P_tile.size == (N // tile_n) * (K // tile_k) and P24.shape == (6, N * K // 4)
    flags = np.empty(P_tile.size, np.uint8)
    patterns = np.empty(N * K // 4, np.uint8)
    _check(lib().oracle_hard_mask(_p(P_tile), _p(P24), ctypes.c_int64(N), ctypes.c_int64(K), tile_n, tile_k,
                                  _p(flags), _p(patterns)), "hard_mask")
    return flags, patterns


def mask_patterns(N, K, flags, patterns, tile_n=128, tile_k=128) -> np.ndarray:
    """Hard mask M* (uint8) with the 2:4 part given as candidate indices."""
    patterns = np.ascontiguousarray(patterns, dtype=np.uint8).reshape(-1)
    out = np.empty((N, K), np.uint8)
    _check(lib().oracle_mask_patterns(ctypes.c_int64(N), ctypes.c_int64(K), _p(_flags(flags)), _p(patterns),
                                      tile_n, tile_k, _p(out)), "mask_patterns")
    return out


def parity_metrics(Y_test_f32, Y_ref_f32):
    """relF = |dY|_F / |Yref|_F and max|dY| / max|Yref| (the two tolerances of the benchmark spec)."""
    d = Y_test_f32.astype(np.float64) - Y_ref_f32.astype(np.float64)
    ref = Y_ref_f32.astype(np.float64)
    nref = float(np.sqrt((ref * ref).sum()))
    relF = float(np.sqrt((d * d).sum())) / nref if nref > 0 else float(np.abs(d).max(initial=0.0))
    mref = float(np.abs(ref).max(initial=0.0))
    maxrel = float(np.abs(d).max(initial=0.0)) / mref if mref > 0 else float(np.abs(d).max(initial=0.0))
    return relF, maxrel
