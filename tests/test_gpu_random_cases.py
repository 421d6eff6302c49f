"""Seeded random cases through the C ABI against the oracle: shapes, tile-kind mixtures, row pitches, magnitudes,
given 2:4 masks, flags in host or device memory, token counts on both sides of every schedule boundary and every
combination of launch promises.  Packing is compared bit for bit, products within the stated tolerance."""
import numpy as np
import pytest

from paper_2509_23410_b200 import inputs
from test_gpu_parity import check_parity, gpu, to_bits, to_dev  # noqa: F401  (gpu is a fixture)

pytestmark = pytest.mark.gpu

TOKENS = [1, 2, 3, 4, 5, 8, 15, 16, 17, 31, 32, 33, 63, 64, 65, 100, 127, 128, 129, 239, 240, 241, 300, 481, 512]


def _case(seed):
    g = inputs.generator(4242, "random-cases", seed)
    TN, TK = int(g.integers(1, 9)), int(g.integers(1, 9))
    T = TN * TK
    mode = ["bf16", "q4", "mixed"][seed % 3]
    flags = (g.random(T) < g.random()).astype(np.uint8)
    if mode == "q4":
        flags |= 2
    if mode == "mixed":
        flags |= (2 * (g.random(T) < 0.5)).astype(np.uint8)
    return g, TN, TK, mode, flags


@pytest.mark.parametrize("seed", range(24))
def test_pack_random_case(gpu, oracle, seed):
    torch, B = gpu
    g, TN, TK, mode, flags = _case(seed)
    N, K = 128 * TN, 128 * TK
    vals = (g.standard_normal((N, K)) * np.exp2(g.integers(-30, 30, (N, 1)))).astype(np.float32)
    W = inputs.f32_to_bf16_bits(vals)
    W[g.random((N, K)) < 0.05] = 0
    pad = int(g.choice([0, 8, 72]))
    Wd = torch.zeros((N, K + pad), dtype=torch.bfloat16, device="cuda")
    Wd[:, :K] = to_dev(torch, W)
    given = bool(g.random() < 0.5)
    pats = g.integers(0, 6, N * K // 4).astype(np.uint8) if given else None
    blob_o, L_o = oracle.pack_patterns(W, flags, pats) if given else oracle.pack(W, flags)
    image = oracle.device_image(blob_o)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    pd = torch.from_numpy(pats).cuda() if given else None
    packed, L = (B.patch_pack_patterns(Wd[:, :K], flags, pd, status=status) if given else B.patch_pack(Wd[:, :K], flags))
    assert (packed.cpu().numpy() == image).all(), "flags on the host"
    out = torch.full((image.size + 4096,), 0xAB, dtype=torch.uint8, device="cuda")
    B.patch_pack_dev(Wd[:, :K], torch.from_numpy(flags).cuda(), patterns=pd, out=out, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert (out[:image.size].cpu().numpy() == image).all(), "flags on the device"
    assert bool((out[image.size:] == 0xAB).all()), "nothing is written past the blob"
    Ld = B.patch_read_layout(out)
    for f, _ in B.Layout._fields_:
        assert getattr(Ld, f) == getattr(L_o, f) == getattr(L, f), f
    un = torch.full((N, K + pad), 3.0, dtype=torch.bfloat16, device="cuda")
    B.patch_unpack(L, packed, out=un[:, :K])
    assert (to_bits(un[:, :K].contiguous()) == oracle.unpack(blob_o)).all()
    assert bool((un[:, K:] == 3.0).all())


@pytest.mark.parametrize("seed", range(24))
def test_gemm_random_case(gpu, oracle, seed):
    torch, B = gpu
    g, TN, TK, mode, flags = _case(seed)
    if mode == "mixed":                      # the matmul serves weights of bf16 tiles or of 4-bit tiles, not both
        flags = flags | 2 if seed % 2 else flags & 1
    q4 = bool(flags[0] & 2)
    N, K = 128 * TN, 128 * TK
    W = inputs.weight(N, K, 4242, "random-gemm", seed)
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    padx, pady = int(g.choice([0, 8, 200])), int(g.choice([0, 8, 200]))
    size = max([B.patch_gemm_workspace_size(L, m) for m in (16, 64, 65)] + [256])
    ws = torch.zeros(size, dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    promises = [0, B.WEIGHTS_STATIC, B.WEIGHTS_STATIC | B.INPUT_STATIC, B.WEIGHTS_STATIC | B.INPUT_STATIC | B.OUTPUT_STATIC]
    for M in sorted(int(m) for m in g.choice(TOKENS, 3, replace=False)):
        X = inputs.activation(M, K, 4242, "random-gemm", seed, M)
        Y32, _ = oracle.gemm_f64(X, What)
        Xd = torch.zeros((M, K + padx), dtype=torch.bfloat16, device="cuda")
        Xd[:, :K] = to_dev(torch, X)
        variants = [B.VARIANT_AUTO | p for p in promises] + [B.VARIANT_MMA]
        if M <= 4 and not q4:
            variants.append(B.VARIANT_GEMV)
        for v in variants:
            Yd = torch.full((M, N + pady), 7.0, dtype=torch.bfloat16, device="cuda")
            for _ in range(2):               # twice: the workspace must come back as the next call needs it
                B.patch_gemm(Xd[:, :K], L, packed, Y=Yd[:, :N], workspace=ws, status=status, variant=v)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            check_parity(oracle, to_bits(Yd[:, :N].contiguous()), Y32, f"seed={seed} N={N} K={K} M={M} q4={q4} variant={v:#x}")
            assert bool((Yd[:, N:] == 7.0).all()), "nothing is written past column N"
