"""GPU parity of the CTA-pair large-M schedule (PATCH_VARIANT_PAIR) against the CPU oracle.

A cluster of two CTAs owns four row-blocks; weights whose tiles are all of one kind run on one kernel, weights
that mix kinds on another (2:4 tiles whose pair partner is dense are expanded to their dense image), so the cases
cover all-dense, all-2:4 and mixed weights, row-block counts that are not multiples of four (a quad with one pair, a pair with one
row-block), ragged token counts, several output tiles per cluster and launches back to back."""
import numpy as np
import pytest

from paper_2509_23410_b200 import inputs
from test_gpu_parity import check_parity, f32, gpu, run_gemm, to_bits, to_dev  # noqa: F401  (gpu is a fixture)

pytestmark = pytest.mark.gpu


def _inputs(N, K, M, p, tag="pair"):
    stream = (tag, N, K, p)
    W = inputs.weight(N, K, inputs.MASTER_SEED, *stream)
    flags = inputs.tile_flags(N, K, p, inputs.MASTER_SEED, *stream)
    X = inputs.activation(M, K, inputs.MASTER_SEED, *stream, M)
    return W, flags, X


@pytest.mark.parametrize("p", [0.0, 1.0, 0.5, 0.2, 0.85])
@pytest.mark.parametrize("N,K,M", [(512, 512, 300), (640, 256, 130), (768, 384, 257), (128, 128, 65),
                                   (1024, 1024, 1000), (1536, 2048, 512)])
def test_pair_schedule_full_output(gpu, oracle, N, K, M, p):
    torch, B = gpu
    W, flags, X = _inputs(N, K, M, p)
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Y = run_gemm(gpu, X, L, packed, B.VARIANT_PAIR)
    Y32, Y16 = oracle.gemm_f64(X, What)
    check_parity(oracle, Y, Y32, f"pair N={N} K={K} M={M} p={p}")
    assert (Y == Y16).mean() >= 0.99
    # deterministic: the same launch again gives the same bits
    assert (run_gemm(gpu, X, L, packed, B.VARIANT_PAIR) == Y).all()


@pytest.mark.parametrize("p", [0.0, 1.0, 0.5])
def test_pair_schedule_identity_probe(gpu, oracle, p):
    """X = I: every output is one product, so Y == What^T exactly; a wrong operand or metadata order shows."""
    torch, B = gpu
    N, K = 768, 512
    W, flags, _ = _inputs(N, K, K, p, "pair-id")
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    X = inputs.f32_to_bf16_bits(np.eye(K, dtype=np.float32))
    Y = run_gemm(gpu, X, L, packed, B.VARIANT_PAIR)
    assert (f32(Y) == f32(What).T).all()


def test_pair_schedule_rejects_small_m(gpu):
    torch, B = gpu
    W, flags, X = _inputs(512, 512, 64, 1.0)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    ws = torch.zeros(B.patch_gemm_workspace_size(L, 64), dtype=torch.uint8, device="cuda")
    with pytest.raises(B.PatchError) as e:
        B.patch_gemm(to_dev(torch, X), L, packed, workspace=ws, variant=B.VARIANT_PAIR)
    assert e.value.status == B.ERR_SHAPE


@pytest.mark.parametrize("p", [0.0, 1.0, 0.5])
def test_pair_schedule_back_to_back(gpu, oracle, p):
    """Twelve launches in a row on one stream, alternating between two weights and writing twelve outputs, then a
    dependent chain: every result is checked, so a launch that disturbed its neighbour would show."""
    torch, B = gpu
    M = 520
    cases = []
    for i, (N, K) in enumerate([(1024, 512), (640, 768)]):
        W, flags, X = _inputs(N, K, M, p, f"pair-b2b{i}")
        packed, L = B.patch_pack(to_dev(torch, W), flags)
        cases.append((oracle.prune(W, flags), packed, L, X, to_dev(torch, X)))
    torch.cuda.synchronize()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    outs = []
    for i in range(12):
        What, packed, L, X, Xd = cases[i % 2]
        # every other launch declared independent of its predecessor (weights and X are not written here): it may
        # start while the launch before it still runs, and only its Y stores wait
        promise = (B.WEIGHTS_STATIC | B.INPUT_STATIC) if i % 2 else 0
        outs.append(B.patch_gemm(Xd, L, packed, status=status, variant=B.VARIANT_PAIR | promise))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    refs = [oracle.gemm_f64(c[3], c[0])[0] for c in cases]
    for i, Y in enumerate(outs):
        check_parity(oracle, to_bits(Y), refs[i % 2], f"launch {i}")
        assert (to_bits(Y) == to_bits(outs[i % 2])).all()
    # chain: Y of one call is X of the next (square weight), interleaved with the other prefill schedules
    N = K = 512
    W, flags, X = _inputs(N, K, M, p, "pair-chain")
    W = inputs.f32_to_bf16_bits(f32(W) * 2.0)
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    bufs = [to_dev(torch, X)] + [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(6)]
    for i in range(6):
        B.patch_gemm(bufs[i], L, packed, Y=bufs[i + 1], status=status,
                     variant=(B.VARIANT_PAIR if i % 3 != 2 else B.VARIANT_MMA | B.WEIGHTS_STATIC))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = X
    for i in range(6):
        Y32, _ = oracle.gemm_f64(ref, What)
        got = to_bits(bufs[i + 1])
        check_parity(oracle, got, Y32, f"chain step {i}")
        ref = got


@pytest.mark.parametrize("N,K,M,p", [(4096, 4096, 2048, 0.0), (11008, 4096, 2048, 1.0), (4096, 11008, 4096, 1.0),
                                     (4096, 4096, 4096, 0.5), (11008, 4096, 2048, 0.35)])
def test_pair_schedule_llama_shapes_sampled(gpu, oracle, N, K, M, p):
    """Full-size shapes: 64 token rows over all N, two whole row-blocks over all tokens (every token tile touched)."""
    torch, B = gpu
    W, flags, X = _inputs(N, K, M, p, "pair-llama")
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Y = run_gemm(gpu, X, L, packed, B.VARIANT_PAIR)
    rng = inputs.generator(inputs.MASTER_SEED, "pair-rows", N, K, M)
    rows = np.unique(np.concatenate([rng.integers(0, M, 60), [0, M - 1, 119, 120, 127, 128, 239, 240, 255, 256]]))
    check_parity(oracle, Y[rows], oracle.gemm_f64_rows(X, rows, What), f"rows N={N} K={K} M={M}")
    for tn in (N // 128 - 1, int(rng.integers(0, N // 128))):
        cols = slice(tn * 128, tn * 128 + 128)
        Yb, _ = oracle.gemm_f64(X, What[cols], want_bf16=False)
        check_parity(oracle, Y[:, cols], Yb, f"row-block {tn} N={N} K={K} M={M}")
