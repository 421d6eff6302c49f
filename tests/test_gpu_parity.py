"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.  Packing is compared bit for bit; GEMM outputs within the stated tolerance
(relative Frobenius error <= 2e-3 and max |dY| <= 1e-2 * max |Yref|)."""
import ctypes

import numpy as np
import pytest

from paper_2509_23410_b200 import inputs

pytestmark = pytest.mark.gpu

REL_F_TOL = 2e-3
MAX_TOL = 1e-2


@pytest.fixture(scope="module")
def gpu():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("no CUDA device: GPU tests must run on a B200")
    from paper_2509_23410_b200 import binding
    binding.lib()   # raises if the CUDA library is missing -- there is no fallback
    return torch, binding


def to_dev(torch, bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def to_bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


f32 = inputs.bf16_bits_to_f32


def check_parity(oracle, Y_bits, Y32, what=""):
    relF, maxrel = oracle.parity_metrics(f32(Y_bits), Y32)
    assert relF <= REL_F_TOL and maxrel <= MAX_TOL, f"{what}: relF={relF:.3e} maxrel={maxrel:.3e}"
    return relF, maxrel


def run_gemm(gpu, X_bits, layout, packed, variant):
    torch, B = gpu
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.zeros(max(B.patch_gemm_workspace_size(layout, X_bits.shape[0]), 1), dtype=torch.uint8, device="cuda")
    Y = B.patch_gemm(to_dev(torch, X_bits), layout, packed, workspace=ws, status=status, variant=variant)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, "device-side wait timed out"
    return to_bits(Y)


# ---------------------------------------------------------------------------------------------
# packing: bit exact, image and round trip


@pytest.mark.parametrize("N,K,p", [(128, 128, 0.0), (128, 128, 1.0), (256, 384, 0.5), (1024, 1024, 0.5),
                                   (640, 256, 0.35), (4096, 4096, 0.7)])
def test_pack_bit_exact(gpu, oracle, N, K, p):
    torch, B = gpu
    W = inputs.weight(N, K, 11, "pack", N, K)
    W[::13, ::7] = 0          # exact zeros and ties
    W[5::17, 3::4] = W[5::17, 2::4]
    flags = inputs.tile_flags(N, K, p, 11, "pack", N, K)
    canon, Lo = oracle.pack(W, flags)
    image = oracle.device_image(canon)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    torch.cuda.synchronize()
    assert (L.n_dense, L.n_sparse, L.total_bytes) == (Lo.n_dense, Lo.n_sparse, Lo.total_bytes)
    got = packed.cpu().numpy()
    assert got.shape == image.shape and (got == image).all()
    What = oracle.prune(W, flags)
    assert (to_bits(B.patch_unpack(L, packed)) == What).all()
    # packing the pruned weight again reproduces the blob (idempotence through the GPU path)
    packed2, _ = B.patch_pack(B.patch_unpack(L, packed), flags)
    assert torch.equal(packed, packed2)


@pytest.mark.parametrize("few_values", [False, True])
def test_pack_arbitrary_bit_patterns(gpu, oracle, few_values):
    """The kept pair is decided on the integer key bits & 0x7FFF with ties to the lower index, whatever the
    bits mean: arbitrary 16-bit patterns (NaN, Inf, +-0, subnormals), and a handful of values so that most
    groups tie."""
    torch, B = gpu
    N, K = 512, 640
    rng = inputs.generator(inputs.MASTER_SEED, "bits", few_values)
    if few_values:
        pool = np.array([0x0000, 0x8000, 0x3C00, 0xBC00, 0x3C01, 0x7F80, 0xFF80, 0x7FC1, 0x0001, 0x8001], np.uint16)
        W = pool[rng.integers(0, len(pool), (N, K))]
    else:
        W = rng.integers(0, 65536, (N, K)).astype(np.uint16)
    flags = inputs.tile_flags(N, K, 0.7, inputs.MASTER_SEED, "bits", few_values)
    image = oracle.device_image(oracle.pack(W, flags)[0])
    Wd = torch.from_numpy(W.view(np.int16)).cuda().view(torch.bfloat16)
    packed, L = B.patch_pack(Wd, flags)
    assert (packed.cpu().numpy() == image).all()
    assert (to_bits(B.patch_unpack(L, packed)) == oracle.prune(W, flags)).all()


def test_pack_with_row_pitch(gpu, oracle):
    torch, B = gpu
    N, K, ld = 256, 256, 320
    W = inputs.weight(N, K, 12, "pitch")
    flags = np.array([[1, 0], [0, 1]], np.uint8)
    big = torch.zeros((N, ld), dtype=torch.bfloat16, device="cuda")
    big[:, :K] = to_dev(torch, W)
    packed, L = B.patch_pack(big[:, :K], flags)
    image = oracle.device_image(oracle.pack(W, flags)[0])
    assert (packed.cpu().numpy() == image).all()
    out = torch.zeros((N, ld), dtype=torch.bfloat16, device="cuda")
    B.patch_unpack(L, packed, out=out[:, :K])
    assert (to_bits(out[:, :K]) == oracle.prune(W, flags)).all()
    assert (to_bits(out[:, K:]) == 0).all()


# ---------------------------------------------------------------------------------------------
# identity probe: X = I makes every output a single product, so Y[m][n] == What[n][m] exactly


@pytest.mark.parametrize("variant", ["gemv", "mma"])
@pytest.mark.parametrize("p", [0.0, 1.0, 0.5])
def test_identity_probe(gpu, oracle, variant, p):
    torch, B = gpu
    N, K = 256, 384
    # weights whose value encodes (row, column): a wrong permutation shows as exact mismatches
    r, c = np.meshgrid(np.arange(N), np.arange(K), indexing="ij")
    Wf = ((1.0 + (c % 128) / 128.0) * np.where(r % 2 == 0, 1.0, -1.0) * (1 + (r % 128) // 16)).astype(np.float32)
    W = inputs.f32_to_bf16_bits(Wf)
    W ^= inputs.weight(N, K, 13, "ident") & 0x0003    # break exact ties differently per element
    flags = inputs.tile_flags(N, K, p, 13, "ident")
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    if variant == "mma":
        X = np.zeros((K, K), np.uint16)
        X[np.arange(K), np.arange(K)] = 0x3F80
        Y = run_gemm(gpu, X, L, packed, B.VARIANT_MMA)
        assert (f32(Y) == f32(What).T).all()
    else:
        for k0 in (0, 1, 2, 3, 127, 128, 255, 383):   # one-hot rows through the decode kernel
            X = np.zeros((2, K), np.uint16)
            X[0, k0] = 0x3F80
            X[1, (k0 + 77) % K] = 0x4000               # 2.0
            Y = run_gemm(gpu, X, L, packed, B.VARIANT_GEMV)
            assert (f32(Y[0]) == f32(What[:, k0])).all()
            assert (f32(Y[1]) == 2.0 * f32(What[:, (k0 + 77) % K])).all()


# ---------------------------------------------------------------------------------------------
# GEMM parity at sizes spanning several tiles and ragged token counts


@pytest.mark.parametrize("M", [1, 2, 3, 4])
@pytest.mark.parametrize("N,K,p", [(384, 640, 0.5), (128, 128, 1.0), (1024, 1024, 0.5)])
def test_gemv_parity(gpu, oracle, M, N, K, p):
    torch, B = gpu
    W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=p, stream=("gemv", N, K)), 21, M)
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Y = run_gemm(gpu, X, L, packed, B.VARIANT_GEMV)
    Y32, _ = oracle.gemm_f64(X, What)
    check_parity(oracle, Y, Y32, f"gemv M={M}")


@pytest.mark.parametrize("M", [1, 5, 16, 17, 32, 33, 64, 65, 100, 128, 129, 256, 300, 513])
@pytest.mark.parametrize("N,K,p", [(384, 640, 0.5), (256, 1152, 0.0), (256, 1152, 1.0)])
def test_mma_parity(gpu, oracle, M, N, K, p):
    torch, B = gpu
    W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=p, stream=("mma", N, K)), 22, M)
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Y = run_gemm(gpu, X, L, packed, B.VARIANT_MMA)
    Y32, Y16 = oracle.gemm_f64(X, What)
    check_parity(oracle, Y, Y32, f"mma M={M}")
    assert (Y == Y16).mean() > 0.99      # fp32 accumulation: almost every output rounds identically


def test_single_gemm_config(gpu, oracle):
    """X [16 x 1024], W [1024 x 1024], Bernoulli(0.5) tiles: all three call forms agree."""
    torch, B = gpu
    case = inputs.single_gemm_case()
    W, flags, X = inputs.make_case_inputs(case)
    What = oracle.prune(W, flags)
    assert 0 < flags.sum() < flags.size
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Y32, _ = oracle.gemm_f64(X, What)
    for variant in (B.VARIANT_AUTO, B.VARIANT_MMA, B.VARIANT_MMA | B.WEIGHTS_STATIC, B.VARIANT_AUTO | B.WEIGHTS_STATIC):
        check_parity(oracle, run_gemm(gpu, X, L, packed, variant), Y32, "single")
    # strided X and Y (row pitch > row length)
    Xd = torch.zeros((16, 1024 + 64), dtype=torch.bfloat16, device="cuda")
    Xd[:, :1024] = to_dev(torch, X)
    Yd = torch.full((16, 1024 + 8), 7.0, dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(B.patch_gemm_workspace_size(L, 16), dtype=torch.uint8, device="cuda")
    B.patch_gemm(Xd[:, :1024], L, packed, Y=Yd[:, :1024], workspace=ws)
    torch.cuda.synchronize()
    check_parity(oracle, to_bits(Yd[:, :1024]), Y32, "strided")
    assert (Yd[:, 1024:] == 7.0).all()


def test_linearity_and_zero(gpu, oracle):
    torch, B = gpu
    W, flags, X = inputs.make_case_inputs(dict(N=256, K=512, p=0.5, stream=("lin",)), 23, 16)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    for variant, Xv in ((B.VARIANT_MMA, X), (B.VARIANT_GEMV, X[:3])):
        Y1 = run_gemm(gpu, Xv, L, packed, variant)
        X2 = inputs.f32_to_bf16_bits(2.0 * f32(Xv))
        Y2 = run_gemm(gpu, X2, L, packed, variant)
        assert (f32(Y2) == 2.0 * f32(Y1)).all()          # power-of-two scaling is exact
        Y0 = run_gemm(gpu, np.zeros_like(Xv), L, packed, variant)
        assert (f32(Y0) == 0).all()
        assert (run_gemm(gpu, Xv, L, packed, variant) == Y1).all()   # deterministic


def test_m_zero_and_errors(gpu):
    torch, B = gpu
    flags = np.zeros((1, 1), np.uint8)
    W = torch.zeros((128, 128), dtype=torch.bfloat16, device="cuda")
    packed, L = B.patch_pack(W, flags)
    Y = B.patch_gemm(torch.zeros((0, 128), dtype=torch.bfloat16, device="cuda"), L, packed)   # M = 0: nothing runs
    assert Y.shape == (0, 128)
    with pytest.raises(B.PatchError) as e:
        B.patch_gemm(torch.zeros((5, 128), dtype=torch.bfloat16, device="cuda"), L, packed, variant=B.VARIANT_GEMV)
    assert e.value.status == B.ERR_SHAPE
    with pytest.raises(B.PatchError) as e:
        B.patch_pack(W, np.ones((1, 1), np.uint8), layout=L)      # flags disagree with the layout
    assert e.value.status == B.ERR_FORMAT
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.PatchError) as e:
        B.patch_pack(W, flags, out=small)
    assert e.value.status == B.ERR_SIZE


def test_host_buffer_entry_point(gpu, oracle):
    torch, B = gpu
    W, flags, X = inputs.make_case_inputs(dict(N=512, K=384, p=0.5, stream=("host",)), 24, 16)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Xh = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).pin_memory()
    Yh = torch.empty((16, 512), dtype=torch.bfloat16).pin_memory()
    Xs = torch.empty((16, 384), dtype=torch.bfloat16, device="cuda")
    Ys = torch.empty((16, 512), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(B.patch_gemm_workspace_size(L, 16), dtype=torch.uint8, device="cuda")
    B.patch_gemm_host(Xh, L, packed, Yh, Xs, Ys, workspace=ws)
    Y32, _ = oracle.gemm_f64(X, oracle.prune(W, flags))
    check_parity(oracle, Yh.view(torch.int16).numpy().view(np.uint16), Y32, "host entry point")


# ---------------------------------------------------------------------------------------------
# full-size shapes in the launch configuration the benchmark times


@pytest.mark.parametrize("shape", ["attn_qkvo", "mlp_gate_up", "mlp_down"])
@pytest.mark.parametrize("p", [0.35, 1.0])
def test_decode_shapes_full_output(gpu, oracle, shape, p):
    torch, B = gpu
    N, K = inputs.LLAMA2_7B_SHAPES[shape]
    case = dict(N=N, K=K, p=p, stream=("decode", shape, p))
    W = inputs.weight(N, K, inputs.MASTER_SEED, *case["stream"])
    flags = inputs.tile_flags(N, K, p, inputs.MASTER_SEED, *case["stream"])
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    assert (to_bits(B.patch_unpack(L, packed)) == What).all()
    for M in (1, 16):
        X = inputs.activation(M, K, inputs.MASTER_SEED, *case["stream"], M)
        Y32, _ = oracle.gemm_f64(X, What)
        check_parity(oracle, run_gemm(gpu, X, L, packed, B.VARIANT_AUTO), Y32, f"{shape} M={M} auto")
        check_parity(oracle, run_gemm(gpu, X, L, packed, B.VARIANT_MMA | B.WEIGHTS_STATIC), Y32, f"{shape} M={M} mma")
    X = inputs.activation(1, K, inputs.MASTER_SEED, *case["stream"], 1)
    check_parity(oracle, run_gemm(gpu, X, L, packed, B.VARIANT_GEMV), oracle.gemm_f64(X, What)[0], "gemv")


@pytest.mark.parametrize("N,K,M,p", [(4096, 4096, 2048, 0.5), (11008, 4096, 512, 0.5), (4096, 11008, 4096, 1.0),
                                     (5120, 13824, 64, 0.6), (13824, 5120, 8, 0.3)])
def test_prefill_shapes_sampled(gpu, oracle, N, K, M, p):
    """Large M: compare 64 random token rows over all N (first / last rows included) and two whole row-blocks of N
    over all tokens."""
    torch, B = gpu
    stream = ("prefill", N, K, p)
    W = inputs.weight(N, K, inputs.MASTER_SEED, *stream)
    flags = inputs.tile_flags(N, K, p, inputs.MASTER_SEED, *stream)
    X = inputs.activation(M, K, inputs.MASTER_SEED, *stream, M)
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Y = run_gemm(gpu, X, L, packed, B.VARIANT_AUTO)
    rng = inputs.generator(inputs.MASTER_SEED, "rows", N, K, M)
    rows = np.unique(np.concatenate([rng.integers(0, M, 60), [0, M - 1, min(M - 1, 127), min(M - 1, 128)]]))
    Y32 = oracle.gemm_f64_rows(X, rows, What)
    check_parity(oracle, Y[rows], Y32, f"sampled rows N={N} K={K} M={M}")
    # two whole 128-row blocks of N over all tokens: every token tile of the schedule is touched
    for tn in np.unique(rng.integers(0, N // 128, 2)):
        cols = slice(int(tn) * 128, int(tn) * 128 + 128)
        Yb, _ = oracle.gemm_f64(X, What[cols], want_bf16=False)
        check_parity(oracle, Y[:, cols], Yb, f"row-block {tn} N={N} K={K} M={M}")
    # property that holds at any size: doubling X doubles every output exactly
    Y2 = run_gemm(gpu, inputs.f32_to_bf16_bits(2.0 * f32(X)), L, packed, B.VARIANT_AUTO)
    assert (f32(Y2) == 2.0 * f32(Y)).all()


@pytest.mark.parametrize("M", [16, 48, 96, 300])
def test_back_to_back_launches_are_ordered(gpu, oracle, M):
    """A chain of dependent GEMMs on one stream (each launched with programmatic dependent
    launch): Y of one call is X of the next, so early starts must still see finished inputs.
    M = 16 / 48: the two small-M schedules; 96 / 300: the one- and two-row-block prefill kernels."""
    torch, B = gpu
    N = K = 512
    W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=0.5, stream=("chain",)), 25, M)
    W = inputs.f32_to_bf16_bits(f32(W) * 2.0)      # keep magnitudes from collapsing along the chain
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    torch.cuda.synchronize()
    bufs = [to_dev(torch, X)] + [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(6)]
    ws = torch.zeros(max(B.patch_gemm_workspace_size(L, M), 1), dtype=torch.uint8, device="cuda")
    for i in range(6):
        B.patch_gemm(bufs[i], L, packed, Y=bufs[i + 1], workspace=ws, variant=B.VARIANT_MMA | B.WEIGHTS_STATIC)
    torch.cuda.synchronize()
    ref = X
    for i in range(6):
        Y32, Y16 = oracle.gemm_f64(ref, What)
        got = to_bits(bufs[i + 1])
        check_parity(oracle, got, Y32, f"chain step {i}")
        ref = got                                   # feed the GPU's own bf16 output forward


# ---------------------------------------------------------------------------------------------
# the benchmark's workloads, case by case, in the launch configuration bench.py times
# (WEIGHTS_STATIC | INPUT_STATIC, automatic kernel choice); large M: sampled token rows


def _check_case(gpu, oracle, W, flags, X, what, n_rows=16):
    torch, B = gpu
    M = X.shape[0]
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Y = run_gemm(gpu, X, L, packed, B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC)
    if M <= 64:
        Y32, _ = oracle.gemm_f64(X, What)
        check_parity(oracle, Y, Y32, what)
    else:
        # sampled: random token rows, one row out of every 128 tokens (so that every token tile of every schedule,
        # whose tiles are at least 128 tokens wide, has a sampled row), the corners of the usual tile widths ...
        rng = inputs.generator(inputs.MASTER_SEED, "rows", what)
        stride_rows = np.arange(0, M, 128) + rng.integers(0, 128, (M + 127) // 128)
        rows = np.unique(np.concatenate([rng.integers(0, M, n_rows), stride_rows[stride_rows < M],
                                         [0, M - 1, 239, 240, 255, 256, M // 2]]))
        check_parity(oracle, Y[rows], oracle.gemm_f64_rows(X, rows, What), what)
        # ... and two whole row-blocks of out-features over ALL tokens (the last one and a random one)
        N = W.shape[0]
        for tn in {N // 128 - 1, int(rng.integers(0, N // 128))}:
            cols = slice(tn * 128, tn * 128 + 128)
            Yb, _ = oracle.gemm_f64(X, What[cols], want_bf16=False)
            check_parity(oracle, Y[:, cols], Yb, f"{what} row-block {tn}")
    return packed, L


@pytest.fixture(scope="module")
def decode_workload(gpu, oracle):
    """The 24 GEMMs of the decode workload as bench.py sets them up: 12 packed matrices (3 shapes x four 2:4-tile
    fractions), M = 1 and 16, with the oracle's result for each."""
    torch, B = gpu
    cases = sorted(inputs.decode_cases(), key=lambda c: c["M"])
    mats, jobs = {}, []
    for c in cases:
        key = c["stream"]
        if key not in mats:
            W = inputs.weight(c["N"], c["K"], inputs.MASTER_SEED, *c["stream"])
            flags = inputs.case_flags(c)
            packed, L = B.patch_pack(to_dev(torch, W), flags)
            mats[key] = (oracle.prune(W, flags), packed, L)
        What, packed, L = mats[key]
        X = inputs.activation(c["M"], c["K"], inputs.MASTER_SEED, *c["stream"], c["M"])
        Y32, Y16 = oracle.gemm_f64(X, What)
        jobs.append(dict(case=c, L=L, packed=packed, X=to_dev(torch, X), Y32=Y32, Y16=Y16,
                         Y=torch.zeros((c["M"], c["N"]), dtype=torch.bfloat16, device="cuda")))
    ws = torch.zeros(B.patch_gemm_workspace_size(jobs[0]["L"], 64), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    return jobs, ws


def test_decode_workload_all_cases_bench_flags(gpu, oracle, decode_workload):
    """Every one of the 24 decode cases, whole output, launched as the benchmark launches them
    (automatic kernel choice with both promises: the row-block / cluster schedule)."""
    torch, B = gpu
    jobs, ws = decode_workload
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for j in jobs:
        j["Y"].zero_()
        B.patch_gemm(j["X"], j["L"], j["packed"], Y=j["Y"], workspace=ws, status=status,
                     variant=B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got = to_bits(j["Y"])
        check_parity(oracle, got, j["Y32"], j["case"]["name"])
        assert (got == j["Y16"]).mean() >= 0.99, j["case"]["name"]


@pytest.mark.parametrize("mode", ["independent", "independent+output", "dependent"])
def test_decode_workload_graph_replay(gpu, oracle, decode_workload, mode):
    """The regime the headline number is timed in: two consecutive steps of the 24 GEMMs captured into one CUDA
    graph (several kernels resident at once, ordered only by their device-side waits), replayed twice; then
    every one of the 24 outputs is compared with the oracle.  Once with both promises, once with the weights
    promise only (every GEMM waits for its predecessor before reading X)."""
    torch, B = gpu
    jobs, ws = decode_workload
    flags = B.WEIGHTS_STATIC | {"independent": B.INPUT_STATIC, "independent+output": B.INPUT_STATIC | B.OUTPUT_STATIC,
                                "dependent": 0}[mode]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # with the output promise every launch between two drains writes a buffer of its own (bench.py does the
    # same): the second step of the graph gets a second set of outputs
    first = [j["Y"] for j in jobs]
    second = [torch.zeros_like(j["Y"]) for j in jobs]

    def step(outs):
        for j, Y in zip(jobs, outs):
            B.patch_gemm(j["X"], j["L"], j["packed"], Y=Y, workspace=ws, status=status, variant=B.VARIANT_AUTO | flags)
    step(first)                              # kernel attributes are set outside the capture
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step(first)
        step(second)
    for Y in first + second:
        Y.zero_()
    torch.cuda.synchronize()
    g.replay()
    g.replay()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for outs in (first, second):
        for j, Y in zip(jobs, outs):
            got = to_bits(Y)
            check_parity(oracle, got, j["Y32"], f"{j['case']['name']} ({mode}, graph)")
            assert (got == j["Y16"]).mean() >= 0.99, j["case"]["name"]


_PREFILL = [(s, p) for s in inputs.LLAMA2_7B_SHAPES for p in (0.0, 0.5, 1.0)]


@pytest.mark.parametrize("shape,p", _PREFILL)
def test_prefill_workload_cases(gpu, oracle, shape, p):
    N, K = inputs.LLAMA2_7B_SHAPES[shape]
    stream = ("prefill", shape, p)
    W = inputs.weight(N, K, inputs.MASTER_SEED, *stream)
    flags = inputs.tile_flags(N, K, p, inputs.MASTER_SEED, *stream)
    for M in (512, 2048, 4096):
        X = inputs.activation(M, K, inputs.MASTER_SEED, *stream, M)
        _check_case(gpu, oracle, W, flags, X, f"7b.{shape}.p{p}.M{M}")


@pytest.mark.parametrize("shape", list(inputs.LLAMA2_13B_SHAPES))
def test_13b_workload_cases(gpu, oracle, shape):
    cases = [c for c in inputs.llama13b_cases() if c["stream"][1] == shape]
    N, K, p = cases[0]["N"], cases[0]["K"], cases[0]["p"]
    W = inputs.weight(N, K, inputs.MASTER_SEED, *cases[0]["stream"])
    flags = inputs.tile_flags(N, K, p, inputs.MASTER_SEED, *cases[0]["stream"])
    assert 0 < flags.mean() < 1
    for c in cases:                                   # M in {1, 8, 64, 512, 4096}
        X = inputs.activation(c["M"], K, inputs.MASTER_SEED, *c["stream"], c["M"])
        _check_case(gpu, oracle, W, flags, X, c["name"])


def test_stack_workload_sample(gpu, oracle):
    """Four matrices of the 224-matrix stack (per-matrix tile fraction ~ U[0,1]) at M = 1 and M = 2048,
    with weights drawn on the device as the benchmark does and copied back for the oracle."""
    torch, B = gpu
    cases = inputs.stack_cases()
    for idx in (0, 5, 118, 223):
        c = cases[idx]
        gen = torch.Generator(device="cuda")
        gen.manual_seed(inputs.MASTER_SEED * 1000 + idx)
        Wd = torch.empty((c["N"], c["K"]), dtype=torch.bfloat16, device="cuda").normal_(0.0, 0.02, generator=gen)
        W = to_bits(Wd)
        flags = inputs.tile_flags(c["N"], c["K"], c["p"], inputs.MASTER_SEED, *c["stream"])
        for M in (1, 2048):
            X = inputs.activation(M, c["K"], inputs.MASTER_SEED, *c["stream"], M)
            _check_case(gpu, oracle, W, flags, X, f"{c['name']}.M{M}", n_rows=8)


def test_stacked_matrices_sample(gpu, oracle):
    """q/k/v and gate/up stored as one matrix each (N = 12288, 22016): the stacked flags are the parts'
    flags, and the GEMM over the stacked weight is checked at M = 1 (whole output) and M = 2048 (sampled rows)."""
    torch, B = gpu
    cases = inputs.stack_fused_cases(n_blocks=2)
    for idx in (0, 6):                                  # block 0 qkv, block 1 gate_up
        c = cases[idx]
        flags = inputs.case_flags(c)
        assert flags.shape == (c["N"] // 128, c["K"] // 128)
        row = 0
        for part in c["parts"]:                         # every part keeps its own matrix's flags
            ref = inputs.tile_flags(part["N"], c["K"], part["p"], inputs.MASTER_SEED, *part["stream"])
            assert np.array_equal(flags[row:row + part["N"] // 128], ref)
            row += part["N"] // 128
        gen = torch.Generator(device="cuda")
        gen.manual_seed(inputs.MASTER_SEED * 1000 + idx)
        Wd = torch.empty((c["N"], c["K"]), dtype=torch.bfloat16, device="cuda").normal_(0.0, 0.02, generator=gen)
        W = to_bits(Wd)
        for M in (1, 2048):
            X = inputs.activation(M, c["K"], inputs.MASTER_SEED, *c["stream"], M)
            _check_case(gpu, oracle, W, flags, X, f"{c['name']}.M{M}", n_rows=8)


def test_workspace_is_shared_across_token_counts_and_layouts(gpu, oracle):
    """One workspace, zeroed once, serves calls of every M <= 64 on two layouts of different N in any
    order: the 32/64-token schedule's partial tiles never reach the 16-token schedule's flag words."""
    torch, B = gpu
    mats = []
    for N, K in ((1792, 1280), (4224, 768)):
        W, flags, _ = inputs.make_case_inputs(dict(N=N, K=K, p=0.4, stream=("ws", N, K)), 31, 1)
        packed, L = B.patch_pack(to_dev(torch, W), flags)
        mats.append((N, K, oracle.prune(W, flags), packed, L))
    ws = torch.zeros(max(B.patch_gemm_workspace_size(m[4], 64) for m in mats), dtype=torch.uint8, device="cuda")
    flagged_end = B.patch_gemm_workspace_size(mats[0][4], 16)     # counters + flag words: same offsets for both
    assert flagged_end == B.patch_gemm_workspace_size(mats[1][4], 16)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for i, M in enumerate((48, 8, 64, 16, 33, 1, 17, 5, 64, 2)):
        N, K, What, packed, L = mats[i % 2]
        X = inputs.activation(M, K, 31, "ws", M, i)
        for variant in (B.VARIANT_AUTO, B.VARIANT_MMA | B.WEIGHTS_STATIC | B.INPUT_STATIC):
            Y = B.patch_gemm(to_dev(torch, X), L, packed, workspace=ws, status=status, variant=variant)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            assert int(ws[:flagged_end].count_nonzero()) == 0, f"counters / flag words not clean after M={M}"
            check_parity(oracle, to_bits(Y), oracle.gemm_f64(X, What)[0], f"shared workspace N={N} M={M}")


def test_random_shapes_and_pitches(gpu, oracle):
    """Seeded random (N, K, M, tile fraction, row pitches of X and Y): every schedule, ragged token counts,
    outputs beyond column N untouched."""
    torch, B = gpu
    rng = inputs.generator(inputs.MASTER_SEED, "fuzz")
    Ms = [1, 3, 4, 15, 16, 17, 33, 63, 64, 65, 100, 128, 129, 239, 240, 241, 300]
    for it in range(24):
        TN, TK = int(rng.integers(1, 14)), int(rng.integers(1, 14))
        N, K, M = 128 * TN, 128 * TK, Ms[int(rng.integers(0, len(Ms)))]
        p = [0.0, 1.0, 0.5, float(rng.random())][int(rng.integers(0, 4))]
        padx, pady = int(rng.choice([0, 8, 200])), int(rng.choice([0, 8, 200]))
        W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=p, stream=("fuzz", it)), inputs.MASTER_SEED, M)
        What = oracle.prune(W, flags)
        Y32 = oracle.gemm_f64(X, What)[0]
        packed, L = B.patch_pack(to_dev(torch, W), flags)
        Xfull = torch.zeros((M, K + padx), dtype=torch.bfloat16, device="cuda")
        Xfull[:, :K] = to_dev(torch, X)
        Yfull = torch.full((M, N + pady), 7.0, dtype=torch.bfloat16, device="cuda")
        ws = torch.zeros(max(B.patch_gemm_workspace_size(L, M), 1), dtype=torch.uint8, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        variants = [B.VARIANT_AUTO, B.VARIANT_MMA | B.WEIGHTS_STATIC | B.INPUT_STATIC] + ([B.VARIANT_GEMV] if M <= 4 else [])
        for variant in variants:
            Yfull.fill_(7.0)
            B.patch_gemm(Xfull[:, :K], L, packed, Y=Yfull[:, :N], workspace=ws, status=status, variant=variant)
            torch.cuda.synchronize()
            what = f"N={N} K={K} M={M} p={p:.2f} pitches +{padx}/+{pady} variant={variant:#x}"
            assert int(status.item()) == 0, what
            assert pady == 0 or bool((Yfull[:, N:] == 7.0).all()), what + ": wrote past column N"
            check_parity(oracle, to_bits(Yfull[:, :N]), Y32, what)


# ---------------------------------------------------------------------------------------------
# gated gate/up product (stacked weight with interleaved row-blocks)


def _gated_case(gpu, oracle, Nh, K, M, pg, pu, rows=None, ws=None, flags_arg=0):
    torch, B = gpu
    Wg = inputs.weight(Nh, K, inputs.MASTER_SEED, "gated", "g", Nh, K)
    Wu = inputs.weight(Nh, K, inputs.MASTER_SEED, "gated", "u", Nh, K)
    Wg = inputs.f32_to_bf16_bits(f32(Wg) * 40.0)      # gate pre-activations of order 1: both tails of silu matter
    fg = inputs.tile_flags(Nh, K, pg, inputs.MASTER_SEED, "gated", "g", Nh, K)
    fu = inputs.tile_flags(Nh, K, pu, inputs.MASTER_SEED, "gated", "u", Nh, K)
    W = B.interleave_row_blocks(Wg, Wu)
    flags = B.interleave_row_blocks(fg, fu, block=1)
    X = inputs.activation(M, K, inputs.MASTER_SEED, "gated", M)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if ws == "own":
        ws = torch.zeros(max(B.patch_gemm_gated_workspace_size(L, M), 1), dtype=torch.uint8, device="cuda")
    Y = B.patch_gemm_gated(to_dev(torch, X), L, packed, workspace=ws, status=status, flags=flags_arg)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and tuple(Y.shape) == (M, Nh)
    if ws is not None:
        assert int(ws.count_nonzero()) == 0, "gate words not left empty"
    What = oracle.prune(W, flags)
    if rows is None:
        ref = oracle.swiglu(oracle.gemm_f64(X, What)[0])
        check_parity(oracle, to_bits(Y), ref, f"gated Nh={Nh} K={K} M={M}")
    else:
        ref = oracle.swiglu(oracle.gemm_f64_rows(X, rows, What))
        check_parity(oracle, to_bits(Y)[rows], ref, f"gated Nh={Nh} K={K} M={M} (sampled rows)")


@pytest.mark.parametrize("M", [1, 16, 100, 300, 513])
@pytest.mark.parametrize("pg,pu", [(0.0, 0.0), (1.0, 1.0), (0.3, 0.8)])
def test_gated_product_parity(gpu, oracle, M, pg, pu):
    _gated_case(gpu, oracle, 1024, 768, M, pg, pu)


def test_gated_product_llama_mlp_shape(gpu, oracle):
    M = 2048
    rows = np.array([0, 1, 239, 240, 1023, 1024, 2047])
    _gated_case(gpu, oracle, 11008, 4096, M, 0.6, 0.9, rows=rows)


def test_gated_product_rejects_bad_shapes(gpu):
    torch, B = gpu
    W = inputs.weight(384, 256, 3, "gated-bad")                   # three row-blocks: no whole pairs
    packed, L = B.patch_pack(to_dev(torch, W), np.zeros((3, 2), np.uint8))
    X = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.PatchError):
        B.patch_gemm_gated(X, L, packed)


@pytest.mark.parametrize("M", [1, 5, 16])
@pytest.mark.parametrize("shape", [(1024, 768), (1408, 4096), (11008, 4096)])
def test_gated_product_small_m_schedule(gpu, oracle, M, shape):
    """M <= 16: without a promise and with a workspace the stream-K schedule, where the gate and up row-blocks of a
    pair are usually finished by different CTAs; with the weights promise a cluster per (gate, up) pair of
    row-blocks (workspace ignored or absent); every launch-flag combination."""
    torch, B = gpu
    Nh, K = shape
    for flags_arg in (0, B.WEIGHTS_STATIC, B.WEIGHTS_STATIC | B.INPUT_STATIC):
        _gated_case(gpu, oracle, Nh, K, M, 0.3, 0.8, ws="own", flags_arg=flags_arg)
    # weights static: a cluster per (gate, up) pair of row-blocks, no workspace needed
    _gated_case(gpu, oracle, Nh, K, M, 0.3, 0.8, ws=None, flags_arg=B.WEIGHTS_STATIC)
    _gated_case(gpu, oracle, Nh, K, M, 0.3, 0.8, ws=None, flags_arg=B.WEIGHTS_STATIC | B.INPUT_STATIC)
    _gated_case(gpu, oracle, Nh, K, M, 1.0, 0.0, ws=None, flags_arg=B.WEIGHTS_STATIC | B.INPUT_STATIC)


@pytest.mark.parametrize("M,shape", [(M, s) for M in (17, 32, 33, 48, 64) for s in ((256, 128), (1024, 768), (1408, 4096))] +
                         [(33, (11008, 4096))])
def test_gated_product_17_to_64_tokens(gpu, oracle, M, shape):
    """17 to 64 tokens: the schedule whose CTA holds the gate and the up accumulator of a pair of row-blocks, under
    every combination of launch promises, on weights from one pair of row-blocks to the LLaMA MLP shape."""
    torch, B = gpu
    Nh, K = shape
    for flags_arg in (0, B.WEIGHTS_STATIC, B.WEIGHTS_STATIC | B.INPUT_STATIC):
        _gated_case(gpu, oracle, Nh, K, M, 0.3, 0.8, ws=None, flags_arg=flags_arg)
    _gated_case(gpu, oracle, Nh, K, M, 1.0, 0.0, ws=None, flags_arg=B.WEIGHTS_STATIC | B.INPUT_STATIC)
    _gated_case(gpu, oracle, Nh, K, M, 0.0, 1.0, ws=None, flags_arg=B.WEIGHTS_STATIC)


def test_gated_and_plain_calls_share_a_workspace(gpu, oracle):
    """The gate words live past everything patch_gemm uses of a workspace: plain calls of any M <= 64
    and gated calls may alternate on one buffer."""
    torch, B = gpu
    Nh, K = 1024, 768
    Wp = inputs.weight(2 * Nh, K, inputs.MASTER_SEED, "gated", "plain")
    fp = inputs.tile_flags(2 * Nh, K, 0.5, inputs.MASTER_SEED, "gated", "plain")
    packed_p, Lp = B.patch_pack(to_dev(torch, Wp), fp)
    What_p = oracle.prune(Wp, fp)
    ws = torch.zeros(B.patch_gemm_gated_workspace_size(Lp, 16), dtype=torch.uint8, device="cuda")
    assert ws.numel() >= B.patch_gemm_workspace_size(Lp, 64)
    for M in (48, 8, 64, 3):
        X = inputs.activation(M, K, inputs.MASTER_SEED, "gated", "plain", M)
        Y = B.patch_gemm(to_dev(torch, X), Lp, packed_p, workspace=ws)
        torch.cuda.synchronize()
        check_parity(oracle, to_bits(Y), oracle.gemm_f64(X, What_p)[0], f"plain M={M} on the shared workspace")
        ws_gate = ws[B.patch_gemm_workspace_size(Lp, 64):]
        assert int(ws_gate.count_nonzero()) == 0
        for Mg in (16, 2):
            Wg = inputs.weight(Nh, K, inputs.MASTER_SEED, "gated", "g", Nh, K)
            Wu = inputs.weight(Nh, K, inputs.MASTER_SEED, "gated", "u", Nh, K)
            fg = inputs.tile_flags(Nh, K, 0.3, inputs.MASTER_SEED, "gated", "g", Nh, K)
            fu = inputs.tile_flags(Nh, K, 0.8, inputs.MASTER_SEED, "gated", "u", Nh, K)
            W = B.interleave_row_blocks(inputs.f32_to_bf16_bits(f32(Wg) * 40.0), Wu)
            flags = B.interleave_row_blocks(fg, fu, block=1)
            packed, L = B.patch_pack(to_dev(torch, W), flags)
            Xg = inputs.activation(Mg, K, inputs.MASTER_SEED, "gated", Mg)
            Yg = B.patch_gemm_gated(to_dev(torch, Xg), L, packed, workspace=ws)
            torch.cuda.synchronize()
            ref = oracle.swiglu(oracle.gemm_f64(Xg, oracle.prune(W, flags))[0])
            check_parity(oracle, to_bits(Yg), ref, f"gated M={Mg} after plain M={M}")
            assert int(ws_gate.count_nonzero()) == 0


def test_host_batch_entry_point(gpu, oracle):
    """patch_gemm_host_batch: a step of GEMMs of mixed sizes with pinned host X / Y, one synchronisation."""
    torch, B = gpu
    jobs, refs = [], []
    for i, (N, K, M, p) in enumerate([(1024, 768, 1, 0.5), (1792, 1280, 16, 0.3), (512, 2048, 48, 1.0), (768, 512, 300, 0.0)]):
        W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=p, stream=("batch", i)), 51, M)
        packed, L = B.patch_pack(to_dev(torch, W), flags)
        Xh = torch.from_numpy(np.ascontiguousarray(X).view(np.int16)).view(torch.bfloat16).pin_memory()
        Yh = torch.zeros((M, N), dtype=torch.bfloat16).pin_memory()
        ws = torch.zeros(max(B.patch_gemm_workspace_size(L, M), 1), dtype=torch.uint8, device="cuda")
        jobs.append(dict(Xh=Xh, layout=L, packed=packed, Yh=Yh, X=torch.empty((M, K), dtype=torch.bfloat16, device="cuda"),
                         Y=torch.empty((M, N), dtype=torch.bfloat16, device="cuda"), ws=ws))
        refs.append(oracle.gemm_f64(X, oracle.prune(W, flags))[0])
    batch = B.make_host_batch(jobs)
    for weights_static in (False, True):
        for j in jobs:
            j["Yh"].zero_()
        B.patch_gemm_host_batch(batch, weights_static=weights_static)      # returns after the stream is synchronised
        for j, ref in zip(jobs, refs):
            check_parity(oracle, j["Yh"].view(torch.int16).numpy().view(np.uint16), ref, "host batch")


def test_host_batch_merges_adjacent_buffers(gpu, oracle):
    """Jobs whose host and staging buffers are adjacent (one arena each) are copied in one transfer; a job in
    between with separate buffers breaks the run.  Results must not depend on how the copies were grouped."""
    torch, B = gpu
    shapes = [(1024, 768, 4, 0.5), (512, 768, 16, 1.0), (768, 512, 7, 0.0), (640, 1024, 2, 0.4), (256, 256, 33, 0.6)]
    cases = []
    for i, (N, K, M, p) in enumerate(shapes):
        W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=p, stream=("arena", i)), 52, M)
        packed, L = B.patch_pack(to_dev(torch, W), flags)
        cases.append((N, K, M, X, L, packed, oracle.gemm_f64(X, oracle.prune(W, flags))[0]))
    nx, ny = sum(M * K for N, K, M, *_ in cases), sum(M * N for N, K, M, *_ in cases)
    xh, yh = torch.empty(nx, dtype=torch.bfloat16).pin_memory(), torch.zeros(ny, dtype=torch.bfloat16).pin_memory()
    xd, yd = torch.empty(nx, dtype=torch.bfloat16, device="cuda"), torch.empty(ny, dtype=torch.bfloat16, device="cuda")
    jobs, ox, oy = [], 0, 0
    for i, (N, K, M, X, L, packed, ref) in enumerate(cases):
        ws = torch.zeros(max(B.patch_gemm_workspace_size(L, M), 1), dtype=torch.uint8, device="cuda")
        j = dict(layout=L, packed=packed, ws=ws, Xh=xh[ox:ox + M * K].view(M, K), Yh=yh[oy:oy + M * N].view(M, N),
                 X=xd[ox:ox + M * K].view(M, K), Y=yd[oy:oy + M * N].view(M, N))
        if i == 2:      # separate buffers in the middle of the arena run
            j.update(Xh=torch.empty((M, K), dtype=torch.bfloat16).pin_memory(), Yh=torch.zeros((M, N), dtype=torch.bfloat16).pin_memory(),
                     X=torch.empty((M, K), dtype=torch.bfloat16, device="cuda"), Y=torch.empty((M, N), dtype=torch.bfloat16, device="cuda"))
        j["Xh"].copy_(torch.from_numpy(np.ascontiguousarray(X).view(np.int16)).view(torch.bfloat16))
        jobs.append(j)
        ox, oy = ox + M * K, oy + M * N
    batch = B.make_host_batch(jobs)
    B.patch_gemm_host_batch(batch, weights_static=True)
    for j, c in zip(jobs, cases):
        check_parity(oracle, j["Yh"].contiguous().view(torch.int16).numpy().view(np.uint16), c[6], "arena batch")
    # the pipelined form: copies in, GEMMs and copies out on three streams, any number of chunks
    first = [j["Yh"].clone() for j in jobs]
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    for n_chunks in (1, 2, 3, 5, 64):
        for j in jobs:
            j["Yh"].zero_()
        B.patch_gemm_host_batch_pipelined(batch, s_in, s_out, n_chunks=n_chunks, weights_static=True)
        for j, f in zip(jobs, first):
            assert torch.equal(j["Yh"], f), n_chunks          # the kernels are deterministic: same bits
    lib = B.lib()
    cur = torch.cuda.current_stream().cuda_stream
    assert lib.patch_gemm_host_batch_pipelined(batch, len(batch), 1, 2, cur, cur, s_out.cuda_stream) == B.ERR_SHAPE
    assert lib.patch_gemm_host_batch_pipelined(batch, len(batch), 1, 0, cur, s_in.cuda_stream, s_out.cuda_stream) == B.ERR_SHAPE


# ---------------------------------------------------------------------------------------------
# the schedule for GEMMs declared independent of their predecessor (one CTA per row-block, or a
# small cluster splitting K where the weight has few row-blocks)


@pytest.mark.parametrize("N,K", [(128, 128), (128, 256), (256, 1024), (512, 2304), (1024, 1024), (2048, 640), (4224, 1152)])
@pytest.mark.parametrize("M", [1, 5, 16, 17, 33, 64])
def test_independent_launch_schedule(gpu, oracle, N, K, M):
    """Row-block counts 1 .. 33: cluster sizes 8, 4, 2 and 1 (capped by the number of K tiles), all token tiles."""
    torch, B = gpu
    p = [0.0, 0.5, 1.0][(N // 128 + K // 128 + M) % 3]
    W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=p, stream=("indep", N, K)), 61, M)
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Y32, _ = oracle.gemm_f64(X, What)
    got = run_gemm(gpu, X, L, packed, B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC)
    check_parity(oracle, got, Y32, f"independent N={N} K={K} M={M} p={p}")
    # the stream-K schedule (no promise) rounds the same sums: both are deterministic, and close
    other = run_gemm(gpu, X, L, packed, B.VARIANT_AUTO)
    check_parity(oracle, other, Y32, "stream-K")
    again = run_gemm(gpu, X, L, packed, B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC)
    assert (again == got).all()
    # with the output promise too (only the launch's first cluster waits for its predecessor): the same bits
    out = run_gemm(gpu, X, L, packed, B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC | B.OUTPUT_STATIC)
    assert (out == got).all()


def test_independent_launches_back_to_back(gpu, oracle):
    """A stream of independent GEMMs of different shapes and token counts, launched without any
    synchronisation in between (several kernels are resident at once), twice over the same outputs."""
    torch, B = gpu
    shapes = [(1024, 768, 1), (4096, 512, 16), (256, 2048, 40), (2304, 1024, 3), (512, 512, 64), (1536, 1280, 9)]
    jobs = []
    for i, (N, K, M) in enumerate(shapes):
        W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=0.5, stream=("indep-b2b", i)), 62, M)
        packed, L = B.patch_pack(to_dev(torch, W), flags)
        jobs.append(dict(X=to_dev(torch, X), L=L, packed=packed, Y=torch.zeros((M, N), dtype=torch.bfloat16, device="cuda"),
                         ref=oracle.gemm_f64(X, oracle.prune(W, flags))[0]))
    ws = torch.zeros(B.patch_gemm_workspace_size(jobs[0]["L"], 64), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for rep in range(3):
        for j in jobs:
            B.patch_gemm(j["X"], j["L"], j["packed"], Y=j["Y"], workspace=ws, status=status,
                         variant=B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC)
        # a dependent GEMM in the middle of the stream (stream-K schedule, same workspace)
        B.patch_gemm(jobs[0]["X"], jobs[0]["L"], jobs[0]["packed"], Y=jobs[0]["Y"], workspace=ws, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for j in jobs:
        check_parity(oracle, to_bits(j["Y"]), j["ref"], "independent stream")
    # the same stream under the output promise: every launch between two synchronisations writes a buffer of its own
    outs = [[torch.zeros_like(j["Y"]) for j in jobs] for _ in range(3)]
    for rep in range(3):
        for j, Y in zip(jobs, outs[rep]):
            B.patch_gemm(j["X"], j["L"], j["packed"], Y=Y, workspace=ws, status=status,
                         variant=B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC | B.OUTPUT_STATIC)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for rep in range(3):
        for j, Y in zip(jobs, outs[rep]):
            assert (to_bits(Y) == to_bits(j["Y"])).all()


@pytest.mark.parametrize("M", [4, 48, 300])
def test_promises_are_bounded_by_other_operations(gpu, oracle, M):
    """A GEMM launched with both promises behind an operation that is not one of the library's GEMMs
    (here: the copy that produces its X) must see that operation's result: the overlap window ends there.
    Five rounds without any synchronisation, each with a different X in the same buffer."""
    torch, B = gpu
    N, K = 1024, 768
    W, flags, _ = inputs.make_case_inputs(dict(N=N, K=K, p=0.5, stream=("window",)), 63, M)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    What = oracle.prune(W, flags)
    Xs = [inputs.activation(M, K, 63, "window", M, i) for i in range(5)]
    Xd = [to_dev(torch, x) for x in Xs]
    Xbuf = torch.zeros((M, K), dtype=torch.bfloat16, device="cuda")
    Ys = [torch.zeros((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(5)]
    ws = torch.zeros(max(B.patch_gemm_workspace_size(L, M), 1), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    for i in range(5):
        Xbuf.copy_(Xd[i])                                        # not a library GEMM: fully ordered
        B.patch_gemm(Xbuf, L, packed, Y=Ys[i], workspace=ws, variant=B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC)
    torch.cuda.synchronize()
    for i in range(5):
        if M <= 64:
            ref = oracle.gemm_f64(Xs[i], What)[0]
            check_parity(oracle, to_bits(Ys[i]), ref, f"window round {i}")
        else:
            rows = np.array([0, 1, M // 2, M - 1])
            check_parity(oracle, to_bits(Ys[i])[rows], oracle.gemm_f64_rows(Xs[i], rows, What), f"window round {i}")


@pytest.mark.parametrize("M", [1, 16, 40, 300])
def test_decoder_block_chain(gpu, oracle, M):
    """The chain `bench.py --workload block` times, on small matrices and without any synchronisation, three blocks
    deep: a stacked q/k/v GEMM with both promises (its X is written by no GEMM), then o on the v slice of that output
    (row pitch 3 d), the gated gate/up product on o's output and down on the gated product, each with the weights
    promise only because it reads what the launch before it wrote.  Every intermediate is checked against the oracle
    fed with the GPU's own bf16 output of the step before."""
    torch, B = gpu
    d, dff = 512, 1024
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.zeros(B.patch_gemm_workspace_size(B.patch_packed_size(3 * d, d, np.zeros((12, 4), np.uint8)), 64),
                     dtype=torch.uint8, device="cuda")
    blocks = []
    for b in range(3):
        mats = {}
        for role, N, K, scale in (("qkv", 3 * d, d, 2.0), ("o", d, d, 2.0), ("gate", dff, d, 40.0), ("up", dff, d, 2.0),
                                  ("down", d, dff, 2.0)):
            W = inputs.f32_to_bf16_bits(f32(inputs.weight(N, K, inputs.MASTER_SEED, "block", b, role)) * scale)
            mats[role] = (W, inputs.tile_flags(N, K, 0.5, inputs.MASTER_SEED, "block", b, role))
        Wgu = B.interleave_row_blocks(mats["gate"][0], mats["up"][0])
        fgu = B.interleave_row_blocks(mats["gate"][1], mats["up"][1], block=1)
        packed = {}
        for role, (W, fl) in (("qkv", mats["qkv"]), ("o", mats["o"]), ("mlp", (Wgu, fgu)), ("down", mats["down"])):
            blob, L = B.patch_pack(to_dev(torch, W), fl)
            packed[role] = (blob, L, oracle.prune(W, fl))
        gws = torch.zeros(max(B.patch_gemm_gated_workspace_size(packed["mlp"][1], M), 256), dtype=torch.uint8, device="cuda")
        X = inputs.activation(M, d, inputs.MASTER_SEED, "block", b, M)
        blocks.append(dict(packed=packed, gws=gws, X=X, Xd=to_dev(torch, X),
                           qkv=torch.zeros((M, 3 * d), dtype=torch.bfloat16, device="cuda"),
                           o=torch.zeros((M, d), dtype=torch.bfloat16, device="cuda"),
                           mlp=torch.zeros((M, dff), dtype=torch.bfloat16, device="cuda"),
                           down=torch.zeros((M, d), dtype=torch.bfloat16, device="cuda")))
    torch.cuda.synchronize()
    both, weights_only = B.WEIGHTS_STATIC | B.INPUT_STATIC, B.WEIGHTS_STATIC
    for blk in blocks:
        p = blk["packed"]
        B.patch_gemm(blk["Xd"], p["qkv"][1], p["qkv"][0], Y=blk["qkv"], workspace=ws, status=status, variant=both)
        B.patch_gemm(blk["qkv"][:, 2 * d:], p["o"][1], p["o"][0], Y=blk["o"], workspace=ws, status=status, variant=weights_only)
        B.patch_gemm_gated(blk["o"], p["mlp"][1], p["mlp"][0], Y=blk["mlp"], workspace=blk["gws"], status=status, flags=weights_only)
        B.patch_gemm(blk["mlp"], p["down"][1], p["down"][0], Y=blk["down"], workspace=ws, status=status, variant=weights_only)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for b, blk in enumerate(blocks):
        p = blk["packed"]
        qkv = to_bits(blk["qkv"])
        check_parity(oracle, qkv, oracle.gemm_f64(blk["X"], p["qkv"][2])[0], f"block {b} qkv")
        o = to_bits(blk["o"])
        check_parity(oracle, o, oracle.gemm_f64(np.ascontiguousarray(qkv[:, 2 * d:]), p["o"][2])[0], f"block {b} o")
        mlp = to_bits(blk["mlp"])
        check_parity(oracle, mlp, oracle.swiglu(oracle.gemm_f64(o, p["mlp"][2])[0]), f"block {b} mlp")
        check_parity(oracle, to_bits(blk["down"]), oracle.gemm_f64(mlp, p["down"][2])[0], f"block {b} down")
