"""GPU parity of the 4-bit tile kinds (2: dense, 3: 2:4, stored values as 4-bit codes with one bf16 scale per tile
row) against the CPU oracle: the packed blob bit for bit, the dequantised matrix bit for bit, and the small-M matmul
on a weight made of such tiles."""
import numpy as np
import pytest

from paper_2509_23410_b200 import inputs
from test_gpu_parity import check_parity, f32, gpu, run_gemm, to_bits, to_dev  # noqa: F401  (gpu is a fixture)

pytestmark = pytest.mark.gpu


def _flags4(N, K, p, seed_tag, q4="all"):
    """Tile kinds: bit 0 drawn with probability p; bit 1 set everywhere ("all") or on a random half ("half")."""
    flags = inputs.tile_flags(N, K, p, inputs.MASTER_SEED, "q4", seed_tag)
    if q4 == "all":
        return flags | 2
    g = inputs.generator(inputs.MASTER_SEED, "q4-bit1", seed_tag, N, K)
    return flags | (2 * (g.random(flags.shape) < 0.5)).astype(np.uint8)


@pytest.mark.parametrize("q4", ["all", "half"])
@pytest.mark.parametrize("p", [0.0, 1.0, 0.45])
@pytest.mark.parametrize("N,K", [(128, 128), (384, 640), (1024, 512)])
def test_pack_bit_exact_and_unpack(gpu, oracle, N, K, p, q4):
    torch, B = gpu
    W = inputs.weight(N, K, 31, "q4-pack", N, K)
    W[::13, ::7] = 0                      # exact zeros and ties in the 2:4 selection
    W[5, :] = 0                           # a row of zeros: scale 0, every code 8
    W[7, 128 * (K // 128 - 1):] = inputs.f32_to_bf16_bits(np.float32(0.0371))   # a constant row: every |q| = 7
    flags = _flags4(N, K, p, (N, K, p), q4)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    blob_o, L_o = oracle.pack(W, flags)
    for f, _ in B.Layout._fields_:
        assert getattr(L, f) == getattr(L_o, f), f
    image = oracle.device_image(blob_o)
    got = packed.cpu().numpy()
    assert got.shape == image.shape
    bad = np.flatnonzero(got != image)
    assert bad.size == 0, f"{bad.size} bytes differ, first at {bad[:8]}"
    # the dequantised matrix: what the layer multiplies by
    What = to_bits(B.patch_unpack(L, packed))
    assert (What == oracle.prune(W, flags)).all()
    assert (What == oracle.unpack(blob_o)).all()


def test_pack_with_row_pitch_and_extreme_values(gpu, oracle):
    """Row pitch > K; magnitudes spanning many binades, so that scales and quotients take many exponents."""
    torch, B = gpu
    N, K, ld = 256, 384, 448
    g = inputs.generator(32, "q4-extreme")
    vals = (g.standard_normal((N, K)) * np.exp2(g.integers(-20, 20, (N, 1)))).astype(np.float32)
    W = inputs.f32_to_bf16_bits(vals)
    flags = _flags4(N, K, 0.5, "pitch")
    Wd = torch.zeros((N, ld), dtype=torch.bfloat16, device="cuda")
    Wd[:, :K] = to_dev(torch, W)
    packed, L = B.patch_pack(Wd[:, :K], flags)
    image = oracle.device_image(oracle.pack(W, flags)[0])
    assert (packed.cpu().numpy() == image).all()
    out = torch.full((N, ld), 7.0, dtype=torch.bfloat16, device="cuda")
    B.patch_unpack(L, packed, out=out[:, :K])
    assert (to_bits(out[:, :K]) == oracle.prune(W, flags)).all()
    assert (out[:, K:] == 7.0).all()


@pytest.mark.parametrize("kind", [2, 3])
def test_pack_quantiser_corner_cases(gpu, oracle, kind):
    """Rows built to sit on the quantiser's decision points: quotients that are exact half-integers (ties go to the
    even code), quotients one bf16 step to either side of a half-integer, scales that are subnormal, zero or near
    the top of the range, and a row whose largest magnitude makes max / 7 round up in bf16."""
    torch, B = gpu
    N, K = 256, 256
    g = inputs.generator(35, "q4-corners", kind)
    vals = np.zeros((N, K), np.float32)
    halves = np.arange(-7, 7, dtype=np.float32) + 0.5                      # -6.5 .. 6.5
    for r in range(N):
        e = [-3, 0, 5, -60, 40, -126, 100][r % 7]
        s = np.float32(2.0) ** e                                           # a scale that max / 7 hits exactly
        row = g.choice(halves, K) * s
        if r % 3 == 1:                                                     # one bf16 step off the tie, either side
            bits = inputs.f32_to_bf16_bits(row).astype(np.int32) + g.choice([-1, 1], K)
            row = (bits.astype(np.uint32) << 16).view(np.float32)
        row[g.integers(0, K, 8)] = 7 * s * g.choice([-1, 1], 8)             # the row maximum, in both tiles
        row[:4], row[128:132] = 7 * s, -7 * s
        vals[r] = row
    W = inputs.f32_to_bf16_bits(vals)
    W[3, :] = 0                                                            # scale 0
    W[4, :] = np.tile(np.arange(1, 65, dtype=np.uint16), 4)                # subnormal values, subnormal scale
    W[5, :] = np.tile(np.arange(0x0080, 0x00C0, dtype=np.uint16), 4)       # smallest normal values
    W[6, :] = np.tile(np.arange(0x7F00, 0x7F40, dtype=np.uint16), 4)       # near the largest finite bf16
    W[7, :] = np.tile(np.array([0x3F80, 0x3E12, 0xBE13, 0x3D55], np.uint16), 64)   # max / 7 = 0.142857: rounds in bf16
    flags = np.full((N // 128) * (K // 128), kind, np.uint8)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    blob_o, _ = oracle.pack(W, flags)
    image = oracle.device_image(blob_o)
    bad = np.flatnonzero(packed.cpu().numpy() != image)
    assert bad.size == 0, f"{bad.size} bytes differ, first at {bad[:8]}"
    assert (to_bits(B.patch_unpack(L, packed)) == oracle.unpack(blob_o)).all()


@pytest.mark.parametrize("M", [1, 5, 16])
@pytest.mark.parametrize("p", [0.0, 1.0, 0.4])
@pytest.mark.parametrize("N,K", [(128, 128), (256, 1152), (640, 384), (4096, 1024), (512, 8192)])
def test_gemm_parity(gpu, oracle, N, K, M, p):
    """Whole output against the oracle's matmul on the dequantised matrix, for all three launch forms (they may split
    K differently, so they agree to the last bit only where the split is the same); each form repeats bit for bit."""
    torch, B = gpu
    W = inputs.weight(N, K, 33, "q4-gemm", N, K)
    X = inputs.activation(M, K, 33, "q4-gemm", N, K, M)
    flags = _flags4(N, K, p, ("gemm", N, K, p))
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    assert B.patch_gemm_workspace_size(L, M) == 0
    Y32, Y16 = oracle.gemm_f64(X, What)
    outs = []
    for promise in (0, B.WEIGHTS_STATIC, B.WEIGHTS_STATIC | B.INPUT_STATIC,
                    B.WEIGHTS_STATIC | B.INPUT_STATIC | B.OUTPUT_STATIC):
        Y = run_gemm(gpu, X, L, packed, B.VARIANT_AUTO | promise)
        check_parity(oracle, Y, Y32, f"q4 N={N} K={K} M={M} p={p} promise={promise:#x}")
        assert (Y == Y16).mean() >= 0.99
        assert (run_gemm(gpu, X, L, packed, B.VARIANT_AUTO | promise) == Y).all()
        outs.append(Y)
    assert (outs[0] == outs[1]).all()              # no promise / weights only: the same split of K
    assert (run_gemm(gpu, X, L, packed, B.VARIANT_MMA) == outs[0]).all()


@pytest.mark.parametrize("p", [0.0, 1.0, 0.5])
def test_gemm_one_hot_probe(gpu, oracle, p):
    """Token m is the unit vector e_k(m): every output is one product with 1, so row m of Y must equal column k(m)
    of the dequantised matrix exactly.  A wrong nibble order, scale row or metadata order shows as exact
    mismatches.  Sixteen columns per launch, chosen to cover every position of a group of eight and several tiles."""
    torch, B = gpu
    N, K = 384, 512
    W = inputs.weight(N, K, 34, "q4-onehot")
    flags = _flags4(N, K, p, ("onehot", p))
    What = f32(oracle.prune(W, flags))
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    for base in (0, 8, 120, 250, 496):
        cols = [(base + 9 * i) % K for i in range(16)]
        X = np.zeros((16, K), np.float32)
        X[np.arange(16), cols] = 1.0
        Y = run_gemm(gpu, inputs.f32_to_bf16_bits(X), L, packed, B.VARIANT_AUTO)
        assert (f32(Y) == What[:, cols].T).all(), base


def test_gemm_back_to_back_and_chain(gpu, oracle):
    """Launches in a row on one stream with and without promises, each into its own output; then a chain in which
    the output of one call is the input of the next (square weight)."""
    torch, B = gpu
    M = 16
    cases = []
    for i, (N, K) in enumerate([(1024, 512), (640, 768)]):
        W = inputs.weight(N, K, 35, "q4-b2b", i)
        X = inputs.activation(M, K, 35, "q4-b2b", i)
        flags = _flags4(N, K, 0.5, ("b2b", i))
        packed, L = B.patch_pack(to_dev(torch, W), flags)
        cases.append((oracle.prune(W, flags), packed, L, X, to_dev(torch, X)))
    torch.cuda.synchronize()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    outs = []
    for i in range(12):
        What, packed, L, X, Xd = cases[i % 2]
        # every launch writes a buffer of its own, so the odd ones may also carry the output promise
        promise = (B.WEIGHTS_STATIC | B.INPUT_STATIC | (B.OUTPUT_STATIC if i % 4 == 1 else 0)) if i % 2 else 0
        outs.append(B.patch_gemm(Xd, L, packed, status=status, variant=B.VARIANT_AUTO | promise))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    refs = [oracle.gemm_f64(c[3], c[0])[0] for c in cases]
    for i, Y in enumerate(outs):
        check_parity(oracle, to_bits(Y), refs[i % 2], f"launch {i}")
    N = K = 512
    W = inputs.f32_to_bf16_bits(f32(inputs.weight(N, K, 35, "q4-chain")) * 2.0)
    X = inputs.activation(M, K, 35, "q4-chain")
    flags = _flags4(N, K, 0.5, "chain")
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    bufs = [to_dev(torch, X)] + [torch.empty((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(6)]
    for i in range(6):
        B.patch_gemm(bufs[i], L, packed, Y=bufs[i + 1], status=status,
                     variant=B.VARIANT_AUTO | (B.WEIGHTS_STATIC if i % 2 else 0))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = X
    for i in range(6):
        Y32, _ = oracle.gemm_f64(ref, What)
        got = to_bits(bufs[i + 1])
        check_parity(oracle, got, Y32, f"chain step {i}")
        ref = got


def test_pack_with_given_patterns_bit_exact(gpu, oracle):
    """patch_pack_patterns on 4-bit kinds: the learned 2:4 mask first, then the quantiser; blob and dequantised
    matrix bit for bit; a candidate index above 5 inside a 2:4 tile is reported."""
    torch, B = gpu
    N, K = 512, 384
    W = inputs.weight(N, K, 39, "q4-patterns")
    g = inputs.generator(39, "q4-patterns-c")
    patterns = g.integers(0, 6, (N, K // 4)).astype(np.uint8)
    flags = _flags4(N, K, 0.6, "patterns", "half")
    pd = torch.from_numpy(patterns.reshape(-1)).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    packed, L = B.patch_pack_patterns(to_dev(torch, W), flags, pd, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    blob_o, _ = oracle.pack_patterns(W, flags, patterns)
    assert (packed.cpu().numpy() == oracle.device_image(blob_o)).all()
    assert (to_bits(B.patch_unpack(L, packed)) == oracle.unpack(blob_o)).all()
    bad = patterns.copy()
    tn, tk = np.argwhere(flags == 3)[0]
    bad[tn * 128 + 3, tk * 32 + 5] = 6
    B.patch_pack_patterns(to_dev(torch, W), flags, torch.from_numpy(bad.reshape(-1)).cuda(), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.ERR_FLAG


@pytest.mark.parametrize("with_patterns", [False, True])
def test_pack_with_flags_in_device_memory(gpu, oracle, with_patterns):
    """patch_pack_dev on all four kinds: header, table and payloads equal to patch_pack's from host flags (which
    equal the oracle's), the layout read back from the blob, a flag above 3 reported and packed as dense."""
    torch, B = gpu
    N, K = 640, 1152
    W = inputs.weight(N, K, 40, "q4-dev")
    flags = _flags4(N, K, 0.5, "dev", "half")
    assert set(np.unique(flags)) == {0, 1, 2, 3}
    Wd = to_dev(torch, W)
    g = inputs.generator(40, "q4-dev-c")
    patterns = g.integers(0, 6, (N, K // 4)).astype(np.uint8)
    pd = torch.from_numpy(patterns.reshape(-1)).cuda() if with_patterns else None
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = B.patch_pack_dev(Wd, torch.from_numpy(flags.reshape(-1)).cuda(), patterns=pd, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    L = B.patch_read_layout(out)
    blob_o, L_o = oracle.pack_patterns(W, flags, patterns) if with_patterns else oracle.pack(W, flags)
    for f, _ in B.Layout._fields_:
        assert getattr(L, f) == getattr(L_o, f), f
    assert (out[:L.total_bytes].cpu().numpy() == oracle.device_image(blob_o)).all()
    # the packed weight is usable as it is: all-4-bit part of the flags through the matmul
    flags4 = flags | 2
    out4 = B.patch_pack_dev(Wd, torch.from_numpy(flags4.reshape(-1)).cuda(), patterns=pd, status=status)
    L4 = B.patch_read_layout(out4)
    X = inputs.activation(8, K, 40, "q4-dev-x")
    Y = run_gemm(gpu, X, L4, out4[:L4.total_bytes], B.VARIANT_AUTO)
    blob4 = oracle.pack_patterns(W, flags4, patterns)[0] if with_patterns else oracle.pack(W, flags4)[0]
    check_parity(oracle, Y, oracle.gemm_f64(X, oracle.unpack(blob4))[0], "matmul on a blob packed from device flags")
    bad = flags.reshape(-1).copy()
    bad[5] = 9
    out_b = B.patch_pack_dev(Wd, torch.from_numpy(bad).cuda(), patterns=pd, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.ERR_FLAG
    good = bad.copy()
    good[5] = 0                                  # the bad flag was packed as dense
    ref = B.patch_pack_dev(Wd, torch.from_numpy(good).cuda(), patterns=pd)
    Lb = B.patch_read_layout(ref)
    assert torch.equal(out_b[:Lb.total_bytes], ref[:Lb.total_bytes])


@pytest.mark.parametrize("M", [17, 40, 64])
def test_gemm_more_than_16_tokens(gpu, oracle, M):
    """17 to 64 tokens are multiplied sixteen at a time (no workspace); every promise; Y with a row pitch."""
    torch, B = gpu
    N, K = 640, 768
    W = inputs.weight(N, K, 38, "q4-chunks")
    X = inputs.activation(M, K, 38, "q4-chunks", M)
    flags = _flags4(N, K, 0.5, "chunks")
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Y32, Y16 = oracle.gemm_f64(X, What)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for promise in (0, B.WEIGHTS_STATIC, B.WEIGHTS_STATIC | B.INPUT_STATIC):
        Ybuf = torch.full((M, N + 64), 3.0, dtype=torch.bfloat16, device="cuda")
        B.patch_gemm(to_dev(torch, X), L, packed, Y=Ybuf[:, :N], status=status, variant=B.VARIANT_AUTO | promise)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got = to_bits(Ybuf[:, :N])
        check_parity(oracle, got, Y32, f"M={M} promise={promise:#x}")
        assert (got == Y16).mean() >= 0.99
        assert (Ybuf[:, N:] == 3.0).all()


@pytest.mark.parametrize("p", [0.0, 1.0, 0.5])
@pytest.mark.parametrize("M", [65, 300, 1000])
def test_gemm_many_tokens(gpu, oracle, M, p):
    """Beyond 64 tokens the weight is rewritten as the bf16 blob of its dequantised values (in the workspace) and the
    large-M schedule multiplies by it: the same matrix, so the same reference."""
    torch, B = gpu
    N, K = 640, 768
    W = inputs.weight(N, K, 44, "q4-many")
    X = inputs.activation(M, K, 44, "q4-many", M)
    flags = _flags4(N, K, p, ("many", p))
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    need = B.patch_gemm_workspace_size(L, M)
    off = 32 << 20                                                          # the blob's place in the workspace
    assert need == off + oracle.packed_size(N, K, flags & 1).total_bytes    # ... and the size of the bf16 blob of the same mask
    Y32, Y16 = oracle.gemm_f64(X, What)
    Y = run_gemm(gpu, X, L, packed, B.VARIANT_AUTO)
    check_parity(oracle, Y, Y32, f"q4 M={M} p={p}")
    assert (Y == Y16).mean() >= 0.99
    assert (run_gemm(gpu, X, L, packed, B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC) == Y).all()
    # what was written to the workspace is the bf16 blob of the dequantised matrix: it unpacks to that matrix
    ws = torch.zeros(need, dtype=torch.uint8, device="cuda")
    B.patch_gemm(to_dev(torch, X), L, packed, workspace=ws)
    torch.cuda.synchronize()
    assert int(ws[:off].count_nonzero()) == 0                               # the part other calls share stays zero
    E = B.patch_read_layout(ws[off:])
    assert (E.n_dense, E.n_sparse, E.n_dense_q4, E.n_sparse_q4) == (L.n_dense_q4, L.n_sparse_q4, 0, 0)
    assert (to_bits(B.patch_unpack(E, ws[off:])) == What).all()
    with pytest.raises(B.PatchError) as e:
        B.patch_gemm(to_dev(torch, X), L, packed, workspace=ws[:need - 256])
    assert e.value.status == B.ERR_SIZE


def test_workspace_shared_between_bf16_and_4bit_calls(gpu, oracle):
    """One workspace for a bf16 weight's small-M calls (which count on its counters and flag words being zero) and a
    4-bit weight's many-token call (which writes a whole blob into it): in any order, every result stays right."""
    torch, B = gpu
    N, K = 512, 1024
    W = inputs.weight(N, K, 46, "q4-shared-ws")
    fb = inputs.tile_flags(N, K, 0.5, inputs.MASTER_SEED, "q4-shared-ws")
    f4 = fb | 2
    pb, Lb = B.patch_pack(to_dev(torch, W), fb)
    p4, L4 = B.patch_pack(to_dev(torch, W), f4)
    size = max(B.patch_gemm_workspace_size(Lb, 64), B.patch_gemm_workspace_size(L4, 200))
    ws = torch.zeros(size, dtype=torch.uint8, device="cuda")
    Xs, Xl = inputs.activation(7, K, 46, "q4-shared-ws", 7), inputs.activation(200, K, 46, "q4-shared-ws", 200)
    Ys32, _ = oracle.gemm_f64(Xs, oracle.prune(W, fb))
    Yl32, _ = oracle.gemm_f64(Xl, oracle.prune(W, f4))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for rnd in range(2):
        Ys = B.patch_gemm(to_dev(torch, Xs), Lb, pb, workspace=ws, status=status, variant=B.VARIANT_MMA)   # the schedule with counters
        Yl = B.patch_gemm(to_dev(torch, Xl), L4, p4, workspace=ws, status=status)
        Ys2 = B.patch_gemm(to_dev(torch, Xs), Lb, pb, workspace=ws, status=status, variant=B.VARIANT_MMA)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        check_parity(oracle, to_bits(Ys), Ys32, f"bf16 before, round {rnd}")
        check_parity(oracle, to_bits(Yl), Yl32, f"4-bit many tokens, round {rnd}")
        assert (Ys2 == Ys).all()


def test_mixed_stream_of_4bit_and_bf16_launches(gpu, oracle):
    """A long stream in which 4-bit GEMMs share the GPU with bf16 GEMMs of other shapes, token counts and launch
    promises (several kernels resident at once, copies completing out of order).  Every job is checked once against
    the oracle; after that every launch must repeat, bit for bit, the first result of its launch form -- the kernels
    are deterministic, so one tile read too early or too late in any launch shows."""
    torch, B = gpu
    g = inputs.generator(47, "mixed-stream")
    jobs = []
    ws = torch.zeros(8192 + 3145728 + 2 * 192 * 64 * 128 * 4, dtype=torch.uint8, device="cuda")
    for it in range(20):
        TN, TK = int(g.integers(8, 60)), int(g.integers(8, 60))
        N, K = 128 * TN, 128 * TK
        q4 = it % 2 == 0
        M = int(g.choice([1, 2, 5, 16] if q4 else [1, 3, 8, 16, 17, 40, 64]))
        flags = inputs.tile_flags(N, K, float(g.choice([0.0, 1.0, 0.5])), 47, "mixed-stream", it) | (2 if q4 else 0)
        W = inputs.weight(N, K, 47, "mixed-stream", it)
        X = inputs.activation(M, K, 47, "mixed-stream", it)
        packed, L = B.patch_pack(to_dev(torch, W), flags)
        rows = np.unique(g.integers(0, M, 2))
        ref_rows = oracle.gemm_f64_rows(X, rows, oracle.prune(W, flags))
        jobs.append(dict(X=to_dev(torch, X), L=L, packed=packed, rows=rows, ref_rows=ref_rows, first={},
                         Ys=[torch.zeros((M, N), dtype=torch.bfloat16, device="cuda") for _ in range(4)], n=0, form=[None] * 4))
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    forms = [B.WEIGHTS_STATIC | B.INPUT_STATIC | B.OUTPUT_STATIC, B.WEIGHTS_STATIC | B.INPUT_STATIC, B.WEIGHTS_STATIC, 0]
    for rnd in range(12):
        order = g.permutation(len(jobs))
        for rep in range(25):
            for i in order:
                j = jobs[i]
                k = j["n"] % 4
                j["n"] += 1
                j["form"][k] = forms[int(g.integers(0, 4))]
                B.patch_gemm(j["X"], j["L"], j["packed"], Y=j["Ys"][k], workspace=ws, status=status,
                             variant=B.VARIANT_AUTO | j["form"][k])
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for j in jobs:
            for k, Y in enumerate(j["Ys"]):
                form = j["form"][k]
                if form not in j["first"]:
                    check_parity(oracle, to_bits(Y)[j["rows"]], j["ref_rows"], f"first result of launch form {form:#x}")
                    j["first"][form] = Y.clone()
                assert torch.equal(Y, j["first"][form]), f"round {rnd}: launch form {form:#x} did not repeat its result"
                Y.zero_()


def test_gemm_many_tokens_llama_shape_sampled(gpu, oracle):
    torch, B = gpu
    N, K, M = 4096, 4096, 2048
    W = inputs.weight(N, K, 45, "q4-many-llama")
    X = inputs.activation(M, K, 45, "q4-many-llama", M)
    flags = _flags4(N, K, 0.5, "many-llama")
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Y = run_gemm(gpu, X, L, packed, B.VARIANT_AUTO)
    rows = np.array([0, 1, 127, 128, 239, 240, 1000, 2047])
    check_parity(oracle, Y[rows], oracle.gemm_f64_rows(X, rows, What), "q4 4096x4096 M=2048, sampled token rows")


def test_unsupported_combinations_are_refused(gpu):
    torch, B = gpu
    N, K = 256, 256
    W = to_dev(torch, inputs.weight(N, K, 36, "q4-err"))
    all_q4 = np.array([[2, 3], [3, 2]], np.uint8)
    mixed = np.array([[2, 0], [3, 1]], np.uint8)
    packed, L = B.patch_pack(W, all_q4)
    packed_m, L_m = B.patch_pack(W, mixed)             # packing and unpacking serve any mixture
    assert (L_m.n_dense, L_m.n_sparse, L_m.n_dense_q4, L_m.n_sparse_q4) == (1, 1, 1, 1)
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    X4 = torch.zeros((4, K), dtype=torch.bfloat16, device="cuda")

    def refused(fn):
        with pytest.raises(B.PatchError) as e:
            fn()
        return e.value.status

    assert refused(lambda: B.patch_gemm(X4, L_m, packed_m, workspace=ws)) == B.ERR_SHAPE       # bf16 and 4-bit tiles
    assert refused(lambda: B.patch_gemm(X4, L, packed, workspace=ws, variant=B.VARIANT_GEMV)) == B.ERR_SHAPE
    assert refused(lambda: B.patch_gemm_gated(X4, L, packed, workspace=ws)) == B.ERR_SHAPE
    assert refused(lambda: B.patch_gemm_noalloc(X4, L, packed, torch.empty((4, N), dtype=torch.bfloat16, device="cuda"))) == B.ERR_SHAPE


def test_bad_table_entries_are_reported(gpu, oracle):
    """A table entry whose kind is not a 4-bit kind, or whose payload lies outside the blob: the launch completes,
    the status word says PATCH_ERR_FORMAT, nothing is read out of range."""
    torch, B = gpu
    N, K, M = 256, 512, 8
    W = inputs.weight(N, K, 37, "q4-bad")
    X = inputs.activation(M, K, 37, "q4-bad")
    flags = _flags4(N, K, 0.5, "bad")
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    good = run_gemm(gpu, X, L, packed, B.VARIANT_AUTO)
    for word, value in ((0, 1), (0, 9), (1, int(L.total_bytes // 16) - 3), (1, 2)):
        blob = packed.clone()
        entry = blob[int(L.table_off) + 16 * 3:int(L.table_off) + 16 * 4].view(torch.int32)
        entry[word] = value
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.patch_gemm(to_dev(torch, X), L, blob, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == B.ERR_FORMAT, (word, value)
    assert (run_gemm(gpu, X, L, packed, B.VARIANT_AUTO) == good).all()
    # the same with many tokens, where the blob is first rewritten as bf16 tiles: also an offset inside the blob that
    # no sequence of tiles before it can add up to
    Xm = inputs.activation(100, K, 37, "q4-bad-many")
    ws = torch.zeros(B.patch_gemm_workspace_size(L, 100), dtype=torch.uint8, device="cuda")
    for word, value in ((0, 1), (0, 9), (1, int(L.total_bytes // 16) - 3), (1, 2), (1, int(L.payload_off // 16) + 1)):
        blob = packed.clone()
        entry = blob[int(L.table_off) + 16 * 3:int(L.table_off) + 16 * 4].view(torch.int32)
        entry[word] = value
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        B.patch_gemm(to_dev(torch, Xm), L, blob, workspace=ws, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == B.ERR_FORMAT, (word, value)
    Ym = run_gemm(gpu, Xm, L, packed, B.VARIANT_AUTO)
    check_parity(oracle, Ym, oracle.gemm_f64(Xm, oracle.prune(W, flags))[0], "after the bad tables")


# ---------------------------------------------------------------------------------------------
# the decode-q4 workload as bench.py runs it


@pytest.fixture(scope="module")
def decode_q4_workload(gpu, oracle):
    """The 24 GEMMs of `bench.py --workload decode-q4`: 12 packed matrices (3 LLaMA-2-7B shapes x four 2:4-tile
    fractions, every tile 4-bit), M = 1 and 16, with the oracle's result for each."""
    torch, B = gpu
    cases = sorted(inputs.decode_q4_cases(), key=lambda c: c["M"])
    mats, jobs = {}, []
    for c in cases:
        key = c["stream"]
        if key not in mats:
            W = inputs.weight(c["N"], c["K"], inputs.MASTER_SEED, *c["stream"])
            flags = inputs.case_flags(c)
            assert ((flags & 2) == 2).all()
            packed, L = B.patch_pack(to_dev(torch, W), flags)
            mats[key] = (oracle.prune(W, flags), packed, L)
        What, packed, L = mats[key]
        X = inputs.activation(c["M"], c["K"], inputs.MASTER_SEED, *c["stream"], c["M"])
        Y32, Y16 = oracle.gemm_f64(X, What)
        jobs.append(dict(case=c, L=L, packed=packed, X=to_dev(torch, X), Y32=Y32, Y16=Y16,
                         Y=torch.zeros((c["M"], c["N"]), dtype=torch.bfloat16, device="cuda")))
    torch.cuda.synchronize()
    return jobs


@pytest.mark.parametrize("mode", ["independent", "independent+output", "dependent", "no promise"])
def test_decode_q4_workload_graph_replay(gpu, oracle, decode_q4_workload, mode):
    """The regime the decode-q4 number is timed in: two consecutive steps of the 24 GEMMs captured into one CUDA
    graph (CTAs of consecutive kernels share SMs, ordered only by their device-side waits), replayed twice; then
    every one of the 24 outputs, whole, against the oracle."""
    torch, B = gpu
    jobs = decode_q4_workload
    flags = {"independent": B.WEIGHTS_STATIC | B.INPUT_STATIC,
             "independent+output": B.WEIGHTS_STATIC | B.INPUT_STATIC | B.OUTPUT_STATIC,
             "dependent": B.WEIGHTS_STATIC, "no promise": 0}[mode]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # the output promise: every launch between two drains writes a buffer of its own (the second step of the
    # graph gets a second set), as bench.py does
    second = [torch.zeros_like(j["Y"]) for j in jobs]

    def step(outs):
        for j, Y in zip(jobs, outs):
            B.patch_gemm(j["X"], j["L"], j["packed"], Y=Y, status=status, variant=B.VARIANT_AUTO | flags)
    first = [j["Y"] for j in jobs]
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


def test_decode_q4_workload_pack_bit_exact(gpu, oracle):
    """The largest matrices of the workload, packed image against the oracle's, bit for bit."""
    torch, B = gpu
    for c in inputs.decode_q4_cases():
        if c["M"] != 1 or c["p"] not in (0.35, 1.0) or c["N"] == c["K"]:
            continue
        W = inputs.weight(c["N"], c["K"], inputs.MASTER_SEED, *c["stream"])
        flags = inputs.case_flags(c)
        packed, L = B.patch_pack(to_dev(torch, W), flags)
        assert (packed.cpu().numpy() == oracle.device_image(oracle.pack(W, flags)[0])).all(), c["name"]
        assert (to_bits(B.patch_unpack(L, packed)) == oracle.prune(W, flags)).all(), c["name"]
