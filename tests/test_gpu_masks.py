"""GPU parity of the mask-learning entry points (hard masks, packing with a given 2:4 mask, the
soft-mask forward and its sums) against the CPU oracle on the same seeded inputs.

Integer and byte results are compared bit for bit.  The soft mask is fp32 arithmetic on the
device against double in the oracle: with the exponents (kappa p + z) / tau reaching a few
hundred at the end of the schedule, fp32 rounding of the exponent and the hardware logarithm
leave a relative error of up to a few 1e-4 in a softmax term, hence |dMt| <= 1e-3; the masked
weight is that times w, rounded to bf16 (one more 2^-9 relative)."""
import numpy as np
import pytest

from paper_2509_23410_b200 import inputs

pytestmark = pytest.mark.gpu

MT_TOL = 1e-3
# gradients of saturated tiles are e^-|d| with |d| in the hundreds: below fp32's range the device returns 0
TINY = 1e-20


@pytest.fixture(scope="module")
def gpu():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("no CUDA device: GPU tests must run on a B200")
    from paper_2509_23410_b200 import binding
    binding.lib()
    return torch, binding


def to_dev(torch, bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def to_bits(t):
    import torch
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


f32 = inputs.bf16_bits_to_f32


def logits(N, K, p_dense, seed, *stream, std=inputs.LOGIT_STD):
    PT = inputs.tile_logits(N // 128, K // 128, p_dense, seed, *stream)
    P6 = inputs.pattern_logits(N, K, seed, *stream, std=std)
    return PT, P6


# ---------------------------------------------------------------------------------------------
# hard masks and packing with them


@pytest.mark.parametrize("N,K", [(128, 128), (256, 384), (640, 256), (4096, 4096)])
def test_hard_mask_bit_exact(gpu, oracle, N, K):
    torch, B = gpu
    PT, P6 = logits(N, K, 0.4, 21, "hard", N, K)
    PT.reshape(-1)[0] = 0.0                     # not positive: 2:4
    P6[:, 5] = 0.125                            # six-way tie -> candidate 0
    P6[[1, 3], 17] = 9.0                        # two-way tie -> the lower index
    P6[5, 33] = 7.0                             # last candidate wins
    flags, patterns = B.patch_hard_mask(torch.from_numpy(PT).cuda(), torch.from_numpy(P6).cuda(), N, K)
    rf, rp = oracle.hard_mask(PT, P6, N, K)
    assert (flags.cpu().numpy() == rf).all()
    got = patterns.cpu().numpy()
    assert (got == rp).all()
    assert got[5] == 0 and got[17] == 1 and got[33] == 5 and got.max() <= 5


@pytest.mark.parametrize("N,K,p", [(128, 128, 0.0), (256, 384, 0.5), (1024, 1024, 0.5), (4096, 4096, 0.3)])
def test_pack_patterns_bit_exact(gpu, oracle, N, K, p):
    torch, B = gpu
    W = inputs.weight(N, K, 22, "pp", N, K)
    W[::13, ::7] = 0
    flags = inputs.tile_flags(N, K, 1.0 - p, 22, "pp", N, K)
    patterns = inputs.generator(22, "pp", "patterns", N, K).integers(0, 6, N * K // 4).astype(np.uint8)
    canon, Lo = oracle.pack_patterns(W, flags, patterns)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    packed, L = B.patch_pack_patterns(to_dev(torch, W), flags, torch.from_numpy(patterns).cuda(), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert (L.n_dense, L.n_sparse, L.total_bytes) == (Lo.n_dense, Lo.n_sparse, Lo.total_bytes)
    assert (packed.cpu().numpy() == oracle.device_image(canon)).all()
    M = oracle.mask_patterns(N, K, flags, patterns)
    assert (to_bits(B.patch_unpack(L, packed)) == np.where(M == 1, W, 0)).all()


def test_pack_patterns_flags_a_bad_index(gpu, oracle):
    torch, B = gpu
    N, K = 256, 256
    W = inputs.weight(N, K, 23, "bad")
    flags = np.array([[1, 0], [0, 1]], np.uint8)
    patterns = np.zeros(N * K // 4, np.uint8)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    bad = patterns.copy()
    bad[(3 * (K // 4)) + 40] = 9                 # row 3, group 40: inside the dense tile (0, 1) -> ignored
    B.patch_pack_patterns(to_dev(torch, W), flags, torch.from_numpy(bad).cuda(), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    bad[(3 * (K // 4)) + 4] = 6                  # inside the 2:4 tile (0, 0)
    packed, L = B.patch_pack_patterns(to_dev(torch, W), flags, torch.from_numpy(bad).cuda(), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.ERR_FLAG
    # the offending group was packed as candidate 0, everything else is unaffected
    canon, _ = oracle.pack_patterns(W, flags, patterns)
    assert (packed.cpu().numpy() == oracle.device_image(canon)).all()


@pytest.mark.parametrize("M", [1, 16, 300])
def test_learned_mask_deployment_chain(gpu, oracle, M):
    """logits -> hard masks -> packed blob -> GEMM, all on the device, against the oracle's chain."""
    torch, B = gpu
    N, K = 512, 768
    W = inputs.weight(N, K, 24, "chain")
    X = inputs.activation(M, K, 24, "chain", M)
    PT, P6 = logits(N, K, 0.5, 24, "chain")
    flags_d, patterns_d = B.patch_hard_mask(torch.from_numpy(PT).cuda(), torch.from_numpy(P6).cuda(), N, K)
    flags = flags_d.cpu().numpy()
    packed, L = B.patch_pack_patterns(to_dev(torch, W), flags, patterns_d)
    ws = torch.zeros(max(B.patch_gemm_workspace_size(L, M), 1), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Y = to_bits(B.patch_gemm(to_dev(torch, X), L, packed, workspace=ws, status=status))
    assert int(status.item()) == 0
    rf, rp = oracle.hard_mask(PT, P6, N, K)
    assert 0 < rf.sum() < rf.size
    What = oracle.unpack(oracle.pack_patterns(W, rf, rp)[0])
    Y32, _ = oracle.gemm_f64(X, What)
    relF, maxrel = oracle.parity_metrics(f32(Y), Y32)
    assert relF <= 2e-3 and maxrel <= 1e-2, (relF, maxrel)


# ---------------------------------------------------------------------------------------------
# soft masks


def run_soft(gpu, W, PT, P6, tau, kappa, seed, noise, want_mt=True, ld_pad=0):
    torch, B = gpu
    N, K = W.shape
    Wd = to_dev(torch, W)
    if ld_pad:
        buf = torch.zeros((N, K + ld_pad), dtype=torch.bfloat16, device="cuda")
        buf[:, :K] = Wd
        Wd = buf[:, :K]
    Mt = torch.full((N, K), -1.0, dtype=torch.float32, device="cuda") if want_mt else None
    Wt, sums = B.patch_soft_mask(Wd, torch.from_numpy(PT).cuda(), torch.from_numpy(P6).cuda(), tau, kappa, seed,
                                 0 if noise else B.MASK_NO_NOISE, Mt=Mt)
    torch.cuda.synchronize()
    return to_bits(Wt), (Mt.cpu().numpy() if want_mt else None), sums.cpu().numpy()


def check_soft(oracle, W, got_Wt, got_Mt, got_sums, ref):
    rMt, rWt, rsums = ref
    w = f32(W).astype(np.float64)
    if got_Mt is not None:
        assert np.abs(got_Mt - rMt).max() <= MT_TOL
    dW = np.abs(f32(got_Wt).astype(np.float64) - rMt * w)
    assert (dW <= np.abs(w) * (MT_TOL + 2.0 ** -8) + 1e-30).all()
    assert (got_Wt == rWt).mean() > 0.97
    assert got_sums[1] == rsums[1]                                  # ||W||_0 is a count
    assert np.allclose(got_sums[[0, 2, 3]], rsums[[0, 2, 3]], rtol=2e-4)
    assert abs(got_sums[3] - rsums[3]) <= 2e-6 * rsums[3]           # no softmax in ||W||^2


@pytest.mark.parametrize("tau,kappa", [inputs.SCHEDULE_START, inputs.SCHEDULE_END, (0.6, 100.0)])
@pytest.mark.parametrize("noise", [False, True])
def test_soft_mask_parity(gpu, oracle, tau, kappa, noise):
    N, K = 384, 640
    W = inputs.weight(N, K, 31, "soft")
    W[::11, ::5] = 0
    PT, P6 = logits(N, K, 0.5, 31, "soft")
    PT *= np.float32(0.004)       # tile values across (0, 1) instead of saturated ones
    ref = oracle.soft_mask(W, PT, P6, tau, kappa, seed=77, noise=noise)
    got = run_soft(gpu, W, PT, P6, tau, kappa, 77, noise)
    check_soft(oracle, W, *got, ref)
    # the same through a padded leading dimension and without the optional mask output
    got2 = run_soft(gpu, W, PT, P6, tau, kappa, 77, noise, want_mt=False, ld_pad=24)
    assert (got2[0] == got[0]).all() and (got2[2] == got[2]).all()


def test_soft_mask_prior_initialised_tiles_and_seeds(gpu, oracle):
    N, K = 256, 512
    W = inputs.weight(N, K, 32, "soft2")
    PT, P6 = logits(N, K, 0.5, 32, "soft2")          # +-3 prior: tiles saturate as kappa grows
    tau, kappa = 1.0, 60.0
    a = run_soft(gpu, W, PT, P6, tau, kappa, 1, True)
    check_soft(oracle, W, *a, oracle.soft_mask(W, PT, P6, tau, kappa, seed=1, noise=True))
    b = run_soft(gpu, W, PT, P6, tau, kappa, 2 ** 63 + 5, True)
    check_soft(oracle, W, *b, oracle.soft_mask(W, PT, P6, tau, kappa, seed=2 ** 63 + 5, noise=True))
    assert np.abs(a[1] - b[1]).max() > 0.1           # a different seed is a different draw
    c = run_soft(gpu, W, PT, P6, tau, kappa, 1, True)
    assert (a[0] == c[0]).all() and (a[1] == c[1]).all() and (a[2] == c[2]).all()     # reproducible, sums included


def test_soft_mask_closed_form_and_hardening(gpu, oracle):
    torch, B = gpu
    N, K = 256, 256
    W = inputs.weight(N, K, 33, "soft3")
    # equal logits, zero tile logit, no noise: Mt = 3/4 everywhere
    Wt, Mt, sums = run_soft(gpu, W, np.zeros((2, 2), np.float32), np.full((6, N * K // 4), 0.3, np.float32),
                            0.7, 9.0, 0, False)
    assert np.abs(Mt - 0.75).max() < 1e-6
    assert abs(sums[0] - 0.75 * N * K) < 1e-3 * N * K
    # tau -> 0 without noise: the soft mask becomes the hard mask of the same logits
    PT = np.array([[2.5, -2.5], [-1.0, 4.0]], np.float32)
    P6 = inputs.pattern_logits(N, K, 33, "soft3", std=1.0)
    top = np.sort(P6, axis=0)
    clear = np.repeat(((top[-1] - top[-2]) > 1e-2).reshape(N, K // 4), 4, axis=1)
    Wt, Mt, _ = run_soft(gpu, W, PT, P6, 1e-3, 1.0, 0, False)
    flags, patterns = B.patch_hard_mask(torch.from_numpy(PT).cuda(), torch.from_numpy(P6).cuda(), N, K)
    Mstar = oracle.mask_patterns(N, K, flags.cpu().numpy(), patterns.cpu().numpy())
    assert clear.mean() > 0.95 and np.abs(Mt - Mstar)[clear].max() < 1e-3


def test_soft_mask_full_size(gpu, oracle):
    """The 4096 x 4096 shape the benchmark times, against the oracle over the whole matrix."""
    N, K = 4096, 4096
    W = inputs.weight(N, K, 34, "soft4")
    PT, P6 = logits(N, K, 0.5, 34, "soft4")
    PT *= np.float32(0.004)
    tau, kappa = 0.5, 120.0
    got = run_soft(gpu, W, PT, P6, tau, kappa, 12345, True)
    check_soft(oracle, W, *got, oracle.soft_mask(W, PT, P6, tau, kappa, seed=12345, noise=True))


def test_mask_entry_points_reject_bad_arguments(gpu):
    torch, B = gpu
    lib = B.lib()
    z = torch.zeros(4096, dtype=torch.float32, device="cuda")
    p = z.data_ptr()
    assert lib.patch_hard_mask(p, p, 128, 100, 128, 128, p, p, None) == B.ERR_SHAPE
    assert lib.patch_hard_mask(p, p, 128, 128, 64, 128, p, p, None) == B.ERR_TILE
    assert lib.patch_hard_mask(p, None, 128, 128, 128, 128, p, p, None) == B.ERR_NULL
    assert lib.patch_hard_mask(p, p + 4, 128, 128, 128, 128, p, p, None) == B.ERR_ALIGN
    args = lambda tau=1.0, ws=128, flags=0: (p, 128, p, p, 128, 128, 128, 128, tau, 1.0, 0, flags, p, 128, None, 0,
                                             p, p, ws, None)
    assert lib.patch_soft_mask(*args(tau=0.0)) == B.ERR_SHAPE
    assert lib.patch_soft_mask(*args(tau=float("nan"))) == B.ERR_SHAPE
    assert lib.patch_soft_mask(*args(ws=8)) == B.ERR_SIZE
    assert lib.patch_soft_mask(*args(flags=4)) == B.ERR_SHAPE


# ---------------------------------------------------------------------------------------------
# backward


@pytest.mark.parametrize("tau,kappa", [inputs.SCHEDULE_START, (0.6, 100.0), inputs.SCHEDULE_END])
@pytest.mark.parametrize("noise", [False, True])
def test_soft_mask_backward_parity(gpu, oracle, tau, kappa, noise):
    """fp32 on the device against the oracle's double gradient: relative Frobenius error <= 1e-3 and
    max |d| <= 2e-3 max |g| (the same exponent-rounding argument as for the forward, times the few terms
    of the chain rule)."""
    torch, B = gpu
    N, K = 384, 640
    W = inputs.weight(N, K, 41, "bwd")
    W[::11, ::5] = 0
    Gw = inputs.normal_bf16((N, K), 1.0, 41, "bwd", "gw")
    PT, P6 = logits(N, K, 0.5, 41, "bwd")
    PT *= np.float32(0.004)
    c1, c2 = 3.0e-6, 0.8
    rt, r6 = oracle.soft_mask_backward(W, PT, P6, tau, kappa, f32(Gw), c1, c2, seed=55, noise=noise)
    gt, g6 = B.patch_soft_mask_backward(to_dev(torch, W), torch.from_numpy(PT).cuda(), torch.from_numpy(P6).cuda(), tau,
                                        kappa, to_dev(torch, Gw), c1, c2, seed=55, flags=0 if noise else B.MASK_NO_NOISE)
    torch.cuda.synchronize()
    # at the end of the schedule (kappa / tau = 7000) the tiles are saturated: their gradient is e^-|d| with
    # |d| in the tens to hundreds, so an absolute error of 1e-3 in the fp32 exponent is a relative error of
    # 1e-3 in the gradient
    tol = 3.0 if kappa / tau > 1000 else 1.0
    for got, ref in ((gt.cpu().numpy().astype(np.float64), rt), (g6.cpu().numpy().astype(np.float64), r6)):
        assert np.isfinite(got).all()
        assert np.abs(got - ref).max() <= tol * 2e-3 * np.abs(ref).max() + TINY
        assert np.sqrt(((got - ref) ** 2).sum()) <= tol * 1e-3 * np.sqrt((ref ** 2).sum()) + TINY
    assert np.abs(r6).max() > 0 and np.abs(rt).max() > 0


def test_soft_mask_backward_full_size_and_determinism(gpu, oracle):
    torch, B = gpu
    N, K = 2048, 4096
    W = inputs.weight(N, K, 42, "bwd2")
    Gw = inputs.normal_bf16((N, K), 1.0, 42, "bwd2", "gw")
    PT, P6 = logits(N, K, 0.5, 42, "bwd2")
    tau, kappa, c1, c2 = 0.5, 120.0, -2.0e-7, 0.05
    args = (to_dev(torch, W), torch.from_numpy(PT).cuda(), torch.from_numpy(P6).cuda(), tau, kappa, to_dev(torch, Gw), c1, c2)
    gt, g6 = B.patch_soft_mask_backward(*args, seed=9)
    gt2, g62 = B.patch_soft_mask_backward(*args, seed=9)
    torch.cuda.synchronize()
    assert torch.equal(gt, gt2) and torch.equal(g6, g62)
    rt, r6 = oracle.soft_mask_backward(W, PT, P6, tau, kappa, f32(Gw), c1, c2, seed=9, noise=True)
    for got, ref in ((gt.cpu().numpy().astype(np.float64), rt), (g6.cpu().numpy().astype(np.float64), r6)):
        assert np.abs(got - ref).max() <= 2e-3 * np.abs(ref).max() + TINY
        assert np.sqrt(((got - ref) ** 2).sum()) <= 1e-3 * np.sqrt((ref ** 2).sum()) + TINY


def test_forward_backward_step_lowers_the_objective(gpu, oracle):
    """One gradient step on the logits, all on the device, lowers F = sum(Gw Mt W) + regularisers' linearisation."""
    torch, B = gpu
    N, K = 256, 512
    W = to_dev(torch, inputs.weight(N, K, 43, "step"))
    Gw = to_dev(torch, inputs.normal_bf16((N, K), 1.0, 43, "step", "gw"))
    PT0, P60 = logits(N, K, 0.5, 43, "step")
    PT = torch.from_numpy(PT0 * np.float32(0.004)).cuda()
    P6 = torch.from_numpy(P60).cuda()
    tau, kappa = 1.0, 30.0

    def objective(pt, p6):
        Mt = torch.empty((N, K), dtype=torch.float32, device="cuda")
        B.patch_soft_mask(W, pt, p6, tau, kappa, 7, 0, Mt=Mt)
        return float((Gw.float() * Mt * W.float()).double().sum())

    f0 = objective(PT, P6)
    gt, g6 = B.patch_soft_mask_backward(W, PT, P6, tau, kappa, Gw, 0.0, 0.0, seed=7)
    lr = 1e-3 / float(g6.abs().max())
    f1 = objective(PT - lr * gt, P6 - lr * g6)
    predicted = -lr * float((gt.double() ** 2).sum() + (g6.double() ** 2).sum())
    assert f1 < f0
    assert (f1 - f0) == pytest.approx(predicted, rel=0.15)       # a small step follows the linearisation


# ---------------------------------------------------------------------------------------------
# packing with the tile flags on the device


@pytest.mark.parametrize("N,K,p", [(128, 128, 1.0), (256, 384, 0.5), (1024, 1024, 0.0), (4096, 11008, 0.6), (11008, 4096, 0.3)])
def test_pack_dev_equals_pack(gpu, oracle, N, K, p):
    """The device-built header and table, and the payloads behind them, are byte for byte those of patch_pack
    (which the other tests compare with the oracle)."""
    torch, B = gpu
    W = to_dev(torch, inputs.weight(N, K, 51, "pdev", N, K))
    flags = inputs.tile_flags(N, K, p, 51, "pdev", N, K)
    ref, L = B.patch_pack(W, flags)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    fd = torch.from_numpy(np.ascontiguousarray(flags).reshape(-1)).cuda()
    out = B.patch_pack_dev(W, fd, status=status)
    Ld = B.patch_read_layout(out)
    assert int(status.item()) == 0
    assert bytes(Ld) == bytes(L)
    assert torch.equal(out[:L.total_bytes], ref)
    # an exactly sized buffer works too, and so does the given-mask variant
    out2 = B.patch_pack_dev(W, fd, out=torch.empty(L.total_bytes, dtype=torch.uint8, device="cuda"), status=status)
    assert int(status.item()) == 0 and torch.equal(out2, ref)
    patterns = torch.from_numpy(inputs.generator(51, "pdev", "pat", N, K).integers(0, 6, N * K // 4).astype(np.uint8)).cuda()
    ref_p, _ = B.patch_pack_patterns(W, flags, patterns)
    out_p = B.patch_pack_dev(W, fd, patterns=patterns, status=status)
    assert int(status.item()) == 0 and torch.equal(out_p[:L.total_bytes], ref_p)


def test_pack_dev_reports_size_and_flag_errors(gpu):
    torch, B = gpu
    N, K = 512, 512
    W = to_dev(torch, inputs.weight(N, K, 52, "pdev2"))
    flags = np.zeros(16, np.uint8)
    flags[[1, 5, 6]] = 1
    L = B.patch_packed_size(N, K, flags)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    fd = torch.from_numpy(flags).cuda()
    small = torch.full((L.total_bytes - 1024,), 0xAB, dtype=torch.uint8, device="cuda")   # above the all-2:4 minimum, below the need
    B.patch_pack_dev(W, fd, out=small, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.ERR_SIZE
    assert (small[L.payload_off:] == 0xAB).all()               # no payload was written
    with pytest.raises(B.PatchError) as e:
        B.patch_read_layout(small)
    assert e.value.status == B.ERR_FORMAT
    with pytest.raises(B.PatchError) as e:                      # below the smallest possible blob: refused on the host
        B.patch_pack_dev(W, fd, out=torch.empty(16 * 6000, dtype=torch.uint8, device="cuda"))
    assert e.value.status == B.ERR_SIZE
    status.zero_()
    bad = flags.copy()
    bad[3] = 7
    out = B.patch_pack_dev(W, torch.from_numpy(bad).cuda(), status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == B.ERR_FLAG
    ref, _ = B.patch_pack(W, flags)                             # the bad flag was packed as dense, which flags[3] is
    assert torch.equal(out[:L.total_bytes], ref)


def test_device_only_deployment_chain(gpu, oracle):
    """logits -> hard masks -> blob -> GEMM with no flag ever visiting the host before the layout read-back."""
    torch, B = gpu
    N, K, M = 768, 512, 5
    W = inputs.weight(N, K, 53, "chain2")
    X = inputs.activation(M, K, 53, "chain2", M)
    PT, P6 = logits(N, K, 0.5, 53, "chain2")
    flags_d, patterns_d = B.patch_hard_mask(torch.from_numpy(PT).cuda(), torch.from_numpy(P6).cuda(), N, K)
    packed = B.patch_pack_dev(to_dev(torch, W), flags_d, patterns=patterns_d)
    L = B.patch_read_layout(packed)
    ws = torch.zeros(max(B.patch_gemm_workspace_size(L, M), 1), dtype=torch.uint8, device="cuda")
    Y = to_bits(B.patch_gemm(to_dev(torch, X), L, packed, workspace=ws))
    rf, rp = oracle.hard_mask(PT, P6, N, K)
    assert (L.n_dense, L.n_sparse) == (int((rf == 0).sum()), int((rf == 1).sum()))
    Y32, _ = oracle.gemm_f64(X, oracle.unpack(oracle.pack_patterns(W, rf, rp)[0]))
    relF, maxrel = oracle.parity_metrics(f32(Y), Y32)
    assert relF <= 2e-3 and maxrel <= 1e-2, (relF, maxrel)


def test_device_only_deployment_chain_with_4bit_tiles(gpu, oracle):
    """The same chain for the 4-bit combination: learned flags and candidates stay on the device, bit 1 is set on the
    device, the blob is the oracle's for the same masks, and the matmul multiplies by its dequantised matrix."""
    torch, B = gpu
    N, K, M = 768, 512, 5
    W = inputs.weight(N, K, 54, "chain4")
    X = inputs.activation(M, K, 54, "chain4", M)
    PT, P6 = logits(N, K, 0.5, 54, "chain4")
    flags_d, patterns_d = B.patch_hard_mask(torch.from_numpy(PT).cuda(), torch.from_numpy(P6).cuda(), N, K)
    packed = B.patch_pack_dev(to_dev(torch, W), flags_d | 2, patterns=patterns_d)
    L = B.patch_read_layout(packed)
    rf, rp = oracle.hard_mask(PT, P6, N, K)
    assert (L.n_dense, L.n_sparse, L.n_dense_q4, L.n_sparse_q4) == (0, 0, int((rf == 0).sum()), int((rf == 1).sum()))
    blob_o, _ = oracle.pack_patterns(W, rf | 2, rp)
    assert (packed[:L.total_bytes].cpu().numpy() == oracle.device_image(blob_o)).all()
    Y = to_bits(B.patch_gemm(to_dev(torch, X), L, packed[:L.total_bytes]))
    Y32, _ = oracle.gemm_f64(X, oracle.unpack(blob_o))
    relF, maxrel = oracle.parity_metrics(f32(Y), Y32)
    assert relF <= 2e-3 and maxrel <= 1e-2, (relF, maxrel)
