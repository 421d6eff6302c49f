"""The entry point for callers that cannot allocate device memory (a plug-in given only pointers
and a stream, code running under a frozen memory pool): it must give the same result as the
regular call that uses a caller-owned workspace, call after call, with no buffer of its own
passed in.  Collected last on purpose: a failure here stops nothing that runs before it."""
import numpy as np
import pytest

from paper_2509_23410_b200 import inputs

pytestmark = pytest.mark.gpu


def test_noalloc_entry_point_matches_regular_call(oracle):
    import torch
    from paper_2509_23410_b200 import binding as B
    assert torch.cuda.is_available(), "GPU tests must run on a B200"
    B.lib()
    to_dev = lambda b: torch.from_numpy(np.ascontiguousarray(b).view(np.int16)).cuda().view(torch.bfloat16)
    f32 = lambda t: inputs.bf16_bits_to_f32(t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16))
    results = []
    for call, (N, K, M, p) in enumerate([(1024, 1024, 16, 0.5), (512, 2304, 5, 0.7)]):   # two calls in a row
        W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=p, stream=("noalloc", call)), 31, M)
        packed, L = B.patch_pack(to_dev(W), flags)
        Xd = to_dev(X)
        ws = torch.zeros(B.patch_gemm_workspace_size(L, M), dtype=torch.uint8, device="cuda")
        Y_ref = B.patch_gemm(Xd, L, packed, workspace=ws, variant=B.VARIANT_MMA)
        Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")     # the caller still owns inputs and outputs
        B.patch_gemm_noalloc(Xd, L, packed, Y)
        torch.cuda.synchronize()
        relF, maxrel = oracle.parity_metrics(f32(Y), f32(Y_ref))
        assert relF <= 2e-3 and maxrel <= 1e-2, (call, relF, maxrel)
        assert torch.equal(Y, Y_ref)          # same kernel, same summation order
        results.append(Y)
        # and against the oracle, like every other GEMM test
        Y32, _ = oracle.gemm_f64(X, oracle.prune(W, flags))
        relF, maxrel = oracle.parity_metrics(f32(Y), Y32)
        assert relF <= 2e-3 and maxrel <= 1e-2, (call, relF, maxrel)
    # sizes beyond the fixed scratch are refused, nothing is launched
    W, flags, X = inputs.make_case_inputs(dict(N=256, K=256, p=0.5, stream=("noalloc", "big")), 31, 17)
    packed, L = B.patch_pack(to_dev(W), flags)
    with pytest.raises(B.PatchError) as e:
        B.patch_gemm_noalloc(to_dev(X), L, packed, torch.empty((17, 256), dtype=torch.bfloat16, device="cuda"))
    assert e.value.status == B.ERR_SIZE
