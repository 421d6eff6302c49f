"""Failure paths on the GPU, exercised without faulting, trapping or hanging anything.

* A bounded device-side wait that really runs out: the fault-injection build of the library (same sources, waits
  limited to 300 us) lets the test tell the stream-K decode kernel, through its status word, to announce sixteen
  bytes more than its first stage will ever receive.  The MMA warp's wait expires, the CTA raises its abort flag,
  reports PATCH_ERR_TIMEOUT, drains, frees its tensor memory and returns; the context stays usable.  The kernel of
  the 4-bit tile kinds has the same hook.
* A tile table that does not belong to the layout: every kernel checks each entry against the blob's extent before
  it requests a byte of the tile, reports PATCH_ERR_FORMAT and reads the first payload instead.  The bad offsets used
  here point inside the test's own over-allocated buffer, so a check that failed to catch them could not fault."""
import ctypes

import numpy as np
import pytest

from paper_2509_23410_b200 import inputs
from test_gpu_parity import check_parity, gpu, to_bits, to_dev  # noqa: F401  (gpu is a fixture)

pytestmark = pytest.mark.gpu

INJECT_MAGIC = 0x7E57


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else ctypes.c_void_p(0)


def test_a_bounded_wait_that_runs_out_is_reported_and_survivable(gpu, oracle):
    torch, B = gpu
    from paper_2509_23410_b200 import build
    fi = B.load(build.build(fault_injection=True))          # built on demand (about a minute), in-tree
    N, K, M = 512, 1024, 16
    W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=0.5, stream=("timeout",)), 71, M)
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Xd = to_dev(torch, X)
    Y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(B.patch_gemm_workspace_size(L, M), dtype=torch.uint8, device="cuda")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

    def call(status):
        rc = fi.patch_gemm_ex(_ptr(Xd), K, M, ctypes.byref(L), _ptr(packed), _ptr(Y), N, _ptr(ws), ws.numel(), _ptr(status),
                              stream, B.VARIANT_MMA)
        assert rc == B.OK
        torch.cuda.synchronize()
        return int(status.item())

    # the same build, no injection: a normal result (the 300 us limit is far above this kernel's few microseconds)
    assert call(torch.zeros(1, dtype=torch.int32, device="cuda")) == B.OK
    check_parity(oracle, to_bits(Y), oracle.gemm_f64(X, What)[0], "fault-injection build, no injection")
    # injection: CTA 0's first stage can never complete; its wait runs out
    status = torch.full((1,), INJECT_MAGIC, dtype=torch.int32, device="cuda")
    assert call(status) == B.ERR_TIMEOUT
    # the context is alive, and after re-initialising the workspace (the aborted CTA left partial sums behind)
    # the next call -- through the product build -- is correct
    B.patch_workspace_init(ws)
    Y.zero_()
    status.zero_()
    B.patch_gemm(Xd, L, packed, Y=Y, workspace=ws, status=status, variant=B.VARIANT_MMA)
    torch.cuda.synchronize()
    assert int(status.item()) == B.OK
    check_parity(oracle, to_bits(Y), oracle.gemm_f64(X, What)[0], "after the timeout")
    # and the injected build again, without injection
    assert call(torch.zeros(1, dtype=torch.int32, device="cuda")) == B.OK


def test_a_wait_of_the_4bit_kernel_that_runs_out(gpu, oracle):
    """The same for the kernel of the 4-bit tile kinds: the group that waits for CTA 0's first payload gives up,
    the CTA's other roles follow, the launch completes with PATCH_ERR_TIMEOUT and the next launch is correct."""
    torch, B = gpu
    from paper_2509_23410_b200 import build
    fi = B.load(build.build(fault_injection=True))
    N, K, M = 512, 2048, 16
    W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=0.5, stream=("timeout-q4",)), 73, M)
    flags = flags | 2
    What = oracle.prune(W, flags)
    packed, L = B.patch_pack(to_dev(torch, W), flags)
    Xd = to_dev(torch, X)
    Y = torch.zeros((M, N), dtype=torch.bfloat16, device="cuda")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    ref = oracle.gemm_f64(X, What)[0]

    def call(status, variant):
        rc = fi.patch_gemm_ex(_ptr(Xd), K, M, ctypes.byref(L), _ptr(packed), _ptr(Y), N, ctypes.c_void_p(0), 0, _ptr(status),
                              stream, variant)
        assert rc == B.OK
        torch.cuda.synchronize()
        return int(status.item())

    for variant in (B.VARIANT_AUTO, B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC):
        assert call(torch.zeros(1, dtype=torch.int32, device="cuda"), variant) == B.OK
        check_parity(oracle, to_bits(Y), ref, "fault-injection build, no injection")
        status = torch.full((1,), INJECT_MAGIC, dtype=torch.int32, device="cuda")
        assert call(status, variant) == B.ERR_TIMEOUT
        Y.zero_()
        status.zero_()
        B.patch_gemm(Xd, L, packed, Y=Y, status=status, variant=variant)
        torch.cuda.synchronize()
        assert int(status.item()) == B.OK
        check_parity(oracle, to_bits(Y), ref, "after the timeout")


@pytest.mark.parametrize("M,variant", [(1, "gemv"), (1, "independent"), (16, "independent"), (16, "streamk"), (48, "streamk"),
                                       (300, "auto"), (700, "auto")])
@pytest.mark.parametrize("corruption", ["kind", "offset_beyond_blob", "offset_before_payloads"])
def test_bad_tile_table_entries_are_reported_not_followed(gpu, oracle, M, variant, corruption):
    torch, B = gpu
    if variant == "streamk" and corruption != "kind" and M != 16:
        # the stream-K schedule also derives its work split from the offsets; one such case is enough (below)
        pytest.skip("covered by the M = 16 case")
    N, K = 1024, 1024
    W, flags, X = inputs.make_case_inputs(dict(N=N, K=K, p=0.5, stream=("badtable",)), 72, M)
    What = oracle.prune(W, flags)
    good, L = B.patch_pack(to_dev(torch, W), flags)
    # the blob sits in the middle of a buffer three times its size: an offset that leaves the blob stays in the buffer
    big = torch.zeros(3 * L.total_bytes, dtype=torch.uint8, device="cuda")
    base = L.total_bytes - L.total_bytes % 1024
    blob = big[base:base + L.total_bytes]
    blob.copy_(good)
    table = blob[L.table_off:L.table_off + 16 * (N // 128) * (K // 128)].view(torch.int32).view(-1, 4)
    t = 37                                                   # some tile in the middle of the matrix
    saved = table[t].clone()
    if corruption == "kind":
        table[t, 0] = 7
    elif corruption == "offset_beyond_blob":
        table[t, 1] = (L.total_bytes + 4096) // 16           # inside `big`, outside the blob
    else:
        table[t, 1] = 0                                      # the header, not a payload
    vflags = {"gemv": B.VARIANT_GEMV, "independent": B.VARIANT_AUTO | B.WEIGHTS_STATIC | B.INPUT_STATIC,
              "streamk": B.VARIANT_MMA, "auto": B.VARIANT_AUTO}[variant]
    Xd = to_dev(torch, X)
    ws = torch.zeros(max(B.patch_gemm_workspace_size(L, M), 1), dtype=torch.uint8, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    B.patch_gemm(Xd, L, blob, workspace=ws, status=status, variant=vflags)
    torch.cuda.synchronize()
    if variant == "streamk" and corruption != "kind":
        # a wrong offset can also upset the split of the work, whose bounded waits then run out: the first error
        # reported is one of the two, and nothing was read out of range either way
        assert int(status.item()) in (B.ERR_FORMAT, B.ERR_TIMEOUT)
    else:
        assert int(status.item()) == B.ERR_FORMAT
    # with the entry restored the same call is clean and correct
    table[t] = saved
    status.zero_()
    B.patch_workspace_init(ws)
    Y = B.patch_gemm(Xd, L, blob, workspace=ws, status=status, variant=vflags)
    torch.cuda.synchronize()
    assert int(status.item()) == B.OK
    if M <= 64:
        check_parity(oracle, to_bits(Y), oracle.gemm_f64(X, What)[0], f"{variant} M={M}")
    else:
        rows = np.array([0, 1, M // 2, M - 1])
        check_parity(oracle, to_bits(Y)[rows], oracle.gemm_f64_rows(X, rows, What), f"{variant} M={M}")
