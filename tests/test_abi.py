"""Host-side checks of the C ABI: the library loads without a GPU, exports every symbol the
header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re
import subprocess

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2509_23410_b200 import build
    build.build()
    from paper_2509_23410_b200 import binding as b
    return b


def declared_functions():
    text = open(os.path.join(ROOT, "include", "patch.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(patch_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(binding):
    names = declared_functions()
    assert "patch_gemm" in names and "patch_pack" in names and len(names) >= 9
    L = binding.lib()
    for n in names:
        assert hasattr(L, n), n
    assert sorted(binding.EXPORTS) == names


def test_layout_struct_matches_header(binding, tmp_path):
    assert ctypes.sizeof(binding.Layout) == 96
    assert binding.patch_version() == 1
    # size and field offsets as a C compiler lays the header's struct out
    src = tmp_path / "layout.c"
    fields = [f for f, _ in binding.Layout._fields_]
    src.write_text('#include <stdio.h>\n#include <stddef.h>\n#include "patch.h"\nint main(void) {\n'
                   '  printf("%zu", sizeof(patch_layout_t));\n' +
                   "".join(f'  printf(" %zu", offsetof(patch_layout_t, {f}));\n' for f in fields) + "  return 0; }\n")
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)], check=True)
    got = [int(v) for v in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
    assert got == [ctypes.sizeof(binding.Layout)] + [getattr(binding.Layout, f).offset for f in fields]


def test_packed_size_and_validation(binding, oracle):
    flags = np.array([[0, 1, 1], [1, 0, 0]], np.uint8)
    L = binding.patch_packed_size(256, 384, flags)
    Lo = oracle.packed_size(256, 384, flags)
    for f, _ in binding.Layout._fields_:
        assert getattr(L, f) == getattr(Lo, f), f
    assert L.payload_bytes == 3 * 32768 + 3 * 18432
    # all four kinds
    flags4 = np.array([[0, 3, 2], [1, 2, 3]], np.uint8)
    L = binding.patch_packed_size(256, 384, flags4)
    Lo = oracle.packed_size(256, 384, flags4)
    for f, _ in binding.Layout._fields_:
        assert getattr(L, f) == getattr(Lo, f), f
    assert L.payload_bytes == 32768 + 18432 + 2 * 8448 + 2 * 6400
    with pytest.raises(binding.PatchError) as e:
        binding.patch_packed_size(256, 384, np.full((2, 3), 4, np.uint8))
    assert e.value.status == binding.ERR_FLAG
    with pytest.raises(binding.PatchError) as e:
        binding.patch_packed_size(250, 384, flags)
    assert e.value.status == binding.ERR_SHAPE
    with pytest.raises(binding.PatchError) as e:
        binding.patch_packed_size(256, 384, flags, 64, 128)
    assert e.value.status == binding.ERR_TILE


def test_gemm_rejects_bad_arguments_on_host(binding):
    lib = binding.lib()
    flags = np.zeros((1, 1), np.uint8)
    L = binding.patch_packed_size(128, 128, flags)
    null = ctypes.c_void_p(0)
    fake = ctypes.c_void_p(1024 * 1024)   # never dereferenced: validation fails first
    args = lambda X, ldx, M, Lp, P, Y, ldy: (X, ldx, M, Lp, P, Y, ldy, null, 0, null, null)
    assert lib.patch_gemm(*args(null, 128, 4, ctypes.byref(L), fake, fake, 128)) == binding.ERR_NULL
    assert lib.patch_gemm(*args(fake, 64, 4, ctypes.byref(L), fake, fake, 128)) == binding.ERR_SHAPE
    assert lib.patch_gemm(*args(fake, 128, 4, ctypes.byref(L), fake, fake, 100)) == binding.ERR_SHAPE
    assert lib.patch_gemm(*args(ctypes.c_void_p(1024 * 1024 + 2), 128, 4, ctypes.byref(L), fake, fake, 128)) == binding.ERR_ALIGN
    assert lib.patch_gemm(*args(fake, 128, -1, ctypes.byref(L), fake, fake, 128)) == binding.ERR_SHAPE
    assert lib.patch_gemm(*args(null, 128, 0, ctypes.byref(L), null, null, 128)) == binding.OK   # M = 0: no launch
    bad = binding.Layout.from_buffer_copy(bytes(L))
    bad.magic = 0
    assert lib.patch_gemm(*args(fake, 128, 4, ctypes.byref(bad), fake, fake, 128)) == binding.ERR_FORMAT
    bad = binding.Layout.from_buffer_copy(bytes(L))
    bad.payload_bytes += 1024
    assert lib.patch_gemm(*args(fake, 128, 4, ctypes.byref(bad), fake, fake, 128)) == binding.ERR_FORMAT
    bad = binding.Layout.from_buffer_copy(bytes(L))
    bad.tile_k = 64
    assert lib.patch_gemm(*args(fake, 128, 4, ctypes.byref(bad), fake, fake, 128)) == binding.ERR_TILE
    assert lib.patch_gemm_ex(*args(fake, 128, 9, ctypes.byref(L), fake, fake, 128), binding.VARIANT_GEMV) == binding.ERR_SHAPE
    assert lib.patch_pack(null, 128, null, ctypes.byref(L), fake, 1 << 20, null) == binding.ERR_NULL
    f = np.zeros(1, np.uint8)
    assert lib.patch_pack(fake, 128, ctypes.c_void_p(f.ctypes.data), ctypes.byref(L), fake, 10, null) == binding.ERR_SIZE
    assert b"timed out" in lib.patch_strerror(binding.ERR_TIMEOUT)


def test_4bit_weights_are_refused_where_no_kernel_serves_them(binding):
    """Weights with 4-bit tiles: mixtures with bf16 tiles, the GEMV variant, the gated product and the
    no-allocation entry point are refused on the host, before any device is touched."""
    lib = binding.lib()
    null = ctypes.c_void_p(0)
    fake = ctypes.c_void_p(1024 * 1024)   # never dereferenced: validation fails first
    L4 = binding.patch_packed_size(256, 256, np.array([[2, 3], [3, 2]], np.uint8))
    Lm = binding.patch_packed_size(256, 256, np.array([[2, 0], [3, 1]], np.uint8))
    args = lambda M, Lp: (fake, 256, M, ctypes.byref(Lp), fake, fake, 256, null, 0, null, null)
    assert lib.patch_gemm(*args(4, Lm)) == binding.ERR_SHAPE
    assert lib.patch_gemm_ex(*args(4, L4), binding.VARIANT_GEMV) == binding.ERR_SHAPE
    assert lib.patch_gemm_gated(*args(4, L4), 0) == binding.ERR_SHAPE
    assert lib.patch_gemm_noalloc(fake, 256, 4, ctypes.byref(L4), fake, fake, 256, null) == binding.ERR_SHAPE
    assert binding.patch_gemm_workspace_size(L4, 16) == 0
    # a layout whose counts do not add up to the tile count, or whose bytes do not follow from the counts
    bad = binding.Layout.from_buffer_copy(bytes(L4))
    bad.n_dense_q4 -= 1
    assert lib.patch_gemm(*args(4, bad)) == binding.ERR_FORMAT
    bad = binding.Layout.from_buffer_copy(bytes(L4))
    bad.n_dense_q4, bad.n_sparse_q4 = bad.n_sparse_q4 + 1, bad.n_dense_q4 - 1
    assert lib.patch_gemm(*args(4, bad)) == binding.ERR_FORMAT


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2509_23410_b200")
    for dirpath, _, files in os.walk(pkg):
        for fn in files:
            if fn.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, fn)).read()
                assert "import oracle" not in text and "from oracle" not in text, fn
                assert "patch_oracle" not in text, fn


def test_library_reads_no_environment_variable():
    """The schedules are fixed in the source: no knob such as PATCH_DECODE_CLUSTER_S can change a launch."""
    csrc = os.path.join(ROOT, "paper_2509_23410_b200", "csrc")
    for fn in os.listdir(csrc):
        text = open(os.path.join(csrc, fn)).read()
        assert "getenv" not in text and "environ" not in text, fn
    build_py = open(os.path.join(ROOT, "paper_2509_23410_b200", "build.py")).read()
    assert "NVCC_FLAGS" not in build_py


def test_stacked_case_flags_concatenate_parts():
    """Input recipe of the stacked-matrix workload: flags of q/k/v (gate/up) stacked along N."""
    import numpy as np
    from paper_2509_23410_b200 import inputs
    plain = {c["name"]: c for c in inputs.stack_cases(n_blocks=1)}
    fused = inputs.stack_fused_cases(n_blocks=1)
    assert [c["N"] for c in fused] == [12288, 4096, 22016, 4096] and len(fused) == 4
    qkv = inputs.case_flags(fused[0])
    parts = [inputs.tile_flags(4096, 4096, plain[f"stack.0.{r}"]["p"], inputs.MASTER_SEED, "stack", 0, r) for r in "qkv"]
    assert np.array_equal(qkv, np.concatenate(parts, axis=0))
    assert abs(fused[0]["p"] - sum(plain[f"stack.0.{r}"]["p"] for r in "qkv") / 3) < 1e-12


def test_gated_entry_validates_on_the_host():
    """patch_gemm_gated: argument errors are reported before any launch (no GPU here)."""
    import ctypes
    import numpy as np
    from paper_2509_23410_b200 import binding as B
    lib = B.lib()
    ok = B.patch_packed_size(512, 256, np.zeros((4, 2), np.uint8))
    odd = B.patch_packed_size(384, 256, np.zeros((3, 2), np.uint8))
    buf = ctypes.create_string_buffer(64)
    p = ctypes.cast(buf, ctypes.c_void_p)

    def call(X, ldx, M, L, Y, ldy, flags=0):
        return lib.patch_gemm_gated(X, ldx, M, ctypes.byref(L), p, Y, ldy, None, 0, None, None, flags)

    assert call(p, 256, 4, odd, p, 192) == B.ERR_SHAPE      # N % 256
    assert call(None, 256, 4, ok, p, 256) == B.ERR_NULL
    assert call(p, 128, 4, ok, p, 256) == B.ERR_SHAPE       # ldx < K
    assert call(p, 256, 4, ok, p, 248) == B.ERR_SHAPE       # ldy < N / 2
    assert call(p, 256, 0, ok, p, 256) == 0                 # M = 0
    assert call(p, 256, -1, ok, p, 256) == B.ERR_SHAPE
    assert call(p, 256, 4, ok, p, 256, flags=1) == B.ERR_SHAPE      # only the two *_STATIC flags
    # workspace of the small-M schedule: past everything patch_gemm uses of a shared buffer, one slot per pair
    assert B.patch_gemm_gated_workspace_size(ok, 16) == B.patch_gemm_workspace_size(ok, 64) + 2 * 128 * 16 * 4
    assert B.patch_gemm_gated_workspace_size(ok, 17) == 0


def test_host_batch_validates_before_enqueueing():
    """patch_gemm_host_batch: an empty batch is a no-op, bad jobs are rejected on the host (no GPU here)."""
    import ctypes
    import numpy as np
    from paper_2509_23410_b200 import binding as B
    lib = B.lib()
    assert lib.patch_gemm_host_batch(None, 0, 0, None) == 0
    assert lib.patch_gemm_host_batch(None, 2, 0, None) == B.ERR_NULL
    assert lib.patch_gemm_host_batch(None, -1, 0, None) == B.ERR_SHAPE
    L = B.patch_packed_size(256, 256, np.zeros((2, 2), np.uint8))
    jobs = (B.HostJob * 2)()
    for j in jobs:
        j.M, j.layout = 4, ctypes.pointer(L)          # every pointer NULL
    assert lib.patch_gemm_host_batch(jobs, 2, 1, None) == B.ERR_NULL
    jobs[1].M = -3
    assert lib.patch_gemm_host_batch(jobs, 2, 1, None) == B.ERR_NULL      # job 0 is checked first
    jobs[0].M = 0
    assert lib.patch_gemm_host_batch(jobs, 2, 1, None) == B.ERR_SHAPE


def test_mask_entry_points_validate_on_the_host():
    """Shape, tile, pointer and alignment errors of the mask entry points are reported before any device is touched."""
    import ctypes
    from paper_2509_23410_b200 import binding as B
    lib = B.lib()
    buf = (ctypes.c_double * 64)()
    p = ctypes.addressof(buf)
    assert lib.patch_hard_mask(p, p, 128, 100, 128, 128, p, p, None) == B.ERR_SHAPE
    assert lib.patch_hard_mask(p, p, 128, 128, 128, 64, p, p, None) == B.ERR_TILE
    assert lib.patch_hard_mask(None, p, 128, 128, 128, 128, p, p, None) == B.ERR_NULL
    n = ctypes.c_size_t(0)
    assert lib.patch_soft_mask_workspace_size(4096, 11008, 128, 128, ctypes.byref(n)) == 0
    assert n.value == 32 * 86 * 32
    assert lib.patch_soft_mask_workspace_size(4096, 11000, 128, 128, ctypes.byref(n)) == B.ERR_SHAPE
    assert lib.patch_soft_mask(p, 128, p, p, 128, 128, 128, 128, -1.0, 1.0, 0, 0, p, 128, None, 0, p, p, 128, None) == B.ERR_SHAPE
    assert lib.patch_soft_mask(p, 120, p, p, 128, 128, 128, 128, 1.0, 1.0, 0, 0, p, 128, None, 0, p, p, 128, None) == B.ERR_SHAPE
    assert lib.patch_soft_mask(p, 128, p, p, 128, 128, 128, 128, 1.0, 1.0, 0, 0, p, 128, None, 0, p, p, 16, None) == B.ERR_SIZE
    assert lib.patch_pack_patterns(p, 128, p, None, None, p, 0, None, None) == B.ERR_NULL
    # the regularisers: 7 |75/100 - 1/2| - 10 * 30/60, and pooled sums over two matrices
    assert B.patch_mask_regularizers([[75, 100, 30, 60]], 0.5, 7, 10) == -3.25
    two = [[10, 40, 1, 4], [50, 60, 5, 6]]
    assert abs(B.patch_mask_regularizers(two, 0.9, 3, 0.1) - (3 * abs(60 / 100 - 0.9) - 0.1 * 6 / 10)) < 1e-15
    out = ctypes.c_double(0)
    assert lib.patch_mask_regularizers(p, 0, 0.5, 1.0, 1.0, ctypes.byref(out)) == B.ERR_SHAPE
    assert lib.patch_mask_regularizers(p, 1, 0.5, 1.0, 1.0, ctypes.byref(out)) == B.ERR_SHAPE   # all-zero sums: no weights


def test_mask_backward_validates_on_the_host():
    import ctypes
    from paper_2509_23410_b200 import binding as B
    lib = B.lib()
    buf = (ctypes.c_double * 64)()
    p = ctypes.addressof(buf)
    ok = (p, 128, p, p, 128, 128, 128, 128, 1.0, 1.0, 0, 0, p, 128, 0.0, 0.0, p, p, None)
    bad = lambda i, v: ok[:i] + (v,) + ok[i + 1:]
    assert lib.patch_soft_mask_backward(*bad(8, 0.0)) == B.ERR_SHAPE            # tau
    assert lib.patch_soft_mask_backward(*bad(14, float("inf"))) == B.ERR_SHAPE  # c1
    assert lib.patch_soft_mask_backward(*bad(13, 100)) == B.ERR_SHAPE           # ldg < K
    assert lib.patch_soft_mask_backward(*bad(12, None)) == B.ERR_NULL           # Gw
    assert lib.patch_soft_mask_backward(*bad(17, p + 4)) == B.ERR_ALIGN         # gP24
    assert lib.patch_soft_mask_backward(*bad(6, 64)) == B.ERR_TILE
    c1, c2 = B.patch_mask_regularizer_coefficients([[60.0, 100, 30, 60], [20.0, 50, 8, 20]], 0.4, 7.0, 10.0)
    assert abs(c1 - 7.0 / 150) < 1e-15 and abs(c2 - 0.25) < 1e-15
    assert B.patch_mask_regularizer_coefficients([[60.0, 100, 30, 60]], 0.9, 7.0, 10.0)[0] == -0.07


def test_pack_dev_validates_on_the_host():
    import ctypes
    from paper_2509_23410_b200 import binding as B
    lib = B.lib()
    buf = (ctypes.c_double * 64)()
    p = ctypes.addressof(buf)
    assert lib.patch_pack_dev(p, 128, None, None, 128, 128, 128, 128, p, 1 << 20, None, None) == B.ERR_NULL
    assert lib.patch_pack_dev(p, 128, p, None, 128, 192, 128, 128, p, 1 << 20, None, None) == B.ERR_SHAPE
    assert lib.patch_pack_dev(p, 120, p, None, 128, 128, 128, 128, p, 1 << 20, None, None) == B.ERR_SHAPE
    assert lib.patch_pack_dev(p, 128, p, None, 128, 128, 128, 64, p, 1 << 20, None, None) == B.ERR_TILE
    assert lib.patch_pack_dev(p, 128, p, p + 2, 128, 128, 128, 128, p, 1 << 20, None, None) == B.ERR_ALIGN
    assert lib.patch_pack_dev(p, 128, p, None, 128, 128, 128, 128, p, 1024 + 6399, None, None) == B.ERR_SIZE
    assert lib.patch_read_layout(None, None, None) == B.ERR_NULL


def test_pipelined_host_batch_validates_before_enqueueing():
    import ctypes
    from paper_2509_23410_b200 import binding as B
    lib = B.lib()
    assert lib.patch_gemm_host_batch_pipelined(None, 0, 0, 4, None, None, None) == 0        # empty batch: nothing to do
    assert lib.patch_gemm_host_batch_pipelined(None, 3, 0, 4, None, None, None) == B.ERR_NULL
    jobs = (B.HostJob * 1)()
    assert lib.patch_gemm_host_batch_pipelined(jobs, 1, 0, 4, None, None, None) == B.ERR_NULL   # no layout
