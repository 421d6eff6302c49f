"""B200-native tile-hybrid linear layer (PATCH deployment path): C-ABI CUDA library + thin binding."""
from .binding import (  # noqa: F401
    Layout, PatchError, TILE_DENSE, TILE_SPARSE_2_4, VARIANT_AUTO, VARIANT_GEMV, VARIANT_MMA, WEIGHTS_STATIC, INPUT_STATIC, OUTPUT_STATIC,
    patch_gemm, patch_gemm_host, patch_gemm_noalloc, patch_gemm_workspace_size, patch_pack, patch_packed_size, patch_unpack,
    patch_version, patch_workspace_init, strerror,
)
