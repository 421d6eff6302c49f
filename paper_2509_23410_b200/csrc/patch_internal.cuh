// Internal definitions shared by the library's translation units (not part of the C ABI).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <atomic>
#include "../../include/patch.h"

namespace patch {

constexpr uint32_t kMagic = 0x48435450u;
constexpr uint32_t kVersion = 1u;
constexpr int kTile = 128;
constexpr uint32_t kDenseBytes = 32768u;    // two 16 KB atoms
constexpr uint32_t kSparseBytes = 18432u;   // one 16 KB atom + 2 KB metadata
constexpr uint32_t kAtomBytes = 16384u;
constexpr uint32_t kMetaBytes = 2048u;
constexpr uint32_t kHeaderBytes = 256u;
// 4-bit kinds: codes (8192 / 4096 B) [+ metadata 2048 B] + 128 bf16 scales
constexpr uint32_t kScaleBytes = 256u;
constexpr uint32_t kDenseQ4CodeBytes = 8192u, kSparseQ4CodeBytes = 4096u;
constexpr uint32_t kDenseQ4Bytes = kDenseQ4CodeBytes + kScaleBytes;                    // 8 448
constexpr uint32_t kSparseQ4Bytes = kSparseQ4CodeBytes + kMetaBytes + kScaleBytes;     // 6 400
__host__ __device__ constexpr uint32_t tile_payload_bytes(uint32_t kind) {
    return kind == PATCH_TILE_DENSE ? kDenseBytes : kind == PATCH_TILE_SPARSE_2_4 ? kSparseBytes
         : kind == PATCH_TILE_DENSE_Q4 ? kDenseQ4Bytes : kSparseQ4Bytes;
}

// One entry of the tile table inside the packed blob.
struct TileDesc {
    uint32_t kind;          // PATCH_TILE_DENSE / PATCH_TILE_SPARSE_2_4
    uint32_t payload_off16; // byte offset / 16 from the start of the blob
    uint32_t meta_off16;    // byte offset / 16 of the metadata block, 0xFFFFFFFF if dense
    uint32_t scales_off16;  // byte offset / 16 of the scales of a 4-bit kind, 0 otherwise
};
static_assert(sizeof(TileDesc) == 16, "tile table entry is 16 bytes");

// Byte offset of 16-byte chunk `c` (0..7) of row `r` (0..127) inside a 128-byte-swizzled
// K-major atom of 128 rows x 128 bytes.
__host__ __device__ inline uint32_t atom_chunk_offset(uint32_t r, uint32_t c) {
    return (r >> 3) * 1024u + (r & 7u) * 128u + ((c ^ (r & 7u)) << 4);
}

// Trap-free check of a tile-table entry read from device memory, made before any byte of the tile is requested.
// The host validates the layout struct, but the table inside the blob is the caller's device memory: an entry
// whose kind is unknown or whose payload does not lie inside [first payload, end of blob) is reported
// (PATCH_ERR_FORMAT in status_dev) and replaced by the first payload read as a 2:4 tile -- 18 432 bytes that lie
// inside every blob -- so that the launch runs to its end with a defined status and an undefined Y instead of
// reading out of range.
__device__ __forceinline__ void sanitize_tile(uint32_t& kind, uint32_t& off16, uint32_t pay0_16, uint32_t end16,
                                              int* status_dev) {
    const uint32_t len16 = (kind == PATCH_TILE_DENSE ? kDenseBytes : kSparseBytes) / 16;
    if (kind > PATCH_TILE_SPARSE_2_4 || off16 < pay0_16 || off16 > end16 || len16 > end16 - off16) {
        if (status_dev) atomicCAS(status_dev, PATCH_OK, PATCH_ERR_FORMAT);
        kind = PATCH_TILE_SPARSE_2_4;
        off16 = pay0_16;
    }
}

// Host-side checks of a layout struct handed in by the caller.
int validate_layout(const patch_layout_t* L);

// Status of the current device: PATCH_OK if it is sm_100, PATCH_ERR_ARCH / PATCH_ERR_CUDA otherwise.
int check_device();

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// What the library remembers between calls is per device: which kernels had their shared-memory limit
// raised there, and the device's SM count.  A process may drive several GPUs from several threads.
constexpr int kMaxDevices = 64;
inline int current_device() {
    int d = -1;
    return (cudaGetDevice(&d) == cudaSuccess && d >= 0 && d < kMaxDevices) ? d : -1;
}
// Number of SMs of the current device (0 on failure).
inline int sm_count() {
    static std::atomic<int> cache[kMaxDevices];
    const int d = current_device();
    if (d < 0) return 0;
    int n = cache[d].load(std::memory_order_relaxed);
    if (n == 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, d) != cudaSuccess) return 0;
        cache[d].store(n, std::memory_order_relaxed);
    }
    return n;
}
// Raises a kernel's dynamic shared-memory limit once per device; `done` is that kernel's bit mask of devices.
template <class Kernel>
inline int allow_dynamic_smem(Kernel kern, uint32_t bytes, std::atomic<uint64_t>& done) {
    const int d = current_device();
    if (d < 0) return PATCH_ERR_CUDA;
    if ((done.load(std::memory_order_acquire) >> d) & 1u) return PATCH_OK;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bytes)) != cudaSuccess)
        return PATCH_ERR_CUDA;
    done.fetch_or(uint64_t(1) << d, std::memory_order_release);
    return PATCH_OK;
}

// Kernel launchers implemented in the .cu files; all return a PATCH_* status.
// `wstatic` / `xstatic`: the packed weight / X was not written by the operation preceding this
// launch in the stream.
int launch_gemv(const __nv_bfloat16* X, int64_t ldx, int M, const patch_layout_t* L,
                const uint8_t* packed, __nv_bfloat16* Y, int64_t ldy, int* status_dev,
                cudaStream_t stream);
int launch_decode(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L,
                  const uint8_t* packed, __nv_bfloat16* Y, int64_t ldy, void* workspace, int* status_dev,
                  cudaStream_t stream, bool wstatic, bool xstatic, bool ystatic = false);
// `independent`: the caller declared the GEMM independent of its predecessor (weights and X static): only its
// Y stores wait for the preceding kernel.
// `force_pair`: only the CTA-pair schedule will do (PATCH_ERR_SHAPE if the weight mixes tile kinds).
int launch_prefill(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L,
                   const uint8_t* packed, __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream,
                   bool independent, bool force_pair = false);
int launch_prefill_gated(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L,
                         const uint8_t* packed, __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream,
                         bool independent);
size_t decode_workspace_bytes(const patch_layout_t* L, int64_t M);
int launch_decode_gated(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L,
                        const uint8_t* packed, __nv_bfloat16* Y, int64_t ldy, void* workspace, int* status_dev,
                        cudaStream_t stream, bool wstatic, bool xstatic);
size_t decode_gated_workspace_bytes(const patch_layout_t* L, int64_t M);   // 0 if the gated decode schedule does not apply
// M <= 16 on a weight whose tiles are all of a 4-bit kind (gemm_decode_q4_sm100.cu)
int launch_decode_q4(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                     __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool wstatic, bool xstatic,
                     bool ystatic = false);
// all-4-bit weight -> bf16 blob of its dequantised values (pack.cu), for the large-M kernels
void q4_expanded_layout(const patch_layout_t* L, patch_layout_t* out);
int launch_expand_q4(const patch_layout_t* L, const uint8_t* packed, const patch_layout_t* out_layout, uint8_t* out,
                     int* status_dev, cudaStream_t stream);
// Where the many-token call on a 4-bit weight puts that weight's bf16 image inside the caller's workspace: past
// every word that other calls keep zero there (arrival counters, flagged partial sums, the gated product's flag
// words: under 20 MB for N <= 131072), so that a workspace shared with them stays valid.
constexpr size_t kQ4ExpandOffset = size_t(32) << 20;
inline bool has_q4_tiles(const patch_layout_t* L) { return L->n_dense_q4 != 0 || L->n_sparse_q4 != 0; }

}  // namespace patch
