// Hybrid dense / 2:4 tile matmul on the sm_100a tensor cores (tcgen05 + TMEM + TMA).
//
// Computes Y^T[N x M] = What[N x K] * X^T[K x M]: the packed weight is the MMA "A" operand
// (the only operand tcgen05.mma.sp accepts in compressed form), out-features ride the 128 TMEM
// lanes, tokens ride the MMA N dimension (16..256).  This is the paper's mixed execution
// "within a single matrix multiplication" (Appendix A): for every 128 x 128 weight tile the
// MMA warp issues either eight dense tcgen05.mma (K = 16 each) or four tcgen05.mma.sp
// (K = 32 each, half the A bytes plus metadata from TMEM) into the same fp32 accumulator.
//
// Warp roles (192 threads): warp 0 streams tiles with TMA (one linear bulk copy per weight
// tile, whose payload is already in the swizzled shared-memory layout, and two tensor copies
// for the activations); warp 1 owns TMEM and issues the MMAs; warps 2..5 read the accumulator
// back (tcgen05.ld), convert to bf16 and store the transposed result.
//
// SPLIT = true is the small-M schedule (Appendix A: "split-K parallelism" for decode): a
// thread-block cluster of S CTAs shares one row-block, each CTA streams a K-slice, and the S
// fp32 partial tiles are summed in fixed slice order through distributed shared memory.
//
// Every wait on an mbarrier is bounded; on expiry the CTA raises an abort flag, reports
// PATCH_ERR_TIMEOUT through status_dev, drains its copies in flight, frees TMEM and returns.
#include <cuda.h>
#include "patch_internal.cuh"

namespace patch {

// ---------------------------------------------------------------------------------------------
// PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s: far beyond any legitimate wait
constexpr uint64_t kDrainLimitNs = 2000000ull;    // 2 ms for copies already in flight

// Bounded wait.  Returns false if the wait was given up (own timeout or another role aborted).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* status_dev) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                if (status_dev) atomicExch(status_dev, PATCH_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

// 1-D bulk copy global -> shared, completion counted on an mbarrier.
__device__ __forceinline__ void tma_bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// 2-D tiled copy global -> shared through a tensor map.
__device__ __forceinline__ void tma_tile_load(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], dense bf16, fp32 accumulate
__device__ __forceinline__ void mma_dense(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// same with A stored 2:4-compressed and its position metadata in TMEM
__device__ __forceinline__ void mma_sparse(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t e_tmem,
                                           uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(e_tmem), "r"(idesc), "r"(accumulate) : "memory");
}
// arrive on an mbarrier once all previously issued tcgen05 operations of this thread completed
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// shared memory (128 rows x 16 bytes) -> TMEM (128 lanes x 4 columns)
__device__ __forceinline__ void tmem_copy_128x128b(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::1.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ float ld_peer_smem_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t remote;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

// Shared-memory matrix descriptor, K-major operand in 128-byte-swizzled atoms
// (8 rows x 128 B = 1024 B per row group): start address, stride between row groups, sm_100
// descriptor version, swizzle mode.
__device__ __forceinline__ uint64_t desc_kmajor_sw128(uint32_t saddr) {
    return uint64_t((saddr & 0x3FFFFu) >> 4) | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) |
           (uint64_t(1) << 46) | (uint64_t(2) << 61);
}
// Unswizzled 128 rows x 16 B block (8-row groups of 128 B): source of the metadata copy.
__device__ __forceinline__ uint64_t desc_rows16(uint32_t saddr) {
    return uint64_t((saddr & 0x3FFFFu) >> 4) | (uint64_t(128 >> 4) << 16) | (uint64_t(128 >> 4) << 32) |
           (uint64_t(1) << 46);
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n_tok.
__host__ __device__ constexpr uint32_t instr_desc(int n_tok, bool sparse) {
    return (sparse ? (1u << 2) : 0u) | (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(n_tok >> 3) << 17) |
           (uint32_t(128 >> 4) << 24);
}

template <int N_TOK, int STAGES>
struct MmaConfig {
    static constexpr uint32_t kXAtomBytes = N_TOK * 128;           // N_TOK rows x 64 bf16
    static constexpr uint32_t kXBytes = 2 * kXAtomBytes;           // 128 columns of K
    static constexpr uint32_t kStageBytes = kDenseBytes + kXBytes;
    static constexpr uint32_t kBarrierOffset = STAGES * kStageBytes;
    static constexpr uint32_t kSmemBytes = kBarrierOffset + 256 + 1024;  // + barriers + alignment slack
    static constexpr uint32_t kTmemNeeded = N_TOK + 4 * STAGES;
    static constexpr uint32_t kTmemCols = kTmemNeeded <= 32 ? 32 : kTmemNeeded <= 64 ? 64 : kTmemNeeded <= 128 ? 128
                                          : kTmemNeeded <= 256 ? 256 : 512;
    static_assert(N_TOK % 16 == 0 && N_TOK >= 16 && N_TOK <= 256, "MMA N must be a multiple of 16 in [16, 256]");
    static_assert(kTmemNeeded <= 512, "accumulator + metadata exceed TMEM");
};

template <int N_TOK, int STAGES, bool SPLIT>
__global__ void __launch_bounds__(192)
mma_kernel(const __grid_constant__ CUtensorMap tmap_x, const uint8_t* __restrict__ blob, uint64_t table_off,
           int TK, int M, __nv_bfloat16* __restrict__ Y, int64_t ldy, int* status_dev) {
    using Cfg = MmaConfig<N_TOK, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_full = smem_base + Cfg::kBarrierOffset;    // STAGES x 8 B
    const uint32_t bar_empty = bar_full + 8 * STAGES;             // STAGES x 8 B
    const uint32_t bar_acc = bar_empty + 8 * STAGES;              // 8 B
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + Cfg::kBarrierOffset + 16 * STAGES + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile uint32_t* stage_kind = reinterpret_cast<volatile uint32_t*>(tmem_slot + 2);  // STAGES words

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    int tn, m0, tk0, tk1, split = 0, n_split = 1;
    if constexpr (SPLIT) {
        n_split = gridDim.x; split = blockIdx.x; tn = blockIdx.y; m0 = 0;
        tk0 = int(int64_t(split) * TK / n_split);
        tk1 = int(int64_t(split + 1) * TK / n_split);
    } else {
        tn = blockIdx.x; m0 = blockIdx.y * N_TOK; tk0 = 0; tk1 = TK;
    }
    const int n_tiles = tk1 - tk0;

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, 1);
        }
        mbar_init(bar_acc, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap_x) : "memory");
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), Cfg::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_acc = tmem_base;                 // columns [0, N_TOK)
    const uint32_t tmem_meta = tmem_base + N_TOK;        // 4 columns per stage

    if (warp == 0) {
        // ---------------- producer: one elected lane issues all copies ----------------
        const TileDesc* table = reinterpret_cast<const TileDesc*>(blob + table_off) + int64_t(tn) * TK + tk0;
        TileDesc mine = TileDesc{0, 0, 0, 0};
        int issued = 0;
        bool ok = true;
        for (int i = 0; i < n_tiles && ok; ++i) {
            if ((i & 31) == 0 && i + lane < n_tiles) mine = table[i + lane];   // 32 descriptors per warp load
            TileDesc d;
            d.kind = __shfl_sync(0xFFFFFFFFu, mine.kind, i & 31);
            d.payload_off16 = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, i & 31);
            if (lane == 0) {
                const int stage = i % STAGES;
                const uint32_t parity = (uint32_t(i / STAGES) & 1u) ^ 1u;
                ok = mbar_wait(bar_empty + 8 * stage, parity, abort_flag, status_dev);
                if (ok) {
                    const uint32_t wbytes = d.kind == PATCH_TILE_DENSE ? kDenseBytes : kSparseBytes;
                    const uint32_t sW = smem_base + stage * Cfg::kStageBytes, sX = sW + kDenseBytes;
                    stage_kind[stage] = d.kind;
                    mbar_expect_tx(bar_full + 8 * stage, wbytes + Cfg::kXBytes);
                    tma_bulk_load(sW, blob + uint64_t(d.payload_off16) * 16, wbytes, bar_full + 8 * stage);
                    const int k = (tk0 + i) * kTile;
                    tma_tile_load(sX, &tmap_x, k, m0, bar_full + 8 * stage);
                    tma_tile_load(sX + Cfg::kXAtomBytes, &tmap_x, k + 64, m0, bar_full + 8 * stage);
                    issued = i + 1;
                }
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
        }
        if (lane == 0 && *abort_flag) {
            // drain: wait (bounded) until the copies this thread started have landed
            const uint64_t t0 = global_timer_ns();
            for (int j = issued > STAGES ? issued - STAGES : 0; j < issued; ++j) {
                const uint32_t bar = bar_full + 8 * (j % STAGES), parity = uint32_t(j / STAGES) & 1u;
                while (!mbar_try_wait(bar, parity) && global_timer_ns() - t0 < kDrainLimitNs) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc_d = instr_desc(N_TOK, false), idesc_s = instr_desc(N_TOK, true);
            bool ok = true;
            for (int i = 0; i < n_tiles && ok; ++i) {
                const int stage = i % STAGES;
                ok = mbar_wait(bar_full + 8 * stage, uint32_t(i / STAGES) & 1u, abort_flag, status_dev);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sW = smem_base + stage * Cfg::kStageBytes, sX = sW + kDenseBytes;
                const uint64_t dA = desc_kmajor_sw128(sW), dB = desc_kmajor_sw128(sX);
                if (stage_kind[stage] == PATCH_TILE_DENSE) {
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {   // K = 16 per instruction: 32 B of each operand row
                        const uint64_t a = dA + uint64_t(((ks >> 2) * kAtomBytes + (ks & 3) * 32) >> 4);
                        const uint64_t b = dB + uint64_t(((ks >> 2) * Cfg::kXAtomBytes + (ks & 3) * 32) >> 4);
                        mma_dense(tmem_acc, a, b, idesc_d, (i | ks) != 0);
                    }
                } else {
                    const uint32_t e = tmem_meta + 4 * stage;
                    tmem_copy_128x128b(e, desc_rows16(sW + kAtomBytes));
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {   // K = 32 per instruction: 32 B of A, 64 B of B per row
                        const uint64_t a = dA + uint64_t((ks * 32) >> 4);
                        const uint64_t b = dB + uint64_t(((ks >> 1) * Cfg::kXAtomBytes + (ks & 1) * 64) >> 4);
                        // metadata column ks of this stage: even column in the address, parity in the selector
                        mma_sparse(tmem_acc, a, b, e + (ks & 2), idesc_s | uint32_t(ks & 1), (i | ks) != 0);
                    }
                }
                mma_commit(bar_empty + 8 * stage);   // frees the stage once these MMAs have read it
            }
            mma_commit(bar_acc);                     // accumulator complete
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: warps 2..5, TMEM lane quadrant = warp % 4 ----------------
        const uint32_t quad = warp & 3u, row = quad * 32 + lane;   // out-feature inside the row-block
        const bool ok = mbar_wait(bar_acc, 0, abort_flag, status_dev);
        tc_fence_after();
        const int valid = M - m0 < N_TOK ? M - m0 : N_TOK;          // tokens of this tile that exist
        float* part = reinterpret_cast<float*>(smem);               // SPLIT: [N_TOK][128] fp32, reuses stage 0
        if (ok) {
#pragma unroll 1
            for (int c0 = 0; c0 < valid; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(tmem_acc + ((quad * 32u) << 16) + uint32_t(c0), v);
                tmem_ld_wait();
                if constexpr (SPLIT) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) part[(c0 + j) * kTile + row] = __uint_as_float(v[j]);
                } else {
                    __nv_bfloat16* y = Y + int64_t(m0 + c0) * ldy + int64_t(tn) * kTile + row;
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (c0 + j < valid) y[int64_t(j) * ldy] = __float2bfloat16_rn(__uint_as_float(v[j]));
                }
            }
        }
    }

    if constexpr (SPLIT) {
        // Every thread of every CTA of the cluster takes part in both cluster barriers, also
        // after an abort, so that no peer is left waiting.
        cluster_arrive();
        cluster_wait();
        if (warp >= 2 && !*abort_flag) {
            const uint32_t row = (warp & 3u) * 32 + lane;
            const uint32_t part_addr = smem_base;
            for (int m = split; m < M; m += n_split) {      // this CTA finishes tokens split, split+S, ...
                float a = 0.f;
                for (int q = 0; q < n_split; ++q) a += ld_peer_smem_f32(part_addr + uint32_t(m * kTile + row) * 4u, q);
                Y[int64_t(m) * ldy + int64_t(tn) * kTile + row] = __float2bfloat16_rn(a);
            }
        }
        cluster_arrive();
        cluster_wait();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

// ---------------------------------------------------------------------------------------------
// host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// Tensor map over X [M x ldx] bf16: box = 64 columns (128 B, one swizzle atom row) x n_tok rows.
static int make_x_map(CUtensorMap* map, const __nv_bfloat16* X, int64_t ldx, int64_t M, int64_t K, int n_tok) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return PATCH_ERR_CUDA;
    const cuuint64_t dims[2] = {cuuint64_t(K), cuuint64_t(M)};
    const cuuint64_t strides[1] = {cuuint64_t(ldx) * 2};
    const cuuint32_t box[2] = {64, cuuint32_t(n_tok)};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<__nv_bfloat16*>(X), dims, strides, box,
                     estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PATCH_OK : PATCH_ERR_CUDA;
}

static int pick_splits(int TN, int TK, int target_ctas) {
    int best = 1;
    for (int S = 1; S <= 8 && S <= TK; ++S)
        if (TN * S <= target_ctas) best = S;
    return best;
}

template <int N_TOK, int STAGES, bool SPLIT>
static int launch_t(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int64_t M,
                    __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, int target_ctas) {
    using Cfg = MmaConfig<N_TOK, STAGES>;
    auto kern = mma_kernel<N_TOK, STAGES, SPLIT>;
    static bool configured = false;   // per-process attribute, idempotent
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess)
            return PATCH_ERR_CUDA;
        configured = true;
    }
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.blockDim = dim3(192, 1, 1);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = stream;
    if (SPLIT) {
        const int S = pick_splits(TN, TK, target_ctas);
        if (TN > 65535) return PATCH_ERR_SHAPE;
        cfg.gridDim = dim3(S, TN, 1);
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = S;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    } else {
        const int64_t MT = (M + N_TOK - 1) / N_TOK;
        if (MT > 65535) return PATCH_ERR_SHAPE;
        cfg.gridDim = dim3(TN, unsigned(MT), 1);
    }
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, map, packed, uint64_t(L->table_off), TK, int(M), Y, ldy, status_dev);
    return e == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

size_t mma_workspace_bytes(const patch_layout_t*, int64_t) { return 0; }

int launch_mma(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
               __nv_bfloat16* Y, int64_t ldy, void*, size_t, int* status_dev, cudaStream_t stream) {
    if (M > 0x7FFFFFFF) return PATCH_ERR_SHAPE;
    const int n_tok = M <= 16 ? 16 : M <= 32 ? 32 : M <= 64 ? 64 : M <= 128 ? 128 : 256;
    CUtensorMap map;
    int rc = make_x_map(&map, X, ldx, M, L->K, n_tok);
    if (rc) return rc;
    switch (n_tok) {
        case 16: return launch_t<16, 3, true>(map, L, packed, M, Y, ldy, status_dev, stream, 296);
        case 32: return launch_t<32, 5, true>(map, L, packed, M, Y, ldy, status_dev, stream, 148);
        case 64: return launch_t<64, 4, true>(map, L, packed, M, Y, ldy, status_dev, stream, 148);
        case 128: return launch_t<128, 3, false>(map, L, packed, M, Y, ldy, status_dev, stream, 0);
        default: return launch_t<256, 2, false>(map, L, packed, M, Y, ldy, status_dev, stream, 0);
    }
}

}  // namespace patch
