// Large-M (prefill) schedule of the hybrid dense / 2:4 tile matmul on the sm_100a tensor cores.
//
// Computes Y^T[N x M] = What[N x K] * X^T[K x M]: the packed weight is the MMA "A" operand
// (the only operand tcgen05.mma.sp accepts in compressed form), out-features ride the 128 TMEM
// lanes, tokens ride the MMA N dimension.  One CTA per (row-block tn, token tile of N_TOK): it
// walks all TK weight tiles of its row-block and issues, per tile, eight dense tcgen05.mma or
// four tcgen05.mma.sp into one fp32 TMEM accumulator -- the paper's mixed execution "within a
// single matrix multiplication" (Appendix A).
//
// Warp roles (192 threads): warp 0 streams tiles with TMA (one linear bulk copy per weight
// tile, whose payload is already in the swizzled shared-memory layout, and two tensor copies
// for the activations); warp 1 owns TMEM and issues the MMAs; warps 2..5 read the accumulator
// back (tcgen05.ld), convert to bf16 and store the transposed result.
//
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, reports
// PATCH_ERR_TIMEOUT through status_dev, drains its copies in flight, frees TMEM and returns.
#include "sm100_ptx.cuh"

namespace patch {

template <int N_TOK, int STAGES>
struct PrefillConfig {
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
    static_assert(STAGES <= 8, "barrier block holds at most 8 stages");
};

template <int N_TOK, int STAGES>
__global__ void __launch_bounds__(192)
prefill_kernel(const __grid_constant__ CUtensorMap tmap_x, const uint8_t* __restrict__ blob, uint64_t table_off,
               int TK, int M, __nv_bfloat16* __restrict__ Y, int64_t ldy, int* status_dev) {
    using Cfg = PrefillConfig<N_TOK, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_full = smem_base + Cfg::kBarrierOffset;    // 8 x 8 B
    const uint32_t bar_empty = bar_full + 64;                     // 8 x 8 B
    const uint32_t bar_acc = bar_empty + 64;                      // 8 B
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + Cfg::kBarrierOffset + 144);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile uint32_t* stage_kind = reinterpret_cast<volatile uint32_t*>(tmem_slot + 2);  // STAGES words

    grid_launch_dependents();
    grid_dependency_wait();     // X, the packed weight and Y may belong to the previous kernel until here

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tn = blockIdx.x, m0 = blockIdx.y * N_TOK;
    const int n_tiles = TK;

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, 1);
        }
        mbar_init(bar_acc, 1);
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_map(&tmap_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), Cfg::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_acc = tmem_base;                 // columns [0, N_TOK)
    const uint32_t tmem_meta = tmem_base + N_TOK;        // 4 columns per stage

    if (warp == 0) {
        // ---------------- producer ----------------
        const uint64_t pol_w = l2_policy_evict_last(), pol_x = l2_policy_evict_last();
        const TileDesc* table = reinterpret_cast<const TileDesc*>(blob + table_off) + int64_t(tn) * TK;
        TileDesc mine = TileDesc{0, 0, 0, 0};
        int issued = 0;
        bool ok = true;
        for (int i = 0; i < n_tiles && ok; ++i) {
            if ((i & 31) == 0 && i + lane < n_tiles) mine = table[i + lane];   // 32 descriptors per warp load
            const uint32_t kind = __shfl_sync(0xFFFFFFFFu, mine.kind, i & 31);
            const uint32_t off16 = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, i & 31);
            if (lane == 0) {
                const int stage = i % STAGES;
                ok = mbar_wait(bar_empty + 8 * stage, (uint32_t(i / STAGES) & 1u) ^ 1u, abort_flag, status_dev);
                if (ok) {
                    const uint32_t wbytes = kind == PATCH_TILE_DENSE ? kDenseBytes : kSparseBytes;
                    const uint32_t sW = smem_base + stage * Cfg::kStageBytes, sX = sW + kDenseBytes;
                    const uint32_t full = bar_full + 8 * stage;
                    stage_kind[stage] = kind;
                    mbar_expect_tx(full, wbytes + Cfg::kXBytes);
                    tma_bulk_load(sW, blob + uint64_t(off16) * 16, wbytes, full, pol_w);
                    tma_tile_load(sX, &tmap_x, i * kTile, m0, full, pol_x);
                    tma_tile_load(sX + Cfg::kXAtomBytes, &tmap_x, i * kTile + 64, m0, full, pol_x);
                    issued = i + 1;
                }
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
        }
        if (lane == 0 && *abort_flag) {
            // drain: wait (bounded) until the copies this thread started have landed
            const uint64_t tstart = global_timer_ns();
            for (int j = issued > STAGES ? issued - STAGES : 0; j < issued; ++j) {
                const uint32_t bar = bar_full + 8 * (j % STAGES), parity = uint32_t(j / STAGES) & 1u;
                while (!mbar_try_wait(bar, parity) && global_timer_ns() - tstart < kDrainLimitNs) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            bool ok = true;
            for (int i = 0; i < n_tiles && ok; ++i) {
                const int stage = i % STAGES;
                ok = mbar_wait(bar_full + 8 * stage, uint32_t(i / STAGES) & 1u, abort_flag, status_dev);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sW = smem_base + stage * Cfg::kStageBytes;
                issue_tile_mma<N_TOK>(stage_kind[stage], sW, sW + kDenseBytes, Cfg::kXAtomBytes, tmem_acc,
                                      tmem_meta + 4 * stage, i == 0);
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
        if (ok) {
#pragma unroll 1
            for (int c0 = 0; c0 < valid; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(tmem_acc + ((quad * 32u) << 16) + uint32_t(c0), v);
                tmem_ld_wait();
                __nv_bfloat16* y = Y + int64_t(m0 + c0) * ldy + int64_t(tn) * kTile + row;
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (c0 + j < valid) y[int64_t(j) * ldy] = __float2bfloat16_rn(__uint_as_float(v[j]));
            }
        }
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

int make_x_tensor_map(CUtensorMap* map, const __nv_bfloat16* X, int64_t ldx, int64_t M, int64_t K, int n_tok) {
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

template <int N_TOK, int STAGES>
static int launch_prefill_t(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int64_t M,
                            __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream) {
    using Cfg = PrefillConfig<N_TOK, STAGES>;
    auto kern = prefill_kernel<N_TOK, STAGES>;
    static bool configured = false;   // per-process attribute, idempotent
    if (!configured) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg::kSmemBytes) != cudaSuccess)
            return PATCH_ERR_CUDA;
        configured = true;
    }
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    const int64_t MT = (M + N_TOK - 1) / N_TOK;
    if (MT > 65535) return PATCH_ERR_SHAPE;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3(TN, unsigned(MT), 1);
    cfg.blockDim = dim3(192, 1, 1);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, map, packed, uint64_t(L->table_off), TK, int(M), Y, ldy, status_dev);
    return e == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

int launch_prefill(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                   __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream) {
    if (M > 0x7FFFFFFF) return PATCH_ERR_SHAPE;
    const int n_tok = M <= 128 ? 128 : 256;
    CUtensorMap map;
    int rc = make_x_tensor_map(&map, X, ldx, M, L->K, n_tok);
    if (rc) return rc;
    if (n_tok == 128) return launch_prefill_t<128, 3>(map, L, packed, M, Y, ldy, status_dev, stream);
    return launch_prefill_t<256, 2>(map, L, packed, M, Y, ldy, status_dev, stream);
}

}  // namespace patch
