// Large-M (prefill) schedule of the hybrid dense / 2:4 tile matmul on the sm_100a tensor cores.
//
// Computes Y^T[N x M] = What[N x K] * X^T[K x M]: the packed weight is the MMA "A" operand
// (the only operand tcgen05.mma.sp accepts in compressed form), out-features ride the 128 TMEM
// lanes, tokens ride the MMA N dimension.  An output tile is (row-block tn) x (n_tok tokens); its
// mainloop walks the TK weight tiles of the row-block and issues, per tile, eight dense
// tcgen05.mma or four tcgen05.mma.sp into one fp32 TMEM accumulator -- dense and 2:4 tiles
// mixed inside one multiplication, as Appendix A describes the deployed kernels.
//
// Persistent kernel: one CTA per SM loops over output tiles (tile index = mt * TN + tn, so CTAs
// running side by side share an X tile in L2 and stream different row-blocks).  Two TMEM
// accumulators: the epilogue of one output tile (tcgen05.ld, bf16, transposed store) overlaps the
// mainloop of the next.  n_tok (a multiple of 16, at most 240) is chosen per problem so that the
// number of output tiles fills whole waves of SMs.
//
// Warp roles (192 threads): warp 0 streams tiles with TMA (one linear bulk copy per weight
// tile, whose payload is already in the swizzled shared-memory layout, and two tensor copies
// for the activations); warp 1 owns TMEM and issues the MMAs; warps 2..5 are the epilogue.
//
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, reports
// PATCH_ERR_TIMEOUT through status_dev, drains its copies in flight, frees TMEM and returns.
#include "sm100_ptx.cuh"

namespace patch {

constexpr int kPrefillMaxTok = 240;      // two accumulators + metadata must fit 512 TMEM columns

// A stage holds a whole weight tile (32 KB reserved) and the n_tok x 128 activation tile; the ring
// takes as many stages as fit: 2 at n_tok = 240 (92 KB each), 3 up to n_tok = 160, 4 at n_tok <= 80.
struct PrefillConfig {
    static constexpr uint32_t kRingBytes = 216 * 1024;
    static constexpr int kMaxStages = 8;
    static constexpr uint32_t kBarrierOffset = kRingBytes;
    static constexpr uint32_t kStageOffset = kBarrierOffset + 256;       // 4 epilogue warps x 1 KB transpose staging
    static constexpr uint32_t kSmemBytes = kStageOffset + 4 * 1024 + 1024;   // + alignment slack
    static constexpr uint32_t kTmemCols = 512;
    static constexpr uint32_t kAcc1Col = 256, kMetaCol = 240;      // acc0 [0,240) acc1 [256,496); metadata, 4 columns per stage: [240,256) then [496,512)
};

__global__ void __launch_bounds__(192)
prefill_kernel(const __grid_constant__ CUtensorMap tmap_x, const uint8_t* __restrict__ blob, uint64_t table_off,
               uint32_t pay0_16, uint32_t end16, int TN, int TK, int M, int n_tok, __nv_bfloat16* __restrict__ Y, int64_t ldy,
               int* status_dev, int independent) {
    using Cfg = PrefillConfig;
    const uint32_t stage_bytes = kDenseBytes + uint32_t(n_tok) * 256u;
    const int STAGES = int(Cfg::kRingBytes / stage_bytes) < Cfg::kMaxStages ? int(Cfg::kRingBytes / stage_bytes) : Cfg::kMaxStages;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_full = smem_base + Cfg::kBarrierOffset;    // 8 x 8 B
    const uint32_t bar_empty = bar_full + 64;                     // 8 x 8 B
    const uint32_t bar_acc_full = bar_empty + 64;                 // 2 x 8 B
    const uint32_t bar_acc_empty = bar_acc_full + 16;             // 2 x 8 B
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + Cfg::kBarrierOffset + 160);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile uint32_t* stage_kind = reinterpret_cast<volatile uint32_t*>(tmem_slot + 2);  // kMaxStages words

    grid_launch_dependents();
    // X, the packed weight and Y may belong to the previous kernel until here -- unless the caller declared
    // this GEMM independent of its predecessor: then only the Y stores (and the exit) wait, and this kernel's
    // CTAs start on whatever SMs the tail of the previous kernel leaves idle
    if (!independent) grid_dependency_wait();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int MT = (M + n_tok - 1) / n_tok;
    const int n_out = TN * MT;                                    // output tiles, index = mt * TN + tn
    const uint32_t x_atom_bytes = uint32_t(n_tok) * 128u;

    if (threadIdx.x == 0) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_acc_full + 8 * i, 1);
            mbar_init(bar_acc_empty + 8 * i, 4);     // one arrival per epilogue warp
        }
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_map(&tmap_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), Cfg::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- producer ----------------
        const uint64_t pol = l2_policy_evict_last();     // weights and activations are both re-read from L2
        const TileDesc* table0 = reinterpret_cast<const TileDesc*>(blob + table_off);
        int issued = 0;      // stage-ring position, continues across output tiles
        bool ok = true;
        for (int t = blockIdx.x; t < n_out && ok; t += gridDim.x) {
            const int tn = t % TN, m0 = (t / TN) * n_tok;
            const TileDesc* table = table0 + int64_t(tn) * TK;
            TileDesc mine = TileDesc{0, 0, 0, 0};
            for (int i = 0; i < TK && ok; ++i) {
                if ((i & 31) == 0 && i + lane < TK) mine = table[i + lane];   // 32 descriptors per warp load
                uint32_t kind = __shfl_sync(0xFFFFFFFFu, mine.kind, i & 31);
                uint32_t off16 = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, i & 31);
                if (lane == 0) {
                    const int stage = issued % STAGES;
                    sanitize_tile(kind, off16, pay0_16, end16, status_dev);
                    ok = mbar_wait(bar_empty + 8 * stage, (uint32_t(issued / STAGES) & 1u) ^ 1u, abort_flag, status_dev);
                    if (ok) {
                        const uint32_t wbytes = kind == PATCH_TILE_DENSE ? kDenseBytes : kSparseBytes;
                        const uint32_t sW = smem_base + stage * stage_bytes, sX = sW + kDenseBytes;
                        const uint32_t full = bar_full + 8 * stage;
                        stage_kind[stage] = kind;
                        mbar_expect_tx(full, wbytes + 2 * x_atom_bytes);
                        tma_bulk_load(sW, blob + uint64_t(off16) * 16, wbytes, full, pol);
                        tma_tile_load(sX, &tmap_x, i * kTile, m0, full, pol);
                        tma_tile_load(sX + x_atom_bytes, &tmap_x, i * kTile + 64, m0, full, pol);
                        ++issued;
                    }
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            }
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
            int step = 0, j = 0;      // stage-ring position; local output-tile counter
            for (int t = blockIdx.x; t < n_out && ok; t += gridDim.x, ++j) {
                const uint32_t acc = tmem_base + (j & 1 ? Cfg::kAcc1Col : 0u);
                // the epilogue must have drained this accumulator (two tiles ago)
                ok = mbar_wait(bar_acc_empty + 8 * (j & 1), (uint32_t(j >> 1) & 1u) ^ 1u, abort_flag, status_dev);
                for (int i = 0; i < TK && ok; ++i, ++step) {
                    const int stage = step % STAGES;
                    ok = mbar_wait(bar_full + 8 * stage, uint32_t(step / STAGES) & 1u, abort_flag, status_dev);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t sW = smem_base + stage * stage_bytes;
                    issue_tile_mma_n(stage_kind[stage], sW, sW + kDenseBytes, x_atom_bytes, acc,
                                     tmem_base + (stage < 4 ? Cfg::kMetaCol + 4 * stage : 496 + 4 * (stage - 4)), i == 0, uint32_t(n_tok));
                    mma_commit(bar_empty + 8 * stage);   // frees the stage once these MMAs have read it
                }
                if (ok) mma_commit(bar_acc_full + 8 * (j & 1));      // accumulator complete
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: warps 2..5, TMEM lane quadrant = warp % 4 ----------------
        const uint32_t quad = warp & 3u;     // this warp's 32 out-features inside the row-block
        bool ok = true;
        int j = 0;
        for (int t = blockIdx.x; t < n_out && ok; t += gridDim.x, ++j) {
            const int tn = t % TN, m0 = (t / TN) * n_tok;
            // one thread polls, the other 127 epilogue threads sleep on a hardware barrier
            ok = group_wait(bar_acc_full + 8 * (j & 1), uint32_t(j >> 1) & 1u, warp == 2 && lane == 0, 1, 128, abort_flag, status_dev);
            if (!ok) break;
            tc_fence_after();
            const uint32_t acc = tmem_base + (j & 1 ? Cfg::kAcc1Col : 0u) + ((quad * 32u) << 16);
            const int valid = M - m0 < n_tok ? M - m0 : n_tok;      // tokens of this tile that exist
            __nv_bfloat16* ytile = Y + int64_t(m0) * ldy + int64_t(tn) * kTile + quad * 32;
            if (independent && j == 0) grid_dependency_wait();      // Y may be in use by the preceding kernel
#pragma unroll 1
            for (int c0 = 0; c0 < valid; c0 += 16) {
                uint32_t v[16];
                tmem_ld16(acc + uint32_t(c0), v);
                tmem_ld_wait();
                store_fragment_transposed(v, smem + Cfg::kStageOffset + (warp - 2) * 1024, lane, ytile + int64_t(c0) * ldy, ldy,
                                          valid - c0);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty + 8 * (j & 1));
        }
    }

    if (independent) grid_dependency_wait();      // every thread passes the dependency before the CTA exits
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

// X as a 3-D tensor (column inside a 64-column chunk, token row, chunk): a box of `chunks` chunks lands in shared
// memory as `chunks` consecutive [n_tok x 128 B] swizzled atoms -- the activations of chunks / 2 weight tiles in one copy.
int make_x_chunk_tensor_map(CUtensorMap* map, const __nv_bfloat16* X, int64_t ldx, int64_t M, int64_t K, int n_tok, int chunks) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return PATCH_ERR_CUDA;
    const cuuint64_t dims[3] = {64, cuuint64_t(M), cuuint64_t(K / 64)};
    const cuuint64_t strides[2] = {cuuint64_t(ldx) * 2, 128};
    const cuuint32_t box[3] = {64, cuuint32_t(n_tok), cuuint32_t(chunks)};
    const cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(X), dims, strides, box,
                     estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PATCH_OK : PATCH_ERR_CUDA;
}

int make_blob_tensor_map(CUtensorMap* map, const uint8_t* blob, uint64_t total_bytes, int box_rows) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return PATCH_ERR_CUDA;
    if (total_bytes % 256 || box_rows < 1 || box_rows > 256) return PATCH_ERR_FORMAT;
    const cuuint64_t dims[2] = {256, cuuint64_t(total_bytes / 256)};
    const cuuint64_t strides[1] = {256};
    const cuuint32_t box[2] = {256, cuuint32_t(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(blob), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? PATCH_OK : PATCH_ERR_CUDA;
}

int launch_prefill2(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int64_t M, int n_tok,
                    int sms, __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool gated,
                    bool independent);

// Schedule choice: token-tile width n (a multiple of 16 in [128, 240]) and one or two row-blocks
// per CTA, by a small cost model -- waves of output tiles over the SMs times the time of one tile,
// which is the slower of the tensor pipe (0.55 us per 128 x 128 x 256 step at full clocks) and
// what one SM pulls from L2 (measured: a step's copies land ~1.75 us after they are issued, so
// the one-row-block ring sustains one step per 1.75 us / stages; ~120 GB/s with the two-ring
// pipeline), plus a per-tile prologue/epilogue cost.
struct PrefillPlan { int n_tok; int schedule; double cost_ns; };   // schedule: row-blocks per CTA (1 or 2), 3 = CTA pairs

static PrefillPlan plan_prefill(int64_t M, int TN, int TK, int sms, bool two_row_blocks_only = false,
                                bool independent = false) {
    PrefillPlan best = {240, 1, 1e300};
    double best_cost = 1e300;
    const int n_hi = M <= 128 ? int((M + 15) / 16 * 16) : kPrefillMaxTok, n_lo = M <= 128 ? n_hi : 128;
    for (int n = n_hi; n >= n_lo; n -= 16) {
        const int64_t MT = (M + n - 1) / n;
        for (int sched = 1; sched <= 2; ++sched) {
            if (two_row_blocks_only && sched != 2) continue;
            const int64_t tiles = int64_t(sched == 1 ? TN : (TN + 1) / 2) * MT;
            const int64_t waves = (tiles + sms - 1) / sms;
            const double mma_ns = (sched == 1 ? 550.0 : 1100.0) * n / 256.0;
            // one row-block: the ring holds `stages` whole steps and a step's copies take ~1.75 us to land
            const double stage_bytes = 32768.0 + n * 256.0;
            const int stages = int(PrefillConfig::kRingBytes / stage_bytes) < PrefillConfig::kMaxStages
                                   ? int(PrefillConfig::kRingBytes / stage_bytes) : PrefillConfig::kMaxStages;
            const double load1_ns = 1750.0 / stages > stage_bytes / 150.0 ? 1750.0 / stages : stage_bytes / 150.0;
            // two row-blocks: the rings hold ~1.5 steps, which bounds a step at ~1.2 us whatever its size
            const double load2_ns = (65536.0 + n * 256.0) / 120.0 > 1200.0 ? (65536.0 + n * 256.0) / 120.0 : 1200.0;
            const double load_ns = sched == 1 ? load1_ns : load2_ns;
            const double tile_ns = TK * (mma_ns > load_ns ? mma_ns : load_ns) + (sched == 1 ? 6000.0 : 10000.0);
            // a GEMM whose successor may start on the SMs its last wave leaves idle pays only part of that wave
            const double frac = double(tiles) / sms > 1.0 ? double(tiles) / sms : 1.0;
            const double eff_waves = independent ? frac : double(waves);
            const double cost = eff_waves * tile_ns + n;          // at equal time, the narrower tile (less padding)
            if (cost < best_cost) { best_cost = cost; best = {n, sched, cost}; }
        }
    }
    return best;
}

// CTA-pair schedule (weights whose tiles are all of one kind): a cluster takes four row-blocks x n tokens, so the
// waves are those of the two-row-block schedule; what a K step costs is the tensor time alone (per CTA the same
// two accumulators, but half the activation bytes), 2:4 tiles at twice the dense rate.
int prefill_pair_clusters(bool sparse);
int prefill_pair_max_tok(bool sparse);
int launch_prefill_pair(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                        int n_tok, __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool independent);

int prefill_pair_mixed_clusters();
int prefill_pair_mixed_max_tok();
int launch_prefill_pair_mixed(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                              int n_tok, __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool independent);

// kind: 0 all dense, 1 all 2:4, 2 mixed (gemm_prefill_pair_mixed_sm100.cu)
static PrefillPlan plan_prefill_pair(int64_t M, int TN, int TK, int kind) {
    PrefillPlan best = {0, 3, 1e300};
    const bool sparse = kind == 1;
    const int clusters = kind == 2 ? prefill_pair_mixed_clusters() : prefill_pair_clusters(sparse);
    if (clusters <= 0) return best;
    const int n_max = kind == 2 ? prefill_pair_mixed_max_tok() : prefill_pair_max_tok(sparse);
    const int n_hi = M < n_max ? int((M + 15) / 16 * 16 < 32 ? 32 : (M + 15) / 16 * 16) : n_max, n_lo = n_hi < 128 ? n_hi : 128;
    for (int n = n_hi; n >= n_lo; n -= 16) {
        const int64_t tiles = int64_t((TN + 3) / 4) * ((M + n - 1) / n);
        const int64_t waves = (tiles + clusters - 1) / clusters;
        // a K step costs the tensor time of n tokens, but not less than the pipeline's latency floor (measured with every
        // SM busy: ~1.3 us on dense, ~0.8 us on 2:4 tiles, whatever the width): at equal cost the wider tile wins
        const double mma_ns = (sparse ? 550.0 : 1100.0) * n / 256.0, floor_ns = sparse ? 800.0 : 1300.0;
        const double cost = double(waves) * (TK * (mma_ns > floor_ns ? mma_ns : floor_ns) + 8000.0) - 1e-3 * n;
        if (cost < best.cost_ns) best = {n, 3, cost};
    }
    return best;
}

int launch_prefill(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                   __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool independent, bool force_pair) {
    if (M > 0x7FFFFFFF) return PATCH_ERR_SHAPE;
    const int sms = sm_count();
    if (sms <= 0) return PATCH_ERR_CUDA;
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    const PrefillPlan plan = plan_prefill(M, TN, TK, sms, false, independent);
    {
        const int kind = L->n_sparse == 0 ? 0 : L->n_dense == 0 ? 1 : 2;
        const PrefillPlan pair = plan_prefill_pair(M, TN, TK, kind);
        // the pair schedule wins wherever every cluster gets a tile of a useful width (measured on the LLaMA shapes:
        // all M >= 2048, and M = 512 on the 11008-row weights)
        const bool enough = M * int64_t((TN + 3) / 4) >= int64_t(sms / 2) * 128;
        // Weights that mix kinds go to the pair schedule only on request: every 2:4 tile whose pair partner is dense
        // has to be expanded first, and the chain [tile lands -> helper warps rewrite it -> arrival crosses the pair]
        // is longer than the four stages can hide (measured on the LLaMA-2-7B shapes at half 2:4 tiles:
        // 900-1020 TFLOP/s against 1200-1640 on the two-row-block schedule).
        if (pair.n_tok && (force_pair || (enough && kind != 2))) {
            if (kind == 2) return launch_prefill_pair_mixed(X, ldx, M, L, packed, pair.n_tok, Y, ldy, status_dev, stream, independent);
            return launch_prefill_pair(X, ldx, M, L, packed, pair.n_tok, Y, ldy, status_dev, stream, independent);
        }
    }
    if (force_pair) return PATCH_ERR_CUDA;       // the schedule is unavailable on this device
    const int n_tok = plan.n_tok;
    CUtensorMap map;
    int rc = make_x_tensor_map(&map, X, ldx, M, L->K, n_tok);
    if (rc) return rc;
    if (plan.schedule == 2) return launch_prefill2(map, L, packed, M, n_tok, sms, Y, ldy, status_dev, stream, false, independent);
    static std::atomic<uint64_t> configured{0};
    if (int rc = allow_dynamic_smem(prefill_kernel, PrefillConfig::kSmemBytes, configured)) return rc;
    const int64_t n_out = int64_t(TN) * ((M + n_tok - 1) / n_tok);
    if (n_out > 0x7FFFFFFF) return PATCH_ERR_SHAPE;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3(unsigned(n_out < sms ? n_out : sms), 1, 1);
    cfg.blockDim = dim3(192, 1, 1);
    cfg.dynamicSmemBytes = PrefillConfig::kSmemBytes;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, prefill_kernel, map, packed, uint64_t(L->table_off), uint32_t(L->payload_off / 16),
                                       uint32_t(L->total_bytes / 16), TN, TK, int(M), n_tok, Y, ldy, status_dev, independent ? 1 : 0);
    return e == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

// Gated product of a stacked gate/up weight whose row-blocks alternate (gate j, up j): always the
// two-row-block kernel, whose CTA holds both accumulators of an output row-block.
int launch_prefill_gated(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                         __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool independent) {
    if (M > 0x7FFFFFFF) return PATCH_ERR_SHAPE;
    const int sms = sm_count();
    if (sms <= 0) return PATCH_ERR_CUDA;
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    const PrefillPlan plan = plan_prefill(M, TN, TK, sms, true, independent);
    CUtensorMap map;
    int rc = make_x_tensor_map(&map, X, ldx, M, L->K, plan.n_tok);
    if (rc) return rc;
    return launch_prefill2(map, L, packed, M, plan.n_tok, sms, Y, ldy, status_dev, stream, true, independent);
}

}  // namespace patch
