// Large-M (prefill) schedule with two row-blocks per CTA: a 256 x n_tok output tile.
//
// Same operation and operand roles as gemm_prefill_sm100.cu (weights are the MMA A operand, dense
// tcgen05.mma or tcgen05.mma.sp per 128 x 128 weight tile, fp32 accumulation in TMEM), but a CTA
// owns the row-block pair (2p, 2p+1) and keeps one accumulator for each, so the activation tile
// it streams is used twice: 496 B of operands per K column and row-block instead of 736 B.  At
// 128 x 240 tiles the single-row-block kernel is bound by what one SM can pull from L2 with two
// 92 KB stages in flight; this one is not.
//
// Shared memory is two rings instead of one ring of whole tiles, so that more, smaller copies
// are in flight:
//   A ring: 6 slots of 18 KB -- one K-half of a dense tile (16 KB atom) or a whole 2:4 tile
//           (16 KB of kept values + 2 KB metadata);
//   B ring: 3 slots of n_tok x 128 B -- one K-half (64 columns) of the activation tile.
// Per weight-tile step k and K-half h the producer issues {A(rb0), A(rb1), B(k,h)} (a 2:4 tile
// only at h = 0) and the MMA warp consumes them in the same order: four K=16 MMAs per dense half,
// two K=32 sparse MMAs per half of a 2:4 tile, each stage released by its own tcgen05.commit.
//
// 320 threads: warp 0 producer, warp 1 MMA + TMEM owner, warps 2..9 epilogue (two warps per TMEM
// lane quadrant, each taking half of the token columns).  Persistent over output tiles; the
// producer prefetches the next tile's first stages while the epilogue drains the accumulators.
//
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, reports
// PATCH_ERR_TIMEOUT through status_dev, drains its copies in flight, frees TMEM and returns.
#include "sm100_ptx.cuh"

namespace patch {

namespace p2 {
constexpr int kMaxTok = 240;
constexpr int NA = 6, NB = 3;
constexpr uint32_t kASlotBytes = kSparseBytes;                 // 18 432
constexpr uint32_t kBSlotBytes = kMaxTok * 128;                // 30 720
constexpr uint32_t kBOffset = NA * kASlotBytes;
constexpr uint32_t kBarrierOffset = kBOffset + NB * kBSlotBytes;
constexpr uint32_t kStageOffset = kBarrierOffset + 512;         // 8 epilogue warps x 1 KB transpose staging
constexpr uint32_t kSmemBytes = kStageOffset + 8 * 1024 + 1024; // + alignment slack
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kAcc1Col = 256;                              // acc0 [0,240)  acc1 [256,496)
// metadata: 4 TMEM columns per A slot, in the gaps [240,256) and [496,512)
__device__ __forceinline__ uint32_t meta_col(int slot) { return slot < 4 ? 240u + 4u * slot : 496u + 4u * (slot - 4); }
// what an A slot holds: 0 / 1 = first / second K-half of a dense tile, 2 = a whole 2:4 tile
constexpr uint32_t kSparse = 2;
}  // namespace p2

__global__ void __launch_bounds__(320)
prefill2_kernel(const __grid_constant__ CUtensorMap tmap_x, const uint8_t* __restrict__ blob, uint64_t table_off,
                uint32_t pay0_16, uint32_t end16, int TN, int TK, int M, int n_tok, __nv_bfloat16* __restrict__ Y, int64_t ldy,
                int* status_dev, int gated, int independent) {
    using namespace p2;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_fullA = smem_base + kBarrierOffset;        // NA x 8 B  (8 reserved)
    const uint32_t bar_emptyA = bar_fullA + 64;
    const uint32_t bar_fullB = bar_emptyA + 64;                   // NB x 8 B  (4 reserved)
    const uint32_t bar_emptyB = bar_fullB + 32;
    const uint32_t bar_acc_full = bar_emptyB + 32;                // 8 B
    const uint32_t bar_acc_empty = bar_acc_full + 8;              // 8 B
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kBarrierOffset + 208);
    uint32_t* tmem_slot = misc;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 1);
    volatile uint32_t* slot_kind = misc + 2;                      // NA words

    grid_launch_dependents();
    // X, the packed weight and Y may belong to the previous kernel until here -- unless the caller declared
    // this GEMM independent of its predecessor: then only the Y stores (and the exit) wait
    if (!independent) grid_dependency_wait();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int TP = (TN + 1) / 2;                                   // row-block pairs
    const int MT = (M + n_tok - 1) / n_tok;
    const int n_out = TP * MT;                                     // output tiles, index = mt * TP + pair
    const uint32_t x_half_bytes = uint32_t(n_tok) * 128u;

    if (threadIdx.x == 0) {
        for (int i = 0; i < NA; ++i) { mbar_init(bar_fullA + 8 * i, 1); mbar_init(bar_emptyA + 8 * i, 1); }
        for (int i = 0; i < NB; ++i) { mbar_init(bar_fullB + 8 * i, 1); mbar_init(bar_emptyB + 8 * i, 1); }
        mbar_init(bar_acc_full, 1);
        mbar_init(bar_acc_empty, 8);       // one arrival per epilogue warp
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_map(&tmap_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- producer ----------------
        const uint64_t pol = l2_policy_evict_last();
        const TileDesc* table0 = reinterpret_cast<const TileDesc*>(blob + table_off);
        int ia = 0, ib = 0;                  // ring positions, continue across output tiles
        bool ok = true;
        for (int t = blockIdx.x; t < n_out && ok; t += gridDim.x) {
            const int pair = t % TP, m0 = (t / TP) * n_tok;
            const int tn0 = 2 * pair;
            const bool has1 = tn0 + 1 < TN;
            // lanes 0..15 hold the next 16 descriptors of row-block tn0, lanes 16..31 those of tn0+1
            const TileDesc* table = table0 + int64_t(tn0 + (lane >> 4 && has1 ? 1 : 0)) * TK;
            // fetched one batch of 16 ahead, so that the table read is never waited for inside the K loop
            TileDesc mine = TileDesc{0, 0, 0, 0}, next = TileDesc{0, 0, 0, 0};
            if ((lane & 15) < TK) next = table[lane & 15];
            for (int k = 0; k < TK && ok; ++k) {
                if ((k & 15) == 0) {
                    mine = next;
                    if (k + 16 + (lane & 15) < TK) next = table[k + 16 + (lane & 15)];
                }
                uint32_t kind[2], off16[2];
                kind[0] = __shfl_sync(0xFFFFFFFFu, mine.kind, k & 15);
                off16[0] = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, k & 15);
                kind[1] = __shfl_sync(0xFFFFFFFFu, mine.kind, 16 + (k & 15));
                off16[1] = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, 16 + (k & 15));
                if (lane == 0) {
                    sanitize_tile(kind[0], off16[0], pay0_16, end16, status_dev);
                    if (has1) sanitize_tile(kind[1], off16[1], pay0_16, end16, status_dev);
#pragma unroll
                    for (int h = 0; h < 2 && ok; ++h) {
#pragma unroll
                        for (int rb = 0; rb < 2 && ok; ++rb) {
                            if (rb == 1 && !has1) continue;
                            const bool dense = kind[rb] == PATCH_TILE_DENSE;
                            if (h == 1 && !dense) continue;          // a 2:4 tile arrived whole at h = 0
                            const int slot = ia % NA;
                            ok = mbar_wait(bar_emptyA + 8 * slot, (uint32_t(ia / NA) & 1u) ^ 1u, abort_flag, status_dev);
                            if (!ok) break;
                            const uint32_t bytes = dense ? kAtomBytes : kSparseBytes;
                            slot_kind[slot] = dense ? uint32_t(h) : kSparse;
                            mbar_expect_tx(bar_fullA + 8 * slot, bytes);
                            tma_bulk_load(smem_base + slot * kASlotBytes,
                                          blob + uint64_t(off16[rb]) * 16 + (dense ? h * kAtomBytes : 0u), bytes,
                                          bar_fullA + 8 * slot, pol);
                            ++ia;
                        }
                        if (!ok) break;
                        const int slot = ib % NB;
                        ok = mbar_wait(bar_emptyB + 8 * slot, (uint32_t(ib / NB) & 1u) ^ 1u, abort_flag, status_dev);
                        if (!ok) break;
                        mbar_expect_tx(bar_fullB + 8 * slot, x_half_bytes);
                        tma_tile_load(smem_base + kBOffset + slot * kBSlotBytes, &tmap_x, k * kTile + 64 * h, m0,
                                      bar_fullB + 8 * slot, pol);
                        ++ib;
                    }
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            }
        }
        if (lane == 0 && *abort_flag) {
            // drain: wait (bounded) until the copies this thread started have landed
            const uint64_t tstart = global_timer_ns();
            for (int j = ia > NA ? ia - NA : 0; j < ia; ++j)
                while (!mbar_try_wait(bar_fullA + 8 * (j % NA), uint32_t(j / NA) & 1u) &&
                       global_timer_ns() - tstart < kDrainLimitNs) {}
            for (int j = ib > NB ? ib - NB : 0; j < ib; ++j)
                while (!mbar_try_wait(bar_fullB + 8 * (j % NB), uint32_t(j / NB) & 1u) &&
                       global_timer_ns() - tstart < kDrainLimitNs) {}
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            const uint32_t idesc_d = instr_desc(0, false) | ((uint32_t(n_tok) >> 3) << 17);
            const uint32_t idesc_s = idesc_d | (1u << 2);
            bool ok = true;
            int ia = 0, ib = 0, j = 0;
            for (int t = blockIdx.x; t < n_out && ok; t += gridDim.x, ++j) {
                const bool has1 = 2 * (t % TP) + 1 < TN;
                // the epilogue must have drained both accumulators of the previous tile
                ok = mbar_wait(bar_acc_empty, (uint32_t(j) & 1u) ^ 1u, abort_flag, status_dev);
                for (int k = 0; k < TK && ok; ++k) {
                    int sp_slot[2] = {-1, -1};       // A slot of a 2:4 tile, kept from h = 0 to h = 1
#pragma unroll
                    for (int h = 0; h < 2 && ok; ++h) {
                        const int bslot = ib % NB;
                        ok = mbar_wait(bar_fullB + 8 * bslot, uint32_t(ib / NB) & 1u, abort_flag, status_dev);
                        if (!ok) break;
                        const uint64_t dB = desc_kmajor_sw128(smem_base + kBOffset + bslot * kBSlotBytes);
#pragma unroll
                        for (int rb = 0; rb < 2 && ok; ++rb) {
                            if (rb == 1 && !has1) continue;
                            const uint32_t acc = tmem_base + (rb ? kAcc1Col : 0u);
                            if (h == 0 || sp_slot[rb] < 0) {
                                // next A slot in ring order: a dense half, or (at h = 0) a whole 2:4 tile
                                const int slot = ia % NA;
                                ok = mbar_wait(bar_fullA + 8 * slot, uint32_t(ia / NA) & 1u, abort_flag, status_dev);
                                if (!ok) break;
                                ++ia;
                                tc_fence_after();
                                const uint64_t dA = desc_kmajor_sw128(smem_base + slot * kASlotBytes);
                                if (slot_kind[slot] != kSparse) {
#pragma unroll
                                    for (int ks = 0; ks < 4; ++ks)     // K = 16 each: 32 B of both operand rows
                                        mma_dense(acc, dA + uint64_t((ks * 32) >> 4), dB + uint64_t((ks * 32) >> 4), idesc_d,
                                                  !(k == 0 && h == 0 && ks == 0));
                                    mma_commit(bar_emptyA + 8 * slot);
                                } else {
                                    sp_slot[rb] = slot;
                                    const uint32_t e = tmem_base + meta_col(slot);
                                    tmem_copy_128x128b(e, desc_rows16(smem_base + slot * kASlotBytes + kAtomBytes));
#pragma unroll
                                    for (int ks = 0; ks < 2; ++ks)     // K = 32 each: 32 B of A, 64 B of B per row
                                        mma_sparse(acc, dA + uint64_t((ks * 32) >> 4), dB + uint64_t((ks * 64) >> 4), e,
                                                   idesc_s | uint32_t(ks & 1), !(k == 0 && ks == 0));
                                }
                            } else {
                                // second half of a 2:4 tile: metadata columns 2 and 3, kept values 64..127 B
                                tc_fence_after();
                                const int slot = sp_slot[rb];
                                const uint64_t dA = desc_kmajor_sw128(smem_base + slot * kASlotBytes);
                                const uint32_t e = tmem_base + meta_col(slot) + 2;
#pragma unroll
                                for (int ks = 0; ks < 2; ++ks)
                                    mma_sparse(acc, dA + uint64_t((64 + ks * 32) >> 4), dB + uint64_t((ks * 64) >> 4), e,
                                               idesc_s | uint32_t(ks & 1), true);
                                mma_commit(bar_emptyA + 8 * slot);
                            }
                        }
                        if (!ok) break;
                        mma_commit(bar_emptyB + 8 * bslot);
                        ++ib;
                    }
                }
                if (ok) mma_commit(bar_acc_full);
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: warps 2..9; lane quadrant = warp % 4, column half = (warp - 2) / 4 ----
        const uint32_t quad = warp & 3u;
        const int half = (warp - 2) >> 2;
        bool ok = true;
        int j = 0;
        for (int t = blockIdx.x; t < n_out && ok; t += gridDim.x, ++j) {
            const int tn0 = 2 * (t % TP), m0 = (t / TP) * n_tok;
            const bool has1 = tn0 + 1 < TN;
            // one thread polls, the other 255 epilogue threads sleep on a hardware barrier
            ok = group_wait(bar_acc_full, uint32_t(j) & 1u, warp == 2 && lane == 0, 1, 256, abort_flag, status_dev);
            if (!ok) break;
            tc_fence_after();
            if (independent && j == 0) grid_dependency_wait();     // Y may be in use by the preceding kernel
            const int valid = M - m0 < n_tok ? M - m0 : n_tok;      // tokens of this tile that exist
            const int chunks = (valid + 15) / 16, c_begin = half == 0 ? 0 : (chunks + 1) / 2,
                      c_end = half == 0 ? (chunks + 1) / 2 : chunks;
            if (gated) {
                // the pair is (gate row-block, up row-block) of the same 128 outputs: Y = silu(gate) * up,
                // one output row-block per pair
                const uint32_t acc_g = tmem_base + ((quad * 32u) << 16), acc_u = acc_g + kAcc1Col;
                __nv_bfloat16* ytile = Y + int64_t(m0) * ldy + int64_t(tn0 >> 1) * kTile + quad * 32;
#pragma unroll 1
                for (int ch = c_begin; ch < c_end; ++ch) {
                    const int c0 = ch * 16;
                    uint32_t g[16], u[16];
                    tmem_ld16(acc_g + uint32_t(c0), g);
                    tmem_ld16(acc_u + uint32_t(c0), u);
                    tmem_ld_wait();
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        const float x = __uint_as_float(g[q]);
                        g[q] = __float_as_uint(__fdividef(x, 1.0f + __expf(-x)) * __uint_as_float(u[q]));   // 2 MUFU ops, ~2 ulp
                    }
                    store_fragment_transposed(g, smem + kStageOffset + (warp - 2) * 1024, lane, ytile + int64_t(c0) * ldy, ldy,
                                              valid - c0);
                }
            }
#pragma unroll 1
            for (int rb = 0; rb < 2 && !gated; ++rb) {
                if (rb == 1 && !has1) break;
                const uint32_t acc = tmem_base + (rb ? kAcc1Col : 0u) + ((quad * 32u) << 16);
                __nv_bfloat16* ytile = Y + int64_t(m0) * ldy + int64_t(tn0 + rb) * kTile + quad * 32;
#pragma unroll 1
                for (int ch = c_begin; ch < c_end; ++ch) {
                    const int c0 = ch * 16;
                    uint32_t v[16];
                    tmem_ld16(acc + uint32_t(c0), v);
                    tmem_ld_wait();
                    store_fragment_transposed(v, smem + kStageOffset + (warp - 2) * 1024, lane, ytile + int64_t(c0) * ldy, ldy,
                                              valid - c0);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acc_empty);
        }
    }

    if (independent) grid_dependency_wait();      // every thread passes the dependency before the CTA exits
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

int launch_prefill2(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int64_t M, int n_tok,
                    int sms, __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool gated,
                    bool independent) {
    static std::atomic<uint64_t> configured{0};
    if (int rc = allow_dynamic_smem(prefill2_kernel, p2::kSmemBytes, configured)) return rc;
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    const int64_t n_out = int64_t((TN + 1) / 2) * ((M + n_tok - 1) / n_tok);
    if (n_out > 0x7FFFFFFF) return PATCH_ERR_SHAPE;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3(unsigned(n_out < sms ? n_out : sms), 1, 1);
    cfg.blockDim = dim3(320, 1, 1);
    cfg.dynamicSmemBytes = p2::kSmemBytes;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, prefill2_kernel, map, packed, uint64_t(L->table_off), uint32_t(L->payload_off / 16),
                                       uint32_t(L->total_bytes / 16), TN, TK, int(M), n_tok, Y, ldy, status_dev, gated ? 1 : 0,
                                       independent ? 1 : 0);
    return e == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

}  // namespace patch
