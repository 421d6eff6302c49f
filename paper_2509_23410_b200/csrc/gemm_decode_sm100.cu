// Small-M (decode) schedule of the hybrid dense / 2:4 tile matmul on the sm_100a tensor cores.
//
// Appendix A singles out decode as the stage that limits generation and split-K as the schedule
// its inspector picks there.  At M <= 64 tokens the layer is bound by the bytes of
// the packed weight, so the whole design serves one purpose: keep HBM busy.
//
//   * Work = the T = TN x TK weight tiles in (tn, tk) order.  One CTA per SM; CTA c streams the
//     contiguous run of tiles whose payload starts in the c-th 1/G of the payload bytes (a
//     byte-balanced split-K: a 2:4 tile costs 9/16 of a dense one).  The run boundaries are
//     found by a two-level warp-parallel search over the tile table.
//   * Per tile the MMA warp issues eight dense tcgen05.mma or four tcgen05.mma.sp (metadata
//     copied to TMEM) into an fp32 TMEM accumulator [128 out-features x N_TOK tokens]; weights
//     are the A operand, tokens ride the MMA N dimension (16/32/64).
//   * A run covers at most one partial row-block at each end; partial sums go through the
//     caller's workspace and are added in ascending K order (deterministic) before the single
//     bf16 rounding.  Up to 16 tokens: the partial-sum words double as flags (0 = empty); the CTA
//     that owns a row-block's first tile finishes it by polling the following CTAs' words (their
//     number follows from inverting the byte partition), then empties them -- one memory round
//     trip between the last MMA and the result.  32 or 64 tokens (partial tiles of 16-32 KB): a
//     64-bit counter per row-block collects {tiles, contributors, first contributor}; every
//     contributor waits for the count and finishes a share of the rows.  Two TMEM accumulators
//     let the epilogue of one row-block overlap the next row-block's MMAs.
//   * The kernel uses half an SM's shared memory and is launched with programmatic dependent
//     launch: the next GEMM's CTAs become resident while this one streams, fetch their first
//     weight tiles, and wait for this grid only where they touch X, Y or the workspace.
//
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, reports
// PATCH_ERR_TIMEOUT through status_dev, drains its copies in flight, frees TMEM and returns.
#include "sm100_ptx.cuh"

namespace patch {

constexpr int kMaxDecodeCtas = 192;      // workspace is sized for this many CTAs
#ifndef PATCH_XSTATIC_STAGES
#define PATCH_XSTATIC_STAGES 3           // ring depth when consecutive kernels stream concurrently (2 measured 2 % slower)
#endif

template <int N_TOK, int STAGES>
struct DecodeConfig {
    static constexpr uint32_t kXAtomBytes = N_TOK * 128;           // N_TOK rows x 64 bf16
    static constexpr uint32_t kXBytes = 2 * kXAtomBytes;           // 128 columns of K
    static constexpr uint32_t kStageBytes = kDenseBytes + kXBytes;
    static constexpr uint32_t kBarrierOffset = STAGES * kStageBytes;
    static constexpr uint32_t kSmemBytes = kBarrierOffset + 256 + 1024;  // + barriers + alignment slack
    static constexpr uint32_t kTmemNeeded = 2 * N_TOK + 4 * STAGES;      // two accumulators + metadata
    static constexpr uint32_t kTmemCols = kTmemNeeded <= 32 ? 32 : kTmemNeeded <= 64 ? 64 : kTmemNeeded <= 128 ? 128
                                          : kTmemNeeded <= 256 ? 256 : 512;
    static_assert(N_TOK % 16 == 0 && N_TOK >= 16 && N_TOK <= 64, "decode schedule: MMA N in {16, 32, 48, 64}");
    static_assert(STAGES >= 2 && STAGES <= 8, "2..8 pipeline stages");
};

// Number of table entries base[i * stride] (i < n) that are < target, over a whole warp.
__device__ __forceinline__ int warp_count_below(const uint32_t* base, int64_t stride_words, int n, uint32_t target,
                                                int lane) {
    int cnt = 0;
    for (int i = lane; i < n; i += 32) cnt += __ldg(base + int64_t(i) * stride_words) < target;
    return __reduce_add_sync(0xFFFFFFFFu, cnt);
}

// First tile whose payload offset (in 16-byte units) is >= target.  Offsets increase with the
// tile index, so: find the last row-block starting below target, then count inside it.
__device__ __forceinline__ int first_tile_at_or_after(const TileDesc* table, int TN, int TK, uint32_t target, int lane) {
    const uint32_t* off = &table[0].payload_off16;
    const int nb = warp_count_below(off, int64_t(TK) * 4, TN, target, lane);
    if (nb == 0) return 0;
    const int jb = nb - 1;
    return jb * TK + warp_count_below(off + int64_t(jb) * TK * 4, 4, TK, target, lane);
}

// t0 / t1 = first tile at or after `lo` / `hi` (as above), and the offset of the last tile of t1's row-block
// (t1 lies strictly inside that row-block whenever the caller needs it).
__device__ __forceinline__ void find_run(const TileDesc* table, int TN, int TK, uint32_t lo, uint32_t hi, int lane,
                                         int& t0, int& t1, uint32_t& off_last) {
    const uint32_t* off = &table[0].payload_off16;
    int c0 = 0, c1 = 0;
    for (int i = lane; i < TN; i += 32) {
        const uint32_t v = __ldg(off + int64_t(i) * TK * 4);
        c0 += v < lo;
        c1 += v < hi;
    }
    const int nb0 = __reduce_add_sync(0xFFFFFFFFu, c0), nb1 = __reduce_add_sync(0xFFFFFFFFu, c1);
    const int jb0 = nb0 ? nb0 - 1 : 0, jb1 = nb1 ? nb1 - 1 : 0;
    const uint32_t* row0 = off + int64_t(jb0) * TK * 4;
    const uint32_t* row1 = off + int64_t(jb1) * TK * 4;
    int d0 = 0, d1 = 0;
    for (int i = lane; i < TK; i += 32) {
        const uint32_t a = __ldg(row0 + i * 4), b = __ldg(row1 + i * 4);
        d0 += a < lo;
        d1 += b < hi;
    }
    off_last = __ldg(row1 + (TK - 1) * 4);
    t0 = nb0 ? jb0 * TK + __reduce_add_sync(0xFFFFFFFFu, d0) : 0;
    t1 = nb1 ? jb1 * TK + __reduce_add_sync(0xFFFFFFFFu, d1) : 0;
}

__device__ __forceinline__ unsigned long long atom_add_acq_rel_gpu(unsigned long long* p, unsigned long long v) {
    unsigned long long old;
    asm volatile("atom.acq_rel.gpu.global.add.u64 %0, [%1], %2;" : "=l"(old) : "l"(p), "l"(v) : "memory");
    return old;
}

// Barrier over the 128 epilogue threads that also ANDs a predicate.
__device__ __forceinline__ bool epilogue_all(bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
        "bar.red.and.pred p, 1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r) : "r"(uint32_t(pred)) : "memory");
    return r != 0;
}

// L2 load that the compiler keeps in program order, so that a batch of them is issued back to
// back before the first result is consumed.
__device__ __forceinline__ uint4 ld_cg_issue(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// 16-byte vector accesses at GPU scope that bypass L1.  A vector access is four 32-bit accesses,
// each single-copy atomic, which is all the flagged-partials protocol needs: every 32-bit word is
// either still empty (0) or the complete partial sum.
__device__ __forceinline__ void st_relaxed_gpu_v4(uint32_t* p, uint4 v) {
    asm volatile("st.relaxed.gpu.global.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint4 ld_relaxed_gpu_v4(const uint32_t* p) {
    uint4 v;
    asm volatile("ld.relaxed.gpu.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
// A partial sum of +0 would look like an empty word; -0 adds to the same result.
__device__ __forceinline__ uint32_t nonempty(uint32_t bits) { return bits == 0u ? 0x80000000u : bits; }

__device__ __forceinline__ unsigned long long ld_acquire_gpu(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}

// Gated mode (stacked gate/up weight, row-blocks interleaved): what the finisher of a row-block does with its 16
// finished fp32 values of one out-feature row.  An even row-block is a gate: its values are published as flagged
// words (0 = not there yet; +0 is stored as -0).  An odd row-block is the matching up projection: its finisher
// fetches the gate values (bounded poll), empties the words again and writes silu(gate) * up.  The gate's
// finisher waits for nothing here, and partial sums are always written before anything is polled, so the waits
// cannot form a cycle.
__device__ __forceinline__ bool finish_gated_row(const float (&a)[16], int tn, int row, int M, __nv_bfloat16* Y, int64_t ldy,
                                                 uint32_t* gate_words, volatile int* abort_flag, int* status_dev) {
    uint32_t* slot = gate_words + (int64_t(tn >> 1) * kTile + row) * 16;
    if ((tn & 1) == 0) {
#pragma unroll
        for (int q = 0; q < 4; ++q)
            st_relaxed_gpu_v4(slot + 4 * q, make_uint4(nonempty(__float_as_uint(a[4 * q])), nonempty(__float_as_uint(a[4 * q + 1])),
                                                      nonempty(__float_as_uint(a[4 * q + 2])), nonempty(__float_as_uint(a[4 * q + 3]))));
        return true;
    }
    uint4 w[4];
    const uint64_t tstart = global_timer_ns();
    for (bool all = false; !all;) {
#pragma unroll
        for (int q = 0; q < 4; ++q) w[q] = ld_relaxed_gpu_v4(slot + 4 * q);
        all = true;
#pragma unroll
        for (int q = 0; q < 4; ++q) all = all && w[q].x != 0u && w[q].y != 0u && w[q].z != 0u && w[q].w != 0u;
        if (!all && (*abort_flag || global_timer_ns() - tstart > kWaitLimitNs)) {
            *abort_flag = 1;
            if (status_dev) atomicCAS(status_dev, PATCH_OK, PATCH_ERR_TIMEOUT);
            return false;
        }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) st_relaxed_gpu_v4(slot + 4 * q, make_uint4(0, 0, 0, 0));   // empty again for the next launch
    const uint32_t g[16] = {w[0].x, w[0].y, w[0].z, w[0].w, w[1].x, w[1].y, w[1].z, w[1].w,
                            w[2].x, w[2].y, w[2].z, w[2].w, w[3].x, w[3].y, w[3].z, w[3].w};
    __nv_bfloat16* ycol = Y + int64_t(tn >> 1) * kTile + row;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float x = __uint_as_float(g[j]);
        if (j < M) ycol[int64_t(j) * ldy] = __float2bfloat16_rn(__fdividef(x, 1.0f + __expf(-x)) * a[j]);
    }
    return true;
}

// Every contributor of a row-block finishes rows [r0, r1) of it: thread `et` (0..127) takes
// (row, 16-token chunk) items, sums the n_contrib partial tiles in ascending K order and writes bf16.
template <int N_TOK>
__device__ __forceinline__ void reduce_row_share(const float* __restrict__ partials, int first_slot, int n_contrib,
                                                 int r0, int r1, int M, __nv_bfloat16* ytile, int64_t ldy, int et) {
    constexpr int CH = N_TOK / 16;
    const int c_lo = first_slot >> 1;
    const int items = (r1 - r0) * CH;
#pragma unroll 1
    for (int it = et; it < items; it += 128) {
        const int row = r0 + it / CH, c0 = (it % CH) * 16;
        if (c0 >= M) continue;
        float a[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) a[i] = 0.f;
#pragma unroll 1
        for (int j0 = 0; j0 < n_contrib; j0 += 8) {
            uint4 q[8][4];
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                const int j = j0 + jj < n_contrib ? j0 + jj : n_contrib - 1;
                const int s = j == 0 ? first_slot : 2 * (c_lo + j);
                const uint4* src = reinterpret_cast<const uint4*>(partials + (int64_t(s) * kTile + row) * N_TOK + c0);
#pragma unroll
                for (int i = 0; i < 4; ++i) q[jj][i] = ld_cg_issue(src + i);
            }
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                if (j0 + jj < n_contrib) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        a[4 * i + 0] += __uint_as_float(q[jj][i].x);
                        a[4 * i + 1] += __uint_as_float(q[jj][i].y);
                        a[4 * i + 2] += __uint_as_float(q[jj][i].z);
                        a[4 * i + 3] += __uint_as_float(q[jj][i].w);
                    }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < 16; ++i)
            if (c0 + i < M) ytile[int64_t(c0 + i) * ldy + row] = __float2bfloat16_rn(a[i]);
    }
}

// XSTATIC: the caller promises that X was not written by the operation preceding this launch
//          in the stream, so activations may be fetched before the grid dependency resolves.
// Weight tiles are always fetched early only if WSTATIC (same promise about the packed blob).
// GATED:   silu(gate) * up epilogue on a stacked gate/up weight (see finish_gated_row); 16-token schedule only.
template <int N_TOK, int STAGES, bool WSTATIC, bool XSTATIC, bool GATED = false>
__global__ void __launch_bounds__(192)
decode_kernel(const __grid_constant__ CUtensorMap tmap_x, const uint8_t* __restrict__ blob, uint64_t table_off,
              uint32_t pay0_16, uint32_t pay_total_16, int TN, int TK, int M,
              __nv_bfloat16* __restrict__ Y, int64_t ldy,
              unsigned long long* __restrict__ counters, float* __restrict__ partials, int* status_dev,
              uint32_t* __restrict__ gate_words) {
    static_assert(!GATED || N_TOK == 16, "the gated epilogue exists for the 16-token schedule");
    using Cfg = DecodeConfig<N_TOK, STAGES>;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_full = smem_base + Cfg::kBarrierOffset;    // 8 x 8 B
    const uint32_t bar_empty = bar_full + 64;                     // 8 x 8 B
    const uint32_t bar_acc_full = bar_empty + 64;                 // 2 x 8 B
    const uint32_t bar_acc_empty = bar_acc_full + 16;             // 2 x 8 B
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + Cfg::kBarrierOffset + 160);
    uint32_t* tmem_slot = misc;                                   // [0]
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 1);
    volatile int* range = reinterpret_cast<volatile int*>(misc + 2);          // [2], [3]: t0, t1
    volatile uint32_t* stage_kind = misc + 4;                                 // [4 .. 4+STAGES)
    volatile unsigned long long* red_info = reinterpret_cast<volatile unsigned long long*>(misc + 12);  // 8-B aligned

    grid_launch_dependents();   // the next kernel in the stream may become resident now

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int c = blockIdx.x, G = gridDim.x;
    const TileDesc* table = reinterpret_cast<const TileDesc*>(blob + table_off);

    if (warp == 0) {
        if constexpr (!WSTATIC) grid_dependency_wait();
        // byte-balanced run of tiles for this CTA
        const uint32_t lo = pay0_16 + uint32_t(uint64_t(c) * pay_total_16 / G);
        const uint32_t hi = pay0_16 + uint32_t(uint64_t(c + 1) * pay_total_16 / G);
        // Both ends of the run in two round trips to the table instead of five dependent ones: the row-block
        // starts serve both searches, the two in-row-block searches and the look-up below are independent.
        int t0, t1;
        uint32_t off_last;      // payload offset of the last tile of the row-block in which the run ends
        find_run(table, TN, TK, lo, hi, lane, t0, t1, off_last);
        if (c + 1 == G) t1 = TN * TK;
        int n_others = -1;
        if constexpr (N_TOK == 16) {
            // Flagged-partials protocol: if this run ends inside a row-block whose first tile it
            // owns, this CTA finishes that row-block.  The other contributors are the next CTAs, up
            // to the owner of the row-block's last tile (inverse of the byte partition above).
            const int tn_b = (t1 - 1) / TK;
            if (t1 > t0 && t1 < (tn_b + 1) * TK && t0 <= tn_b * TK) {
                const uint32_t d = off_last - pay0_16;
                int c_last = int(((uint64_t(d) + 1) * uint64_t(G) - 1) / pay_total_16);
                c_last = c_last < c ? c : c_last > G - 1 ? G - 1 : c_last;     // whatever the table says, a CTA of this grid
                n_others = c_last - c;
            }
        }
        if (lane == 0) { range[0] = t0; range[1] = t1; misc[16] = uint32_t(n_others); }
    }
    if (threadIdx.x == 64) {       // a thread outside warp 0, whose lanes are busy with the search
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
    const int t0 = range[0], t1 = range[1], n_tiles = t1 - t0;
    const uint32_t tmem_meta = tmem_base + 2 * N_TOK;    // 4 columns per stage; accumulators at 0 and N_TOK

    if (warp == 0) {
        // ---------------- producer: streams tiles t0 .. t1-1 through the stage ring ----------------
        const uint64_t pol_w = l2_policy_evict_first(), pol_x = l2_policy_evict_last();
        TileDesc mine = TileDesc{0, 0, 0, 0};
        int issued = 0;
        bool ok = true;
#ifdef PATCH_FAULT_INJECTION
        uint32_t inject_bytes = 0u;
        if (c == 0 && status_dev && *status_dev == kInjectMagic) {
            inject_bytes = 16u;
            __syncwarp();
            if (lane == 0) *status_dev = PATCH_OK;       // the word then reports like any other launch's
        }
#else
        constexpr uint32_t inject_bytes = 0u;
#endif
        // Weight tiles of the first STAGES steps may be requested before the grid dependency is
        // resolved (WSTATIC); their activations follow once it is (unless XSTATIC).
        const int n_early = (WSTATIC && !XSTATIC) ? (n_tiles < STAGES ? n_tiles : STAGES) : 0;
        for (int i = 0; i < n_tiles && ok; ++i) {
            if ((i & 31) == 0 && i + lane < n_tiles) mine = table[t0 + i + lane];   // 32 descriptors per load
            uint32_t kind = __shfl_sync(0xFFFFFFFFu, mine.kind, i & 31);
            uint32_t off16 = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, i & 31);
            if (lane == 0) {
                const int stage = i % STAGES;
                sanitize_tile(kind, off16, pay0_16, pay0_16 + pay_total_16, status_dev);
                const uint32_t wbytes = kind == PATCH_TILE_DENSE ? kDenseBytes : kSparseBytes;
                const uint32_t sW = smem_base + stage * Cfg::kStageBytes;
                const uint32_t full = bar_full + 8 * stage;
                if (i >= n_early)
                    ok = mbar_wait(bar_empty + 8 * stage, (uint32_t(i / STAGES) & 1u) ^ 1u, abort_flag, status_dev);
                if (ok) {
                    stage_kind[stage] = kind;
                    mbar_expect_tx(full, wbytes + Cfg::kXBytes + (i == 0 ? inject_bytes : 0u));
                    tma_bulk_load(sW, blob + uint64_t(off16) * 16, wbytes, full, pol_w);
                    if (i < n_early) {
                        if (i + 1 == n_early) {
                            grid_dependency_wait();
                            for (int j = 0; j < n_early; ++j) {
                                const uint32_t sX = smem_base + j * Cfg::kStageBytes + kDenseBytes;
                                const int k = ((t0 + j) % TK) * kTile;
                                tma_tile_load(sX, &tmap_x, k, 0, bar_full + 8 * j, pol_x);
                                tma_tile_load(sX + Cfg::kXAtomBytes, &tmap_x, k + 64, 0, bar_full + 8 * j, pol_x);
                            }
                        }
                    } else {
                        const uint32_t sX = sW + kDenseBytes;
                        const int k = ((t0 + i) % TK) * kTile;
                        tma_tile_load(sX, &tmap_x, k, 0, full, pol_x);
                        tma_tile_load(sX + Cfg::kXAtomBytes, &tmap_x, k + 64, 0, full, pol_x);
                    }
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
            int seg = 0, tk = t0 % TK;
            bool first = true, ok = true;
            for (int i = 0; i < n_tiles && ok; ++i) {
                const int stage = i % STAGES;
                if (first)   // the accumulator of segment `seg` must have been drained by the epilogue
                    ok = mbar_wait(bar_acc_empty + 8 * (seg & 1), (uint32_t(seg >> 1) & 1u) ^ 1u, abort_flag, status_dev);
                if (ok) ok = mbar_wait(bar_full + 8 * stage, uint32_t(i / STAGES) & 1u, abort_flag, status_dev);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sW = smem_base + stage * Cfg::kStageBytes;
                issue_tile_mma<N_TOK>(stage_kind[stage], sW, sW + kDenseBytes, Cfg::kXAtomBytes,
                                      tmem_base + uint32_t(seg & 1) * N_TOK, tmem_meta + 4 * stage, first);
                mma_commit(bar_empty + 8 * stage);            // frees the stage once these MMAs have read it
                const bool last = (tk == TK - 1) || (i == n_tiles - 1);
                if (last) { mma_commit(bar_acc_full + 8 * (seg & 1)); ++seg; }
                first = last;
                tk = (tk == TK - 1) ? 0 : tk + 1;
            }
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: warps 2..5, TMEM lane quadrant = warp % 4 ----------------
        const uint32_t quad = warp & 3u, row = quad * 32 + lane;   // out-feature inside the row-block
        const int et = threadIdx.x - 64;                           // 0..127
        bool waited = false, ok = true;
        int seg = 0;
        // A run has at most two partial row-blocks: its first segment (k = 0) and its last (k = 1).
        // Thread 32k updates the counter of partial k; the result is looked at only after every
        // segment of the run is out, so the two updates and the second segment's writes overlap.
        int part_tn[2] = {-1, -1};
        unsigned long long seen = 0ull;
        for (int ts = t0; ts < t1 && ok; ++seg) {
            const int tn = ts / TK;
            const int te = (tn + 1) * TK < t1 ? (tn + 1) * TK : t1;
            const int ntiles = te - ts;
            ok = mbar_wait(bar_acc_full + 8 * (seg & 1), uint32_t(seg >> 1) & 1u, abort_flag, status_dev);
            ok = epilogue_all(ok);      // same decision in all 128 threads: they share barriers below
            if (!ok) break;
            tc_fence_after();
            if (!waited) {              // Y and the workspace may be in use by the previous kernel until here
                grid_dependency_wait();
                waited = true;
            }
            const uint32_t acc = tmem_base + uint32_t(seg & 1) * N_TOK + ((quad * 32u) << 16);
            if (GATED && ntiles == TK) {
                // whole row-block in this run: its values are final
                uint32_t v[16];
                tmem_ld16(acc, v);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty + 8 * (seg & 1));
                float a[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) a[j] = __uint_as_float(v[j]);
                ok = finish_gated_row(a, tn, row, M, Y, ldy, gate_words, abort_flag, status_dev);
            } else if (ntiles == TK) {
                // whole row-block in this run: finish it here
                __nv_bfloat16* ycol = Y + int64_t(tn) * kTile + row;
#pragma unroll 1
                for (int c0 = 0; c0 < M; c0 += 16) {
                    uint32_t v[16];
                    tmem_ld16(acc + uint32_t(c0), v);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        if (c0 + j < M) ycol[int64_t(c0 + j) * ldy] = __float2bfloat16_rn(__uint_as_float(v[j]));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty + 8 * (seg & 1));
            } else if constexpr (N_TOK == 16) {
                // Partial row-block, flagged-partials protocol.  A slot is [CTA][row][16 tokens] fp32 whose
                // words double as flags: 0 = not written yet (+0 is stored as -0).  The finishing CTA polls
                // the words themselves, so no fence, counter or second round trip separates writer and reader.
                uint32_t* words = reinterpret_cast<uint32_t*>(partials);
                uint32_t v[16];
                tmem_ld16(acc, v);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty + 8 * (seg & 1));
                if (seg == 0 && t0 > tn * TK) {
                    // the run starts inside this row-block: hand the partial to the CTA that owns its first tile
                    uint32_t* mine = words + (int64_t(c) * kTile + row) * 16;
#pragma unroll
                    for (int j = 0; j < 16; j += 4)
                        st_relaxed_gpu_v4(mine + j, make_uint4(nonempty(v[j]), nonempty(v[j + 1]), nonempty(v[j + 2]),
                                                               nonempty(v[j + 3])));
                } else {
                    // this run owns the row-block's first tile and ends inside it: add the following CTAs'
                    // partials in ascending K order, five contributors in flight at a time
                    constexpr int kBatch = 5;     // covers the usual 148 / TN + 1 contributors in one round trip
                    const int n_others = int(misc[16]);
                    float a[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) a[j] = __uint_as_float(v[j]);
#pragma unroll 1
                    for (int j0 = 0; j0 < n_others && ok; j0 += kBatch) {
                        uint4 w[kBatch][4];
                        const uint64_t tstart = global_timer_ns();
                        for (bool all = false; !all;) {
#pragma unroll
                            for (int jj = 0; jj < kBatch; ++jj) {
                                const int cj = c + 1 + (j0 + jj < n_others ? j0 + jj : n_others - 1);
                                const uint32_t* src = words + (int64_t(cj) * kTile + row) * 16;
#pragma unroll
                                for (int q = 0; q < 4; ++q) w[jj][q] = ld_relaxed_gpu_v4(src + 4 * q);
                            }
                            all = true;
#pragma unroll
                            for (int jj = 0; jj < kBatch; ++jj)
#pragma unroll
                                for (int q = 0; q < 4; ++q)
                                    all = all && w[jj][q].x != 0u && w[jj][q].y != 0u && w[jj][q].z != 0u && w[jj][q].w != 0u;
                            if (!all && (*abort_flag || global_timer_ns() - tstart > kWaitLimitNs)) {
                                *abort_flag = 1;
                                if (status_dev) atomicCAS(status_dev, PATCH_OK, PATCH_ERR_TIMEOUT);
                                ok = false;
                                break;
                            }
                        }
                        if (!ok) break;
#pragma unroll
                        for (int jj = 0; jj < kBatch; ++jj) {
                            if (j0 + jj < n_others) {
                                uint32_t* src = words + (int64_t(c + 1 + j0 + jj) * kTile + row) * 16;
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    a[4 * q + 0] += __uint_as_float(w[jj][q].x);
                                    a[4 * q + 1] += __uint_as_float(w[jj][q].y);
                                    a[4 * q + 2] += __uint_as_float(w[jj][q].z);
                                    a[4 * q + 3] += __uint_as_float(w[jj][q].w);
                                    st_relaxed_gpu_v4(src + 4 * q, make_uint4(0, 0, 0, 0));   // empty again for the next launch
                                }
                            }
                        }
                    }
                    if (ok && GATED) {
                        ok = finish_gated_row(a, tn, row, M, Y, ldy, gate_words, abort_flag, status_dev);
                    } else if (ok) {
                        __nv_bfloat16* ycol = Y + int64_t(tn) * kTile + row;
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (j < M) ycol[int64_t(j) * ldy] = __float2bfloat16_rn(a[j]);
                    }
                }
            } else {
                // partial row-block: write fp32 partial sums ([slot][row][token]), then count in
                const int k = seg == 0 ? 0 : 1;
                float* slot = partials + (int64_t(2 * c + k) * kTile + row) * N_TOK;
#pragma unroll 1
                for (int c0 = 0; c0 < M; c0 += 16) {
                    uint32_t v[16];
                    tmem_ld16(acc + uint32_t(c0), v);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; j += 4)
                        __stcg(reinterpret_cast<uint4*>(slot + c0 + j), make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]));
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty + 8 * (seg & 1));
                asm volatile("bar.sync 1, 128;" ::: "memory");      // all 128 epilogue threads have written
                part_tn[k] = tn;
                if (et == 32 * k) {
                    // {tiles : 16, contributors : 16, first contributor's slot + 1 : 16, finished readers : 16}
                    unsigned long long add = (unsigned long long)ntiles | (1ull << 16);
                    if (ts == tn * TK) add |= (unsigned long long)(2 * c + k + 1) << 32;
                    // release: publishes the partial sums written before the barrier;
                    // acquire: the last contributor then sees every other contributor's
                    seen = atom_add_acq_rel_gpu(&counters[tn], add) + add;
                }
            }
            ts = te;
        }
        if constexpr (N_TOK > 16) {
            // large partial tiles (32 or 64 tokens): every contributor finishes a share of the rows.  All
            // partials of this CTA are already published above, so waiting here cannot form a cycle.
#pragma unroll 1
            for (int k = 0; k < 2 && ok; ++k) {
                if (part_tn[k] < 0) continue;
                unsigned long long* ctr = &counters[part_tn[k]];
                if (et == 32 * k) {
                    unsigned long long cur = seen;
                    const uint64_t tstart = global_timer_ns();
                    while (int(cur & 0xFFFFu) != TK) {                 // bounded wait for the other contributors
                        cur = ld_acquire_gpu(ctr);
                        if (*abort_flag || global_timer_ns() - tstart > kWaitLimitNs) {
                            *abort_flag = 1;
                            if (status_dev) atomicCAS(status_dev, PATCH_OK, PATCH_ERR_TIMEOUT);
                            cur = 0ull;
                            break;
                        }
                    }
                    red_info[k] = cur;
                }
                asm volatile("bar.sync 1, 128;" ::: "memory");
                const unsigned long long info = red_info[k];
                ok = info != 0ull;
                if (ok) {
                    const int n_contrib = int((info >> 16) & 0xFFFFu);
                    const int first_slot = int((info >> 32) & 0xFFFFu) - 1;
                    const int mine = (2 * c + k == first_slot) ? 0 : c - (first_slot >> 1);   // position in K order
                    reduce_row_share<N_TOK>(partials, first_slot, n_contrib, kTile * mine / n_contrib,
                                            kTile * (mine + 1) / n_contrib, M, Y + int64_t(part_tn[k]) * kTile, ldy, et);
                    asm volatile("bar.sync 1, 128;" ::: "memory");     // every thread has read its partials
                    if (et == 32 * k) {
                        // count finished readers in bits 48..63; the last one clears the counter for the next launch
                        const unsigned long long old = atomicAdd(ctr, 1ull << 48);
                        if (int(old >> 48) + 1 == n_contrib) *ctr = 0ull;
                    }
                }
            }
        }
    }

    grid_dependency_wait();     // completion of this grid implies completion of its predecessors
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, Cfg::kTmemCols);
}

// ---------------------------------------------------------------------------------------------
// host side

static int decode_n_tok(int64_t M) { return M <= 16 ? 16 : M <= 32 ? 32 : 64; }

// Workspace layout: [arrival counters | flagged partial sums of the 16-token schedule | partial tiles of the
// 32/64-token schedule].  The flagged words must be zero between calls (the schedule that uses them leaves
// them so); the partial tiles need not be (they are written before they are read and are never taken for
// flags), so the two regions are disjoint.  The counter region is 8 KB for every N <= 131072, which makes
// the offsets the same for all such layouts: one workspace, zeroed once, serves any mix of them and of M.
static size_t counters_bytes(const patch_layout_t* L) {
    const size_t need = (size_t(L->N / kTile) * 8 + 255) / 256 * 256;
    return need > 8192 ? need : 8192;
}
constexpr size_t kFlaggedBytes = size_t(2) * kMaxDecodeCtas * 16 * kTile * sizeof(float);

// Gated mode: one slot of [128 rows][16 tokens] flag words per (gate, up) pair of row-blocks, past everything
// the plain schedules use of the same workspace (their partial tiles are not kept zero).
static size_t gate_words_offset(const patch_layout_t* L) {
    return counters_bytes(L) + kFlaggedBytes + size_t(2) * kMaxDecodeCtas * 64 * kTile * sizeof(float);
}
size_t decode_gated_workspace_bytes(const patch_layout_t* L, int64_t M) {
    if (M > 16) return 0;
    return gate_words_offset(L) + size_t(L->N / (2 * kTile)) * kTile * 16 * sizeof(float);
}

size_t decode_workspace_bytes(const patch_layout_t* L, int64_t M) {
    if (M > 64) return 0;
    const int n_tok = decode_n_tok(M);
    return counters_bytes(L) + kFlaggedBytes + (n_tok > 16 ? size_t(2) * kMaxDecodeCtas * n_tok * kTile * sizeof(float) : 0);
}

template <int N_TOK, int STAGES, bool WSTATIC, bool XSTATIC, bool GATED = false>
static int launch_decode_t(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int M,
                           __nv_bfloat16* Y, int64_t ldy, void* workspace, int* status_dev, cudaStream_t stream) {
    using Cfg = DecodeConfig<N_TOK, STAGES>;
    auto kern = decode_kernel<N_TOK, STAGES, WSTATIC, XSTATIC, GATED>;
    static std::atomic<uint64_t> configured{0};
    if (int rc = allow_dynamic_smem(kern, Cfg::kSmemBytes, configured)) return rc;
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    if (TK > 65535) return PATCH_ERR_SHAPE;
    int G = sm_count();
    if (G <= 0) return PATCH_ERR_CUDA;
    if (G > kMaxDecodeCtas) G = kMaxDecodeCtas;
    // every CTA's byte range must be longer than the largest tile so that no run is empty
    // (the reduction assumes the contributors of a row-block are consecutive CTAs)
    const uint64_t by_bytes = L->payload_bytes / (2 * kDenseBytes);
    if (uint64_t(G) > by_bytes) G = by_bytes ? int(by_bytes) : 1;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3(G, 1, 1);
    cfg.blockDim = dim3(192, 1, 1);
    cfg.dynamicSmemBytes = Cfg::kSmemBytes;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    unsigned long long* counters = static_cast<unsigned long long*>(workspace);
    float* partials = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + counters_bytes(L) + (N_TOK > 16 ? kFlaggedBytes : 0));
    uint32_t* gate_words = GATED ? reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(workspace) + gate_words_offset(L)) : nullptr;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, map, packed, uint64_t(L->table_off),
                                       uint32_t(L->payload_off / 16), uint32_t(L->payload_bytes / 16), TN, TK, M, Y,
                                       ldy, counters, partials, status_dev, gate_words);
    return e == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

template <int N_TOK, int STAGES>
static int launch_decode_f(bool wstatic, bool xstatic, const CUtensorMap& map, const patch_layout_t* L,
                           const uint8_t* packed, int M, __nv_bfloat16* Y, int64_t ldy, void* workspace,
                           int* status_dev, cudaStream_t stream) {
    if (wstatic && xstatic) return launch_decode_t<N_TOK, STAGES, true, true>(map, L, packed, M, Y, ldy, workspace, status_dev, stream);
    if (wstatic) return launch_decode_t<N_TOK, STAGES, true, false>(map, L, packed, M, Y, ldy, workspace, status_dev, stream);
    // X may only be fetched early if the weight may be as well (the flag alone changes nothing)
    return launch_decode_t<N_TOK, STAGES, false, false>(map, L, packed, M, Y, ldy, workspace, status_dev, stream);
}

// Which small-M schedule serves a launch: stream-K over all SMs (a lone or dependent GEMM gets the whole
// GPU's bandwidth) or one CTA per row-block / small cluster (independent GEMMs: several of them are resident
// at once and together stream faster).  With the weights promise alone (X may be the predecessor's output) the
// row-block schedule still wins, with more CTAs per GEMM: its split-K sums meet in shared memory instead of
// travelling through L2 behind the predecessor's completion (24-GEMM step: 0.322 against 0.339 ms).
static bool use_rowblock_schedule(bool wstatic, bool xstatic) { (void)xstatic; return wstatic; }

int launch_decode(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                  __nv_bfloat16* Y, int64_t ldy, void* workspace, int* status_dev, cudaStream_t stream,
                  bool wstatic, bool xstatic, bool ystatic) {
    const int n_tok = decode_n_tok(M);
    CUtensorMap map;
    int rc = make_x_tensor_map(&map, X, ldx, M, L->K, n_tok);
    if (rc) return rc;
    if (use_rowblock_schedule(wstatic, xstatic))
        return launch_decode_cluster(map, L, packed, int(M), n_tok, Y, ldy, status_dev, stream, wstatic, xstatic, ystatic);
    switch (n_tok) {
        case 16:
            if (wstatic && xstatic)
                return launch_decode_f<16, PATCH_XSTATIC_STAGES>(wstatic, xstatic, map, L, packed, int(M), Y, ldy, workspace, status_dev, stream);
            return launch_decode_f<16, 3>(wstatic, xstatic, map, L, packed, int(M), Y, ldy, workspace, status_dev, stream);
        case 32: return launch_decode_f<32, 2>(wstatic, xstatic, map, L, packed, int(M), Y, ldy, workspace, status_dev, stream);
        default: return launch_decode_f<64, 2>(wstatic, xstatic, map, L, packed, int(M), Y, ldy, workspace, status_dev, stream);
    }
}

// silu(gate) * up on a stacked gate/up weight with interleaved row-blocks, M <= 16: Y is [M x N / 2].
int launch_decode_gated(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                        __nv_bfloat16* Y, int64_t ldy, void* workspace, int* status_dev, cudaStream_t stream,
                        bool wstatic, bool xstatic) {
    CUtensorMap map;
    int rc = make_x_tensor_map(&map, X, ldx, M, L->K, 16);
    if (rc) return rc;
    if (wstatic && xstatic)
        return launch_decode_t<16, PATCH_XSTATIC_STAGES, true, true, true>(map, L, packed, int(M), Y, ldy, workspace, status_dev, stream);
    if (wstatic) return launch_decode_t<16, 3, true, false, true>(map, L, packed, int(M), Y, ldy, workspace, status_dev, stream);
    return launch_decode_t<16, 3, false, false, true>(map, L, packed, int(M), Y, ldy, workspace, status_dev, stream);
}

}  // namespace patch

// ---------------------------------------------------------------------------------------------
// Entry point that brings its own scratch memory (see include/patch.h: patch_gemm_noalloc).

namespace {

constexpr int kNoAllocMaxTokens = 16;         // decode only
constexpr int kNoAllocMaxRowBlocks = 1024;    // N <= 131072
constexpr size_t kNoAllocCounterBytes = size_t(kNoAllocMaxRowBlocks) * 8;
constexpr size_t kNoAllocScratchBytes =
    kNoAllocCounterBytes + size_t(2) * patch::kMaxDecodeCtas * kNoAllocMaxTokens * patch::kTile * sizeof(float);

// Lives in the library image: every GPU that loads the library holds these ~3.2 MB until exit.
// In host code this name is only a handle; the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

std::atomic<void*> g_noalloc_ptr[patch::kMaxDevices];   // device address of the array, per device, once known

}  // namespace

extern "C" int patch_gemm_noalloc(const void* X_dev, int64_t ldx, int64_t M, const patch_layout_t* L,
                                  const void* packed_dev, void* Y_dev, int64_t ldy, void* stream) {
    using namespace patch;
    if (!L) return PATCH_ERR_NULL;
    int rc = validate_layout(L);
    if (rc) return rc;
    if (M < 0) return PATCH_ERR_SHAPE;
    if (M == 0) return PATCH_OK;
    if (has_q4_tiles(L)) return PATCH_ERR_SHAPE;
    if (M > kNoAllocMaxTokens || L->N / kTile > kNoAllocMaxRowBlocks) return PATCH_ERR_SIZE;
    if (!X_dev || !packed_dev || !Y_dev) return PATCH_ERR_NULL;
    if (ldx < L->K || ldy < L->N || ldx % 8 || ldy % 8) return PATCH_ERR_SHAPE;
    if (!aligned16(X_dev) || !aligned16(Y_dev) || !aligned16(packed_dev)) return PATCH_ERR_ALIGN;
    rc = check_device();
    if (rc) return rc;
    const int dev = current_device();
    if (dev < 0) return PATCH_ERR_CUDA;
    void* scratch = g_noalloc_ptr[dev].load(std::memory_order_acquire);
    if (!scratch) {
        // set-up, once per device, with that device current (two threads racing here store the same address)
        if (cudaGetSymbolAddress(&scratch, g_noalloc_scratch) != cudaSuccess || !scratch) return PATCH_ERR_CUDA;
        g_noalloc_ptr[dev].store(scratch, std::memory_order_release);
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The whole array is cleared on every call: counters and partial-sum flags must start at zero, and the array
    // keeps whatever the last call left -- also a call that was aborted or that raced with another one.
    if (cudaMemsetAsync(scratch, 0, kNoAllocScratchBytes, s) != cudaSuccess) return PATCH_ERR_CUDA;
    return launch_decode(static_cast<const __nv_bfloat16*>(X_dev), ldx, M, L, static_cast<const uint8_t*>(packed_dev),
                         static_cast<__nv_bfloat16*>(Y_dev), ldy, scratch, nullptr, s, false, false);
}
