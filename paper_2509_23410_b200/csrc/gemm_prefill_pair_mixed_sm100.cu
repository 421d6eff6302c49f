// CTA-pair large-M schedule for weights that MIX dense and 2:4 tiles (the hybrid case proper of Appendix A).
//
// Same ownership and pair protocol as gemm_prefill_pair_sm100.cu: a cluster of two CTAs owns four row-blocks
// (pair j = row-blocks 4q + 2j and 4q + 2j + 1, one in each CTA) and one token tile, one thread of the leader
// issues cta_group::2 MMAs over 256 out-features, every copy is a pair-form tiled TMA load (no multicast).
//
// One pair instruction has one kind, but the two tiles of a pair choose theirs independently.  Per K step and pair:
//   * both dense   -> tcgen05.mma, one 16 KB K-half of each tile per stage;
//   * both 2:4     -> tcgen05.mma.sp: each whole tile (16 KB kept values + 2 KB metadata) arrives with the
//                     stage of the first K-half and stays until the second K-half is done;
//   * one of each  -> the pair runs dense, and the CTA that holds the 2:4 tile expands it to its dense image
//                     W (.) M* (kept values at their positions, zeros elsewhere -- Algorithm 1's pruned tile).
// The expansion needs no extra buffer.  The compressed tile lands in the A region of the first K-half's stage;
// thread r of four helper warps reads row r (64 kept values + its position codes) into registers, writes the
// dense first half of that row over it and the dense second half into the same row of the next stage's A
// region: a row is touched by one thread only, so the rewrite in place is safe, and the metadata behind the
// 16 KB of values is not overwritten.  Nothing else is decompressed, and the bytes fetched are the packed ones.
//
// Stages: one K-half (64 columns) each, [A region pair 0 | A region pair 1 | B] = 18 + 18 + 15 KB, four deep.
// The leader's "full" barrier of a stage collects: its producer's byte count (the pair-form copies of both CTAs)
// and one arrival per CTA and pair -- from that CTA's helper warps where they fill the A region, from the LEADER's
// producer otherwise (it reads the tile kinds of both CTAs, so nothing crosses the pair unless a tile was expanded).
// A compressed tile that awaits expansion is counted on a barrier of its own CTA.
//
// 448 threads: warp 0 producer, warp 1 MMA issuer (leader) and TMEM owner, warps 2..9 epilogue, warps 10..13
// expansion.  Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, reports
// PATCH_ERR_TIMEOUT through status_dev, and every role still runs to the common cluster barrier at the end.
#include "sm100_ptx.cuh"

namespace patch {

namespace pm {
constexpr int kThreads = 448;
constexpr int NST = 4;
constexpr int kMaxTok = 240;                                     // two accumulators + 32 metadata columns = 512
constexpr uint32_t kARegionBytes = kSparseBytes;                 // 18 432: a dense K-half or a whole 2:4 tile
constexpr uint32_t kBRegionBytes = (kMaxTok / 2) * 128;          // 15 360
constexpr uint32_t kBOffset = 2 * kARegionBytes;
constexpr uint32_t kStageBytes = kBOffset + kBRegionBytes;       // 52 224
constexpr uint32_t kBarrierOffset = NST * kStageBytes;
constexpr uint32_t kEpiOffset = kBarrierOffset + 256;            // 8 epilogue warps x 1 KB transpose staging
constexpr uint32_t kSmemBytes = kEpiOffset + 8 * 1024 + 1024;    // + alignment slack
static_assert(kStageBytes % 1024 == 0 && kSmemBytes <= 227 * 1024, "shared memory layout");
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kAcc1Col = 256;
constexpr int kExpandWarp0 = 10, kExpandThreads = 128;
// metadata: 4 TMEM columns per (stage, pair), in the gaps [240,256) and [496,512)
__device__ __forceinline__ uint32_t meta_col(int stage, int j) {
    const int i = 2 * stage + j;
    return i < 4 ? 240u + 4u * i : 496u + 4u * (i - 4);
}

// The row-blocks of a quad as seen from one CTA (clamped to TN - 1 where they do not exist: such a tile is loaded
// and multiplied like any other and never stored, so that both CTAs run the same sequence).
struct Quad { int own[2], peer[2], npairs; };
__device__ __forceinline__ Quad make_quad(int q, int TN, uint32_t rank) {
    Quad Q;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        const int a = 4 * q + 2 * j + int(rank), b = 4 * q + 2 * j + 1 - int(rank);
        Q.own[j] = a < TN ? a : TN - 1;
        Q.peer[j] = b < TN ? b : TN - 1;
    }
    Q.npairs = 4 * q + 2 < TN ? 2 : 1;
    return Q;
}
// lanes 8i .. 8i+7 hold the table entries of K steps k0 .. k0+7 of {own[0], own[1], peer[0], peer[1]}[i]
__device__ __forceinline__ TileDesc load_step_descs(const TileDesc* table0, int TK, const Quad& Q, int k0, int lane) {
    const int i = lane >> 3, kk = k0 + (lane & 7);
    const int rb = i == 0 ? Q.own[0] : i == 1 ? Q.own[1] : i == 2 ? Q.peer[0] : Q.peer[1];
    TileDesc d = TileDesc{0, 0, 0, 0};
    if (kk < TK) d = table0[int64_t(rb) * TK + kk];
    return d;
}
// What one K step looks like from this CTA.  A kind other than DENSE counts as 2:4 here; the host has checked
// the table against the layout, and every address derived from it goes through a tensor map, which cannot fault.
struct Step {
    bool own_sparse[2], peer_sparse[2];
    uint32_t off256[2];                    // payload offset / 256 of this CTA's tile of pair j
    __device__ __forceinline__ bool sparse_pair(int j) const { return own_sparse[j] && peer_sparse[j]; }
    __device__ __forceinline__ bool expand(int j) const { return own_sparse[j] && !peer_sparse[j]; }
};
__device__ __forceinline__ Step step_info(const TileDesc& mine, int k) {      // all 32 lanes call this
    Step s;
#pragma unroll
    for (int j = 0; j < 2; ++j) {
        s.off256[j] = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, 8 * j + (k & 7)) >> 4;
        s.own_sparse[j] = __shfl_sync(0xFFFFFFFFu, mine.kind, 8 * j + (k & 7)) != PATCH_TILE_DENSE;
        s.peer_sparse[j] = __shfl_sync(0xFFFFFFFFu, mine.kind, 8 * (2 + j) + (k & 7)) != PATCH_TILE_DENSE;
    }
    return s;
}
// bytes that the pair-form copies of one CTA bring into a stage for its tile of pair j (counted on the leader's barrier)
__device__ __forceinline__ uint32_t pair_form_bytes(bool mine_sparse, bool other_sparse, int h) {
    if (!mine_sparse) return kAtomBytes;                           // a dense K-half
    if (other_sparse) return h == 0 ? kSparseBytes : 0u;           // a whole 2:4 tile with the first K-half
    return 0u;                                                     // awaits expansion: counted on this CTA's own barrier
}
}  // namespace pm

__global__ void __launch_bounds__(pm::kThreads)
prefill_pair_mixed_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w16,
                          const __grid_constant__ CUtensorMap tmap_w18, const uint8_t* __restrict__ blob, uint64_t table_off,
                          int TN, int TK, int M, int n_tok, __nv_bfloat16* __restrict__ Y, int64_t ldy, int* status_dev,
                          int independent) {
    using namespace pm;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_full = smem_base + kBarrierOffset;         // NST x 8 B; waited for in the leader only
    const uint32_t bar_empty = bar_full + 32;                     // NST x 8 B
    const uint32_t bar_land = bar_empty + 32;                     // NST x 2 x 8 B: compressed tile (stage, pair) has landed here
    const uint32_t bar_acc_full = bar_land + 64;                  // 8 B
    const uint32_t bar_acc_empty = bar_acc_full + 8;              // 8 B, used in the leader only
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kBarrierOffset + 160);
    uint32_t* tmem_slot = misc;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const bool leader = rank == 0;
    const int TQ = (TN + 3) / 4;                                   // quads of row-blocks
    const int MT = (M + n_tok - 1) / n_tok;
    const int n_out = TQ * MT;                                     // output tiles, index = mt * TQ + quad
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    const int n_half = n_tok >> 1;
    const uint32_t x_half_bytes = uint32_t(n_half) * 128u;
    const TileDesc* table0 = reinterpret_cast<const TileDesc*>(blob + table_off);

    if (threadIdx.x == 0) {
        for (int i = 0; i < NST; ++i) {
            // the leader producer's arrive.expect_tx + one arrival per CTA and pair (producer or helper warps)
            mbar_init(bar_full + 8 * i, 5);
            mbar_init(bar_empty + 8 * i, 1);     // one commit of the issuing thread, delivered to both CTAs
            mbar_init(bar_land + 16 * i, 1);
            mbar_init(bar_land + 16 * i + 8, 1);
        }
        mbar_init(bar_acc_full, 1);              // one commit, delivered to both CTAs
        mbar_init(bar_acc_empty, 16);            // one arrival per epilogue warp of both CTAs
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_map(&tmap_x);
        tma_prefetch_map(&tmap_w16);
        tma_prefetch_map(&tmap_w18);
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();     // both CTAs' barriers and tensor memory exist before anything crosses the pair
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // programmatic dependent launch, as in the one-kind pair kernel
    grid_launch_dependents();
    if (!independent) grid_dependency_wait();

    if (warp == 0) {
        // ---------------- producer ----------------
        const uint64_t pol = l2_policy_evict_last();
        const uint32_t leader_full = map_to_rank(bar_full, 0);
        int g = 0;                           // stage counter, continues across output tiles
        bool ok = true;
        for (int t = cluster_id; t < n_out && ok; t += n_clusters) {
            const Quad Q = make_quad(t % TQ, TN, rank);
            const int m0 = (t / TQ) * n_tok + int(rank) * n_half;
            TileDesc mine, next = load_step_descs(table0, TK, Q, 0, lane);
            for (int k = 0; k < TK && ok; ++k) {
                if ((k & 7) == 0) { mine = next; next = load_step_descs(table0, TK, Q, k + 8, lane); }   // one batch ahead
                const Step s = step_info(mine, k);
                if (lane == 0) {
#pragma unroll
                    for (int h = 0; h < 2; ++h, ++g) {
                        if (!ok) continue;
                        const int st = g % NST;
                        const uint32_t stage = smem_base + st * kStageBytes, full = leader_full + 8 * st;
                        ok = mbar_wait(bar_empty + 8 * st, (uint32_t(g / NST) & 1u) ^ 1u, abort_flag, status_dev);
                        if (!ok) continue;
                        if (leader) {
                            uint32_t bytes = 2 * x_half_bytes;
#pragma unroll
                            for (int j = 0; j < 2; ++j)
                                if (j < Q.npairs)
                                    bytes += pair_form_bytes(s.own_sparse[j], s.peer_sparse[j], h) +
                                             pair_form_bytes(s.peer_sparse[j], s.own_sparse[j], h);
                            mbar_expect_tx(bar_full + 8 * st, bytes);
                            // A regions that no helper warp fills, here or in the other CTA (whose tile kinds this
                            // thread knows as well): their arrivals are made here, locally -- an arrival that crosses
                            // the pair costs about a microsecond and must stay off the path of the copies
#pragma unroll
                            for (int j = 0; j < 2; ++j) {
                                if (!(j < Q.npairs && s.expand(j))) mbar_arrive(bar_full + 8 * st);
                                if (!(j < Q.npairs && s.peer_sparse[j] && !s.own_sparse[j])) mbar_arrive(bar_full + 8 * st);
                            }
                        }
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            const bool expanding = j < Q.npairs && s.expand(j);
                            if (j >= Q.npairs) continue;
                            const uint32_t dst = stage + j * kARegionBytes;
                            if (!s.own_sparse[j]) {
                                tma_tile_load_pair(dst, &tmap_w16, 0, int(s.off256[j]) + h * int(kAtomBytes / 256), full, pol);
                            } else if (h == 0) {
                                if (!expanding) {
                                    tma_tile_load_pair(dst, &tmap_w18, 0, int(s.off256[j]), full, pol);
                                } else {
                                    // 2:4 tile of a dense pair: lands here, counted here; the helper warps take it from there
                                    const uint32_t land = bar_land + 16 * st + 8 * j;
                                    mbar_expect_tx(land, kSparseBytes);
                                    tma_tile_load(dst, &tmap_w18, 0, int(s.off256[j]), land, pol);
                                }
                            }
                        }
                        tma_tile_load_pair(stage + kBOffset, &tmap_x, k * kTile + 64 * h, m0, full, pol);
                    }
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            }
        }
        if (lane == 0) {
            // The release of the last stages reaches both CTAs from the leader's commits: take every stage once
            // more, so that no arrival is still on its way when this CTA exits.
            for (int gg = g; gg < g + NST && ok; ++gg)
                if (gg >= NST) ok = mbar_wait(bar_empty + 8 * (gg % NST), (uint32_t(gg / NST) & 1u) ^ 1u, abort_flag, status_dev);
            if (*abort_flag) {
                const uint64_t tstart = global_timer_ns();
                while (global_timer_ns() - tstart < kDrainLimitNs) {}
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer: one thread of the leader CTA drives both CTAs ----------------
        if (leader) {
            const uint32_t idesc_d = instr_desc_pair(0, false) | ((uint32_t(n_tok) >> 3) << 17);
            const uint32_t idesc_s = idesc_d | (1u << 2);
            bool ok = true;
            int g = 0, jt = 0;
            for (int t = cluster_id; t < n_out && ok; t += n_clusters, ++jt) {
                const Quad Q = make_quad(t % TQ, TN, rank);
                // both CTAs' epilogues must have drained the accumulators of the previous tile
                if (lane == 0) ok = mbar_wait(bar_acc_empty, (uint32_t(jt) & 1u) ^ 1u, abort_flag, status_dev);
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                tc_fence_after();
                TileDesc mine, next = load_step_descs(table0, TK, Q, 0, lane);
                for (int k = 0; k < TK && ok; ++k) {
                    if ((k & 7) == 0) { mine = next; next = load_step_descs(table0, TK, Q, k + 8, lane); }
                    const Step s = step_info(mine, k);
                    if (lane == 0) {
                        const bool sp0 = s.sparse_pair(0), sp1 = Q.npairs > 1 && s.sparse_pair(1);
                        const int st0 = g % NST;
#pragma unroll
                        for (int h = 0; h < 2; ++h, ++g) {
                            if (!ok) continue;
                            const int st = g % NST;
                            const uint32_t stage = smem_base + st * kStageBytes;
                            ok = mbar_wait(bar_full + 8 * st, uint32_t(g / NST) & 1u, abort_flag, status_dev);
                            if (!ok) continue;
                            tc_fence_after();
                            const uint64_t dB = desc_kmajor_sw128(stage + kBOffset);
#pragma unroll
                            for (int j = 0; j < 2; ++j) {
                                if (j >= Q.npairs) continue;
                                const uint32_t acc = tmem_base + (j ? kAcc1Col : 0u);
                                if (j == 0 ? sp0 : sp1) {
                                    // 2:4 pair: the whole tile sits in the first K-half's stage
                                    const uint32_t a_region = smem_base + st0 * kStageBytes + j * kARegionBytes;
                                    const uint64_t dA = desc_kmajor_sw128(a_region);
                                    const uint32_t e = tmem_base + meta_col(st0, j) + 2u * h;
                                    if (h == 0) tmem_copy_pair_128x128b(e, desc_rows16(a_region + kAtomBytes));
#pragma unroll
                                    for (int ks = 0; ks < 2; ++ks)     // K = 32 each: 32 B of A, 64 B of B per row
                                        mma_sparse_pair(acc, dA + uint64_t((64 * h + ks * 32) >> 4), dB + uint64_t((ks * 64) >> 4), e,
                                                        idesc_s | uint32_t(ks & 1), !(k == 0 && h == 0 && ks == 0));
                                } else {
                                    // dense pair (either tile may be an expanded 2:4 tile): one K-half per stage
                                    const uint64_t dA = desc_kmajor_sw128(stage + j * kARegionBytes);
#pragma unroll
                                    for (int ks = 0; ks < 4; ++ks)     // K = 16 each: 32 B of both operand rows
                                        mma_dense_pair(acc, dA + uint64_t((ks * 32) >> 4), dB + uint64_t((ks * 32) >> 4), idesc_d,
                                                       !(k == 0 && h == 0 && ks == 0));
                                }
                            }
                            // a stage that holds a whole 2:4 tile is released with the second K-half
                            if (h == 0) {
                                if (!(sp0 || sp1)) mma_commit_pair(bar_empty + 8 * st);
                            } else {
                                if (sp0 || sp1) mma_commit_pair(bar_empty + 8 * st0);
                                mma_commit_pair(bar_empty + 8 * st);
                            }
                        }
                    }
                    ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
                }
                if (ok && lane == 0) mma_commit_pair(bar_acc_full);
            }
            // the epilogue warps of the other CTA arrive on this CTA's barrier: wait for the last tile's arrivals too
            if (ok && lane == 0 && jt > 0) mbar_wait(bar_acc_empty, (uint32_t(jt) & 1u) ^ 1u, abort_flag, status_dev);
        }
        __syncwarp();
    } else if (warp < kExpandWarp0) {
        // ---------------- epilogue: warps 2..9; lane quadrant = warp % 4, column half = (warp - 2) / 4 ----
        const uint32_t quad = warp & 3u;
        const int half = (warp - 2) >> 2;
        const uint32_t leader_acc_empty = map_to_rank(bar_acc_empty, 0);
        bool ok = true;
        int jt = 0;
        for (int t = cluster_id; t < n_out && ok; t += n_clusters, ++jt) {
            const int q = t % TQ, m0 = (t / TQ) * n_tok;
            ok = group_wait(bar_acc_full, uint32_t(jt) & 1u, warp == 2 && lane == 0, 1, 256, abort_flag, status_dev);
            if (!ok) break;
            tc_fence_after();
            if (independent && jt == 0) grid_dependency_wait();     // Y may be in use by the preceding kernel
            const int valid = M - m0 < n_tok ? M - m0 : n_tok;      // tokens of this tile that exist
            const int chunks = (valid + 15) / 16, c_begin = half == 0 ? 0 : (chunks + 1) / 2,
                      c_end = half == 0 ? (chunks + 1) / 2 : chunks;
#pragma unroll 1
            for (int j = 0; j < 2; ++j) {
                const int rb = 4 * q + 2 * j + int(rank);
                if (rb >= TN) continue;
                const uint32_t acc = tmem_base + (j ? kAcc1Col : 0u) + ((quad * 32u) << 16);
                __nv_bfloat16* ytile = Y + int64_t(m0) * ldy + int64_t(rb) * kTile + quad * 32;
#pragma unroll 1
                for (int ch = c_begin; ch < c_end; ++ch) {
                    const int c0 = ch * 16;
                    uint32_t v[16];
                    tmem_ld16(acc + uint32_t(c0), v);
                    tmem_ld_wait();
                    store_fragment_transposed(v, smem + kEpiOffset + (warp - 2) * 1024, lane, ytile + int64_t(c0) * ldy, ldy,
                                              valid - c0);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_acc_empty);
        }
    } else {
        // ---------------- expansion warps: 2:4 tile of a dense pair -> dense image, in place ----------------
        const int r = threadIdx.x - kExpandWarp0 * 32;               // this thread's row of the tile, 0..127
        const uint32_t leader_full = map_to_rank(bar_full, 0);
        uint32_t land_phase = 0;                                     // bit 2 st + j: parity of the next use of bar_land[st][j]
        bool ok = true;
        int g = 0;
        for (int t = cluster_id; t < n_out && ok; t += n_clusters) {
            const Quad Q = make_quad(t % TQ, TN, rank);
            TileDesc mine, next = load_step_descs(table0, TK, Q, 0, lane);
            for (int k = 0; k < TK && ok; ++k, g += 2) {
                if ((k & 7) == 0) { mine = next; next = load_step_descs(table0, TK, Q, k + 8, lane); }
                const Step s = step_info(mine, k);
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    if (!ok || j >= Q.npairs || !s.expand(j)) continue;
                    const int st0 = g % NST, st1 = (g + 1) % NST;
                    const uint32_t bit = 1u << (2 * st0 + j);
                    bool fail = false;
                    if (r == 0) {
                        // the compressed tile has landed, and the next stage (whose A region gets the second half) is free
                        fail = !mbar_wait(bar_land + 16 * st0 + 8 * j, (land_phase & bit) ? 1u : 0u, abort_flag, status_dev) ||
                               !mbar_wait(bar_empty + 8 * st1, (uint32_t((g + 1) / NST) & 1u) ^ 1u, abort_flag, status_dev);
                    }
                    land_phase ^= bit;
                    if (barrier_any(fail, 2, kExpandThreads)) { ok = false; continue; }
                    uint8_t* a0 = smem + st0 * kStageBytes + j * kARegionBytes;      // compressed tile; becomes dense half 0
                    uint8_t* a1 = smem + st1 * kStageBytes + j * kARegionBytes;      // receives dense half 1
                    const uint8_t* meta = a0 + kAtomBytes;
                    // row r: eight 16-byte chunks of kept values (chunk u = 8 values = 16 dense columns) and their codes
                    uint4 v[8];
                    uint32_t code[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        v[u] = *reinterpret_cast<const uint4*>(a0 + atom_chunk_offset(uint32_t(r), uint32_t(u)));
                        // codes of tile row r, columns [16u, 16u + 16): metadata row 16 (r / 16) + 8 (u % 2) + r % 8, word u / 2,
                        // low half for the rows r % 16 < 8, high half for the others
                        const uint32_t Lrow = (uint32_t(r) & ~15u) + 8u * (uint32_t(u) & 1u) + (uint32_t(r) & 7u);
                        code[u] = *reinterpret_cast<const uint16_t*>(meta + Lrow * 16 + (u >> 1) * 4 + ((r >> 3) & 1) * 2);
                    }
                    asm volatile("bar.sync 2, 128;" ::: "memory");    // every row has been read before any row is overwritten
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        const uint32_t in[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                        uint32_t out[8];
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            const uint32_t nib = (code[u] >> (4 * q4)) & 0xFu, i0 = nib & 3u, i1 = nib >> 2;
                            const uint32_t v0 = in[q4] & 0xFFFFu, v1 = in[q4] >> 16;
                            uint32_t w[4];
#pragma unroll
                            for (uint32_t pz = 0; pz < 4; ++pz) w[pz] = pz == i0 ? v0 : pz == i1 ? v1 : 0u;
                            out[2 * q4] = w[0] | (w[1] << 16);
                            out[2 * q4 + 1] = w[2] | (w[3] << 16);
                        }
                        // dense chunks 2u and 2u + 1 of the 128-column row: K-half u / 4, chunks (2u) % 8 and (2u) % 8 + 1 of it
                        uint8_t* dst = u < 4 ? a0 : a1;
                        const uint32_t c = (2u * uint32_t(u)) & 7u;
                        *reinterpret_cast<uint4*>(dst + atom_chunk_offset(uint32_t(r), c)) = make_uint4(out[0], out[1], out[2], out[3]);
                        *reinterpret_cast<uint4*>(dst + atom_chunk_offset(uint32_t(r), c + 1)) = make_uint4(out[4], out[5], out[6], out[7]);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the MMA's reads
                    asm volatile("bar.sync 2, 128;" ::: "memory");
                    if (r == 0) {
                        if (leader) {
                            mbar_arrive(bar_full + 8 * st0);
                            mbar_arrive(bar_full + 8 * st1);
                        } else {
                            mbar_arrive_cluster(leader_full + 8 * st0);
                            mbar_arrive_cluster(leader_full + 8 * st1);
                        }
                    }
                }
            }
        }
    }

    if (independent) grid_dependency_wait();      // every thread passes the dependency before the CTA exits
    // every role of both CTAs ends here: nothing crosses the pair after this barrier
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();
    if (warp == 1) tmem_dealloc_pair(tmem_base, kTmemCols);
}

// ---------------------------------------------------------------------------------------------
// host side

int prefill_pair_mixed_clusters() {
    static std::atomic<int> cache[kMaxDevices];
    const int d = current_device();
    if (d < 0) return 0;
    int n = cache[d].load(std::memory_order_acquire);
    if (n) return n;
    if (cudaFuncSetAttribute(prefill_pair_mixed_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(pm::kSmemBytes)) != cudaSuccess)
        return 0;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3(2, 1, 1);
    cfg.blockDim = dim3(pm::kThreads, 1, 1);
    cfg.dynamicSmemBytes = pm::kSmemBytes;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&n, prefill_pair_mixed_kernel, &cfg) != cudaSuccess || n <= 0) return 0;
    cache[d].store(n, std::memory_order_release);
    return n;
}

int prefill_pair_mixed_max_tok() { return pm::kMaxTok; }

int launch_prefill_pair_mixed(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                              int n_tok, __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool independent) {
    const int clusters = prefill_pair_mixed_clusters();
    if (clusters <= 0) return PATCH_ERR_CUDA;
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    const int64_t n_out = int64_t((TN + 3) / 4) * ((M + n_tok - 1) / n_tok);
    if (n_out > 0x3FFFFFFF || L->total_bytes / 256 > 0x7FFFFFFFull) return PATCH_ERR_SHAPE;
    if (n_tok % 16 || n_tok < 32 || n_tok > pm::kMaxTok) return PATCH_ERR_SHAPE;
    CUtensorMap map_x, map_w16, map_w18;
    int rc = make_x_tensor_map(&map_x, X, ldx, M, L->K, n_tok / 2);
    if (rc) return rc;
    rc = make_blob_tensor_map(&map_w16, packed, L->total_bytes, int(kAtomBytes / 256));
    if (rc) return rc;
    rc = make_blob_tensor_map(&map_w18, packed, L->total_bytes, int(kSparseBytes / 256));
    if (rc) return rc;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    cfg.gridDim = dim3(2u * unsigned(n_out < clusters ? n_out : clusters), 1, 1);
    cfg.blockDim = dim3(pm::kThreads, 1, 1);
    cfg.dynamicSmemBytes = pm::kSmemBytes;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, prefill_pair_mixed_kernel, map_x, map_w16, map_w18, packed, uint64_t(L->table_off),
                                       TN, TK, int(M), n_tok, Y, ldy, status_dev, independent ? 1 : 0);
    return e == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

}  // namespace patch
