// Large-M (prefill) schedule on CTA pairs: every MMA is a cta_group::2 instruction over 256 out-features.
//
// Same operation and operand roles as the other prefill kernels (the packed weight is the MMA A operand,
// dense tcgen05.mma or tcgen05.mma.sp per 128 x 128 weight tile, fp32 accumulation in tensor memory, dense
// and 2:4 tiles mixed inside one multiplication as Appendix A describes the deployed kernels).  What
// changes is who holds what.  A cluster of two CTAs (the two SMs of one TPC) owns four row-blocks and one
// token tile:
//   * pair j (j = 0, 1) of quad q is the row-blocks (4q + 2j, 4q + 2j + 1); CTA rank r holds row-block
//     4q + 2j + r and its accumulator (128 TMEM lanes x n_tok columns);
//   * the activation tile is split by tokens: CTA r loads rows [m0 + r n_tok/2, m0 + (r + 1) n_tok/2) and
//     the pair MMA reads one half from each CTA.
// Per weight tile and token a CTA therefore reads half as many activation bytes from shared memory (and
// from L2) as a one-CTA MMA does.  That is what bounds the one-CTA kernels: operand reads plus the copies
// landing come to ~160 B/clock on dense tiles against the 128 B/clock a shared memory delivers, and the
// one-CTA 2:4 MMA alone needs 118 B/clock, which holds it at 1.47x the dense rate instead of 2x.
//
// Synchronisation is the standard pair protocol and nothing else:
//   * every copy is a tiled TMA load of the pair form (cp.async.bulk.tensor ... cta_group::2, no multicast)
//     whose bytes are counted on the LEADER's (rank 0) "full" barrier of the stage -- the weight tiles through
//     a tensor map that views the packed blob as rows of 256 bytes, so that a box lands like a linear copy;
//     the leader's producer posts the byte count of both CTAs;
//   * ONE thread of the leader issues every MMA and releases a stage in both CTAs with one
//     tcgen05.commit (CTA mask 0b11) on the "empty" barriers; the same for "accumulators complete";
//   * the epilogue warps of both CTAs arrive on the leader's "accumulators drained" barrier;
//   * tensor memory is allocated and freed with the pair allocator by one warp of each CTA; before the
//     CTAs part, every arrival that crosses the pair has been waited for and a cluster barrier has passed.
//
// This kernel serves weights whose tiles are all of one kind (all dense: stages of one K-half, four deep,
// up to 256 tokens; all 2:4: stages of one whole tile, three deep, up to 240 tokens because the metadata
// needs tensor-memory columns too).  Weights that mix kinds run on the two-row-block kernel.
//
// 320 threads: warp 0 producer, warp 1 MMA issuer (leader) and TMEM owner, warps 2..9 epilogue (two warps
// per TMEM lane quadrant, each taking half of the token columns).  Persistent over output tiles.
//
// Tried and dropped (each measured against this form on the LLaMA-2-7B shapes at M = 2048 / 4096, same GPU, runs
// interleaved): cutting the token axis into nearly equal tiles whose count is a multiple of the cluster count (the
// K steps are bound by the latency of the copies, not by the tensor time of the tile's width, so narrower tiles cost
// the same per step and balance bought nothing); and an epilogue of sixteen warps that pulls both accumulators into
// registers, hands them back at once and writes Y while the next tile's MMAs run (no gain on dense, a loss on 2:4
// weights, whose short stages are the most sensitive to anything else that runs on the SM).
//
// Every mbarrier wait is bounded; on expiry the CTA raises an abort flag, reports PATCH_ERR_TIMEOUT through
// status_dev, and every role still runs to the common cluster barrier at the end before TMEM is freed.
#include "sm100_ptx.cuh"

namespace patch {

namespace pp {
constexpr int kThreads = 320;
enum { kDense = 0, kSparse = 1 };
template <int KIND_>
struct Cfg {
    static constexpr int KIND = KIND_;
    static constexpr int NST = KIND_ == kDense ? 4 : 3;                       // stages
    static constexpr int kMaxTok = KIND_ == kDense ? 256 : 240;
    static constexpr int kHalves = KIND_ == kDense ? 1 : 2;                   // K-halves of X per stage
    static constexpr uint32_t kARegionBytes = KIND_ == kDense ? kAtomBytes : kSparseBytes;
    static constexpr uint32_t kBRegionBytes = (kMaxTok / 2) * 128;            // one K-half of this CTA's tokens
    static constexpr uint32_t kBOffset = 2 * kARegionBytes;
    static constexpr uint32_t kStageBytes = kBOffset + kHalves * kBRegionBytes;
    static constexpr uint32_t kBarrierOffset = NST * kStageBytes;
    static constexpr uint32_t kEpiOffset = kBarrierOffset + 256;              // 8 epilogue warps x 1 KB transpose staging
    static constexpr uint32_t kSmemBytes = kEpiOffset + 8 * 1024 + 1024;      // + alignment slack
    static_assert(kStageBytes % 1024 == 0 && kARegionBytes % 1024 == 0 && kBRegionBytes % 1024 == 0, "swizzle atoms");
    static_assert(kSmemBytes <= 227 * 1024, "shared memory per CTA");
};
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kAcc1Col = 256;                 // acc0 [0, n_tok)   acc1 [256, 256 + n_tok)
// metadata of the 2:4 schedule: 4 TMEM columns per (stage, pair), in the gaps [240,256) and [496,512)
__device__ __forceinline__ uint32_t meta_col(int stage, int j) {
    const int i = 2 * stage + j;
    return i < 4 ? 240u + 4u * i : 496u + 4u * (i - 4);
}
}  // namespace pp

template <class C>
__global__ void __launch_bounds__(pp::kThreads)
prefill_pair_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                    uint32_t pay0_256, int TN, int TK, int M, int n_tok, __nv_bfloat16* __restrict__ Y, int64_t ldy,
                    int* status_dev, int independent) {
    using namespace pp;
    constexpr int KIND = C::KIND, NST = C::NST;
    constexpr uint32_t kTileRows256 = (KIND == kDense ? kDenseBytes : kSparseBytes) / 256;   // blob rows per tile
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_full = smem_base + C::kBarrierOffset;      // NST x 8 B (4 reserved); waited for in the leader only
    const uint32_t bar_empty = bar_full + 32;                     // NST x 8 B
    const uint32_t bar_acc_full = bar_empty + 32;                 // 8 B
    const uint32_t bar_acc_empty = bar_acc_full + 8;              // 8 B, used in the leader only
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + C::kBarrierOffset + 96);
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

    if (threadIdx.x == 0) {
        for (int i = 0; i < NST; ++i) {
            mbar_init(bar_full + 8 * i, 1);      // the leader producer's arrive.expect_tx; the bytes of both CTAs complete it
            mbar_init(bar_empty + 8 * i, 1);     // one commit of the issuing thread, delivered to both CTAs
        }
        mbar_init(bar_acc_full, 1);              // one commit, delivered to both CTAs
        mbar_init(bar_acc_empty, 16);            // one arrival per epilogue warp of both CTAs
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_map(&tmap_x);
        tma_prefetch_map(&tmap_w);
    }
    if (warp == 1) tmem_alloc_pair(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();     // both CTAs' barriers and tensor memory exist before anything crosses the pair
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    // Programmatic dependent launch: the next kernel in the stream may become resident from here on (its CTAs fit
    // on an SM only once this kernel's have left it).  X, the packed weight and Y may belong to the previous
    // kernel until the wait -- unless the caller declared this GEMM independent of its predecessor: then only the
    // Y stores (and the exit) wait.
    grid_launch_dependents();
    if (!independent) grid_dependency_wait();

    if (warp == 0) {
        // ---------------- producer: this CTA's two weight tiles and its half of the tokens, per stage ----------------
        if (lane == 0) {
            const uint64_t pol = l2_policy_evict_last();     // weights and activations are both re-read from L2
            const uint32_t leader_full = map_to_rank(bar_full, 0);
            // bytes one stage brings into ONE CTA; the leader posts twice that
            const uint32_t stage_tx = 2 * C::kARegionBytes + C::kHalves * x_half_bytes;
            int g = 0;                           // stage counter, continues across output tiles
            bool ok = true;
            for (int t = cluster_id; t < n_out && ok; t += n_clusters) {
                const int q = t % TQ, m0 = (t / TQ) * n_tok + int(rank) * n_half;
                // row-blocks held here (clamped: a missing one is loaded from the last row-block and never stored)
                int rb[2];
#pragma unroll
                for (int j = 0; j < 2; ++j) { const int a = 4 * q + 2 * j + int(rank); rb[j] = a < TN ? a : TN - 1; }
                for (int k = 0; k < TK && ok; ++k) {
                    // tiles of one kind are equally long and stored in (tn, tk) order: their place follows from the index
                    const int row0 = int(pay0_256 + uint32_t(rb[0] * TK + k) * kTileRows256);
                    const int row1 = int(pay0_256 + uint32_t(rb[1] * TK + k) * kTileRows256);
                    if (KIND == kDense) {
#pragma unroll
                        for (int h = 0; h < 2; ++h, ++g) {
                            if (!ok) continue;
                            const int st = g % NST;
                            const uint32_t stage = smem_base + st * C::kStageBytes, full = leader_full + 8 * st;
                            ok = mbar_wait(bar_empty + 8 * st, (uint32_t(g / NST) & 1u) ^ 1u, abort_flag, status_dev);
                            if (!ok) continue;
                            if (leader) mbar_expect_tx(bar_full + 8 * st, 2 * stage_tx);
                            tma_tile_load_pair(stage, &tmap_w, 0, row0 + h * int(kAtomBytes / 256), full, pol);
                            tma_tile_load_pair(stage + C::kARegionBytes, &tmap_w, 0, row1 + h * int(kAtomBytes / 256), full, pol);
                            tma_tile_load_pair(stage + C::kBOffset, &tmap_x, k * kTile + 64 * h, m0, full, pol);
                        }
                    } else {
                        const int st = g % NST;
                        const uint32_t stage = smem_base + st * C::kStageBytes, full = leader_full + 8 * st;
                        ok = mbar_wait(bar_empty + 8 * st, (uint32_t(g / NST) & 1u) ^ 1u, abort_flag, status_dev);
                        if (ok) {
                            if (leader) mbar_expect_tx(bar_full + 8 * st, 2 * stage_tx);
                            tma_tile_load_pair(stage, &tmap_w, 0, row0, full, pol);
                            tma_tile_load_pair(stage + C::kARegionBytes, &tmap_w, 0, row1, full, pol);
                            tma_tile_load_pair(stage + C::kBOffset, &tmap_x, k * kTile, m0, full, pol);
                            tma_tile_load_pair(stage + C::kBOffset + C::kBRegionBytes, &tmap_x, k * kTile + 64, m0, full, pol);
                            ++g;
                        }
                    }
                }
            }
            // The release of the last stages reaches both CTAs from the leader's commits: take every stage once
            // more, so that no arrival is still on its way when this CTA exits.
            for (int gg = g; gg < g + NST && ok; ++gg)
                if (gg >= NST) ok = mbar_wait(bar_empty + 8 * (gg % NST), (uint32_t(gg / NST) & 1u) ^ 1u, abort_flag, status_dev);
            if (*abort_flag) {
                // give the copies this thread started a bounded time to land
                const uint64_t tstart = global_timer_ns();
                while (global_timer_ns() - tstart < kDrainLimitNs) {}
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer: one thread of the leader CTA drives both CTAs ----------------
        if (leader && lane == 0) {
            const uint32_t idesc = instr_desc_pair(0, KIND == kSparse) | ((uint32_t(n_tok) >> 3) << 17);
            bool ok = true;
            int g = 0, jt = 0;
            for (int t = cluster_id; t < n_out && ok; t += n_clusters, ++jt) {
                const int npairs = 4 * (t % TQ) + 2 < TN ? 2 : 1;
                // both CTAs' epilogues must have drained the accumulators of the previous tile
                ok = mbar_wait(bar_acc_empty, (uint32_t(jt) & 1u) ^ 1u, abort_flag, status_dev);
                if (!ok) break;
                tc_fence_after();
                for (int k = 0; k < TK && ok; ++k) {
                    if (KIND == kDense) {
#pragma unroll
                        for (int h = 0; h < 2; ++h, ++g) {
                            if (!ok) continue;
                            const int st = g % NST;
                            const uint32_t stage = smem_base + st * C::kStageBytes;
                            ok = mbar_wait(bar_full + 8 * st, uint32_t(g / NST) & 1u, abort_flag, status_dev);
                            if (!ok) continue;
                            tc_fence_after();
                            const uint64_t dB = desc_kmajor_sw128(stage + C::kBOffset);
#pragma unroll
                            for (int j = 0; j < 2; ++j) {
                                if (j >= npairs) continue;
                                const uint64_t dA = desc_kmajor_sw128(stage + j * C::kARegionBytes);
#pragma unroll
                                for (int ks = 0; ks < 4; ++ks)     // K = 16 each: 32 B of both operand rows
                                    mma_dense_pair(tmem_base + (j ? kAcc1Col : 0u), dA + uint64_t((ks * 32) >> 4),
                                                   dB + uint64_t((ks * 32) >> 4), idesc, !(k == 0 && h == 0 && ks == 0));
                            }
                            mma_commit_pair(bar_empty + 8 * st);   // frees the stage in both CTAs once these MMAs have read it
                        }
                    } else {
                        const int st = g % NST;
                        const uint32_t stage = smem_base + st * C::kStageBytes;
                        ok = mbar_wait(bar_full + 8 * st, uint32_t(g / NST) & 1u, abort_flag, status_dev);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t dB = desc_kmajor_sw128(stage + C::kBOffset);
#pragma unroll
                        for (int j = 0; j < 2; ++j) {
                            if (j >= npairs) continue;
                            const uint32_t a_region = stage + j * C::kARegionBytes;
                            const uint64_t dA = desc_kmajor_sw128(a_region);
                            const uint32_t e = tmem_base + meta_col(st, j);
                            tmem_copy_pair_128x128b(e, desc_rows16(a_region + kAtomBytes));   // each CTA's metadata -> its TMEM
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks)         // K = 32 each: 32 B of A, 64 B of B per row
                                mma_sparse_pair(tmem_base + (j ? kAcc1Col : 0u), dA + uint64_t((ks * 32) >> 4),
                                                dB + uint64_t(((ks >> 1) * C::kBRegionBytes + (ks & 1) * 64) >> 4),
                                                e + (ks & 2), idesc | uint32_t(ks & 1), !(k == 0 && ks == 0));
                        }
                        mma_commit_pair(bar_empty + 8 * st);
                        ++g;
                    }
                }
                if (ok) mma_commit_pair(bar_acc_full);
            }
            // the epilogue warps of the other CTA arrive on this CTA's barrier: wait for the last tile's arrivals too
            if (ok && jt > 0) mbar_wait(bar_acc_empty, (uint32_t(jt) & 1u) ^ 1u, abort_flag, status_dev);
        }
        __syncwarp();
    } else {
        // ---------------- epilogue: warps 2..9; lane quadrant = warp % 4, column half = (warp - 2) / 4 ----
        const uint32_t quad = warp & 3u;
        const int half = (warp - 2) >> 2;
        const uint32_t leader_acc_empty = map_to_rank(bar_acc_empty, 0);
        bool ok = true;
        int jt = 0;
        for (int t = cluster_id; t < n_out && ok; t += n_clusters, ++jt) {
            const int q = t % TQ, m0 = (t / TQ) * n_tok;
            // one thread polls the barrier (sleeping in between); the other 255 wait on a hardware barrier, which
            // costs the shared-memory port nothing while the MMAs run
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
                    store_fragment_transposed(v, smem + C::kEpiOffset + (warp - 2) * 1024, lane, ytile + int64_t(c0) * ldy, ldy,
                                              valid - c0);
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_acc_empty);
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

template <class C>
static int max_clusters_of(std::atomic<int>* cache) {
    const int d = current_device();
    if (d < 0) return 0;
    int n = cache[d].load(std::memory_order_acquire);
    if (n) return n;
    if (cudaFuncSetAttribute(prefill_pair_kernel<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(C::kSmemBytes)) != cudaSuccess)
        return 0;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3(2, 1, 1);
    cfg.blockDim = dim3(pp::kThreads, 1, 1);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaOccupancyMaxActiveClusters(&n, prefill_pair_kernel<C>, &cfg) != cudaSuccess || n <= 0) return 0;
    cache[d].store(n, std::memory_order_release);
    return n;
}

// Number of CTA pairs that can be resident at once on the current device (0: the schedule is not available).
int prefill_pair_clusters(bool sparse) {
    static std::atomic<int> cache_d[kMaxDevices], cache_s[kMaxDevices];
    return sparse ? max_clusters_of<pp::Cfg<pp::kSparse>>(cache_s) : max_clusters_of<pp::Cfg<pp::kDense>>(cache_d);
}

int prefill_pair_max_tok(bool sparse) { return sparse ? pp::Cfg<pp::kSparse>::kMaxTok : pp::Cfg<pp::kDense>::kMaxTok; }

template <class C>
static int launch_pair_t(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                         int n_tok, int clusters, __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream,
                         bool independent) {
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    const int64_t n_out = int64_t((TN + 3) / 4) * ((M + n_tok - 1) / n_tok);
    if (n_out > 0x3FFFFFFF || L->total_bytes / 256 > 0x7FFFFFFFull) return PATCH_ERR_SHAPE;
    if (n_tok % 16 || n_tok < 32 || n_tok > C::kMaxTok) return PATCH_ERR_SHAPE;
    CUtensorMap map_x, map_w;
    int rc = make_x_tensor_map(&map_x, X, ldx, M, L->K, n_tok / 2);
    if (rc) return rc;
    rc = make_blob_tensor_map(&map_w, packed, L->total_bytes, int(C::kARegionBytes / 256));
    if (rc) return rc;
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    cfg.gridDim = dim3(2u * unsigned(n_out < clusters ? n_out : clusters), 1, 1);
    cfg.blockDim = dim3(pp::kThreads, 1, 1);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, prefill_pair_kernel<C>, map_x, map_w, uint32_t(L->payload_off / 256), TN, TK,
                                       int(M), n_tok, Y, ldy, status_dev, independent ? 1 : 0);
    return e == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

// The weight must hold tiles of one kind only (n_dense == 0 or n_sparse == 0).
int launch_prefill_pair(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                        int n_tok, __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool independent) {
    if (L->n_dense && L->n_sparse) return PATCH_ERR_FORMAT;
    const bool sparse = L->n_sparse != 0;
    const int clusters = prefill_pair_clusters(sparse);
    if (clusters <= 0) return PATCH_ERR_CUDA;
    if (sparse) return launch_pair_t<pp::Cfg<pp::kSparse>>(X, ldx, M, L, packed, n_tok, clusters, Y, ldy, status_dev, stream, independent);
    return launch_pair_t<pp::Cfg<pp::kDense>>(X, ldx, M, L, packed, n_tok, clusters, Y, ldy, status_dev, stream, independent);
}

}  // namespace patch
