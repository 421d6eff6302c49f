// Small-M schedule for SMALL weights: fixed split-K over a thread-block cluster, partial sums
// exchanged through distributed shared memory.
//
// The stream-K decode kernel hands its split-K partial sums over through global memory.  With
// consecutive GEMMs overlapped (programmatic dependent launch), those words travel through L2
// queues that the next kernels' weight stream keeps full, and they may only be written once the
// preceding kernel has completed (they share the workspace): for a weight that streams in ~5 us
// the chain [wait for the predecessor -> write partial sums -> finishing CTA sees them] of 6-7 us
// per launch is longer than the stream itself.  Here a cluster of S CTAs owns one row-block, CTA s
// streams the s-th K-slice of its tiles, and the S partial accumulators meet in shared memory:
//   accumulate (tcgen05.mma / .mma.sp into TMEM)  ->  own partial to own shared memory
//   -> cluster barrier -> every CTA sums 128 / S rows over the S partials (ld.shared::cluster, in K
//   order: deterministic) -> wait for the predecessor kernel -> bf16 stores -> cluster barrier.
// Nothing but Y is written to global memory, so only the Y stores wait for the predecessor.
// This is the split-K schedule Appendix A mentions for decode, in the form the hardware offers for it.
//
// Measured (B200, the 24 decode GEMMs of the LLaMA-2-7B workload launched back to back as independent
// GEMMs): with S chosen as small as possible -- S = 1 wherever the weight has 32 or more row-blocks, i.e. one
// CTA per row-block and no split at all -- a kernel occupies only a fraction of the CTA slots, so four to
// nine consecutive GEMMs are resident at once, and the step runs at 6.6 TB/s (0.202 ms, 83 % of the 8 TB/s
// roofline) against 5.6 TB/s (0.238 ms) for the stream-K kernel, which fills every SM with one GEMM.  A GEMM
// whose successor has to wait for it is the opposite case (few CTAs means low bandwidth for a lone kernel):
// the launcher uses this schedule only when the caller has declared the GEMMs independent
// (PATCH_GEMM_WEIGHTS_STATIC | PATCH_GEMM_INPUT_STATIC).
//
// Same operand roles, tile format, ring of whole-tile stages, bounded waits and launch flags as the
// stream-K kernel; M <= 64 tokens (MMA N = 16, 32 or 64).
#include "sm100_ptx.cuh"

namespace patch {

namespace dc {
template <int N_TOK, int STAGES, bool GATED = false>
struct Cfg {
    static constexpr uint32_t kXAtomBytes = N_TOK * 128;                  // N_TOK rows x 64 bf16
    static constexpr uint32_t kXBytes = 2 * kXAtomBytes;
    static constexpr uint32_t kStageBytes = kDenseBytes + kXBytes;
    static constexpr uint32_t kBarrierOffset = STAGES * kStageBytes;
    static constexpr uint32_t kSmemBytes = kBarrierOffset + 256 + 1024;   // + barriers + alignment slack
    static constexpr int kAccs = GATED ? 2 : 1;                           // gated: gate and up accumulators
    static constexpr uint32_t kTmemNeeded = kAccs * N_TOK + 4 * STAGES;   // accumulators + metadata (4 columns per stage)
    static constexpr uint32_t kTmemCols = kTmemNeeded <= 32 ? 32 : kTmemNeeded <= 64 ? 64 : 128;
    static constexpr uint32_t kPartialRowBytes = N_TOK * 4;               // fp32 partial: [128 rows][N_TOK]
    static_assert(N_TOK == 16 || N_TOK == 32 || N_TOK == 64, "MMA N in {16, 32, 64}");
    static_assert(STAGES >= 2 && STAGES <= 4, "ring depth");
    static constexpr uint32_t kPartialBytes = 128 * kPartialRowBytes;     // per accumulator
    static_assert(kAccs * kPartialBytes <= kDenseBytes, "the partials take the place of the first stage's weight tile");
    static_assert(!GATED || N_TOK == 16, "the gated product exists for the 16-token schedule");
};

__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// 16 bytes from the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ float4 ld_peer_f4(uint32_t saddr, uint32_t rank) {
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(saddr), "r"(rank));
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a) : "memory");
    return v;
}
}  // namespace dc

// GATED: the weight stacks a gate and an up projection with their row-blocks interleaved (2j: gate, 2j + 1: up);
// a cluster owns the pair j, streams the gate tiles of its K-slice into one accumulator and the up tiles into a
// second one, and writes silu(gate) * up for out-feature block j of Y [M x N / 2].
// YSTATIC: the caller also promised that nothing in the overlap window touches Y: only the launch's first cluster
// waits for the preceding kernel (so that launches still complete in order); every other CTA stores Y and leaves
// as soon as it is done instead of holding its shared memory until then.
template <int N_TOK, int STAGES, bool WSTATIC, bool XSTATIC, bool GATED = false, bool YSTATIC = false>
__global__ void __launch_bounds__(192)
decode_cluster_kernel(const __grid_constant__ CUtensorMap tmap_x, const uint8_t* __restrict__ blob, uint64_t table_off,
                      uint32_t pay0_16, uint32_t end16, int TK, int S, int M, __nv_bfloat16* __restrict__ Y, int64_t ldy,
                      int* status_dev) {
    using namespace dc;
    using C = Cfg<N_TOK, STAGES, GATED>;
    constexpr uint32_t kStageBytes = C::kStageBytes, kXAtomBytes = C::kXAtomBytes, kXBytes = C::kXBytes;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_full = smem_base + C::kBarrierOffset;      // STAGES x 8 B (4 reserved)
    const uint32_t bar_empty = bar_full + 32;
    const uint32_t bar_acc_full = bar_empty + 32;
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + C::kBarrierOffset + 96);
    uint32_t* tmem_slot = misc;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 1);
    volatile uint32_t* stage_kind = misc + 4;                     // [STAGES]

    grid_launch_dependents();   // the next kernel in the stream may become resident now

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t s = cluster_ctarank();
    const int tn = blockIdx.x / S;
    // K-slice of this CTA: tiles [k0, k1) of row-block tn
    const int k0 = int(int64_t(s) * TK / S), k1 = int(int64_t(s + 1) * TK / S), n_slice = k1 - k0;
    constexpr int kAccs = C::kAccs;
    const int n_tiles = kAccs * n_slice;             // gated: the slice of the gate row-block, then of the up row-block
    const TileDesc* table = reinterpret_cast<const TileDesc*>(blob + table_off) + int64_t(kAccs) * tn * TK + k0;

    if (threadIdx.x == 64) {
        for (int i = 0; i < STAGES; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, 1);
        }
        mbar_init(bar_acc_full, 1);
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_map(&tmap_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), C::kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_meta = tmem_base + kAccs * N_TOK;         // 4 columns per stage behind the accumulators

    if (warp == 0) {
        // ---------------- producer ----------------
        if constexpr (!WSTATIC) grid_dependency_wait();
        const uint64_t pol_w = l2_policy_evict_first(), pol_x = l2_policy_evict_last();
        TileDesc mine = TileDesc{0, 0, 0, 0};
        int issued = 0;
        bool ok = true;
        // weight tiles of the first STAGES steps may be requested before the grid dependency is
        // resolved (WSTATIC); their activations follow once it is (unless XSTATIC)
        const int n_early = (WSTATIC && !XSTATIC) ? (n_tiles < STAGES ? n_tiles : STAGES) : 0;
        for (int i = 0; i < n_tiles && ok; ++i) {
            const int half = (GATED && i >= n_slice) ? 1 : 0, idx = i - half * n_slice;   // tile idx of row-block `half`
            if ((idx & 31) == 0 && idx + lane < n_slice) mine = table[int64_t(half) * TK + idx + lane];
            uint32_t kind = __shfl_sync(0xFFFFFFFFu, mine.kind, idx & 31);
            uint32_t off16 = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, idx & 31);
            if (lane == 0) {
                const int stage = i % STAGES;
                sanitize_tile(kind, off16, pay0_16, end16, status_dev);
                const uint32_t wbytes = kind == PATCH_TILE_DENSE ? kDenseBytes : kSparseBytes;
                const uint32_t sW = smem_base + stage * kStageBytes, full = bar_full + 8 * stage;
                if (i >= STAGES)
                    ok = mbar_wait(bar_empty + 8 * stage, (uint32_t(i / STAGES) & 1u) ^ 1u, abort_flag, status_dev);
                if (ok) {
                    stage_kind[stage] = kind;
                    mbar_expect_tx(full, wbytes + kXBytes);
                    tma_bulk_load(sW, blob + uint64_t(off16) * 16, wbytes, full, pol_w);
                    if (i < n_early) {
                        if (i + 1 == n_early) {
                            grid_dependency_wait();
                            for (int j = 0; j < n_early; ++j) {
                                const uint32_t sX = smem_base + j * kStageBytes + kDenseBytes;
                                const int k = (k0 + (GATED && j >= n_slice ? j - n_slice : j)) * kTile;
                                tma_tile_load(sX, &tmap_x, k, 0, bar_full + 8 * j, pol_x);
                                tma_tile_load(sX + kXAtomBytes, &tmap_x, k + 64, 0, bar_full + 8 * j, pol_x);
                            }
                        }
                    } else {
                        const uint32_t sX = sW + kDenseBytes;
                        const int k = (k0 + idx) * kTile;
                        tma_tile_load(sX, &tmap_x, k, 0, full, pol_x);
                        tma_tile_load(sX + kXAtomBytes, &tmap_x, k + 64, 0, full, pol_x);
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
            bool ok = true;
            for (int i = 0; i < n_tiles && ok; ++i) {
                const int stage = i % STAGES;
                ok = mbar_wait(bar_full + 8 * stage, uint32_t(i / STAGES) & 1u, abort_flag, status_dev);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sW = smem_base + stage * kStageBytes;
                const int half = (GATED && i >= n_slice) ? 1 : 0;
                issue_tile_mma<N_TOK>(stage_kind[stage], sW, sW + kDenseBytes, kXAtomBytes, tmem_base + uint32_t(half) * N_TOK,
                                      tmem_meta + 4 * stage, i == half * n_slice);
                mma_commit(bar_empty + 8 * stage);
            }
            if (ok && n_tiles > 0) mma_commit(bar_acc_full);      // every MMA of the slice has completed
        }
        __syncwarp();
    } else {
        // ---------------- epilogue warps 2..5: own partial -> own shared memory ----------------
        // The ring is free once the accumulator is complete (every stage has been read by then);
        // the partial [128 rows][16 tokens] fp32 takes the first 8 KB of it.
        const uint32_t quad = warp & 3u, row = quad * 32 + lane;
        bool ok = true;
        if (n_tiles > 0) {
            if (lane == 0) ok = mbar_wait(bar_acc_full, 0, abort_flag, status_dev);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            tc_fence_after();
        }
#pragma unroll
        for (int c0 = 0; c0 < kAccs * N_TOK; c0 += 16) {
            // accumulator c0 / N_TOK, its columns (c0 % N_TOK) .. + 15: partial [acc][row][token]
            float4* dst = reinterpret_cast<float4*>(smem + (c0 / N_TOK) * C::kPartialBytes + row * C::kPartialRowBytes) +
                          (c0 % N_TOK) / 4;
            uint32_t v[16];
            if (n_tiles > 0 && ok) {
                tmem_ld16(tmem_base + ((quad * 32u) << 16) + uint32_t(c0), v);
                tmem_ld_wait();
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) v[j] = 0u;
            }
#pragma unroll
            for (int q = 0; q < 4; ++q)
                dst[q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                              __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
        }
        tc_fence_before();
    }

    // every partial of the cluster is in place (on a timeout the partials are zeros or garbage,
    // and status_dev says so)
    __syncthreads();
    dc::cluster_barrier();

    if (warp >= 2) {
        // ---------------- reduction: this CTA finishes rows [128 s / S, 128 (s + 1) / S) ----------------
        const int e = threadIdx.x - 64;                            // 0..127
        const int rows = kTile / S;                                // S in {1, 2, 4, 8}
        constexpr int kGroups = N_TOK / 4;                         // groups of four tokens per row
        const int n_out = rows * kGroups;
        if (!YSTATIC || int(blockIdx.x) < S) grid_dependency_wait();   // Y may be in use by the preceding kernel
        for (int o = e; o < n_out; o += 128) {
            // consecutive threads take consecutive rows of one token group: their stores are neighbours in Y
            const int r = int(s) * rows + (o % rows), tg = o / rows;
            const uint32_t addr = smem_base + uint32_t(r) * C::kPartialRowBytes + uint32_t(tg) * 16u;
            float4 acc = dc::ld_peer_f4(addr, 0);
            for (int q = 1; q < S; ++q) {                          // ascending K: a fixed summation order
                const float4 p = dc::ld_peer_f4(addr, uint32_t(q));
                acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
            }
            float a[4] = {acc.x, acc.y, acc.z, acc.w};
            if (GATED) {
                float4 up = dc::ld_peer_f4(addr + C::kPartialBytes, 0);
                for (int q = 1; q < S; ++q) {
                    const float4 p = dc::ld_peer_f4(addr + C::kPartialBytes, uint32_t(q));
                    up.x += p.x; up.y += p.y; up.z += p.z; up.w += p.w;
                }
                const float u[4] = {up.x, up.y, up.z, up.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) a[j] = __fdividef(a[j], 1.0f + __expf(-a[j])) * u[j];   // silu(gate) * up
            }
            __nv_bfloat16* y = Y + int64_t(tn) * kTile + r;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int m = 4 * tg + j;
                if (m < M) y[int64_t(m) * ldy] = __float2bfloat16_rn(a[j]);
            }
        }
    } else {
        if (!YSTATIC || int(blockIdx.x) < S) grid_dependency_wait();   // every thread passes the dependency before the CTA exits
    }

    // nobody leaves while a peer may still read its shared memory
    tc_fence_before();
    __syncthreads();
    dc::cluster_barrier();
    if (warp == 1) tmem_dealloc(tmem_base, C::kTmemCols);
}

template <int N_TOK, int STAGES, bool WSTATIC, bool XSTATIC, bool GATED = false, bool YSTATIC = false>
static int launch_dc_t(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int M, int S,
                       __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream) {
    using C = dc::Cfg<N_TOK, STAGES, GATED>;
    auto kern = decode_cluster_kernel<N_TOK, STAGES, WSTATIC, XSTATIC, GATED, YSTATIC>;
    static std::atomic<uint64_t> configured{0};
    if (int rc = allow_dynamic_smem(kern, C::kSmemBytes, configured)) return rc;
    const int TN = int(L->N / kTile) / (GATED ? 2 : 1), TK = int(L->K / kTile);     // gated: pairs of row-blocks
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    cfg.gridDim = dim3(unsigned(TN) * unsigned(S), 1, 1);
    cfg.blockDim = dim3(192, 1, 1);
    cfg.dynamicSmemBytes = C::kSmemBytes;
    cfg.stream = stream;
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = unsigned(S);
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, map, packed, uint64_t(L->table_off), uint32_t(L->payload_off / 16),
                                       uint32_t(L->total_bytes / 16), TK, S, M, Y, ldy, status_dev);
    return e == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

// Cluster size for a weight of TN x TK tiles: the smallest power of two that gives the kernel at least 32
// CTAs (fewer would leave a short stream of GEMMs without enough bytes in flight) and at most 48 tiles per CTA
// (a longer run holds back the completion of every kernel behind it), at most 8 and at most TK.
int decode_cluster_split(int TN, int TK) {
    constexpr int kMaxTilesPerCta = 48;
    int S = 1;
    while (S < 8 && (TN * S < 32 || TK > kMaxTilesPerCta * S)) S *= 2;
    while (S > 1 && S > TK) S /= 2;
    return S;
}

template <int N_TOK, int STAGES>
static int launch_dc_f(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int M, int S,
                       __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool wstatic, bool xstatic,
                       bool ystatic) {
    if (wstatic && xstatic && ystatic)
        return launch_dc_t<N_TOK, STAGES, true, true, false, true>(map, L, packed, M, S, Y, ldy, status_dev, stream);
    if (wstatic && xstatic) return launch_dc_t<N_TOK, STAGES, true, true>(map, L, packed, M, S, Y, ldy, status_dev, stream);
    if (wstatic) return launch_dc_t<N_TOK, STAGES, true, false>(map, L, packed, M, S, Y, ldy, status_dev, stream);
    return launch_dc_t<N_TOK, STAGES, false, false>(map, L, packed, M, S, Y, ldy, status_dev, stream);
}

int launch_decode_cluster(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int M, int n_tok,
                          __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool wstatic,
                          bool xstatic, bool ystatic) {
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    int S = decode_cluster_split(TN, TK);
    if (!xstatic) {
        // a GEMM that waits for its predecessor streams alone for a while: at least 128 CTAs, so that its own loads
        // can keep HBM busy (the independent schedule wants few CTAs per GEMM and several GEMMs resident instead).
        // Tried on top of this and dropped: asking L2 for the rest of the CTA's weight tiles before the wait
        // (0.332 against 0.322 ms on the 24-GEMM step) -- a three-stage ring drains L2 hardly faster than HBM.
        // Also tried: at least one CTA per SM instead of 128 (the 4096-row weights then split K eight ways, 256 CTAs):
        // 0.303 ms on that step, but the decoder-block chain, where independent launches of the next block already
        // hold SM slots, goes from 1.99 to 2.20 ms -- the chain is the case that matters, so 128 stays.
        S = 1;
        while (S < 8 && TN * S < 128 && 2 * S <= TK) S *= 2;
    }
    switch (n_tok) {
        case 16: return launch_dc_f<16, 3>(map, L, packed, M, S, Y, ldy, status_dev, stream, wstatic, xstatic, ystatic);
        case 32: return launch_dc_f<32, 2>(map, L, packed, M, S, Y, ldy, status_dev, stream, wstatic, xstatic, ystatic);
        default: return launch_dc_f<64, 2>(map, L, packed, M, S, Y, ldy, status_dev, stream, wstatic, xstatic, ystatic);
    }
}

// silu(gate) * up on a stacked gate/up weight (row-blocks interleaved), M <= 16, weights static: independent launches
// (few CTAs, several GEMMs resident) or, with `xstatic` false, a launch that streams alone once its predecessor is
// done (at least 128 CTAs) -- the gated product of a decoder block reads the output of the projection before it.
int launch_decode_cluster_gated(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int M,
                                __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool xstatic) {
    const int TN = int(L->N / kTile) / 2, TK = int(L->K / kTile);
    int S = decode_cluster_split(TN, 2 * TK);                         // a CTA streams the slices of two row-blocks
    if (!xstatic) {
        S = 1;
        while (S < 8 && TN * S < 128 && 2 * S <= TK) S *= 2;
    }
    while (S > 1 && S > TK) S /= 2;
    if (xstatic) return launch_dc_t<16, 3, true, true, true>(map, L, packed, M, S, Y, ldy, status_dev, stream);
    return launch_dc_t<16, 3, true, false, true>(map, L, packed, M, S, Y, ldy, status_dev, stream);
}

}  // namespace patch
