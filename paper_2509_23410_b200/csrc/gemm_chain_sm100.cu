// A chain of small-M matmuls in ONE persistent launch: job i + 1 may read, as its X, what job i wrote as its Y.
//
// Launched one after the other, dependent decode GEMMs leave HBM idle at every hand-over: the last tiles of one
// kernel drain, the kernel completes and is flushed, the next one's wait returns, its activations arrive, and only
// then does its weight stream start again (~5 us per GEMM against 8-10 us of streaming; the stream of dependent
// launches reaches 52 % of the HBM roofline).  Here the GEMMs of the chain are jobs of one cooperative kernel with
// one CTA per SM:
//   * every job's tiles, in (row-block, K) order, are cut into one contiguous range per CTA (tile counts equal to
//     within one); a range that covers only part of a row-block yields a partial sum, written to the workspace, and
//     the CTA that is LAST to deliver a part of a row-block (an arrival counter per row-block) sums the parts in CTA
//     order -- a fixed order, whoever does it -- and stores bf16.  Nobody waits for anybody inside a job.
//   * between jobs the CTAs meet at a grid barrier (one counter per job in global memory -- a CTA without tiles in a
//     job is through with it at once, so a single running count would open early -- and a bounded spin).  Only the warp that
//     fetches ACTIVATIONS waits there.  The warp that fetches WEIGHTS never does: weights are static, so it runs on
//     into the next job as stages free up, and the ring (5 stages of a whole tile, 180 KB per SM, 26 MB on the chip)
//     is full of the next job's weights when the barrier opens.  HBM keeps streaming through the hand-over.
//
// warp 0: weight producer (one cp.async.bulk per tile)      warp 6: activation producer (two tiled copies per tile)
// warp 1: MMA issuer (tcgen05.mma / .mma.sp, two accumulators so that the next range starts while one drains)
// warps 2-5: epilogue (accumulator -> Y, or -> workspace + arrival counter + reduction by the last to arrive)
//
// Deterministic; M <= 16; bf16 tile kinds.  Every wait is bounded (shared-memory barriers as elsewhere, the grid
// barrier by the same clock); a CTA that gives up raises the status word and leaves, the others give up at their
// next barrier.  The cooperative launch fails up front if the CTAs cannot all be resident, so the grid barrier
// cannot wait for a CTA that has not started.
#include <cstring>
#include "sm100_ptx.cuh"

namespace patch {

namespace ch {
constexpr int kStages = 5;
constexpr int kThreads = 224;
constexpr int kMaxJobs = 16;                                  // per launch (kernel parameter space)
constexpr int kMaxGrid = 256;                                 // CTAs the workspace is sized for
constexpr uint32_t kXAtomBytes = 16 * 128, kXBytes = 2 * kXAtomBytes;
constexpr uint32_t kStageBytes = kDenseBytes + kXBytes;
constexpr uint32_t kBarrierOffset = kStages * kStageBytes;
constexpr uint32_t kStagingOffset = kBarrierOffset + 256;     // 4 epilogue warps x 1 KB transpose staging
constexpr uint32_t kSmemBytes = kStagingOffset + 4 * 1024 + 1024;
constexpr uint32_t kTmemCols = 64;                            // two accumulators of 16 columns, 4 metadata columns per stage
constexpr uint32_t kPartialFloats = 128 * 16;                 // one partial: [128 rows][16 tokens] fp32
static_assert(32 + 4 * kStages <= kTmemCols, "TMEM columns");
static_assert(kSmemBytes <= 227 * 1024, "shared memory");

struct alignas(64) Job {
    CUtensorMap tmap_x;            // X [M x K] bf16, box 64 columns x 16 rows, 128-byte swizzle
    const uint8_t* blob;
    __nv_bfloat16* Y;
    int64_t ldy;
    uint32_t table_off, pay0_16, end16;
    int TN, TK;
    uint32_t counter_base;         // index of the job's first row-block counter
};
struct Params {
    Job jobs[kMaxJobs];
    int n_jobs, M;
    uint32_t* counters;            // one per row-block of every job, zero at launch
    float* partials;               // [grid][2][128][16]
    unsigned int* grid_bar;        // [kMaxJobs], zero at launch: CTAs that are through with job j
    int* status;
};

// first tile of CTA c's range when T tiles are cut into G ranges (G <= T, so no range is empty), and the CTA
// whose range holds tile t
__device__ __forceinline__ int range_start(int c, int T, int G) { return int(int64_t(c) * T / G); }
__device__ __forceinline__ int range_owner(int t, int T, int G) { return int((int64_t(t + 1) * G - 1) / T); }

__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu_add(unsigned int* p, unsigned int v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ float4 ld_cg_f4(const float* p) {
    float4 v;
    asm volatile("ld.global.cg.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
    return v;
}
// writes of the generic proxy (other CTAs' Y stores, seen through the grid barrier) ordered before this thread's
// tiled copies, which read through the async proxy
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
}  // namespace ch

__global__ void __launch_bounds__(ch::kThreads, 1)
chain_kernel(const __grid_constant__ ch::Params P) {
    using namespace ch;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_wfull = smem_base + kBarrierOffset;        // kStages x 8 B (8 reserved for each array)
    const uint32_t bar_xfull = bar_wfull + 64;
    const uint32_t bar_empty = bar_xfull + 64;
    const uint32_t bar_acc_full = bar_empty + 64;                 // 2 x 8 B
    const uint32_t bar_acc_empty = bar_acc_full + 16;             // 2 x 8 B
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kBarrierOffset + 224);
    uint32_t* tmem_slot = misc;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 1);
    volatile uint32_t* last_flag = misc + 2;                      // epilogue: "this CTA delivered the last part"
    volatile uint32_t* stage_kind = misc + 3;                     // [kStages] (224 + 32 = 256 bytes in all)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int c = int(blockIdx.x), G = int(gridDim.x);

    if (threadIdx.x == 64) {
        for (int i = 0; i < kStages; ++i) {
            mbar_init(bar_wfull + 8 * i, 1);
            mbar_init(bar_xfull + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar_acc_full + 8 * i, 1);
            mbar_init(bar_acc_empty + 8 * i, 4);                  // the four epilogue warps
        }
        *abort_flag = 0;
        mbar_init_fence();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_meta = tmem_base + 32;

    if (warp == 0) {
        // ---------------- weight producer: never waits for another CTA ----------------
        const uint64_t pol_w = l2_policy_evict_first();
        int seq = 0;                                               // tiles of this CTA so far, over all jobs
        bool ok = true;
        for (int j = 0; j < P.n_jobs && ok; ++j) {
            const Job& J = P.jobs[j];
            const int T = J.TN * J.TK, Ge = min(G, T);           // a job with fewer tiles than CTAs uses the first T of them
            const int t0 = c < Ge ? range_start(c, T, Ge) : 0, n = c < Ge ? range_start(c + 1, T, Ge) - t0 : 0;
            const TileDesc* table = reinterpret_cast<const TileDesc*>(J.blob + J.table_off) + t0;
            TileDesc mine = TileDesc{0, 0, 0, 0};
            for (int i = 0; i < n && ok; ++i, ++seq) {
                if ((i & 31) == 0 && i + lane < n) mine = table[i + lane];
                uint32_t kind = __shfl_sync(0xFFFFFFFFu, mine.kind, i & 31);
                uint32_t off16 = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, i & 31);
                if (lane == 0) {
                    const int stage = seq % kStages;
                    sanitize_tile(kind, off16, J.pay0_16, J.end16, P.status);
                    const uint32_t wbytes = kind == PATCH_TILE_DENSE ? kDenseBytes : kSparseBytes;
                    if (seq >= kStages)
                        ok = mbar_wait(bar_empty + 8 * stage, (uint32_t(seq / kStages) & 1u) ^ 1u, abort_flag, P.status);
                    if (ok) {
                        stage_kind[stage] = kind;
                        mbar_expect_tx(bar_wfull + 8 * stage, wbytes);
                        tma_bulk_load(smem_base + stage * kStageBytes, J.blob + uint64_t(off16) * 16, wbytes, bar_wfull + 8 * stage, pol_w);
                    }
                }
                ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            }
        }
        if (lane == 0 && *abort_flag) {
            // drain: wait (bounded) until the copies this thread started have landed
            const uint64_t tstart = global_timer_ns();
            for (int q = seq > kStages ? seq - kStages : 0; q < seq; ++q)
                while (!mbar_try_wait(bar_wfull + 8 * (q % kStages), uint32_t(q / kStages) & 1u) && global_timer_ns() - tstart < kDrainLimitNs) {}
        }
    } else if (warp == 6) {
        // ---------------- activation producer: the one role that waits at the grid barrier ----------------
        if (lane == 0) {
            const uint64_t pol_x = l2_policy_evict_last();
            int seq = 0;
            bool ok = true;
            for (int j = 0; j < P.n_jobs && ok; ++j) {
                const Job& J = P.jobs[j];
                const int T = J.TN * J.TK, Ge = min(G, T);           // a job with fewer tiles than CTAs uses the first T of them
            const int t0 = c < Ge ? range_start(c, T, Ge) : 0, n = c < Ge ? range_start(c + 1, T, Ge) - t0 : 0;
                if (j > 0 && n > 0) {
                    // job j - 1 is complete everywhere once every CTA has added one to its counter
                    const unsigned int target = unsigned(G);
                    const uint64_t t_start = global_timer_ns();
                    while (ld_acquire_gpu(P.grid_bar + (j - 1)) < target) {
                        if (*abort_flag) { ok = false; break; }
                        if (global_timer_ns() - t_start > kWaitLimitNs) {
                            *abort_flag = 1;
                            if (P.status) atomicCAS(P.status, PATCH_OK, PATCH_ERR_TIMEOUT);
                            ok = false;
                            break;
                        }
                        __nanosleep(100);
                    }
                    fence_proxy_async_global();
                }
                for (int i = 0; i < n && ok; ++i, ++seq) {
                    const int stage = seq % kStages, k = ((t0 + i) % J.TK) * kTile;
                    if (seq >= kStages)
                        ok = mbar_wait(bar_empty + 8 * stage, (uint32_t(seq / kStages) & 1u) ^ 1u, abort_flag, P.status);
                    if (!ok) break;
                    const uint32_t sX = smem_base + stage * kStageBytes + kDenseBytes;
                    mbar_expect_tx(bar_xfull + 8 * stage, kXBytes);
                    tma_tile_load(sX, &J.tmap_x, k, 0, bar_xfull + 8 * stage, pol_x);
                    tma_tile_load(sX + kXAtomBytes, &J.tmap_x, k + 64, 0, bar_xfull + 8 * stage, pol_x);
                }
            }
            if (*abort_flag) {
                const uint64_t tstart = global_timer_ns();
                for (int q = seq > kStages ? seq - kStages : 0; q < seq; ++q)
                    while (!mbar_try_wait(bar_xfull + 8 * (q % kStages), uint32_t(q / kStages) & 1u) && global_timer_ns() - tstart < kDrainLimitNs) {}
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            int seq = 0, seg = 0;                                  // tiles and ranges-within-a-row-block so far
            bool ok = true;
            for (int j = 0; j < P.n_jobs && ok; ++j) {
                const Job& J = P.jobs[j];
                const int T = J.TN * J.TK, Ge = min(G, T);
                const int t0 = c < Ge ? range_start(c, T, Ge) : 0, t1 = c < Ge ? range_start(c + 1, T, Ge) : 0;
                for (int t = t0; t < t1 && ok;) {
                    const int tn = t / J.TK, t_end = min(t1, (tn + 1) * J.TK), b = seg & 1;
                    if (seg >= 2) ok = mbar_wait(bar_acc_empty + 8 * b, (uint32_t(seg / 2) & 1u) ^ 1u, abort_flag, P.status);
                    if (!ok) break;
                    tc_fence_after();
                    for (int u = t; u < t_end && ok; ++u, ++seq) {
                        const int stage = seq % kStages;
                        const uint32_t parity = uint32_t(seq / kStages) & 1u;
                        ok = mbar_wait(bar_wfull + 8 * stage, parity, abort_flag, P.status);
                        if (ok) ok = mbar_wait(bar_xfull + 8 * stage, parity, abort_flag, P.status);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t sW = smem_base + stage * kStageBytes;
                        issue_tile_mma<16>(stage_kind[stage], sW, sW + kDenseBytes, kXAtomBytes, tmem_base + 16u * b,
                                           tmem_meta + 4 * stage, u == t);
                        mma_commit(bar_empty + 8 * stage);
                    }
                    if (ok) mma_commit(bar_acc_full + 8 * b);
                    t = t_end;
                    ++seg;
                }
            }
        }
        __syncwarp();
    } else if (warp >= 2 && warp < 6) {
        // ---------------- epilogue ----------------
        const uint32_t quad = warp & 3u, row = quad * 32 + lane;
        const int e = threadIdx.x - 64;                            // 0..127
        uint8_t* staging = smem + kStagingOffset + (warp - 2) * 1024;
        int seg = 0;
        bool ok = true;
#ifdef PATCH_FAULT_INJECTION
        // test build: a status word holding kInjectMagic keeps CTA 0 away from the first grid barrier, so that the
        // other CTAs' wait there runs out (see sm100_ptx.cuh)
        bool inject = false;
        if (c == 0 && P.status && *P.status == kInjectMagic) {
            inject = true;
            asm volatile("barrier.cta.sync 1, 128;" ::: "memory");
            if (e == 0) *P.status = PATCH_OK;
        }
#else
        constexpr bool inject = false;
#endif
        for (int j = 0; j < P.n_jobs && ok; ++j) {
            const Job& J = P.jobs[j];
            const int T = J.TN * J.TK, Ge = min(G, T);
            const int t0 = c < Ge ? range_start(c, T, Ge) : 0, t1 = c < Ge ? range_start(c + 1, T, Ge) : 0;
            for (int t = t0; t < t1 && ok; ++seg) {
                const int tn = t / J.TK, t_end = min(t1, (tn + 1) * J.TK), b = seg & 1;
                // one thread polls, the others wait on hardware barrier 1: all 128 learn of a wait given up together,
                // so nobody is left alone at one of the barriers below
                ok = group_wait(bar_acc_full + 8 * b, uint32_t(seg / 2) & 1u, e == 0, 1, 128, abort_flag, P.status);
                if (!ok) break;
                tc_fence_after();
                uint32_t v[16];
                tmem_ld16(tmem_base + ((quad * 32u) << 16) + 16u * uint32_t(b), v);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acc_empty + 8 * b);
                __nv_bfloat16* y = J.Y + int64_t(tn) * kTile + quad * 32;
                const int first = range_owner(tn * J.TK, T, Ge), last = range_owner((tn + 1) * J.TK - 1, T, Ge);
                if (first == last) {
                    store_fragment_transposed(v, staging, lane, y, J.ldy, P.M);     // the whole row-block was this CTA's
                } else {
                    // this CTA's part: slot 0 if the row-block is the one its range starts in, else slot 1
                    float* mine = P.partials + (size_t(c) * 2 + (tn == t0 / J.TK ? 0 : 1)) * kPartialFloats + row * 16;
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        reinterpret_cast<float4*>(mine)[q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                                                          __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                    __threadfence();
                    asm volatile("barrier.cta.sync 1, 128;" ::: "memory");
                    if (e == 0) *last_flag = atomicAdd(P.counters + J.counter_base + tn, 1u) == unsigned(last - first) ? 1u : 0u;
                    asm volatile("barrier.cta.sync 1, 128;" ::: "memory");
                    if (*last_flag) {
                        // every part has been delivered (each behind a fence): sum them in CTA order
                        __threadfence();
                        float acc[16];
#pragma unroll
                        for (int q = 0; q < 16; ++q) acc[q] = 0.0f;
                        for (int cc = first; cc <= last; ++cc) {
                            const int slot = tn == range_start(cc, T, Ge) / J.TK ? 0 : 1;
                            const float* part = P.partials + (size_t(cc) * 2 + slot) * kPartialFloats + row * 16;
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const float4 p = ld_cg_f4(part + 4 * q);
                                acc[4 * q] += p.x; acc[4 * q + 1] += p.y; acc[4 * q + 2] += p.z; acc[4 * q + 3] += p.w;
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 16; ++q) v[q] = __float_as_uint(acc[q]);
                        store_fragment_transposed(v, staging, lane, y, J.ldy, P.M);
                    }
                    asm volatile("barrier.cta.sync 1, 128;" ::: "memory");       // last_flag may be rewritten
                }
                t = t_end;
            }
            // this CTA's share of job j is written (or handed to the row-block's last contributor): tell the grid
            __threadfence();
            asm volatile("barrier.cta.sync 1, 128;" ::: "memory");
            if (e == 0 && !(inject && j == 0)) red_release_gpu_add(P.grid_bar + j, 1u);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, ch::kTmemCols);
}

// ---------------------------------------------------------------------------------------------

static int chain_grid() {
    static std::atomic<int> cached[kMaxDevices];
    const int dev = current_device();
    if (dev < 0) return 0;
    int g = cached[dev].load(std::memory_order_acquire);
    if (g > 0) return g;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, chain_kernel, ch::kThreads, ch::kSmemBytes) != cudaSuccess || per_sm < 1)
        return 0;
    g = sm_count();                                               // one CTA per SM
    cached[dev].store(g, std::memory_order_release);
    return g;
}

static size_t chain_head_bytes(const patch_chain_job_t* jobs, int n_jobs) {
    size_t counters = ch::kMaxJobs;                               // the first words are the grid barriers of one launch
    for (int i = 0; i < n_jobs; ++i) counters += size_t(jobs[i].layout->N / kTile);
    return (counters * 4 + 255) / 256 * 256;
}

size_t chain_workspace_bytes(const patch_chain_job_t* jobs, int n_jobs) {
    return chain_head_bytes(jobs, n_jobs) + size_t(ch::kMaxGrid) * 2 * ch::kPartialFloats * sizeof(float);
}

int launch_chain(const patch_chain_job_t* jobs, int n_jobs, int64_t M, void* workspace, int* status_dev, cudaStream_t stream) {
    static std::atomic<uint64_t> configured{0};
    if (int rc = allow_dynamic_smem(chain_kernel, ch::kSmemBytes, configured)) return rc;
    const int G = chain_grid();
    if (G < 1 || G > ch::kMaxGrid) return PATCH_ERR_CUDA;
    const size_t head = chain_head_bytes(jobs, n_jobs);
    // counters and the grid barrier start from zero at every call
    if (cudaMemsetAsync(workspace, 0, head, stream) != cudaSuccess) return PATCH_ERR_CUDA;
    uint32_t* words = static_cast<uint32_t*>(workspace);
    uint32_t counter_base = ch::kMaxJobs;
    for (int first = 0; first < n_jobs; first += ch::kMaxJobs) {
        ch::Params P;
        std::memset(&P, 0, sizeof P);
        P.n_jobs = n_jobs - first < ch::kMaxJobs ? n_jobs - first : ch::kMaxJobs;
        P.M = int(M);
        P.counters = words;
        P.partials = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + head);
        P.grid_bar = reinterpret_cast<unsigned int*>(words);      // one launch after the other uses them in turn
        P.status = status_dev;
        for (int i = 0; i < P.n_jobs; ++i) {
            const patch_chain_job_t& src = jobs[first + i];
            ch::Job& J = P.jobs[i];
            int rc = make_x_tensor_map(&J.tmap_x, static_cast<const __nv_bfloat16*>(src.X_dev), src.ldx, M, src.layout->K, 16);
            if (rc) return rc;
            J.blob = static_cast<const uint8_t*>(src.packed_dev);
            J.Y = static_cast<__nv_bfloat16*>(src.Y_dev);
            J.ldy = src.ldy;
            J.table_off = uint32_t(src.layout->table_off);
            J.pay0_16 = uint32_t(src.layout->payload_off / 16);
            J.end16 = uint32_t(src.layout->total_bytes / 16);
            J.TN = int(src.layout->N / kTile);
            J.TK = int(src.layout->K / kTile);
            J.counter_base = counter_base;
            counter_base += uint32_t(J.TN);
        }
        if (first > 0 && cudaMemsetAsync(workspace, 0, ch::kMaxJobs * 4, stream) != cudaSuccess) return PATCH_ERR_CUDA;   // the grid barriers again
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        cfg.gridDim = dim3(unsigned(G), 1, 1);
        cfg.blockDim = dim3(ch::kThreads, 1, 1);
        cfg.dynamicSmemBytes = ch::kSmemBytes;
        cfg.stream = stream;
        attr[0].id = cudaLaunchAttributeCooperative;
        attr[0].val.cooperative = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, chain_kernel, P) != cudaSuccess) return PATCH_ERR_CUDA;
    }
    return PATCH_OK;
}

}  // namespace patch
