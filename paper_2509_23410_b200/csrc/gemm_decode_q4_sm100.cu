// Small-M matmul on a weight whose tiles are stored with 4-bit values (tile kinds 2 and 3: the 4-bit weight-only
// quantisation table of the paper's section on combining the method with other compression).
//
// The layer multiplies by the DEQUANTISED weight v^ = bf16(q * s) (public header), so the kernel turns every tile
// back into the bf16 operand image the tensor core reads -- two swizzled K-major atoms for a dense tile, one atom
// plus the 2 KB metadata block for a 2:4 tile -- in shared memory, and runs the same tcgen05.mma / .mma.sp as the
// bf16 kinds on it.  HBM only ever sees 0.52 B (dense) or 0.39 B (2:4) per weight element.
//
//   warp 0       producer: cp.async.bulk of the tile's payload (8 448 / 6 400 B: codes [, metadata], scales) into a
//                ring of kRaw slots, and the two activation atoms of the tile's K range into the slot's X buffer
//   warps 6..13  dequantise: slot -> operand stage.  A thread owns one 32-bit word of codes at a time = eight
//                consecutive stored values of one row = one 16-byte chunk of the atom: the word's nibbles are
//                ordered (pack.cu) so that (w >> 4j) & 0x000F000F | 0x43004300 is the bf16 pair (128 + n, 128 + n'),
//                then (x - 136) * s in two bf16x2 instructions, both exact or correctly rounded:
//                128 + n and n - 8 are integers below 256, and bf16(q * s) is one rounding of the exact product.
//   warp 1       MMA issuer: operand stage x X buffer -> TMEM accumulator [128 rows x 16 tokens]
//   warps 2..5   epilogue: accumulator -> shared memory; then, as in the bf16 row-block schedule, the S CTAs of a
//                cluster (split-K) sum their partials through distributed shared memory in K order and write Y.
//
// What bounds it: with ~2.2 instructions per value the dequantisation of a dense tile keeps the SM's four issue
// ports busy for ~350 cycles, about what its 8 448 bytes take to arrive at this SM's share of the HBM bandwidth,
// so the kernel sits where the ALU and the HBM roofs meet (2:4 tiles: 64 values per row, memory-bound).
//
// Same bounded waits, table checks, launch flags and determinism as the other decode kernels; M <= 16.
#include "sm100_ptx.cuh"

namespace patch {

namespace dq {
constexpr int kRaw = 8;                                   // payload ring
constexpr int kOps = 3;                                   // operand ring
constexpr int kDequantWarps = 8;
constexpr int kThreads = 192 + 32 * kDequantWarps;
constexpr uint32_t kRawBytes = kDenseQ4Bytes;             // slot size: the larger of the two payloads
constexpr uint32_t kXAtomBytes = 16 * 128, kXBytes = 2 * kXAtomBytes;
constexpr uint32_t kOpBytes = kDenseBytes;                // two atoms, or one atom + metadata
constexpr uint32_t kXOffset = kOps * kOpBytes;
constexpr uint32_t kRawOffset = kXOffset + kRaw * kXBytes;
constexpr uint32_t kBarrierOffset = kRawOffset + kRaw * kRawBytes;
constexpr uint32_t kSmemBytes = kBarrierOffset + 256 + 1024;
constexpr uint32_t kTmemCols = 32;                        // 16 accumulator columns + 4 metadata columns per operand stage
constexpr uint32_t kPartialRowBytes = 16 * 4;
static_assert(16 + 4 * kOps <= kTmemCols, "TMEM columns");
static_assert(kRawBytes % 128 == 0 && kSparseQ4Bytes <= kRawBytes, "payload slots");
static_assert(kSmemBytes <= 227 * 1024, "shared memory");

__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float4 ld_peer_f4(uint32_t saddr, uint32_t rank) {
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(saddr), "r"(rank));
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a) : "memory");
    return v;
}
// generic-proxy writes to shared memory become visible to the async proxy (tcgen05.mma, tcgen05.cp)
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// A table entry of a 4-bit weight, checked before a byte of it is requested: the kind must be one of the two
// 4-bit kinds and the payload must lie inside the blob; otherwise the status word says so and the blob's first
// payload is read as a 2:4 tile (the smaller one) in its place.
__device__ __forceinline__ void sanitize_q4_tile(uint32_t& kind, uint32_t& off16, uint32_t pay0_16, uint32_t end16, int* status_dev) {
    const uint32_t len16 = (kind == PATCH_TILE_DENSE_Q4 ? kDenseQ4Bytes : kSparseQ4Bytes) / 16;
    if (kind < PATCH_TILE_DENSE_Q4 || kind > PATCH_TILE_SPARSE_2_4_Q4 || off16 < pay0_16 || off16 > end16 || len16 > end16 - off16) {
        if (status_dev) atomicCAS(status_dev, PATCH_OK, PATCH_ERR_FORMAT);
        kind = PATCH_TILE_SPARSE_2_4_Q4;
        off16 = pay0_16;
    }
}

// Eight codes -> eight bf16 values (one 16-byte chunk of an atom).  s2 = the row's scale in both halves.
__device__ __forceinline__ uint4 dequant_word(uint32_t w, __nv_bfloat162 s2) {
    const uint32_t kMagic = 0x43004300u;                         // bf16 128.0 twice: 128 + n in the low mantissa bits
    const uint32_t kBias = 0x43084308u;                          // bf16 136.0 twice
    const __nv_bfloat162 bias = *reinterpret_cast<const __nv_bfloat162*>(&kBias);
    uint32_t out[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t p = ((w >> (4 * j)) & 0x000F000Fu) | kMagic;
        const __nv_bfloat162 v = __hmul2(__hsub2(*reinterpret_cast<const __nv_bfloat162*>(&p), bias), s2);
        out[j] = *reinterpret_cast<const uint32_t*>(&v);
    }
    return make_uint4(out[0], out[1], out[2], out[3]);
}
}  // namespace dq

template <bool WSTATIC, bool XSTATIC>
__global__ void __launch_bounds__(dq::kThreads)
decode_q4_kernel(const __grid_constant__ CUtensorMap tmap_x, const uint8_t* __restrict__ blob, uint64_t table_off,
                 uint32_t pay0_16, uint32_t end16, int TK, int S, int M, __nv_bfloat16* __restrict__ Y, int64_t ldy,
                 int* status_dev) {
    using namespace dq;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    const uint32_t bar_raw_full = smem_base + kBarrierOffset;     // kRaw x 8 B
    const uint32_t bar_raw_empty = bar_raw_full + 64;             // kRaw x 8 B
    const uint32_t bar_op_full = bar_raw_empty + 64;              // kOps x 8 B (4 reserved)
    const uint32_t bar_op_empty = bar_op_full + 32;
    const uint32_t bar_acc_full = bar_op_empty + 32;
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kBarrierOffset + 200);
    uint32_t* tmem_slot = misc;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 1);
    volatile uint32_t* slot_kind = misc + 4;                      // [kRaw]

    grid_launch_dependents();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t s = cluster_ctarank();
    const int tn = blockIdx.x / S;
    const int k0 = int(int64_t(s) * TK / S), k1 = int(int64_t(s + 1) * TK / S), n_tiles = k1 - k0;
    const TileDesc* table = reinterpret_cast<const TileDesc*>(blob + table_off) + int64_t(tn) * TK + k0;

    if (threadIdx.x == 64) {
        for (int i = 0; i < kRaw; ++i) {
            mbar_init(bar_raw_full + 8 * i, 1);
            mbar_init(bar_raw_empty + 8 * i, kDequantWarps + 1);   // the dequantising warps (codes) + the MMAs (X)
        }
        for (int i = 0; i < kOps; ++i) {
            mbar_init(bar_op_full + 8 * i, kDequantWarps);
            mbar_init(bar_op_empty + 8 * i, 1);
        }
        mbar_init(bar_acc_full, 1);
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_map(&tmap_x);
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tmem_meta = tmem_base + 16;

    if (warp == 0) {
        // ---------------- producer ----------------
        if constexpr (!WSTATIC) grid_dependency_wait();
        const uint64_t pol_w = l2_policy_evict_first(), pol_x = l2_policy_evict_last();
        TileDesc mine = TileDesc{0, 0, 0, 0};
        int issued = 0;
        bool ok = true;
        // payloads of the first kRaw tiles may be requested before the grid dependency is resolved (WSTATIC);
        // their activations follow once it is (unless XSTATIC)
        const int n_early = (WSTATIC && !XSTATIC) ? (n_tiles < kRaw ? n_tiles : kRaw) : 0;
        for (int i = 0; i < n_tiles && ok; ++i) {
            if ((i & 31) == 0 && i + lane < n_tiles) mine = table[i + lane];
            uint32_t kind = __shfl_sync(0xFFFFFFFFu, mine.kind, i & 31);
            uint32_t off16 = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, i & 31);
            if (lane == 0) {
                const int slot = i % kRaw;
                sanitize_q4_tile(kind, off16, pay0_16, end16, status_dev);
                const uint32_t wbytes = kind == PATCH_TILE_DENSE_Q4 ? kDenseQ4Bytes : kSparseQ4Bytes;
                const uint32_t full = bar_raw_full + 8 * slot;
                if (i >= kRaw) ok = mbar_wait(bar_raw_empty + 8 * slot, (uint32_t(i / kRaw) & 1u) ^ 1u, abort_flag, status_dev);
                if (ok) {
                    slot_kind[slot] = kind;
                    mbar_expect_tx(full, wbytes + kXBytes);
                    tma_bulk_load(smem_base + kRawOffset + slot * kRawBytes, blob + uint64_t(off16) * 16, wbytes, full, pol_w);
                    if (i < n_early) {
                        if (i + 1 == n_early) {
                            grid_dependency_wait();
                            for (int j = 0; j < n_early; ++j) {
                                const uint32_t sX = smem_base + kXOffset + j * kXBytes;
                                tma_tile_load(sX, &tmap_x, (k0 + j) * kTile, 0, bar_raw_full + 8 * j, pol_x);
                                tma_tile_load(sX + kXAtomBytes, &tmap_x, (k0 + j) * kTile + 64, 0, bar_raw_full + 8 * j, pol_x);
                            }
                        }
                    } else {
                        const uint32_t sX = smem_base + kXOffset + slot * kXBytes;
                        tma_tile_load(sX, &tmap_x, (k0 + i) * kTile, 0, full, pol_x);
                        tma_tile_load(sX + kXAtomBytes, &tmap_x, (k0 + i) * kTile + 64, 0, full, pol_x);
                    }
                    issued = i + 1;
                }
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
        }
        if (lane == 0 && *abort_flag) {
            // drain: wait (bounded) until the copies this thread started have landed
            const uint64_t tstart = global_timer_ns();
            for (int j = issued > kRaw ? issued - kRaw : 0; j < issued; ++j) {
                const uint32_t bar = bar_raw_full + 8 * (j % kRaw), parity = uint32_t(j / kRaw) & 1u;
                while (!mbar_try_wait(bar, parity) && global_timer_ns() - tstart < kDrainLimitNs) {}
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            bool ok = true;
            for (int i = 0; i < n_tiles && ok; ++i) {
                const int slot = i % kRaw, op = i % kOps;
                ok = mbar_wait(bar_op_full + 8 * op, uint32_t(i / kOps) & 1u, abort_flag, status_dev);
                // the slot's activations arrived with its payload, which the dequantising warps have consumed: this
                // wait returns at once, and makes the async-proxy writes of X visible to this thread's MMAs
                if (ok) ok = mbar_wait(bar_raw_full + 8 * slot, uint32_t(i / kRaw) & 1u, abort_flag, status_dev);
                if (!ok) break;
                tc_fence_after();
                const uint32_t sW = smem_base + op * kOpBytes, sX = smem_base + kXOffset + slot * kXBytes;
                issue_tile_mma<16>(slot_kind[slot] & 1u, sW, sX, kXAtomBytes, tmem_base, tmem_meta + 4 * op, i == 0);
                mma_commit(bar_op_empty + 8 * op);
                mma_commit(bar_raw_empty + 8 * slot);
            }
            if (ok && n_tiles > 0) mma_commit(bar_acc_full);
        }
        __syncwarp();
    } else if (warp >= 6) {
        // ---------------- dequantisation: payload slot -> operand stage ----------------
        const uint32_t dt = threadIdx.x - 192;                    // 0 .. 32 * kDequantWarps - 1
        constexpr uint32_t kDt = 32 * kDequantWarps;
        bool ok = true;
        for (int i = 0; i < n_tiles && ok; ++i) {
            const int slot = i % kRaw, op = i % kOps;
            if (lane == 0) {
                ok = mbar_wait(bar_raw_full + 8 * slot, uint32_t(i / kRaw) & 1u, abort_flag, status_dev);
                if (ok && i >= kOps)
                    ok = mbar_wait(bar_op_empty + 8 * op, (uint32_t(i / kOps) & 1u) ^ 1u, abort_flag, status_dev);
            }
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            if (!ok) break;
            const uint8_t* raw = smem + kRawOffset + slot * kRawBytes;
            uint8_t* dst = smem + op * kOpBytes;
            const uint32_t* words = reinterpret_cast<const uint32_t*>(raw);
            if (slot_kind[slot] == PATCH_TILE_DENSE_Q4) {
                const uint16_t* scales = reinterpret_cast<const uint16_t*>(raw + kDenseQ4CodeBytes);
#pragma unroll
                for (uint32_t it = 0; it < 2048 / kDt; ++it) {
                    const uint32_t idx = it * kDt + dt, r = idx >> 4, c = idx & 15u;
                    const uint32_t sb = scales[r] * 0x00010001u;
                    const uint4 v = dequant_word(words[idx], *reinterpret_cast<const __nv_bfloat162*>(&sb));
                    *reinterpret_cast<uint4*>(dst + (c >> 3) * kAtomBytes + atom_chunk_offset(r, c & 7u)) = v;
                }
            } else {
                const uint16_t* scales = reinterpret_cast<const uint16_t*>(raw + kSparseQ4CodeBytes + kMetaBytes);
#pragma unroll
                for (uint32_t it = 0; it < 1024 / kDt; ++it) {
                    const uint32_t idx = it * kDt + dt, r = idx >> 3, c = idx & 7u;
                    const uint32_t sb = scales[r] * 0x00010001u;
                    const uint4 v = dequant_word(words[idx], *reinterpret_cast<const __nv_bfloat162*>(&sb));
                    *reinterpret_cast<uint4*>(dst + atom_chunk_offset(r, c)) = v;
                }
                // the metadata block follows the atom, as in a bf16 2:4 payload
                if (dt < kMetaBytes / 16)
                    reinterpret_cast<uint4*>(dst + kAtomBytes)[dt] = reinterpret_cast<const uint4*>(raw + kSparseQ4CodeBytes)[dt];
            }
            fence_proxy_async();
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(bar_op_full + 8 * op);
                mbar_arrive(bar_raw_empty + 8 * slot);
            }
        }
    } else {
        // ---------------- epilogue warps 2..5: own partial -> own shared memory ----------------
        // The operand ring is free once the accumulator is complete; the partial [128 rows][16 tokens] fp32
        // takes the first 8 KB of it.
        const uint32_t quad = warp & 3u, row = quad * 32 + lane;
        bool ok = true;
        if (n_tiles > 0) {
            if (lane == 0) ok = mbar_wait_relaxed(bar_acc_full, 0, abort_flag, status_dev);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            tc_fence_after();
        }
        float4* dst = reinterpret_cast<float4*>(smem + row * kPartialRowBytes);
        uint32_t v[16];
        if (n_tiles > 0 && ok) {
            tmem_ld16(tmem_base + ((quad * 32u) << 16), v);
            tmem_ld_wait();
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = 0u;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q)
            dst[q] = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]), __uint_as_float(v[4 * q + 2]),
                                 __uint_as_float(v[4 * q + 3]));
        tc_fence_before();
    }

    // every partial of the cluster is in place (on a timeout the partials are zeros or garbage, and status_dev says so)
    __syncthreads();
    dq::cluster_barrier();

    if (warp >= 2 && warp < 6) {
        // ---------------- reduction: this CTA finishes rows [128 s / S, 128 (s + 1) / S) ----------------
        const int e = threadIdx.x - 64;                            // 0..127
        const int rows = kTile / S;                                // S in {1, 2, 4, 8}
        const int n_out = rows * 4;                                // groups of four tokens
        grid_dependency_wait();                                    // Y may be in use by the preceding kernel
        for (int o = e; o < n_out; o += 128) {
            const int r = int(s) * rows + (o % rows), tg = o / rows;
            const uint32_t addr = smem_base + uint32_t(r) * kPartialRowBytes + uint32_t(tg) * 16u;
            float4 acc = dq::ld_peer_f4(addr, 0);
            for (int q = 1; q < S; ++q) {                          // ascending K: a fixed summation order
                const float4 p = dq::ld_peer_f4(addr, uint32_t(q));
                acc.x += p.x; acc.y += p.y; acc.z += p.z; acc.w += p.w;
            }
            const float a[4] = {acc.x, acc.y, acc.z, acc.w};
            __nv_bfloat16* y = Y + int64_t(tn) * kTile + r;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int m = 4 * tg + j;
                if (m < M) y[int64_t(m) * ldy] = __float2bfloat16_rn(a[j]);
            }
        }
    } else {
        grid_dependency_wait();     // every thread passes the dependency before the CTA exits
    }

    // nobody leaves while a peer may still read its shared memory
    tc_fence_before();
    __syncthreads();
    dq::cluster_barrier();
    if (warp == 1) tmem_dealloc(tmem_base, dq::kTmemCols);
}

template <bool WSTATIC, bool XSTATIC>
static int launch_q4_t(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int M, int S,
                       __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream) {
    auto kern = decode_q4_kernel<WSTATIC, XSTATIC>;
    static std::atomic<uint64_t> configured{0};
    if (int rc = allow_dynamic_smem(kern, dq::kSmemBytes, configured)) return rc;
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    cfg.gridDim = dim3(unsigned(TN) * unsigned(S), 1, 1);
    cfg.blockDim = dim3(dq::kThreads, 1, 1);
    cfg.dynamicSmemBytes = dq::kSmemBytes;
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

int launch_decode_q4(const __nv_bfloat16* X, int64_t ldx, int64_t M, const patch_layout_t* L, const uint8_t* packed,
                     __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool wstatic, bool xstatic) {
    CUtensorMap map;
    int rc = make_x_tensor_map(&map, X, ldx, M, L->K, 16);
    if (rc) return rc;
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    // The smallest power-of-two split of K that makes at least 128 CTAs, at most 8 and at most TK.
    int S = 1;
    while (S < 8 && TN * S < 128 && 2 * S <= TK) S *= 2;
    if (wstatic && xstatic) return launch_q4_t<true, true>(map, L, packed, int(M), S, Y, ldy, status_dev, stream);
    if (wstatic) return launch_q4_t<true, false>(map, L, packed, int(M), S, Y, ldy, status_dev, stream);
    return launch_q4_t<false, false>(map, L, packed, int(M), S, Y, ldy, status_dev, stream);
}

}  // namespace patch
