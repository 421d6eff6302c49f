// Small-M matmul on a weight whose tiles are stored with 4-bit values (tile kinds 2 and 3: the 4-bit weight-only
// quantisation table of the paper's section on combining the method with other compression).
//
// The layer multiplies by the DEQUANTISED weight v^ = bf16(q * s) (public header).  The kernel rebuilds each tile's
// bf16 A operand in TENSOR MEMORY -- tcgen05.mma / .mma.sp take A from there -- so a weight value crosses shared
// memory once, as half a byte on its way in: HBM sees 0.52 B (dense) or 0.39 B (2:4) per weight element, and shared
// memory sees the same.  (Rebuilding the operand image in shared memory instead costs 32 KB of stores and 32 KB of
// tensor-core reads per dense tile, ~700 cycles of the shared-memory port against ~310 cycles of HBM time: that
// version ran at 1.5 TB/s.)
//
//   warp 0        producer, in rounds of kBatch tiles: lane i requests tile i of the round -- one cp.async.bulk of its
//                 payload (8 448 / 6 400 B: codes [, metadata], scales) into a ring of kRaw slots -- and lane 0 the
//                 round's activations, 2 kBatch atoms in one 3-D tiled copy into the slots' X buffers (one lane
//                 per tile and three copies each took ~1 000 cycles a tile, three times the tile's HBM time)
//   warps 5..     kGroups groups of four warps; group g takes tiles g, g + kGroups, ... and owns 64 TMEM columns (its
//                 operand stage) and an accumulator [128 rows x 16 tokens] of its own.
//                 Dequantise: thread = tile row = TMEM lane.  It reads its row's codes 16 bytes at a time (the image
//                 stores them so that the 32 threads of a warp read 512 consecutive bytes), turns each 32-bit word
//                 into eight bf16 -- the nibbles are ordered (pack.cu) so that (w >> 4j) & 0x000F000F | 0x43004300
//                 is the bf16 pair (128 + n, 128 + n'), then (x - 136) * s in two bf16x2 instructions, exact:
//                 128 + n and n - 8 are small integers and bf16(q * s) is one rounding of the exact product -- and
//                 writes 16 columns (32 values) per tcgen05.st.
//                 Multiply: one thread of the group (of a different warp in each group, so that the issuers sit on
//                 different schedulers) issues the tile's MMAs: A = the group's TMEM columns, B = the slot's X
//                 buffer in shared memory; the metadata of a 2:4 tile goes from the payload slot to TMEM with
//                 tcgen05.cp.  Issuing from one thread for all tiles took ~1 100 cycles per tile next to the
//                 dequantising warps it shares issue slots with, and bounded the kernel at 1.7 TB/s.
//                 Inside a group one thread waits on the mbarriers; the other 127 wait on a hardware barrier.
//   warps 1..4    epilogue: sum of the groups' accumulators (ascending group) -> shared memory; then, as in the bf16
//                 row-block schedule, the S CTAs of a cluster (split-K) sum their partials through distributed
//                 shared memory in K order and write Y.
//
// What bounds it: instruction issue.  A dense tile costs ~1 750 warp instructions (~2 per dequantised value: mask,
// shift, subtract, multiply, the last two at half rate, plus synchronisation), i.e. ~440 cycles of the SM's four
// schedulers, against the ~310 cycles its 8 448 bytes take at this SM's share of 8 TB/s; measured in steady state:
// 425-460 cycles per tile.  A 2:4 tile has half the values but the same fixed work per tile.
//
// Two CTAs per SM: while one is being set up, drains its last tiles or waits for the preceding kernel before it may
// write Y, the other streams (one CTA with twice the groups and ring: 0.150 ms on the 24-GEMM decode step, two: 0.130;
// with the output promise, under which finished CTAs do not wait at all: 0.110, and 0.107 with no split of K;
// 0.111 when every group first waited for the consumption of its slot's previous tile, the first fix of the
// ordering described below).
// A CTA allocates 256 TMEM columns, so the two allocations always fit -- an allocation that had to wait for the
// columns of a CTA whose cluster peer waits for this cluster's would never return -- and a third CTA never fits in
// shared memory.
// Tried on top of this and dropped (24-GEMM decode step without the output promise, 0.130 ms): splitting the tile
// into two K-halves with separate completion tracking, so that a group never waits for its own MMAs (0.142 ms: a third barrier and a second
// issue sequence per tile cost more than the wait); dequantising the next tile's first 32 values before that wait
// (0.138 ms: every warp polls again, registers spill); six groups in one CTA per SM (0.150 ms, see above).
// A slot of the payload ring serves the groups in turn (eight slots, three groups), so the thread that waits for a
// slot's "full" phase is not the one that waited for its previous phase, and an mbarrier wait names a phase by its
// parity only.  Without further ordering, a group that ran ahead of the slot's previous user could take that tile's
// unfinished phase for its own finished one and read the slot before anything had landed: one wrong tile in one
// row-block, seen about once in 10^5 launches, and only in streams where kernels of other kinds share the SMs and
// delay single copies (a launch that ended with "unspecified launch failure" in the same runs fits the barrier
// protocol going wrong after such a read).  A slot now alternates between two "full" barriers -- see the comment
// at the waits.  The kernels with one consuming thread per ring cannot meet this.
// Same bounded waits, table checks, launch flags and determinism as the other decode kernels; M <= 16.
#include "sm100_ptx.cuh"

namespace patch {

namespace dq {
constexpr int kRaw = 8;                                   // payload ring
constexpr int kBatch = 4;                                 // tiles requested per producer round
constexpr int kGroups = 3;                                // dequantising groups = operand stages in TMEM
constexpr int kThreads = 160 + 128 * kGroups;
constexpr uint32_t kRawBytes = kDenseQ4Bytes;             // slot size: the larger of the two payloads
constexpr uint32_t kXAtomBytes = 16 * 128, kXBytes = 2 * kXAtomBytes;
constexpr uint32_t kPartialBytes = 128 * 16 * 4;          // fp32 partial [128 rows][16 tokens]
constexpr uint32_t kXOffset = kPartialBytes;
constexpr uint32_t kRawOffset = kXOffset + kRaw * kXBytes;
constexpr uint32_t kBarrierOffset = kRawOffset + kRaw * kRawBytes;
constexpr uint32_t kSmemBytes = kBarrierOffset + 512 + 1024;
constexpr uint32_t kTmemCols = 256;                       // accumulator 16g, metadata 48 + 4g, operand stage 64 + 64g
constexpr uint32_t kPartialRowBytes = 16 * 4;
static_assert(64 + 64 * kGroups <= kTmemCols && 16 * kGroups <= 48 && 48 + 4 * kGroups <= 64, "TMEM columns");
static_assert(kRawBytes % 128 == 0 && kSparseQ4Bytes <= kRawBytes, "payload slots");
static_assert(2 * kSmemBytes <= 227 * 1024 && 3 * kSmemBytes > 228 * 1024 && 2 * kTmemCols <= 512, "two CTAs per SM, see above");
static_assert(2 * kRaw <= 16 && kGroups <= 8 && kThreads <= 1024, "barrier block, CTA size");
static_assert(32 % kBatch == 0 && kRaw % kBatch == 0 && 2 * kRaw / kBatch <= 8, "producer rounds");

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
// 16 registers per thread -> 32 lanes x 16 consecutive 32-bit columns (thread = lane)
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// D[tmem] (+)= A[tmem] * B[smem]: lane = row of A, a 32-bit column holds two consecutive K elements
__device__ __forceinline__ void mma_dense_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_sparse_ta(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t e_tmem,
                                              uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], [%1], %2, [%3], %4, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(e_tmem), "r"(idesc), "r"(accumulate) : "memory");
}

// true in one lane of the (converged) warp
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xFFFFFFFF;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(pred));
    return pred != 0;
}
// hardware barrier `id` over the 128 threads of a group
__device__ __forceinline__ void group_barrier(int id) { asm volatile("barrier.cta.sync %0, 128;" ::"r"(id) : "memory"); }

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

// Eight codes -> eight bf16 values in four registers.  s2 = the row's scale in both halves.
__device__ __forceinline__ void dequant_word(uint32_t w, __nv_bfloat162 s2, uint32_t* out) {
    const uint32_t kMagic = 0x43004300u;                         // bf16 128.0 twice: 128 + n in the low mantissa bits
    const uint32_t kBias = 0x43084308u;                          // bf16 136.0 twice
    const __nv_bfloat162 bias = *reinterpret_cast<const __nv_bfloat162*>(&kBias);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        uint32_t p;                                              // ((w >> 4j) & 0x000F000F) | magic in one instruction
        asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(p) : "r"(w >> (4 * j)), "r"(0x000F000Fu), "r"(kMagic));
        const __nv_bfloat162 v = __hmul2(__hsub2(*reinterpret_cast<const __nv_bfloat162*>(&p), bias), s2);
        out[j] = *reinterpret_cast<const uint32_t*>(&v);
    }
}
// 32 codes (16 bytes) -> 16 columns of this thread's TMEM lane
__device__ __forceinline__ void dequant_store16(uint4 cw, __nv_bfloat162 s2, uint32_t taddr) {
    uint32_t v[16];
    dequant_word(cw.x, s2, v);
    dequant_word(cw.y, s2, v + 4);
    dequant_word(cw.z, s2, v + 8);
    dequant_word(cw.w, s2, v + 12);
    tmem_st16(taddr, v);
}
}  // namespace dq

// YSTATIC: nothing in the overlap window touches Y (third launch promise): only the launch's first cluster waits for
// the preceding kernel, so that launches still complete in order; every other CTA stores Y and leaves when it is done.
template <bool WSTATIC, bool XSTATIC, bool YSTATIC>
__global__ void __launch_bounds__(dq::kThreads, 2)
decode_q4_kernel(const __grid_constant__ CUtensorMap tmap_x, const uint8_t* __restrict__ blob, uint64_t table_off,
                 uint32_t pay0_16, uint32_t end16, int TK, int S, int M, __nv_bfloat16* __restrict__ Y, int64_t ldy,
                 int* status_dev) {
    using namespace dq;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    // "Full" barriers come in two sets that a slot (a round) uses alternately -- see the consumers' waits for why.
    const uint32_t bar_raw_full = smem_base + kBarrierOffset;     // 2 kRaw x 8 B (16 reserved)
    const uint32_t bar_raw_empty = bar_raw_full + 128;            // kRaw x 8 B (16 reserved)
    const uint32_t bar_x_full = bar_raw_empty + 128;              // 2 kRaw / kBatch x 8 B (8 reserved)
    const uint32_t bar_op_empty = bar_x_full + 64;                // 8 x 8 B reserved
    const uint32_t bar_acc_full = bar_op_empty + 64;
    uint32_t* misc = reinterpret_cast<uint32_t*>(smem + kBarrierOffset + 392);
    uint32_t* tmem_slot = misc;
    volatile int* abort_flag = reinterpret_cast<volatile int*>(misc + 1);
    volatile uint32_t* slot_kind = misc + 2;                      // [kRaw] (392 + 8 + 64 <= 512)

    grid_launch_dependents();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t s = cluster_ctarank();
    const int tn = blockIdx.x / S;
    const int k0 = int(int64_t(s) * TK / S), k1 = int(int64_t(s + 1) * TK / S), n_tiles = k1 - k0;
    const int n_groups = n_tiles < kGroups ? n_tiles : kGroups;   // groups that get a tile: their accumulators count
    const TileDesc* table = reinterpret_cast<const TileDesc*>(blob + table_off) + int64_t(tn) * TK + k0;

    if (threadIdx.x == 32) {
        for (int i = 0; i < kRaw; ++i) {
            mbar_init(bar_raw_full + 8 * i, 1);
            mbar_init(bar_raw_full + 8 * (kRaw + i), 1);
            mbar_init(bar_raw_empty + 8 * i, 1);                   // the tile's MMAs (they follow the group's reads)
        }
        for (int i = 0; i < 2 * kRaw / kBatch; ++i) mbar_init(bar_x_full + 8 * i, 1);
        for (int i = 0; i < kGroups; ++i) mbar_init(bar_op_empty + 8 * i, 1);
        mbar_init(bar_acc_full, n_groups > 0 ? n_groups : 1);
        *abort_flag = 0;
        mbar_init_fence();
        tma_prefetch_map(&tmap_x);
    }
    if (warp == 0) tmem_alloc(smem_u32(tmem_slot), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = __shfl_sync(0xFFFFFFFFu, *tmem_slot, 0);

    if (warp == 0) {
        // ---------------- producer ----------------
        // Lanes 0 .. kBatch-1 each request one tile per round: the round's waits, barrier updates and copy
        // instructions are issued once for all of them (one lane per tile took ~1 000 cycles a tile, four times
        // what the tile's bytes take to arrive).  A round goes out when its last slot is free, so between
        // kRaw - kBatch and kRaw tiles are in flight.
        if constexpr (!WSTATIC) grid_dependency_wait();
        const uint64_t pol_w = l2_policy_evict_first(), pol_x = l2_policy_evict_last();
        TileDesc mine = TileDesc{0, 0, 0, 0};
        int issued = 0;
        bool ok = true;
        // payloads of the first kRaw tiles may be requested before the grid dependency is resolved (WSTATIC);
        // their activations follow once it is (unless XSTATIC)
        const int n_early = (WSTATIC && !XSTATIC) ? (n_tiles < kRaw ? n_tiles : kRaw) : 0;
#ifdef PATCH_FAULT_INJECTION
        // test build: a status word holding kInjectMagic makes CTA 0 announce sixteen bytes more than its first
        // slot will ever receive, so that a wait of this kernel runs out (see sm100_ptx.cuh)
        uint32_t inject_bytes = 0u;
        if (blockIdx.x == 0 && status_dev && *status_dev == kInjectMagic) {
            inject_bytes = 16u;
            __syncwarp();
            if (lane == 0) *status_dev = PATCH_OK;
        }
#else
        constexpr uint32_t inject_bytes = 0u;
#endif
        for (int base = 0; base < n_tiles && ok; base += kBatch) {
            if ((base & 31) == 0 && base + lane < n_tiles) mine = table[base + lane];
            const int i = base + lane, src = i & 31;               // kBatch divides 32: the round's entries sit in one load
            uint32_t kind = __shfl_sync(0xFFFFFFFFu, mine.kind, src);
            uint32_t off16 = __shfl_sync(0xFFFFFFFFu, mine.payload_off16, src);
            bool mine_ok = true;
            if (lane < kBatch) {
                const int slot = i % kRaw;
                // the slot's previous tile (also where this round has no tile for it: its X buffer is overwritten)
                if (i >= kRaw) mine_ok = mbar_wait_suspended(bar_raw_empty + 8 * slot, (uint32_t(i / kRaw) & 1u) ^ 1u, abort_flag, status_dev);
                if (mine_ok && i < n_tiles) {
                    sanitize_q4_tile(kind, off16, pay0_16, end16, status_dev);
                    const uint32_t wbytes = kind == PATCH_TILE_DENSE_Q4 ? kDenseQ4Bytes : kSparseQ4Bytes;
                    const uint32_t full = bar_raw_full + 8 * (i % (2 * kRaw));
                    slot_kind[slot] = kind;
                    mbar_expect_tx(full, wbytes + (i == 0 ? inject_bytes : 0u));
                    tma_bulk_load(smem_base + kRawOffset + slot * kRawBytes, blob + uint64_t(off16) * 16, wbytes, full, pol_w);
                }
            }
            ok = __all_sync(0xFFFFFFFFu, mine_ok);
            if (ok) issued = base + kBatch < n_tiles ? base + kBatch : n_tiles;
            // the round's activations: one copy of 2 kBatch atoms into the X buffers of its kBatch slots
            if (ok && lane == 0 && base >= n_early) {
                const uint32_t xb = bar_x_full + 8 * ((base / kBatch) % (2 * kRaw / kBatch));
                mbar_expect_tx(xb, kBatch * kXBytes);
                tma_tile_load_3d(smem_base + kXOffset + (base % kRaw) * kXBytes, &tmap_x, 0, 0, (k0 + base) * 2, xb, pol_x);
            }
            if (ok && base < n_early && base + kBatch >= n_early) {
                // the last early payload is on its way: now the activations of all early rounds
                grid_dependency_wait();
                if (lane * kBatch < n_early) {
                    const uint32_t xb = bar_x_full + 8 * lane;
                    mbar_expect_tx(xb, kBatch * kXBytes);
                    tma_tile_load_3d(smem_base + kXOffset + lane * kBatch * kXBytes, &tmap_x, 0, 0, (k0 + lane * kBatch) * 2, xb, pol_x);
                }
            }
        }
        if (lane == 0 && *abort_flag) {
            // drain: wait (bounded) until the copies this warp started have landed
            const uint64_t tstart = global_timer_ns();
            for (int j = issued > kRaw ? issued - kRaw : 0; j < issued; ++j) {
                const uint32_t bar = bar_raw_full + 8 * (j % (2 * kRaw)), parity = uint32_t(j / (2 * kRaw)) & 1u;
                while (!mbar_try_wait(bar, parity) && global_timer_ns() - tstart < kDrainLimitNs) {}
                const uint32_t xb = bar_x_full + 8 * ((j / kBatch) % (2 * kRaw / kBatch));
                while (!mbar_try_wait(xb, parity) && global_timer_ns() - tstart < kDrainLimitNs) {}
            }
        }
    } else if (warp >= 5) {
        // ---------------- group g: dequantise tile i into its operand stage, then multiply ----------------
        const int g = (warp - 5) >> 2;
        const bool issuer = ((warp - 5) & 3) == (g & 3);           // one warp of the group also issues its MMAs (the groups' issuers sit on different schedulers)
        const uint32_t quarter = warp & 3u, r = quarter * 32u + lane;         // tile row = TMEM lane
        const uint32_t a_tmem = tmem_base + 64u + 64u * uint32_t(g);
        const uint32_t a_lane = a_tmem + ((quarter * 32u) << 16);
        const uint32_t acc_tmem = tmem_base + 16u * uint32_t(g), e_tmem = tmem_base + 48u + 4u * uint32_t(g);
        constexpr uint32_t idesc_d = instr_desc(16, false), idesc_s = instr_desc(16, true);
        for (int i = g, n = 0; i < n_tiles; i += kGroups, ++n) {
            const int slot = i % kRaw;
            // One thread of the group waits for the tile's payload and for the MMAs that read the operand stage; the
            // other 127 wait on a hardware barrier, which costs no issue slots (24 polling warps did: a third of
            // all instructions).  The barrier also tells everyone if the wait was given up.
            bool failed = false;
            if (issuer && lane == 0) {
                // A slot's successive tiles belong to DIFFERENT groups (kRaw is not a multiple of kGroups), and a wait
                // names a phase by its parity only.  With one "full" barrier per slot, a group that ran ahead of the
                // slot's previous user -- whose payload may still be on its way when later ones have landed and been
                // multiplied -- took that tile's unfinished phase for its own finished one and read the slot too
                // early.  Hence two barriers per slot, used alternately: the phase before this tile's on ITS barrier is
                // the slot's tile before last, which was consumed before the previous one was even requested, and
                // that request precedes the request of this group's last tile.  The same for the rounds' activations.
                const uint32_t par = uint32_t(i / (2 * kRaw)) & 1u;
                failed = !mbar_wait_suspended(bar_raw_full + 8 * (i % (2 * kRaw)), par, abort_flag, status_dev);
                if (!failed)
                    failed = !mbar_wait_suspended(bar_x_full + 8 * ((i / kBatch) % (2 * kRaw / kBatch)), par, abort_flag, status_dev);
                if (!failed && n > 0)
                    failed = !mbar_wait_suspended(bar_op_empty + 8 * g, (uint32_t(n) & 1u) ^ 1u, abort_flag, status_dev);
            }
            if (barrier_any(failed, 1 + g, 128)) break;
            tc_fence_after();                                      // the MMAs that read this stage have completed
            const uint32_t sRaw = smem_base + kRawOffset + slot * kRawBytes;
            const uint8_t* raw = smem + kRawOffset + slot * kRawBytes;
            const uint4* codes = reinterpret_cast<const uint4*>(raw) + r;      // unit j of the row at codes[128 j]
            const bool dense = slot_kind[slot] == PATCH_TILE_DENSE_Q4;
            if (dense) {
                const uint32_t sb = reinterpret_cast<const uint16_t*>(raw + kDenseQ4CodeBytes)[r] * 0x00010001u;
                const __nv_bfloat162 s2 = *reinterpret_cast<const __nv_bfloat162*>(&sb);
#pragma unroll
                for (int j = 0; j < 4; ++j) dequant_store16(codes[128 * j], s2, a_lane + 16u * j);
            } else {
                const uint32_t sb = reinterpret_cast<const uint16_t*>(raw + kSparseQ4CodeBytes + kMetaBytes)[r] * 0x00010001u;
                const __nv_bfloat162 s2 = *reinterpret_cast<const __nv_bfloat162*>(&sb);
#pragma unroll
                for (int j = 0; j < 2; ++j) dequant_store16(codes[128 * j], s2, a_lane + 16u * j);
            }
            tmem_st_wait();
            tc_fence_before();
            group_barrier(8 + g);                                  // all four warps have written their rows
            if (issuer) {
                tc_fence_after();
                if (elect_one()) {
                    {
                        const uint64_t dB = desc_kmajor_sw128(smem_base + kXOffset + slot * kXBytes);
                        if (dense) {
#pragma unroll
                            for (int ks = 0; ks < 8; ++ks) {       // K = 16 per MMA: 8 columns of A, 32 B of every X row
                                const uint64_t b = dB + uint64_t(((ks >> 2) * kXAtomBytes + (ks & 3) * 32) >> 4);
                                mma_dense_ta(acc_tmem, a_tmem + 8u * ks, b, idesc_d, !(n == 0 && ks == 0));
                            }
                        } else {
                            tmem_copy_128x128b(e_tmem, desc_rows16(sRaw + kSparseQ4CodeBytes));
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks) {       // K = 32 per MMA: 16 kept values = 8 columns of A
                                const uint64_t b = dB + uint64_t(((ks >> 1) * kXAtomBytes + (ks & 1) * 64) >> 4);
                                mma_sparse_ta(acc_tmem, a_tmem + 8u * ks, b, e_tmem + (ks & 2), idesc_s | uint32_t(ks & 1),
                                              !(n == 0 && ks == 0));
                            }
                        }
                        mma_commit(bar_op_empty + 8 * g);
                        mma_commit(bar_raw_empty + 8 * slot);
                        if (i + kGroups >= n_tiles) mma_commit(bar_acc_full);    // the group's last tile
                    }
                }
                __syncwarp();
            }
        }
    } else {
        // ---------------- epilogue warps 1..4: sum of the groups' accumulators -> own shared memory ----------------
        const uint32_t quad = warp & 3u, row = quad * 32 + lane;
        bool ok = true;
        if (n_tiles > 0) {
            if (lane == 0) ok = mbar_wait_suspended(bar_acc_full, 0, abort_flag, status_dev);
            ok = __shfl_sync(0xFFFFFFFFu, ok ? 1 : 0, 0) != 0;
            tc_fence_after();
        }
        float acc[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) acc[j] = 0.0f;
        if (ok) {
            for (int gq = 0; gq < n_groups; ++gq) {                // ascending group: a fixed summation order
                uint32_t v[16];
                tmem_ld16(tmem_base + ((quad * 32u) << 16) + 16u * uint32_t(gq), v);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 16; ++j) acc[j] = gq == 0 ? __uint_as_float(v[j]) : acc[j] + __uint_as_float(v[j]);
            }
        }
        float4* dst = reinterpret_cast<float4*>(smem + row * kPartialRowBytes);
#pragma unroll
        for (int q = 0; q < 4; ++q) dst[q] = make_float4(acc[4 * q], acc[4 * q + 1], acc[4 * q + 2], acc[4 * q + 3]);
        tc_fence_before();
    }

    // every partial of the cluster is in place (on a timeout the partials are zeros or garbage, and status_dev says so)
    __syncthreads();
    dq::cluster_barrier();

    if (warp >= 1 && warp < 5) {
        // ---------------- reduction: this CTA finishes rows [128 s / S, 128 (s + 1) / S) ----------------
        const int e = threadIdx.x - 32;                            // 0..127
        const int rows = kTile / S;                                // S in {1, 2, 4, 8}
        const int n_out = rows * 4;                                // groups of four tokens
        if (!YSTATIC || int(blockIdx.x) < S) grid_dependency_wait();   // Y may be in use by the preceding kernel
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
        if (!YSTATIC || int(blockIdx.x) < S) grid_dependency_wait();   // every thread passes the dependency before the CTA exits
    }

    // nobody leaves while a peer may still read its shared memory
    tc_fence_before();
    __syncthreads();
    dq::cluster_barrier();
    if (warp == 0) tmem_dealloc(tmem_base, dq::kTmemCols);
}

template <bool WSTATIC, bool XSTATIC, bool YSTATIC = false>
static int launch_q4_t(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int M, int S,
                       __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream) {
    auto kern = decode_q4_kernel<WSTATIC, XSTATIC, YSTATIC>;
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
                     __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool wstatic, bool xstatic,
                     bool ystatic) {
    CUtensorMap map;
    int rc = make_x_chunk_tensor_map(&map, X, ldx, M, L->K, 16, 2 * dq::kBatch);
    if (rc) return rc;
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    // Split of K.  Independent of its predecessor (several GEMMs resident at once): as few, long CTAs as possible --
    // a CTA's set-up and drain cost about as much as a dozen tiles -- but at least 32 CTAs and at most 96 tiles each
    // (measured on the 24-GEMM step: 48 tiles 0.110 ms, 96 tiles 0.107 ms, 24 tiles 0.142 ms).
    int S = 1;
    while (S < 8 && (TN * S < 32 || TK > 96 * S)) S *= 2;
    while (S > 1 && S > TK) S /= 2;
    // Streaming alone once its predecessor is done: see below.
    if (!xstatic) {
        // alone on the GPU, two CTAs per SM: waves of CTAs x (tiles per CTA x ~0.35 us, 0.46 us where two CTAs share
        // an SM, + ~4 us of set-up, pipeline fill and reduction), over the power-of-two splits
        const int sms = sm_count();
        double best = 1e300;
        for (int s2 = 1; s2 <= 8 && s2 <= TK; s2 *= 2) {
            const int ctas = TN * s2, waves = (ctas + 2 * sms - 1) / (2 * sms);
            const double t = waves * (double((TK + s2 - 1) / s2) * (ctas > sms ? 0.46 : 0.35) + 4.0);
            if (t < best) { best = t; S = s2; }
        }
    }
    if (wstatic && xstatic && ystatic) return launch_q4_t<true, true, true>(map, L, packed, int(M), S, Y, ldy, status_dev, stream);
    if (wstatic && xstatic) return launch_q4_t<true, true>(map, L, packed, int(M), S, Y, ldy, status_dev, stream);
    if (wstatic) return launch_q4_t<true, false>(map, L, packed, int(M), S, Y, ldy, status_dev, stream);
    return launch_q4_t<false, false>(map, L, packed, int(M), S, Y, ldy, status_dev, stream);
}

}  // namespace patch
