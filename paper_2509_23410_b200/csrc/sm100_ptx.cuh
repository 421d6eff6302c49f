// Inline-PTX wrappers for sm_100a: mbarriers, TMA (bulk and tensor copies), tcgen05 (TMEM
// allocation, MMA, sparse MMA, copies, loads), programmatic dependent launch.
#pragma once
#include <cuda.h>
#include <stdint.h>
#include "patch_internal.cuh"

namespace patch {

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_init_fence() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// The same with a suspend-time hint: the thread may stay suspended in hardware for up to `hint_ns` (it is woken
// when the phase completes), so a long wait costs few issue slots.
__device__ __forceinline__ bool mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(hint_ns) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

#ifdef PATCH_FAULT_INJECTION
// Test build (libpatch_b200_fi.so, see build.py): waits give up after 300 us, and a launch of the stream-K decode
// kernel or of the 4-bit decode kernel whose status word holds kInjectMagic announces, in CTA 0, sixteen bytes more
// than its first stage will ever receive -- the one way the tests make a bounded wait run out.  Nothing faults,
// traps or spins for ever.
constexpr uint64_t kWaitLimitNs = 300000ull;
constexpr int kInjectMagic = 0x7E57;
#else
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s: far beyond any legitimate wait
#endif
constexpr uint64_t kDrainLimitNs = 2000000ull;    // 2 ms for copies already in flight

// Bounded wait.  Returns false if the wait was given up (own timeout, or another role of this
// CTA raised the abort flag).  On timeout the flag is raised and the status word is set.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                          int* status_dev) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 63u) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                if (status_dev) atomicCAS(status_dev, PATCH_OK, PATCH_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

// The same for a wait that is expected to last long (tens of microseconds): the thread sleeps between polls, so
// that its polling does not compete for the shared-memory port with the operand traffic of the running MMAs.
__device__ __forceinline__ bool mbar_wait_relaxed(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                  int* status_dev) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t spin = 1;; ++spin) {
        __nanosleep(200);
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 15u) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                if (status_dev) atomicCAS(status_dev, PATCH_OK, PATCH_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

// Bounded wait for warps that share their issue port with busy ones: suspended in hardware between polls.
__device__ __forceinline__ bool mbar_wait_suspended(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                    int* status_dev) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait_hint(bar, parity, 20000u)) return true;
        if ((spin & 3u) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                *abort_flag = 1;
                if (status_dev) atomicCAS(status_dev, PATCH_OK, PATCH_ERR_TIMEOUT);
                return false;
            }
        }
    }
}

// Hardware barrier `id` over `threads` threads of the CTA that also ORs a predicate (the same decision in all of them).
__device__ __forceinline__ bool barrier_any(bool pred, int id, int threads) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\t"
        "barrier.cta.red.or.pred p, %2, %3, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(out) : "r"(uint32_t(pred)), "r"(id), "r"(threads) : "memory");
    return out != 0;
}
// A group of warps waits for an mbarrier: the thread with `poller` set polls it (sleeping in between), the others
// wait on hardware barrier `id`, which costs the shared-memory port nothing while the MMAs run.  False if given up.
__device__ __forceinline__ bool group_wait(uint32_t bar, uint32_t parity, bool poller, int id, int threads,
                                           volatile int* abort_flag, int* status_dev) {
    bool failed = false;
    if (poller) failed = !mbar_wait_relaxed(bar, parity, abort_flag, status_dev);
    return !barrier_any(failed, id, threads);
}

// L2 eviction policies for streamed-once (weights) and reused (activations) data.
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// 1-D bulk copy global -> shared, completion counted on an mbarrier.
__device__ __forceinline__ void tma_bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar,
                                              uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(policy) : "memory");
}
// 2-D tiled copy global -> shared through a tensor map.
__device__ __forceinline__ void tma_tile_load(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar,
                                              uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar), "l"(policy) : "memory");
}
// 3-D tiled copy
__device__ __forceinline__ void tma_tile_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_prefetch_map(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], dense bf16, fp32 accumulate
__device__ __forceinline__ void mma_dense(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// same with A stored 2:4-compressed and its position metadata in TMEM
__device__ __forceinline__ void mma_sparse(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t e_tmem,
                                           uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(e_tmem), "r"(idesc), "r"(accumulate) : "memory");
}
// arrive on an mbarrier once all previously issued tcgen05 operations of this thread completed
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// shared memory (128 rows x 16 bytes) -> TMEM (128 lanes x 4 columns)
__device__ __forceinline__ void tmem_copy_128x128b(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::1.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns -> 16 registers per thread (thread = lane)
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// ---- CTA pairs (cluster of two CTAs on the two SMs of one TPC; cta_group::2 instructions) ----
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t saddr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(saddr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// 2-D tiled copy global -> own shared memory whose completion is counted on a barrier that may live in the
// other CTA of the pair (`bar` is a shared::cluster address).  No multicast: every CTA fetches its own box.
__device__ __forceinline__ void tma_tile_load_pair(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar,
                                                   uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar), "l"(policy) : "memory");
}
// Tensor memory of both CTAs of the pair, same columns in each; executed by one warp of EACH CTA.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// 256 x N x 16 (dense) / 256 x N x 32 (2:4): each CTA supplies its 128 rows of A and N/2 rows of B and
// receives its 128 rows of D; issued by ONE thread of the leader CTA (rank 0), same addresses in both CTAs.
__device__ __forceinline__ void mma_dense_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_sparse_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t e_tmem,
                                                uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
        "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(e_tmem), "r"(idesc), "r"(accumulate) : "memory");
}
// each CTA's 128 rows x 16 B of shared memory -> its own TMEM, 4 columns
__device__ __forceinline__ void tmem_copy_pair_128x128b(uint32_t taddr, uint64_t sdesc) {
    asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
// one arrival on the barrier at this shared-memory offset in BOTH CTAs once all tcgen05 operations issued so
// far by this thread have completed
__device__ __forceinline__ void mma_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(uint16_t(3)) : "memory");
}
// Instruction descriptor of the pair MMA: bf16 x bf16 -> fp32, K-major operands, M = 256, N = n_tok.
__host__ __device__ constexpr uint32_t instr_desc_pair(int n_tok, bool sparse) {
    return (sparse ? (1u << 2) : 0u) | (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(n_tok >> 3) << 17) |
           (uint32_t(256 >> 4) << 24);
}

// programmatic dependent launch: allow the next kernel to start / wait for the previous one
__device__ __forceinline__ void grid_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Shared-memory matrix descriptor, K-major operand in 128-byte-swizzled atoms
// (8 rows x 128 B = 1024 B per row group): start address, stride between row groups, sm_100
// descriptor version, swizzle mode.
__device__ __forceinline__ uint64_t desc_kmajor_sw128(uint32_t saddr) {
    return uint64_t((saddr & 0x3FFFFu) >> 4) | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) |
           (uint64_t(1) << 46) | (uint64_t(2) << 61);
}
// Unswizzled 128 rows x 16 B block (8-row groups of 128 B): source of the metadata copy.
__device__ __forceinline__ uint64_t desc_rows16(uint32_t saddr) {
    return uint64_t((saddr & 0x3FFFFu) >> 4) | (uint64_t(128 >> 4) << 16) | (uint64_t(128 >> 4) << 32) |
           (uint64_t(1) << 46);
}

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n_tok.
__host__ __device__ constexpr uint32_t instr_desc(int n_tok, bool sparse) {
    return (sparse ? (1u << 2) : 0u) | (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(n_tok >> 3) << 17) |
           (uint32_t(128 >> 4) << 24);
}

// Issues the MMAs of one 128 x 128 weight tile held in shared memory at sW (payload image)
// against the activation tile at sX (two K-halves of x_atom_bytes each).
//   dense: eight tcgen05.mma, K = 16 each (32 B of every operand row per step)
//   2:4  : metadata block -> TMEM columns e_tmem..e_tmem+3, then four tcgen05.mma.sp, K = 32 each
//          (32 B of A, 64 B of B per row); metadata column ks is addressed as the even column
//          in the TMEM address plus the column's parity in the descriptor's selector field.
template <int N_TOK>
__device__ __forceinline__ void issue_tile_mma(uint32_t kind, uint32_t sW, uint32_t sX, uint32_t x_atom_bytes,
                                               uint32_t acc_tmem, uint32_t e_tmem, bool first) {
    constexpr uint32_t idesc_d = instr_desc(N_TOK, false), idesc_s = instr_desc(N_TOK, true);
    const uint64_t dA = desc_kmajor_sw128(sW), dB = desc_kmajor_sw128(sX);
    if (kind == PATCH_TILE_DENSE) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint64_t a = dA + uint64_t(((ks >> 2) * kAtomBytes + (ks & 3) * 32) >> 4);
            const uint64_t b = dB + uint64_t(((ks >> 2) * x_atom_bytes + (ks & 3) * 32) >> 4);
            mma_dense(acc_tmem, a, b, idesc_d, !(first && ks == 0));
        }
    } else {
        tmem_copy_128x128b(e_tmem, desc_rows16(sW + kAtomBytes));
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            const uint64_t a = dA + uint64_t((ks * 32) >> 4);
            const uint64_t b = dB + uint64_t(((ks >> 1) * x_atom_bytes + (ks & 1) * 64) >> 4);
            mma_sparse(acc_tmem, a, b, e_tmem + (ks & 2), idesc_s | uint32_t(ks & 1), !(first && ks == 0));
        }
    }
}

// Same with the token count of the MMA (its N dimension) chosen at run time.
__device__ __forceinline__ void issue_tile_mma_n(uint32_t kind, uint32_t sW, uint32_t sX, uint32_t x_atom_bytes,
                                                 uint32_t acc_tmem, uint32_t e_tmem, bool first, uint32_t n_tok) {
    const uint32_t idesc_d = instr_desc(0, false) | ((n_tok >> 3) << 17);
    const uint32_t idesc_s = idesc_d | (1u << 2);
    const uint64_t dA = desc_kmajor_sw128(sW), dB = desc_kmajor_sw128(sX);
    if (kind == PATCH_TILE_DENSE) {
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            const uint64_t a = dA + uint64_t(((ks >> 2) * kAtomBytes + (ks & 3) * 32) >> 4);
            const uint64_t b = dB + uint64_t(((ks >> 2) * x_atom_bytes + (ks & 3) * 32) >> 4);
            mma_dense(acc_tmem, a, b, idesc_d, !(first && ks == 0));
        }
    } else {
        tmem_copy_128x128b(e_tmem, desc_rows16(sW + kAtomBytes));
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            const uint64_t a = dA + uint64_t((ks * 32) >> 4);
            const uint64_t b = dB + uint64_t(((ks >> 1) * x_atom_bytes + (ks & 1) * 64) >> 4);
            mma_sparse(acc_tmem, a, b, e_tmem + (ks & 2), idesc_s | uint32_t(ks & 1), !(first && ks == 0));
        }
    }
}

// Epilogue helper.  A warp holds a 32-row x 16-token fp32 fragment (thread = out-feature row,
// v[j] = token j) and Y is [token][out-feature]: storing straight from registers would be sixteen
// 2-byte stores per thread.  The fragment is converted to bf16, transposed through 1 KB of this
// warp's shared memory and written as two 16-byte vectors per thread (64 contiguous bytes per token).
//   stage   this warp's 1 KB staging buffer      y   &Y[first token of the fragment][first row of the warp]
__device__ __forceinline__ void store_fragment_transposed(const uint32_t (&v)[16], uint8_t* stage, int lane,
                                                          __nv_bfloat16* y, int64_t ldy, int n_valid) {
#pragma unroll
    for (int j = 0; j < 16; ++j)
        *reinterpret_cast<__nv_bfloat16*>(stage + j * 64 + lane * 2) = __float2bfloat16_rn(__uint_as_float(v[j]));
    __syncwarp();
#pragma unroll
    for (int p = 0; p < 2; ++p) {
        const int tok = p * 8 + (lane >> 2), chunk = lane & 3;
        const uint4 q = *reinterpret_cast<const uint4*>(stage + tok * 64 + chunk * 16);
        if (tok < n_valid) *reinterpret_cast<uint4*>(y + int64_t(tok) * ldy + chunk * 8) = q;
    }
    __syncwarp();
}

// Host: tensor map over X [M x ldx] bf16 with a box of 64 columns (128 B) x n_tok rows,
// 128-byte swizzle, zero fill outside the matrix.
int make_x_tensor_map(CUtensorMap* map, const __nv_bfloat16* X, int64_t ldx, int64_t M, int64_t K, int n_tok);
// Host: the same matrix as (column in a 64-column chunk, token row, chunk) with a box of `chunks` chunks: one copy
// brings `chunks` consecutive atoms of n_tok rows x 128 B.
int make_x_chunk_tensor_map(CUtensorMap* map, const __nv_bfloat16* X, int64_t ldx, int64_t M, int64_t K, int n_tok, int chunks);
// Host: tensor map over a packed blob seen as rows of 256 bytes, box = `box_rows` whole rows, no swizzle: a
// tiled copy at row (byte offset / 256) lands in shared memory exactly like a linear copy of box_rows * 256 bytes.
int make_blob_tensor_map(CUtensorMap* map, const uint8_t* blob, uint64_t total_bytes, int box_rows);

// Row-block / cluster split-K schedule for M <= 64 (gemm_decode_cluster_sm100.cu), used for GEMMs the caller
// declared independent of their predecessor (`map`: X tensor map with a box of `n_tok` token rows).
int launch_decode_cluster(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int M, int n_tok,
                          __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool wstatic,
                          bool xstatic, bool ystatic = false);
int decode_cluster_split(int TN, int TK);     // cluster size of the row-block schedule for independent GEMMs
int launch_decode_cluster_gated(const CUtensorMap& map, const patch_layout_t* L, const uint8_t* packed, int M,
                                __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream, bool xstatic = true);


}  // namespace patch
