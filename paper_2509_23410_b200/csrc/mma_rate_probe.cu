// Standalone probe (not part of the library): tcgen05 dense vs 2:4-sparse MMA rate with operands resident
// in shared memory, one CTA per SM: cta_group::1, and cta_group::2 (a CTA pair computes 256 rows, each
// CTA holding its own 128 weight rows and half of the tokens).  Build: python -m paper_2509_23410_b200.build --probe
#include <cstdio>
#include <cuda_runtime.h>
#include "sm100_ptx.cuh"
using namespace patch;
int patch::make_x_tensor_map(CUtensorMap*, const __nv_bfloat16*, int64_t, int64_t, int64_t, int) { return 0; }

__global__ void __launch_bounds__(128) rate_kernel(int mode, int n_tok, int iters, long long* out) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - smem_u32(smem_raw));
    __shared__ uint32_t tmem_slot; __shared__ __align__(8) unsigned long long bar;
    const int warp = threadIdx.x >> 5;
    // zero operands (values irrelevant; metadata must be legal codes: use 0x4 nibble = (0,1))
    for (int i = threadIdx.x; i < (32768 + 65536) / 4; i += 128) ((uint32_t*)smem)[i] = 0;
    for (int i = threadIdx.x; i < 512; i += 128) ((uint32_t*)(smem + 16384))[i] = 0x44444444u;
    if (threadIdx.x == 0) { mbar_init(smem_u32(&bar), 1); mbar_init_fence(); }
    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 512);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before(); __syncthreads(); tc_fence_after();
    const uint32_t tm = tmem_slot;
    long long t0 = 0, t1 = 0;
    if (threadIdx.x == 32) {
        const uint32_t sW = base, sX = base + 32768, xat = n_tok * 128;
        t0 = clock64();
        for (int it = 0; it < iters; ++it) {
            if (mode == 0) issue_tile_mma_n(PATCH_TILE_DENSE, sW, sX, xat, tm, tm + 496, it == 0, n_tok);
            else if (mode == 1) issue_tile_mma_n(PATCH_TILE_SPARSE_2_4, sW, sX, xat, tm, tm + 496, it == 0, n_tok);
            else { // two accumulators alternating (dense)
                issue_tile_mma_n(PATCH_TILE_DENSE, sW, sX, xat, tm + (it & 1) * 256, tm + 496, it < 2, n_tok);
            }
        }
        mma_commit(smem_u32(&bar));
        for (long long spin = 0; spin < (1ll << 26) && !mbar_try_wait(smem_u32(&bar), 0); ++spin) {}   // bounded
        t1 = clock64();
        out[blockIdx.x] = t1 - t0;
    }
    tc_fence_before(); __syncthreads();
    if (warp == 0) tmem_dealloc(tm, 512);
}

// CTA pair: M = 256 MMAs issued by the leader CTA; each CTA supplies its own A tile and n_tok/2 rows of B.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(128) pair_kernel(int sparse, int n_tok, int iters, long long* out) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - smem_u32(smem_raw));
    __shared__ uint32_t tmem_slot; __shared__ __align__(8) unsigned long long bar;
    const int warp = threadIdx.x >> 5;
    uint32_t rank; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    for (int i = threadIdx.x; i < (32768 + 65536) / 4; i += 128) ((uint32_t*)smem)[i] = 0;
    for (int i = threadIdx.x; i < 512; i += 128) ((uint32_t*)(smem + 16384))[i] = 0x44444444u;
    if (threadIdx.x == 0) { mbar_init(smem_u32(&bar), 1); mbar_init_fence(); }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    tc_fence_before(); __syncthreads(); cluster_sync_all(); tc_fence_after();
    const uint32_t tm = tmem_slot;
    if (rank == 0 && threadIdx.x == 32) {
        const uint32_t sW = base, sX = base + 32768, xat = (n_tok / 2) * 128;
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(n_tok >> 3) << 17) | (uint32_t(256 >> 4) << 24);
        const uint64_t dA = desc_kmajor_sw128(sW), dB = desc_kmajor_sw128(sX);
        const uint32_t e_tmem = tm + 496;
        const long long t0 = clock64();
        for (int it = 0; it < iters; ++it) {
            if (!sparse) {
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint64_t a = dA + uint64_t(((ks >> 2) * kAtomBytes + (ks & 3) * 32) >> 4);
                    const uint64_t b = dB + uint64_t(((ks >> 2) * xat + (ks & 3) * 32) >> 4);
                    const uint32_t acc = !(it == 0 && ks == 0);
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                                 "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                 ::"r"(tm), "l"(a), "l"(b), "r"(idesc), "r"(acc) : "memory");
                }
            } else {
                asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(e_tmem), "l"(desc_rows16(sW + kAtomBytes)) : "memory");
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint64_t a = dA + uint64_t((ks * 32) >> 4);
                    const uint64_t b = dB + uint64_t(((ks >> 1) * xat + (ks & 1) * 64) >> 4);
                    const uint32_t acc = !(it == 0 && ks == 0);
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %5, 0;\n\t"
                                 "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n\t}"
                                 ::"r"(tm), "l"(a), "l"(b), "r"(e_tmem + (ks & 2)), "r"(idesc | (1u << 2) | uint32_t(ks & 1)), "r"(acc) : "memory");
                }
            }
        }
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bar)) : "memory");
        for (long long spin = 0; spin < (1ll << 26) && !mbar_try_wait(smem_u32(&bar), 0); ++spin) {}   // bounded
        out[blockIdx.x >> 1] = clock64() - t0;
    }
    tc_fence_before(); __syncthreads(); cluster_sync_all();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(512) : "memory");
}

int main() {
    long long* out; cudaMalloc(&out, 148 * 8);
    cudaFuncSetAttribute(rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    const int iters = 2000;
    for (int n_tok : {32, 64, 128, 240, 256}) for (int mode = 0; mode < 3; ++mode) {
        for (int rep = 0; rep < 2; ++rep) {
            cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
            cudaEventRecord(e0);
            rate_kernel<<<148, 128, 100 * 1024>>>(mode, n_tok, iters, out);
            cudaEventRecord(e1); cudaEventSynchronize(e1);
            float ms; cudaEventElapsedTime(&ms, e0, e1);
            long long h[148]; cudaMemcpy(h, out, sizeof h, cudaMemcpyDeviceToHost);
            if (rep == 1) {
                double clk = double(h[0]) / iters;
                double flops = 2.0 * 128 * n_tok * 128 * iters * 148;
                printf("n_tok=%3d mode=%s: %.0f clk per 128x%dx128 tile-step, kernel %.3f ms -> %.0f TFLOP/s (dense-equivalent)  err=%d\n",
                       n_tok, mode == 0 ? "dense " : mode == 1 ? "sparse" : "dense2", clk, n_tok, ms, flops / ms / 1e9, (int)cudaGetLastError());
            }
        }
    }
    cudaFuncSetAttribute(pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    for (int n_tok : {32, 64, 128, 224, 256}) for (int sparse = 0; sparse < 2; ++sparse) {
        for (int rep = 0; rep < 2; ++rep) {
            cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
            cudaEventRecord(e0);
            pair_kernel<<<148, 128, 100 * 1024>>>(sparse, n_tok, iters, out);
            cudaEventRecord(e1); cudaEventSynchronize(e1);
            float ms; cudaEventElapsedTime(&ms, e0, e1);
            long long h[74]; cudaMemcpy(h, out, sizeof h, cudaMemcpyDeviceToHost);
            if (rep == 1) {
                double clk = double(h[0]) / iters;
                double flops = 2.0 * 256 * n_tok * 128 * iters * 74;
                printf("pair n_tok=%3d %s: %.0f clk per 256x%dx128 step, kernel %.3f ms -> %.0f TFLOP/s (dense-equivalent)  err=%d\n",
                       n_tok, sparse ? "sparse" : "dense ", clk, n_tok, ms, flops / ms / 1e9, (int)cudaGetLastError());
            }
        }
    }
    return 0;
}
