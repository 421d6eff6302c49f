// Standalone probe (not part of the library): tcgen05 dense vs 2:4-sparse MMA rate with operands resident
// in shared memory, one CTA per SM, cta_group::1.  Build: python -m paper_2509_23410_b200.build --probe
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

int main() {
    long long* out; cudaMalloc(&out, 148 * 8);
    cudaFuncSetAttribute(rate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
    const int iters = 2000;
    for (int n_tok : {64, 128, 240, 256}) for (int mode = 0; mode < 3; ++mode) {
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
    return 0;
}
