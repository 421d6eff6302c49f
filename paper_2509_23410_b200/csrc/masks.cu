// Mask learning kernels: the Gumbel-softmax soft masks of Eq. 2-4 applied to W, the per-matrix
// sums the regularisers of Eq. 5 need, and the hard masks Algorithm 1 reads off the logits after
// training.  All of it is elementwise work over W and the 2:4 logits.
//
// Per element of W the soft-mask kernel reads 2 B of W and 6 B of logits (six fp32 logits per
// group of four) and writes 2 B of masked weight: 10 B.  The hard-mask kernel reads 24 B and
// writes 1 B per group.  Both stream every byte exactly once.
#include <cmath>
#include "patch_internal.cuh"

namespace patch {

// ---------------------------------------------------------------------------------------------
// Gumbel noise (Eq. 1): z = -log(-log(u)), u uniform in (0, 1) from a counter-based generator.
// One 64-bit mix of (seed, stream, idx / 2) serves the counters 2i and 2i + 1: the even one takes
// the top 23 bits, the odd one bits 9..31; the 23 bits are centred in their cell.

constexpr uint64_t kGolden = 0x9E3779B97F4A7C15ull, kStreamStep = 0xD1B54A32D192ED03ull;

// finaliser of the mix; its argument is seed + kGolden * (idx / 2 + 1) + kStreamStep * stream
__device__ __forceinline__ uint64_t mix_final(uint64_t x) {
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

// -log2(-ln(u)) for u = (bits + 0.5) / 2^23.  With v = 1 - u, -ln(u) = -ln(1 - v): a short series
// where v is small (there the hardware logarithm of a number next to 1 has no relative accuracy
// left, and these are the large noise values that decide a Gumbel-max draw), the hardware
// logarithm elsewhere.  u and v are built from the bits without an integer-to-float conversion:
// 1.b (binary) minus 1 is b / 2^23 exactly, and adding 2^-24 centres it in its cell; both stay
// within 24 significant bits, so both are exact.
__device__ __forceinline__ float lg2_approx(float x) {   // log2 of a normal positive number
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float gumbel_log2(uint32_t bits) {
    const float u = (__uint_as_float(0x3F800000u | bits) - 1.0f) + 5.9604645e-8f;
    const float v = (__uint_as_float(0x3F800000u | (bits ^ 0x7FFFFFu)) - 1.0f) + 5.9604645e-8f;
    const float series = v * (1.0f + v * (0.5f + v * 0.33333334f));      // v < 2^-6: the next term is below 2^-20 relative
    const float direct = -0.69314718f * lg2_approx(u);
    return -lg2_approx(v < 0.015625f ? series : direct);
}

__device__ __forceinline__ float ex2_approx(float x) {   // 2^x; results below 2^-126 flush to zero
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// GS(p; tau, kappa) over n classes in base-2 form: GS_k = 2^(a_k - max a) / sum, with
// a_k = (kappa p_k + z_k) / tau * log2(e) = p_k * sp + zl_k * sz, where zl_k = -log2(-ln u_k),
// sp = kappa log2(e) / tau and sz = 1 / tau (z = zl * ln 2, and ln 2 * log2(e) = 1).
// Leaves the unnormalised terms in a[] and returns 1 / sum.
template <int NCLS>
__device__ __forceinline__ float softmax2_terms(float (&a)[NCLS]) {
    float top = a[0];
#pragma unroll
    for (int k = 1; k < NCLS; ++k) top = fmaxf(top, a[k]);
    float sum = 0.f;
#pragma unroll
    for (int k = 0; k < NCLS; ++k) { a[k] = ex2_approx(a[k] - top); sum += a[k]; }
    float inv;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(sum));      // sum is in [1, NCLS]
    return inv;
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }
// two floats -> two bf16 (round to nearest even) in one word, `lo` in the low half
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

// One CTA per 128 x 128 tile of W; thread (r, u) of an iteration owns the 16 elements (four
// groups) [16u, 16u + 16) of tile row r.  The tile's soft value Mt_tile is computed once per CTA.
// partials[t] = { sum Mt, ||W||_0, ||Mt (.) W||^2, ||W||^2 } over the tile.
template <bool NOISE, bool WRITE_MT>
__global__ void __launch_bounds__(256)
soft_mask_kernel(const uint16_t* __restrict__ W, int64_t ldw, const float* __restrict__ P_tile,
                 const float* __restrict__ P24, int TK, int64_t G, float sp, float sz, uint64_t seed,
                 uint64_t candidate_step /* kGolden * (G / 2) */, uint16_t* __restrict__ Wt, int64_t ldo, float* __restrict__ Mt, int64_t ldm,
                 double* __restrict__ partials) {
    __shared__ float s_mt, s_omt;
    __shared__ double s_red[8][4];
    const int t = blockIdx.x, tn = t / TK, tk = t - tn * TK;
    if (threadIdx.x == 0) {
        float a[2] = {P_tile[t] * sp, 0.f};
        if (NOISE) {
            const uint64_t h = mix_final(seed + kGolden * (uint64_t(t) + 1));   // stream 0, counters 2t (dense class) and 2t + 1
            a[0] += gumbel_log2(uint32_t(h >> 41)) * sz;
            a[1] += gumbel_log2(uint32_t(h >> 9) & 0x7FFFFFu) * sz;
        }
        const float inv = softmax2_terms(a);
        s_mt = a[0] * inv;
        s_omt = a[1] * inv;     // 1 - Mt_tile as the other softmax term: no cancellation when Mt_tile is next to 1
    }
    __syncthreads();
    const float mt = s_mt, one_minus_mt = s_omt;
    float acc_mw2 = 0.f, acc_w2 = 0.f;
    uint32_t acc_nz = 0;
#pragma unroll 1
    for (int it = 0; it < 4; ++it) {
        const uint32_t idx = it * 256 + threadIdx.x, r = idx >> 3, u = idx & 7u;
        const int64_t n = int64_t(tn) * kTile + r;
        const int64_t grp = n * (int64_t(TK) * 32) + tk * 32 + u * 4;     // first of this thread's four groups
        const uint16_t* src = W + n * ldw + int64_t(tk) * kTile + u * 16;
        const uint4 wa = *reinterpret_cast<const uint4*>(src), wb = *reinterpret_cast<const uint4*>(src + 8);
        float a[4][6];      // a[group][candidate]
        // stream 1, counters c*G + grp .. + 3 (c*G and grp are even): the mix argument of candidate c is the one of
        // candidate 0 plus c * kGolden * (G / 2), and the second pair of groups adds kGolden once more
        uint64_t x0 = seed + kStreamStep + kGolden * (uint64_t(grp >> 1) + 1);
#pragma unroll
        for (int c = 0; c < 6; ++c) {
            const float4 p = *reinterpret_cast<const float4*>(P24 + int64_t(c) * G + grp);
            a[0][c] = p.x * sp; a[1][c] = p.y * sp; a[2][c] = p.z * sp; a[3][c] = p.w * sp;
            if (NOISE) {
                const uint64_t h0 = mix_final(x0), h1 = mix_final(x0 + kGolden);
                x0 += candidate_step;
                a[0][c] += gumbel_log2(uint32_t(h0 >> 41)) * sz;
                a[1][c] += gumbel_log2(uint32_t(h0 >> 9) & 0x7FFFFFu) * sz;
                a[2][c] += gumbel_log2(uint32_t(h1 >> 41)) * sz;
                a[3][c] += gumbel_log2(uint32_t(h1 >> 9) & 0x7FFFFFu) * sz;
            }
        }
        const uint32_t in[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
        uint32_t out[8];
        float mvals[16];
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            // (1 - Mt_tile) / sum: normalisation of the softmax and the factor of Eq. 4 in one
            const float scale = one_minus_mt * softmax2_terms(a[g]);
            // GS x S: position j is kept by the candidates whose pair contains j
            const float m24[4] = {a[g][0] + a[g][1] + a[g][2], a[g][0] + a[g][3] + a[g][4],
                                  a[g][1] + a[g][3] + a[g][5], a[g][2] + a[g][4] + a[g][5]};
            float mw[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t pair = in[2 * g + (j >> 1)];               // a bf16 is the upper half of its fp32
                const float w = __uint_as_float(j & 1 ? pair & 0xFFFF0000u : pair << 16);
                const float m = fmaf(scale, m24[j], mt);                   // Eq. 4
                mw[j] = m * w;
                mvals[4 * g + j] = m;
                acc_nz += w != 0.0f;                                       // -0 is zero
                acc_mw2 = fmaf(mw[j], mw[j], acc_mw2);
                acc_w2 = fmaf(w, w, acc_w2);
            }
            out[2 * g] = pack_bf16x2(mw[0], mw[1]);
            out[2 * g + 1] = pack_bf16x2(mw[2], mw[3]);
        }
        uint16_t* dst = Wt + n * ldo + int64_t(tk) * kTile + u * 16;
        *reinterpret_cast<uint4*>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
        *reinterpret_cast<uint4*>(dst + 8) = make_uint4(out[4], out[5], out[6], out[7]);
        if (WRITE_MT) {
            float* md = Mt + n * ldm + int64_t(tk) * kTile + u * 16;
#pragma unroll
            for (int q = 0; q < 4; ++q)
                *reinterpret_cast<float4*>(md + 4 * q) = make_float4(mvals[4 * q], mvals[4 * q + 1], mvals[4 * q + 2], mvals[4 * q + 3]);
        }
    }
    // fixed-order reduction: lanes by shuffle, warps in index order
    // sum Mt needs no pass over the elements: every candidate keeps two of four, so a group's 2:4 part sums
    // to 2 and the tile's soft mask to 128 * 128 * (Mt_tile + (1 - Mt_tile) / 2); thread 0 contributes it
    double v[4] = {threadIdx.x == 0 ? 16384.0 * double(mt) + 8192.0 * (1.0 - double(mt)) : 0.0,
                   double(acc_nz), double(acc_mw2), double(acc_w2)};
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v[q] += __shfl_xor_sync(0xFFFFFFFFu, v[q], off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0)
#pragma unroll
        for (int q = 0; q < 4; ++q) s_red[warp][q] = v[q];
    __syncthreads();
    if (threadIdx.x < 4) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += s_red[w][threadIdx.x];
        partials[int64_t(t) * 4 + threadIdx.x] = s;
    }
}

// Gradient with respect to the logits of  F = sum Gw Mt W + c1 sum Mt - (c2 / 2) sum (Mt W)^2  ("Update
// P_tile, P_2:4 via backpropagation", Algorithm 1), the forward recomputed on the fly with the same noise.
// Same work split as the forward: one CTA per tile, four groups per thread and iteration.  Per element it
// reads 2 B of W, 2 B of Gw and 6 B of logits and writes 6 B of logit gradient.
template <bool NOISE>
__global__ void __launch_bounds__(256)
soft_mask_backward_kernel(const uint16_t* __restrict__ W, int64_t ldw, const uint16_t* __restrict__ Gw, int64_t ldg,
                          const float* __restrict__ P_tile, const float* __restrict__ P24, int TK, int64_t G, float sp,
                          float sz, float kappa_over_tau, uint64_t seed, uint64_t candidate_step, float c1, float c2,
                          float* __restrict__ gP_tile, float* __restrict__ gP24) {
    __shared__ float s_mt, s_omt;
    __shared__ double s_red[8];
    const int t = blockIdx.x, tn = t / TK, tk = t - tn * TK;
    if (threadIdx.x == 0) {
        float a[2] = {P_tile[t] * sp, 0.f};
        if (NOISE) {
            const uint64_t h = mix_final(seed + kGolden * (uint64_t(t) + 1));
            a[0] += gumbel_log2(uint32_t(h >> 41)) * sz;
            a[1] += gumbel_log2(uint32_t(h >> 9) & 0x7FFFFFu) * sz;
        }
        const float inv = softmax2_terms(a);
        s_mt = a[0] * inv;
        s_omt = a[1] * inv;     // 1 - Mt_tile as the other softmax term: no cancellation when Mt_tile is next to 1
    }
    __syncthreads();
    const float mt = s_mt, one_minus_mt = s_omt;
    float acc_gmt = 0.f;     // sum of gM (1 - Mt_2:4) over this thread's elements
#pragma unroll 1
    for (int it = 0; it < 4; ++it) {
        const uint32_t idx = it * 256 + threadIdx.x, r = idx >> 3, u = idx & 7u;
        const int64_t n = int64_t(tn) * kTile + r;
        const int64_t grp = n * (int64_t(TK) * 32) + tk * 32 + u * 4;
        const uint16_t* src = W + n * ldw + int64_t(tk) * kTile + u * 16;
        const uint16_t* gsrc = Gw + n * ldg + int64_t(tk) * kTile + u * 16;
        const uint4 wa = *reinterpret_cast<const uint4*>(src), wb = *reinterpret_cast<const uint4*>(src + 8);
        const uint4 ga = *reinterpret_cast<const uint4*>(gsrc), gb = *reinterpret_cast<const uint4*>(gsrc + 8);
        float a[4][6];
        uint64_t x0 = seed + kStreamStep + kGolden * (uint64_t(grp >> 1) + 1);
#pragma unroll
        for (int c = 0; c < 6; ++c) {
            const float4 p = *reinterpret_cast<const float4*>(P24 + int64_t(c) * G + grp);
            a[0][c] = p.x * sp; a[1][c] = p.y * sp; a[2][c] = p.z * sp; a[3][c] = p.w * sp;
            if (NOISE) {
                const uint64_t h0 = mix_final(x0), h1 = mix_final(x0 + kGolden);
                x0 += candidate_step;
                a[0][c] += gumbel_log2(uint32_t(h0 >> 41)) * sz;
                a[1][c] += gumbel_log2(uint32_t(h0 >> 9) & 0x7FFFFFu) * sz;
                a[2][c] += gumbel_log2(uint32_t(h1 >> 41)) * sz;
                a[3][c] += gumbel_log2(uint32_t(h1 >> 9) & 0x7FFFFFu) * sz;
            }
        }
        const uint32_t win[8] = {wa.x, wa.y, wa.z, wa.w, wb.x, wb.y, wb.z, wb.w};
        const uint32_t gin[8] = {ga.x, ga.y, ga.z, ga.w, gb.x, gb.y, gb.z, gb.w};
        float gout[6][4];   // gout[candidate][group]
#pragma unroll
        for (int g = 0; g < 4; ++g) {
            const float inv = softmax2_terms(a[g]);
#pragma unroll
            for (int c = 0; c < 6; ++c) a[g][c] *= inv;                        // GS_c
            const float m24[4] = {a[g][0] + a[g][1] + a[g][2], a[g][0] + a[g][3] + a[g][4],
                                  a[g][1] + a[g][3] + a[g][5], a[g][2] + a[g][4] + a[g][5]};
            float gM[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t wbits = j & 1 ? win[2 * g + (j >> 1)] >> 16 : win[2 * g + (j >> 1)] & 0xFFFFu;
                const uint32_t gbits = j & 1 ? gin[2 * g + (j >> 1)] >> 16 : gin[2 * g + (j >> 1)] & 0xFFFFu;
                const float w = bf16_bits_to_float(wbits), gw = bf16_bits_to_float(gbits);
                const float m = fmaf(one_minus_mt, m24[j], mt);
                gM[j] = fmaf(gw, w, c1) - c2 * m * w * w;
                acc_gmt = fmaf(gM[j], 1.0f - m24[j], acc_gmt);
            }
            // h_c = (1 - Mt_tile) (gM of the two kept positions of candidate c); gP_c = kappa/tau GS_c (h_c - sum GS h)
            const float h[6] = {gM[0] + gM[1], gM[0] + gM[2], gM[0] + gM[3], gM[1] + gM[2], gM[1] + gM[3], gM[2] + gM[3]};
            float hbar = 0.f;
#pragma unroll
            for (int c = 0; c < 6; ++c) hbar = fmaf(a[g][c], h[c], hbar);
            const float scale = kappa_over_tau * one_minus_mt;
#pragma unroll
            for (int c = 0; c < 6; ++c) gout[c][g] = scale * a[g][c] * (h[c] - hbar);
        }
#pragma unroll
        for (int c = 0; c < 6; ++c)
            *reinterpret_cast<float4*>(gP24 + int64_t(c) * G + grp) = make_float4(gout[c][0], gout[c][1], gout[c][2], gout[c][3]);
    }
    double v = double(acc_gmt);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, off);
    if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += s_red[w];
        gP_tile[t] = float(s * double(kappa_over_tau) * double(mt) * double(one_minus_mt));
    }
}

// sums[q] = sum over tiles of partials[t][q], tiles taken in a fixed order by one CTA.
__global__ void __launch_bounds__(256)
reduce_partials_kernel(const double* __restrict__ partials, int64_t T, double* __restrict__ sums) {
    __shared__ double s_red[8][4];
    double v[4] = {0, 0, 0, 0};
    for (int64_t t = threadIdx.x; t < T; t += 256)
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] += partials[t * 4 + q];
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) v[q] += __shfl_xor_sync(0xFFFFFFFFu, v[q], off);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (lane == 0)
#pragma unroll
        for (int q = 0; q < 4; ++q) s_red[warp][q] = v[q];
    __syncthreads();
    if (threadIdx.x < 4) {
        double s = 0.0;
        for (int w = 0; w < 8; ++w) s += s_red[w][threadIdx.x];
        sums[threadIdx.x] = s;
    }
}

// Hard masks.  Thread i owns groups [16i, 16i + 16): six rows of four 16-byte loads, one 16-byte
// store of candidate indices.  The first T threads also write the tile flags.
__global__ void __launch_bounds__(256)
hard_mask_kernel(const float* __restrict__ P_tile, const float* __restrict__ P24, int64_t T, int64_t G,
                 uint8_t* __restrict__ flags, uint8_t* __restrict__ patterns) {
    const int64_t i = int64_t(blockIdx.x) * 256 + threadIdx.x;
    if (i < T) flags[i] = P_tile[i] > 0.0f ? PATCH_TILE_DENSE : PATCH_TILE_SPARSE_2_4;
    if (i * 16 >= G) return;
    float best[16];
    uint32_t arg[16];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float4 p = *reinterpret_cast<const float4*>(P24 + i * 16 + 4 * q);
        best[4 * q] = p.x; best[4 * q + 1] = p.y; best[4 * q + 2] = p.z; best[4 * q + 3] = p.w;
        arg[4 * q] = arg[4 * q + 1] = arg[4 * q + 2] = arg[4 * q + 3] = 0;
    }
#pragma unroll
    for (int c = 1; c < 6; ++c)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float4 p = *reinterpret_cast<const float4*>(P24 + int64_t(c) * G + i * 16 + 4 * q);
            const float v[4] = {p.x, p.y, p.z, p.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (v[e] > best[4 * q + e]) { best[4 * q + e] = v[e]; arg[4 * q + e] = c; }   // first of equals stays
        }
    uint32_t o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) o[q] = arg[4 * q] | (arg[4 * q + 1] << 8) | (arg[4 * q + 2] << 16) | (arg[4 * q + 3] << 24);
    *reinterpret_cast<uint4*>(patterns + i * 16) = make_uint4(o[0], o[1], o[2], o[3]);
}

static int check_mask_shape(int64_t N, int64_t K, int tile_n, int tile_k) {
    if (tile_n != kTile || tile_k != kTile) return PATCH_ERR_TILE;
    if (N <= 0 || K <= 0 || N % kTile || K % kTile) return PATCH_ERR_SHAPE;
    if ((N / kTile) * (K / kTile) > 0x7FFFFFFF) return PATCH_ERR_SHAPE;
    return PATCH_OK;
}

}  // namespace patch

using namespace patch;

extern "C" int patch_hard_mask(const float* P_tile_dev, const float* P24_dev, int64_t N, int64_t K, int tile_n,
                               int tile_k, uint8_t* tile_flags_dev, uint8_t* patterns_dev, void* stream) {
    int rc = check_mask_shape(N, K, tile_n, tile_k);
    if (rc) return rc;
    if (!P_tile_dev || !P24_dev || !tile_flags_dev || !patterns_dev) return PATCH_ERR_NULL;
    if (!aligned16(P24_dev) || !aligned16(patterns_dev) || (reinterpret_cast<uintptr_t>(P_tile_dev) & 3u))
        return PATCH_ERR_ALIGN;
    rc = check_device();
    if (rc) return rc;
    const int64_t T = (N / kTile) * (K / kTile), G = N * (K / 4);      // G is a multiple of 4096
    hard_mask_kernel<<<unsigned(G / 16 / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        P_tile_dev, P24_dev, T, G, tile_flags_dev, patterns_dev);
    return cudaGetLastError() == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

extern "C" int patch_soft_mask_workspace_size(int64_t N, int64_t K, int tile_n, int tile_k, size_t* bytes_out) {
    if (!bytes_out) return PATCH_ERR_NULL;
    int rc = check_mask_shape(N, K, tile_n, tile_k);
    if (rc) return rc;
    *bytes_out = size_t((N / kTile) * (K / kTile)) * 4 * sizeof(double);
    return PATCH_OK;
}

extern "C" int patch_soft_mask(const void* W_dev, int64_t ldw, const float* P_tile_dev, const float* P24_dev,
                               int64_t N, int64_t K, int tile_n, int tile_k, float tau, float kappa, uint64_t seed,
                               int flags, void* Wt_dev, int64_t ldo, float* Mt_dev, int64_t ldm, double* sums_dev,
                               void* workspace_dev, size_t workspace_bytes, void* stream) {
    int rc = check_mask_shape(N, K, tile_n, tile_k);
    if (rc) return rc;
    if (!W_dev || !P_tile_dev || !P24_dev || !Wt_dev || !sums_dev || !workspace_dev) return PATCH_ERR_NULL;
    if (!(tau > 0.0f) || !std::isfinite(tau) || !std::isfinite(kappa)) return PATCH_ERR_SHAPE;
    if (flags & ~PATCH_MASK_NO_NOISE) return PATCH_ERR_SHAPE;
    if (ldw < K || ldo < K || ldw % 8 || ldo % 8) return PATCH_ERR_SHAPE;
    if (Mt_dev && (ldm < K || ldm % 4)) return PATCH_ERR_SHAPE;
    if (!aligned16(W_dev) || !aligned16(Wt_dev) || !aligned16(P24_dev) || (Mt_dev && !aligned16(Mt_dev)) ||
        (reinterpret_cast<uintptr_t>(P_tile_dev) & 3u) || (reinterpret_cast<uintptr_t>(sums_dev) & 7u) ||
        (reinterpret_cast<uintptr_t>(workspace_dev) & 7u))
        return PATCH_ERR_ALIGN;
    const int64_t TK = K / kTile, T = (N / kTile) * TK, G = N * (K / 4);
    if (workspace_bytes < size_t(T) * 4 * sizeof(double)) return PATCH_ERR_SIZE;
    rc = check_device();
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const float sz = 1.0f / tau, sp = kappa * 1.44269504f * sz;
    const uint16_t* W = static_cast<const uint16_t*>(W_dev);
    uint16_t* Wt = static_cast<uint16_t*>(Wt_dev);
    double* partials = static_cast<double*>(workspace_dev);
    const bool noise = !(flags & PATCH_MASK_NO_NOISE);
#define PATCH_LAUNCH_SOFT(NOISE_, MT_)                                                                            \
    soft_mask_kernel<NOISE_, MT_><<<unsigned(T), 256, 0, s>>>(W, ldw, P_tile_dev, P24_dev, int(TK), G, sp, sz, seed, \
                                                              kGolden * uint64_t(G / 2), Wt, ldo, Mt_dev, ldm, partials)
    if (noise) { if (Mt_dev) PATCH_LAUNCH_SOFT(true, true); else PATCH_LAUNCH_SOFT(true, false); }
    else       { if (Mt_dev) PATCH_LAUNCH_SOFT(false, true); else PATCH_LAUNCH_SOFT(false, false); }
#undef PATCH_LAUNCH_SOFT
    if (cudaGetLastError() != cudaSuccess) return PATCH_ERR_CUDA;
    reduce_partials_kernel<<<1, 256, 0, s>>>(partials, T, sums_dev);
    return cudaGetLastError() == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

extern "C" int patch_soft_mask_backward(const void* W_dev, int64_t ldw, const float* P_tile_dev, const float* P24_dev,
                                        int64_t N, int64_t K, int tile_n, int tile_k, float tau, float kappa,
                                        uint64_t seed, int flags, const void* Gw_dev, int64_t ldg, double c1, double c2,
                                        float* gP_tile_dev, float* gP24_dev, void* stream) {
    int rc = check_mask_shape(N, K, tile_n, tile_k);
    if (rc) return rc;
    if (!W_dev || !P_tile_dev || !P24_dev || !Gw_dev || !gP_tile_dev || !gP24_dev) return PATCH_ERR_NULL;
    if (!(tau > 0.0f) || !std::isfinite(tau) || !std::isfinite(kappa) || !std::isfinite(c1) || !std::isfinite(c2))
        return PATCH_ERR_SHAPE;
    if (flags & ~PATCH_MASK_NO_NOISE) return PATCH_ERR_SHAPE;
    if (ldw < K || ldg < K || ldw % 8 || ldg % 8) return PATCH_ERR_SHAPE;
    if (!aligned16(W_dev) || !aligned16(Gw_dev) || !aligned16(P24_dev) || !aligned16(gP24_dev) ||
        (reinterpret_cast<uintptr_t>(P_tile_dev) & 3u) || (reinterpret_cast<uintptr_t>(gP_tile_dev) & 3u))
        return PATCH_ERR_ALIGN;
    rc = check_device();
    if (rc) return rc;
    const int64_t TK = K / kTile, T = (N / kTile) * TK, G = N * (K / 4);
    const float sz = 1.0f / tau, sp = kappa * 1.44269504f * sz;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const uint16_t* W = static_cast<const uint16_t*>(W_dev);
    const uint16_t* Gw = static_cast<const uint16_t*>(Gw_dev);
    if (flags & PATCH_MASK_NO_NOISE)
        soft_mask_backward_kernel<false><<<unsigned(T), 256, 0, s>>>(W, ldw, Gw, ldg, P_tile_dev, P24_dev, int(TK), G, sp, sz,
                                                                     kappa * sz, seed, kGolden * uint64_t(G / 2), float(c1),
                                                                     float(c2), gP_tile_dev, gP24_dev);
    else
        soft_mask_backward_kernel<true><<<unsigned(T), 256, 0, s>>>(W, ldw, Gw, ldg, P_tile_dev, P24_dev, int(TK), G, sp, sz,
                                                                    kappa * sz, seed, kGolden * uint64_t(G / 2), float(c1),
                                                                    float(c2), gP_tile_dev, gP24_dev);
    return cudaGetLastError() == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

extern "C" int patch_mask_regularizer_coefficients(const double* sums_host, int n, double rho, double lambda1,
                                                   double lambda2, double* c1_host, double* c2_host) {
    if (!sums_host || !c1_host || !c2_host) return PATCH_ERR_NULL;
    if (n <= 0) return PATCH_ERR_SHAPE;
    double m = 0, nz = 0, w2 = 0;
    for (int i = 0; i < n; ++i) { m += sums_host[4 * i]; nz += sums_host[4 * i + 1]; w2 += sums_host[4 * i + 3]; }
    if (!(nz > 0) || !(w2 > 0)) return PATCH_ERR_SHAPE;
    const double dev = m / nz - rho;
    *c1_host = lambda1 * (dev > 0 ? 1.0 : dev < 0 ? -1.0 : 0.0) / nz;
    *c2_host = 2.0 * lambda2 / w2;
    return PATCH_OK;
}

extern "C" int patch_mask_regularizers(const double* sums_host, int n, double rho, double lambda1, double lambda2,
                                       double* out_host) {
    if (!sums_host || !out_host) return PATCH_ERR_NULL;
    if (n <= 0) return PATCH_ERR_SHAPE;
    double m = 0, nz = 0, mw2 = 0, w2 = 0;
    for (int i = 0; i < n; ++i) {
        m += sums_host[4 * i]; nz += sums_host[4 * i + 1]; mw2 += sums_host[4 * i + 2]; w2 += sums_host[4 * i + 3];
    }
    if (!(nz > 0) || !(w2 > 0)) return PATCH_ERR_SHAPE;
    *out_host = lambda1 * std::fabs(m / nz - rho) - lambda2 * (mw2 / w2);
    return PATCH_OK;
}
