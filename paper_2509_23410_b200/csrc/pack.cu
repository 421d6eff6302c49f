// patch_packed_size / patch_pack / patch_unpack: the per-tile compression of the hybrid weight.
//
// Semantics follow the last lines of Algorithm 1 of the paper (hard mask
// M* = M*_tile + (1 - M*_tile) (.) M*_2:4, What = W (.) M*) with magnitude top-2 selection per
// group of four along K, and Appendix A's "compress" step (values + metadata per tile).
// Both kernels are pure data movement plus integer compares, bound by HBM bandwidth:
// per element of W they read 2 B and write 2 B (dense tile) or 1.125 B (2:4 tile).
// Tiles of the 4-bit kinds (the 4-bit weight-only quantisation table of the paper's section on combining the
// method with other compression; the quantiser is this library's reading, stated in the public header) are
// written by a kernel of their own: one warp per tile row, 0.52 B (dense) or 0.39 B (2:4) per element.
#include <vector>
#include <cstring>
#include "patch_internal.cuh"

namespace patch {

int validate_layout(const patch_layout_t* L) {
    if (!L) return PATCH_ERR_NULL;
    if (L->magic != kMagic || L->version != kVersion) return PATCH_ERR_FORMAT;
    if (L->tile_n != kTile || L->tile_k != kTile) return PATCH_ERR_TILE;
    if (L->N <= 0 || L->K <= 0 || L->N % kTile || L->K % kTile) return PATCH_ERR_SHAPE;
    if (L->n_dense < 0 || L->n_sparse < 0 || L->n_dense_q4 < 0 || L->n_sparse_q4 < 0) return PATCH_ERR_FORMAT;
    uint64_t T = uint64_t(L->N / kTile) * uint64_t(L->K / kTile);
    if (uint64_t(L->n_dense) + uint64_t(L->n_sparse) + uint64_t(L->n_dense_q4) + uint64_t(L->n_sparse_q4) != T)
        return PATCH_ERR_FORMAT;
    if (L->table_off != kHeaderBytes) return PATCH_ERR_FORMAT;
    uint64_t pay = (kHeaderBytes + 16 * T + 1023) / 1024 * 1024;
    if (L->payload_off != pay) return PATCH_ERR_FORMAT;
    if (L->payload_bytes != uint64_t(kDenseBytes) * L->n_dense + uint64_t(kSparseBytes) * L->n_sparse +
                                uint64_t(kDenseQ4Bytes) * L->n_dense_q4 + uint64_t(kSparseQ4Bytes) * L->n_sparse_q4)
        return PATCH_ERR_FORMAT;
    if (L->total_bytes != L->payload_off + L->payload_bytes) return PATCH_ERR_FORMAT;
    if (L->total_bytes / 16 > 0xFFFFFFF0ull) return PATCH_ERR_SHAPE;  // offsets are stored as u32 * 16
    return PATCH_OK;
}

int check_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return PATCH_ERR_CUDA;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
        return PATCH_ERR_CUDA;
    return major == 10 ? PATCH_OK : PATCH_ERR_ARCH;
}

// ---------------------------------------------------------------------------------------------

__device__ __forceinline__ uint4 ld_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

// The two kept positions i0 < i1 of a group whose four bf16 values are the halves of (x0, x1):
// the two largest magnitudes, equal magnitudes ordered by position (lower first).  Each value gets the
// sort key  magnitude << 2 | (3 - position): keys are distinct, and the two largest of four come out of a
// five-comparator network with their positions in the low bits.
__device__ __forceinline__ void top2_positions(uint32_t x0, uint32_t x1, uint32_t& i0, uint32_t& i1) {
    const uint32_t k0 = ((x0 & 0x7FFFu) << 2) | 3u, k1 = ((x0 >> 14) & 0x1FFFCu) | 2u;
    const uint32_t k2 = ((x1 & 0x7FFFu) << 2) | 1u, k3 = (x1 >> 14) & 0x1FFFCu;
    const uint32_t hi01 = max(k0, k1), lo01 = min(k0, k1), hi23 = max(k2, k3), lo23 = min(k2, k3);
    const uint32_t first = max(hi01, hi23);
    // the runner-up is the loser of the final or the partner the winner beat in its own pair
    const uint32_t second = max(min(hi01, hi23), hi01 > hi23 ? lo01 : lo23);
    const uint32_t pa = 3u - (first & 3u), pb = 3u - (second & 3u);
    i0 = min(pa, pb);
    i1 = max(pa, pb);
}

// {value at position i1 : value at position i0} of the group (x0, x1): element j is bytes 2j, 2j + 1 of the pair
__device__ __forceinline__ uint32_t gather_pair(uint32_t x0, uint32_t x1, uint32_t i0, uint32_t i1) {
    return __byte_perm(x0, x1, (i0 | (i1 << 8)) * 0x22u + 0x1010u);
}

// The two kept positions of candidate c (row c of the matrix S of the six 2:4 masks, rows in
// lexicographic order of the kept positions) as the position code i0 | (i1 << 2), one nibble per candidate.
constexpr uint32_t kCandidateCodes = 0xED9C84u;

// Tile flags in device memory (patch_pack_dev): what the pack kernel needs to know about the blob.
struct DeviceFlags {
    const uint8_t* flags;   // [T]; NULL = the table in the blob was written by the host
    int64_t T, N, K;
    uint64_t capacity;
};

// Descriptor of tile t from the flags alone: the CTA sums the payload sizes of the tiles before t (its
// offset) and of all tiles (does the blob fit?).  A few KB of flags per CTA, served by L2.  CTA 0 also
// writes the header and the padding behind the table; every CTA writes its own table entry.
// Returns false if the blob does not fit `capacity` (then only a header without magic number is written).
__device__ __forceinline__ bool descriptor_from_flags(const DeviceFlags& F, int t, uint8_t* blob, int* status, TileDesc& d) {
    // per warp: tiles before t and in total whose flag has bit 0 (2:4), bit 1 (4-bit values), both
    __shared__ unsigned long long s_part[8][6];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long cnt[6] = {0, 0, 0, 0, 0, 0};          // {bit0, bit1, both} before t, then in total
    bool bad = false;
    // four flags per load where the array is word aligned
    const int64_t words = (reinterpret_cast<uintptr_t>(F.flags) & 3u) == 0 ? F.T / 4 : 0;
    for (int64_t i = tid; i < words; i += 256) {
        uint32_t w = reinterpret_cast<const uint32_t*>(F.flags)[i];
        if (w & 0xFCFCFCFCu) {          // a byte above 3: an error, packed as dense
            bad = true;
            uint32_t clean = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) { const uint32_t b = (w >> (8 * q)) & 0xFFu; clean |= (b <= 3u ? b : 0u) << (8 * q); }
            w = clean;
        }
        const uint32_t b0 = w & 0x01010101u, b1 = (w >> 1) & 0x01010101u, bb = b0 & b1;
        const int64_t first = 4 * i;                      // flags first .. first + 3; those below t count as "before"
        const uint32_t below = first + 4 <= t ? 0xFFFFFFFFu : first >= t ? 0u : (1u << (8 * uint32_t(t - first))) - 1u;
        cnt[0] += __popc(b0 & below); cnt[1] += __popc(b1 & below); cnt[2] += __popc(bb & below);
        cnt[3] += __popc(b0); cnt[4] += __popc(b1); cnt[5] += __popc(bb);
    }
    for (int64_t i = 4 * words + tid; i < F.T; i += 256) {
        uint32_t f = F.flags[i];
        if (f > 3u) { bad = true; f = 0; }
        const uint32_t b0 = f & 1u, b1 = f >> 1, bb = b0 & b1, before = i < t ? 1u : 0u;
        cnt[0] += b0 & before; cnt[1] += b1 & before; cnt[2] += bb & before;
        cnt[3] += b0; cnt[4] += b1; cnt[5] += bb;
    }
#pragma unroll
    for (int q = 0; q < 6; ++q) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) cnt[q] += __shfl_xor_sync(0xFFFFFFFFu, cnt[q], off);
        if (lane == 0) s_part[warp][q] = cnt[q];
    }
    bad = __syncthreads_or(bad) != 0;
#pragma unroll
    for (int q = 0; q < 6; ++q) {
        cnt[q] = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) cnt[q] += s_part[w][q];
    }
    // tiles of each kind before t and in total: {dense, 2:4, dense 4-bit, 2:4 4-bit}
    const unsigned long long nb[4] = {(unsigned long long)t - cnt[0] - cnt[1] + cnt[2], cnt[0] - cnt[2], cnt[1] - cnt[2], cnt[2]};
    const unsigned long long nt[4] = {(unsigned long long)F.T - cnt[3] - cnt[4] + cnt[5], cnt[3] - cnt[5], cnt[4] - cnt[5], cnt[5]};
    unsigned long long before = 0, total = 0;
#pragma unroll
    for (uint32_t k = 0; k < 4; ++k) { before += nb[k] * tile_payload_bytes(k); total += nt[k] * tile_payload_bytes(k); }
    const uint64_t payload_off = (kHeaderBytes + 16 * uint64_t(F.T) + 1023) / 1024 * 1024;
    const uint64_t size = payload_off + total;
    const bool fits = size <= F.capacity && size / 16 <= 0xFFFFFFF0ull;
    if (t == 0) {
        if (bad && status && tid == 0) *status = PATCH_ERR_FLAG;     // every CTA sees all flags; one reports
        if (!fits && status && tid == 0) *status = PATCH_ERR_SIZE;
        if (tid == 0) {
            patch_layout_t L;
            L.magic = fits ? kMagic : 0u; L.version = kVersion;
            L.N = F.N; L.K = F.K; L.tile_n = kTile; L.tile_k = kTile;
            L.n_dense = int64_t(nt[0]); L.n_sparse = int64_t(nt[1]);
            L.n_dense_q4 = int64_t(nt[2]); L.n_sparse_q4 = int64_t(nt[3]);
            L.table_off = kHeaderBytes; L.payload_off = payload_off; L.payload_bytes = total; L.total_bytes = size;
            uint32_t* h = reinterpret_cast<uint32_t*>(blob);
            const uint32_t* src = reinterpret_cast<const uint32_t*>(&L);
            for (uint32_t i = 0; i < kHeaderBytes / 4; ++i) h[i] = i < sizeof(L) / 4 ? src[i] : 0u;
        }
        if (fits) {
            uint32_t* pad = reinterpret_cast<uint32_t*>(blob + kHeaderBytes + 16 * uint64_t(F.T));
            for (uint64_t i = tid; i < (payload_off - kHeaderBytes - 16 * uint64_t(F.T)) / 4; i += 256) pad[i] = 0u;
        }
    }
    if (!fits) return false;
    const uint64_t off = payload_off + before;
    uint32_t kind = F.flags[t];
    if (kind > PATCH_TILE_SPARSE_2_4_Q4) kind = PATCH_TILE_DENSE;
    d = TileDesc{kind, uint32_t(off / 16), 0xFFFFFFFFu, 0};
    if (kind == PATCH_TILE_SPARSE_2_4) {
        d.meta_off16 = uint32_t((off + kAtomBytes) / 16);
    } else if (kind == PATCH_TILE_DENSE_Q4) {
        d.scales_off16 = uint32_t((off + kDenseQ4CodeBytes) / 16);
    } else if (kind == PATCH_TILE_SPARSE_2_4_Q4) {
        d.meta_off16 = uint32_t((off + kSparseQ4CodeBytes) / 16);
        d.scales_off16 = uint32_t((off + kSparseQ4CodeBytes + kMetaBytes) / 16);
    }
    if (tid == 0) reinterpret_cast<TileDesc*>(blob + kHeaderBytes)[t] = d;
    return true;
}

// ---------------------------------------------------------------------------------------------
// 4-bit kinds.  Sixteen lanes per tile row (a warp works on two rows at a time); a lane holds eight consecutive
// elements of its row: one 32-bit word of codes of a dense tile, half a word of a 2:4 tile.
//   scale  s = bf16(max|v| / 7) over the row's stored values (all 128, or the 64 the 2:4 selection keeps)
//   code   q + 8 with q = clamp(rint(v / s), -7, 7), 0 where s = 0; fp32 arithmetic, IEEE division
// Codes are stored eight to a 32-bit word, in the row's order of stored values: the even ones of a word in nibbles
// 0..3, the odd ones in nibbles 4..7, so that (word >> 4j) & 0x000F000F is the pair (2j, 2j + 1) in the two halves
// of a register -- what the dequantising GEMM kernel turns into two bf16 with one instruction.  Four words (32
// values) make a 16-byte unit; unit j of tile row r lives at byte (128 j + r) * 16, so the 32 threads of a warp
// that each own a row read 512 consecutive bytes.

__device__ __forceinline__ float bf16_bits_to_f32(uint32_t h) { return __uint_as_float(h << 16); }
// bit position, inside its 32-bit word, of the code of stored value c (c & 7 decides)
__host__ __device__ constexpr uint32_t q4_code_shift(uint32_t c) { return 4u * (((c & 1u) << 2) | ((c & 7u) >> 1)); }
// q = clamp(rint(v / s), -7, 7) with the IEEE quotient; 0 where s = 0
__device__ __forceinline__ int q4_quantise_exact(float v, float s) {
    if (s == 0.0f) return 0;
    return int(fminf(fmaxf(rintf(__fdiv_rn(v, s)), -7.0f), 7.0f));
}
__host__ __device__ constexpr uint32_t q4_sum_shifted(uint32_t x, uint32_t n) {   // sum of x << shift(i), i < n, modulo 2^32
    uint32_t acc = 0;
    for (uint32_t i = 0; i < n; ++i) acc += x << q4_code_shift(i);
    return acc;
}
// Scale of a row whose largest magnitude is m (a bf16 value): bf16(fp32(m / 7)).  m * fp32(1/7) is within two
// fp32 steps of the quotient, and the quotient a / 7 of an 8-bit significand a stays at least 1 / 1792 (relative)
// away from every point c / 2^k, c odd with nine bits, where the rounding to bf16 changes (the difference is
// |2^j a - 7 c| / 1792 with an even and an odd term), so the product rounds to the same bf16 as the quotient; the
// division is kept for magnitudes near the bottom of the range, where m may be subnormal.
__device__ __forceinline__ __nv_bfloat16 q4_scale(float m) {
    return __float2bfloat16_rn(m >= 0x1p-90f ? m * (1.0f / 7.0f) : __fdiv_rn(m, 7.0f));
}
// Codes q + 8 of NV stored values of one row (the first NV of a word), each at its bit position, summed.
// v and s are bf16 values: significands a, b < 256.  The exact quotient v / s is then either a half-integer or at
// least 1 / 1020 away from the nearest one (|a 2^j - (2k + 1) b| >= 1 over a denominator 2 b 2^i <= 1020 for
// quotients above 1/4), and s = bf16(max / 7) keeps every quotient of the row below 7.02, so nothing needs
// clamping.  t = v * (1 / s), with the reciprocal good to 2^-23, is within 1.3e-6 of the exact quotient.  Adding
// and subtracting 1.5 * 2^13 snaps t to the grid of 2^-10: onto the half-integer exactly if the quotient is one,
// never onto or across it otherwise.  Adding 1.5 * 2^23 then rounds to the nearest integer, ties to even -- the
// result of rint on the IEEE quotient -- and leaves q in the low mantissa bits.  Rows whose scale is zero,
// subnormal or huge, and lanes that hold a NaN (`numbers` false), take the division itself.
template <uint32_t NV>
__device__ __forceinline__ uint32_t q4_codes(const float (&v)[NV], float s, bool numbers) {
    constexpr float kSnap = 12288.0f, kRound = 12582912.0f;
    constexpr uint32_t kRoundBits = 0x4B400000u;
    constexpr uint32_t kBias = q4_sum_shifted(8u - kRoundBits, NV);
    uint32_t word;
    if (numbers && s >= 0x1p-100f && s <= 0x1p100f) {
        float inv;
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(inv) : "f"(s));
        word = kBias;
#pragma unroll
        for (uint32_t i = 0; i < NV; ++i) {
            const float t = v[i] * inv;
            const float snapped = (t + kSnap) - kSnap;
            word += __float_as_uint(snapped + kRound) << q4_code_shift(i);
        }
    } else {
        word = 0;
#pragma unroll
        for (uint32_t i = 0; i < NV; ++i) word += uint32_t(q4_quantise_exact(v[i], s) + 8) << q4_code_shift(i);
    }
    return word;
}
// nibble index inside its 32-bit word of stored value c
__device__ __forceinline__ uint32_t q4_nibble_slot(uint32_t c) { return ((c & 1u) << 2) | ((c & 7u) >> 1); }

// One tile of a 4-bit kind, by the 256 threads of a CTA.
// GIVEN: the 2:4 mask of a 2:4 tile comes from `patterns` (one candidate index per group of four, as for
// the bf16 kinds) instead of the magnitude rule; an index above 5 raises PATCH_ERR_FLAG in *status.
template <bool GIVEN>
__device__ __forceinline__ void pack_q4_tile(const TileDesc& d, const uint16_t* __restrict__ W, int64_t ldw, int TK, int t,
                                             uint8_t* __restrict__ blob, const uint8_t* __restrict__ patterns, int* status) {
    const bool sparse = d.kind == PATCH_TILE_SPARSE_2_4_Q4;
    const int tn = t / TK, tk = t - tn * TK;
    const uint16_t* wt = W + int64_t(tn) * kTile * ldw + int64_t(tk) * kTile;
    uint32_t* codes = reinterpret_cast<uint32_t*>(blob + uint64_t(d.payload_off16) * 16);
    uint8_t* meta = blob + uint64_t(d.meta_off16) * 16;                    // only used if sparse
    uint16_t* scales = reinterpret_cast<uint16_t*>(blob + uint64_t(d.scales_off16) * 16);
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u, c = lane & 15u;
    const uint32_t r0 = warp * 2 + (lane >> 4);           // this lane's rows: r0 + 16 it
    // all eight loads of the lane are issued before the first row is quantised: 4 KB in flight per warp
    uint4 xs[8];
    uint32_t given[8] = {0, 0, 0, 0, 0, 0, 0, 0};
#pragma unroll
    for (uint32_t it = 0; it < 8; ++it) {
        const uint32_t r = r0 + 16 * it;
        xs[it] = ld_stream(wt + int64_t(r) * ldw + c * 8);
        if (GIVEN && sparse)   // the candidate indices of this lane's two groups: one aligned 2-byte load
            given[it] = *reinterpret_cast<const uint16_t*>(patterns + (int64_t(tn) * kTile + r) * (int64_t(TK) * 32) + tk * 32 + c * 2);
    }
#pragma unroll
    for (uint32_t it = 0; it < 8; ++it) {
        const uint32_t r = r0 + 16 * it;
        const uint32_t in[4] = {xs[it].x, xs[it].y, xs[it].z, xs[it].w};
        // a bf16 is a NaN iff its magnitude bits exceed 0x7F80: adding 0x7F then carries into bit 15
        const bool numbers = (((((in[0] & 0x7FFF7FFFu) + 0x007F007Fu) | ((in[1] & 0x7FFF7FFFu) + 0x007F007Fu)) |
                               (((in[2] & 0x7FFF7FFFu) + 0x007F007Fu) | ((in[3] & 0x7FFF7FFFu) + 0x007F007Fu))) & 0x80008000u) == 0;
        if (!sparse) {
            float v[8];
            float m = 0.0f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                v[2 * i] = __uint_as_float(in[i] << 16);
                v[2 * i + 1] = __uint_as_float(in[i] & 0xFFFF0000u);
                m = fmaxf(m, fmaxf(fabsf(v[2 * i]), fabsf(v[2 * i + 1])));
            }
#pragma unroll
            for (int off = 8; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
            const __nv_bfloat16 sb = q4_scale(m);
            if (c == 0) scales[r] = __bfloat16_as_ushort(sb);
            codes[((c >> 2) * 128 + r) * 4 + (c & 3u)] = q4_codes<8>(v, __bfloat162float(sb), numbers);
        } else {
            float v[4];
            uint32_t pos = 0;            // position codes of the lane's two groups, four bits each
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                uint32_t i0, i1;
                if (GIVEN) {
                    uint32_t cand = (given[it] >> (8 * g)) & 0xFFu;
                    if (cand > 5u) { if (status) *status = PATCH_ERR_FLAG; cand = 0; }
                    const uint32_t nib = (kCandidateCodes >> (4 * cand)) & 0xFu;
                    i0 = nib & 3u;
                    i1 = nib >> 2;
                } else {
                    top2_positions(in[2 * g], in[2 * g + 1], i0, i1);
                }
                const uint32_t kept = gather_pair(in[2 * g], in[2 * g + 1], i0, i1);
                v[2 * g] = __uint_as_float(kept << 16);
                v[2 * g + 1] = __uint_as_float(kept & 0xFFFF0000u);
                pos |= (i0 | (i1 << 2)) << (4 * g);
            }
            float m = fmaxf(fmaxf(fabsf(v[0]), fabsf(v[1])), fmaxf(fabsf(v[2]), fabsf(v[3])));
#pragma unroll
            for (int off = 8; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, off));
            const __nv_bfloat16 sb = q4_scale(m);
            if (c == 0) scales[r] = __bfloat16_as_ushort(sb);
            // stored values 4c .. 4c + 3 of the row: half of word c / 2 (values 0..3 of a word sit in bits 0-7 and
            // 16-23, values 4..7 eight bits higher); the even lane of a pair stores the word and the metadata
            uint32_t half = q4_codes<4>(v, __bfloat162float(sb), numbers) << (8 * (c & 1u));
            pos <<= 8 * (c & 1u);
            const uint32_t word = half | __shfl_xor_sync(0xFFFFFFFFu, half, 1);
            const uint32_t code = pos | __shfl_xor_sync(0xFFFFFFFFu, pos, 1);
            if ((c & 1u) == 0) {
                const uint32_t w = c >> 1;                     // word of the row (0..7) = 16-column chunk u
                codes[((w >> 2) * 128 + r) * 4 + (w & 3u)] = word;
                // metadata row L = 16q + 8h + i, word j, low half for tile rows 16q+i, high for 16q+8+i
                const uint32_t Lr = (r & ~15u) + 8u * (w & 1u) + (r & 7u), j = w >> 1, hi = (r >> 3) & 1u;
                *reinterpret_cast<uint16_t*>(meta + Lr * 16 + j * 4 + hi * 2) = uint16_t(code);
            }
        }
    }
}

// One CTA per tile.  W is read with 16-byte loads, the payload is written with 16-byte stores.
// GIVEN: the 2:4 mask comes from `patterns` (one candidate index per group of four, [N x K/4]
// row-major) instead of the magnitude rule; an index above 5 raises PATCH_ERR_FLAG in *status.
// DEVFLAGS: the tile's descriptor is computed from tile flags in device memory instead of read
// from a table the host wrote.
template <bool GIVEN, bool DEVFLAGS>
__global__ void __launch_bounds__(256, 4)
pack_kernel(const uint16_t* __restrict__ W, int64_t ldw, int TK, uint8_t* __restrict__ blob,
            uint64_t table_off, const uint8_t* __restrict__ patterns, int* status, DeviceFlags F) {
    const int t = blockIdx.x;
    TileDesc d;
    if (DEVFLAGS) {
        if (!descriptor_from_flags(F, t, blob, status, d)) return;
    } else {
        d = reinterpret_cast<const TileDesc*>(blob + table_off)[t];
    }
    if (d.kind > PATCH_TILE_SPARSE_2_4) {                // a 4-bit kind
        pack_q4_tile<GIVEN>(d, W, ldw, TK, t, blob, patterns, status);
        return;
    }
    const int tn = t / TK, tk = t - tn * TK;
    const uint16_t* wt = W + int64_t(tn) * kTile * ldw + int64_t(tk) * kTile;
    uint8_t* pay = blob + uint64_t(d.payload_off16) * 16;
    if (d.kind == PATCH_TILE_DENSE) {
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const uint32_t idx = it * 256 + threadIdx.x, r = idx >> 4, c = idx & 15u;
            const uint4 v = ld_stream(wt + int64_t(r) * ldw + c * 8);
            *reinterpret_cast<uint4*>(pay + (c >> 3) * kAtomBytes + atom_chunk_offset(r, c & 7u)) = v;
        }
    } else {
        uint8_t* meta = blob + uint64_t(d.meta_off16) * 16;
        // all of the thread's loads are issued before any of the selection work: 128 bytes in flight per thread
        uint4 va[4], vb[4];
        uint32_t vgiven[4] = {0, 0, 0, 0};
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const uint32_t idx = it * 256 + threadIdx.x, r = idx >> 3, u = idx & 7u;
            const uint16_t* src = wt + int64_t(r) * ldw + u * 16;
            va[it] = ld_stream(src);
            vb[it] = ld_stream(src + 8);
            if (GIVEN)   // the four candidate indices of this thread's groups: one aligned 4-byte load
                vgiven[it] = *reinterpret_cast<const uint32_t*>(patterns + (int64_t(tn) * kTile + r) * (int64_t(TK) * 32) +
                                                                tk * 32 + u * 4);
        }
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            // 16 consecutive elements of one row: four groups -> 8 kept values + 16 metadata bits
            const uint32_t idx = it * 256 + threadIdx.x, r = idx >> 3, u = idx & 7u;
            const uint4 a = va[it], b = vb[it];
            const uint32_t in[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
            uint32_t out[4], code = 0;
            const uint32_t given = vgiven[it];
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint32_t i0, i1;
                if (GIVEN) {
                    uint32_t c = (given >> (8 * g)) & 0xFFu;
                    if (c > 5u) { if (status) *status = PATCH_ERR_FLAG; c = 0; }
                    const uint32_t nib = (kCandidateCodes >> (4 * c)) & 0xFu;
                    i0 = nib & 3u;
                    i1 = nib >> 2;
                } else {
                    top2_positions(in[2 * g], in[2 * g + 1], i0, i1);
                }
                code |= (i0 | (i1 << 2)) << (4 * g);
                out[g] = gather_pair(in[2 * g], in[2 * g + 1], i0, i1);
            }
            *reinterpret_cast<uint4*>(pay + atom_chunk_offset(r, u)) = make_uint4(out[0], out[1], out[2], out[3]);
            // metadata row L = 16q + 8h + i, word j, low half for tile rows 16q+i, high for 16q+8+i
            const uint32_t L = (r & ~15u) + 8u * (u & 1u) + (r & 7u), j = u >> 1, hi = (r >> 3) & 1u;
            *reinterpret_cast<uint16_t*>(meta + L * 16 + j * 4 + hi * 2) = uint16_t(code);
        }
    }
}

// Dequantised value of the code nibble n with the row's scale s: bf16(q * s), q = n - 8 (the product is exact in fp32)
__device__ __forceinline__ uint32_t q4_dequant_bits(uint32_t n, float s) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(float(int(n) - 8) * s));
}

__device__ __forceinline__ void unpack_q4_tile(const TileDesc& d, const uint8_t* __restrict__ blob, uint16_t* wt, int64_t ldw) {
    const bool sparse = d.kind == PATCH_TILE_SPARSE_2_4_Q4;
    const uint32_t* codes = reinterpret_cast<const uint32_t*>(blob + uint64_t(d.payload_off16) * 16);
    const uint8_t* meta = blob + uint64_t(d.meta_off16) * 16;
    const uint16_t* scales = reinterpret_cast<const uint16_t*>(blob + uint64_t(d.scales_off16) * 16);
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    for (uint32_t rr = 0; rr < 16; ++rr) {
        const uint32_t r = rr * 8 + warp;
        const float s = bf16_bits_to_f32(scales[r]);
        uint32_t out[4] = {0, 0, 0, 0};
        if (sparse) {
            const uint32_t word = codes[((lane >> 4) * 128 + r) * 4 + ((lane & 15u) >> 2)];
            const uint32_t u = lane >> 2;
            const uint32_t Lr = (r & ~15u) + 8u * (u & 1u) + (r & 7u), j = u >> 1, hi = (r >> 3) & 1u;
            const uint32_t code = *reinterpret_cast<const uint16_t*>(meta + Lr * 16 + j * 4 + hi * 2);
            const uint32_t nib = (code >> (4 * (lane & 3u))) & 0xFu, i0 = nib & 3u, i1 = nib >> 2;
            const uint32_t a = q4_dequant_bits((word >> (4 * q4_nibble_slot(2 * lane))) & 0xFu, s);
            const uint32_t b = q4_dequant_bits((word >> (4 * q4_nibble_slot(2 * lane + 1))) & 0xFu, s);
#pragma unroll
            for (uint32_t p = 0; p < 4; ++p) out[p] = p == i0 ? a : p == i1 ? b : 0u;
        } else {
            const uint32_t word = codes[((lane >> 3) * 128 + r) * 4 + ((lane & 7u) >> 1)];
#pragma unroll
            for (uint32_t p = 0; p < 4; ++p) out[p] = q4_dequant_bits((word >> (4 * q4_nibble_slot(4 * lane + p))) & 0xFu, s);
        }
        *reinterpret_cast<uint2*>(wt + int64_t(r) * ldw + lane * 4) = make_uint2(out[0] | (out[1] << 16), out[2] | (out[3] << 16));
    }
}

// A weight of 4-bit tiles rewritten as the blob of bf16 tiles with the same dequantised values: what the large-M
// kernels multiply by when the layer has many tokens (the dequantisation of a tile is then paid once per call
// instead of once per token tile).  One CTA per tile, one warp per tile row as above; the output offset of tile t
// follows from its 4-bit offset (the payloads of both blobs are laid out in tile order, so the number of dense
// tiles before t is (off4 - 6400 t) / 2048 in units of the two payload sizes' difference).
__global__ void __launch_bounds__(256)
expand_q4_kernel(const uint8_t* __restrict__ blob, uint64_t table_off, uint32_t pay0, uint32_t end16, uint8_t* __restrict__ out,
                 patch_layout_t out_layout, int* status) {
    const int t = blockIdx.x;
    const TileDesc d = reinterpret_cast<const TileDesc*>(blob + table_off)[t];
    const bool sparse = d.kind == PATCH_TILE_SPARSE_2_4_Q4;
    // The entry is checked before a byte of the tile is read: a 4-bit kind, the payload inside the blob and at an
    // offset that tiles of the two sizes before it can add up to.  Otherwise the status word says so, nothing is
    // read, and the tile's entry in the new table points at the first payload as a 2:4 tile (its contents are
    // unspecified, but every later read stays inside the new blob).
    const uint32_t len16 = (sparse ? kSparseQ4Bytes : kDenseQ4Bytes) / 16, pay0_16 = pay0 / 16;
    bool bad = d.kind < PATCH_TILE_DENSE_Q4 || d.kind > PATCH_TILE_SPARSE_2_4_Q4 || d.payload_off16 < pay0_16 ||
               d.payload_off16 > end16 || len16 > end16 - d.payload_off16;
    const int64_t rest = int64_t(d.payload_off16) * 16 - int64_t(pay0) - int64_t(kSparseQ4Bytes) * t;
    constexpr int64_t kStep = int64_t(kDenseQ4Bytes) - int64_t(kSparseQ4Bytes);
    bad = bad || rest < 0 || rest % kStep != 0 || rest / kStep > t;
    if (bad) {
        if (threadIdx.x == 0) {
            if (status) atomicCAS(status, PATCH_OK, PATCH_ERR_FORMAT);
            reinterpret_cast<TileDesc*>(out + table_off)[t] =
                TileDesc{uint32_t(PATCH_TILE_SPARSE_2_4), pay0_16, uint32_t((pay0 + kAtomBytes) / 16), 0};
        }
        if (t != 0) return;
    }
    const uint64_t n_dense_before = bad ? 0 : uint64_t(rest / kStep);
    const uint64_t off = pay0 + n_dense_before * kDenseBytes + (uint64_t(t) - n_dense_before) * kSparseBytes;
    if (threadIdx.x == 0) {
        if (!bad)
            reinterpret_cast<TileDesc*>(out + table_off)[t] =
                TileDesc{sparse ? uint32_t(PATCH_TILE_SPARSE_2_4) : uint32_t(PATCH_TILE_DENSE), uint32_t(off / 16),
                         sparse ? uint32_t((off + kAtomBytes) / 16) : 0xFFFFFFFFu, 0};
        if (t == 0) {
            uint32_t* h = reinterpret_cast<uint32_t*>(out);
            const uint32_t* src = reinterpret_cast<const uint32_t*>(&out_layout);
            for (uint32_t i = 0; i < kHeaderBytes / 4; ++i) h[i] = i < sizeof(out_layout) / 4 ? src[i] : 0u;
        }
    }
    if (bad) return;
    // metadata and scales follow the codes (the table's own offsets for them are not used)
    const uint8_t* src = blob + uint64_t(d.payload_off16) * 16;
    const uint32_t* codes = reinterpret_cast<const uint32_t*>(src);
    const uint16_t* scales = reinterpret_cast<const uint16_t*>(src + (sparse ? kSparseQ4CodeBytes + kMetaBytes : kDenseQ4CodeBytes));
    uint8_t* pay = out + off;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31u;
    if (sparse)   // the metadata block is already in hardware order
        reinterpret_cast<uint2*>(pay + kAtomBytes)[threadIdx.x] = reinterpret_cast<const uint2*>(src + kSparseQ4CodeBytes)[threadIdx.x];
    for (uint32_t rr = 0; rr < 16; ++rr) {
        const uint32_t r = rr * 8 + warp;
        const float s = bf16_bits_to_f32(scales[r]);
        if (sparse) {
            // kept values 2 lane, 2 lane + 1 of the row: four bytes of the atom
            const uint32_t word = codes[((lane >> 4) * 128 + r) * 4 + ((lane & 15u) >> 2)];
            const uint32_t a = q4_dequant_bits((word >> (4 * q4_nibble_slot(2 * lane))) & 0xFu, s);
            const uint32_t b = q4_dequant_bits((word >> (4 * q4_nibble_slot(2 * lane + 1))) & 0xFu, s);
            *reinterpret_cast<uint32_t*>(pay + atom_chunk_offset(r, lane >> 2) + (lane & 3u) * 4) = a | (b << 16);
        } else {
            // columns 4 lane .. 4 lane + 3: eight bytes of atom (column / 64)
            const uint32_t word = codes[((lane >> 3) * 128 + r) * 4 + ((lane & 7u) >> 1)];
            uint32_t o[4];
#pragma unroll
            for (uint32_t p = 0; p < 4; ++p) o[p] = q4_dequant_bits((word >> (4 * q4_nibble_slot(4 * lane + p))) & 0xFu, s);
            *reinterpret_cast<uint2*>(pay + (lane >> 4) * kAtomBytes + atom_chunk_offset(r, (lane & 15u) >> 1) + (lane & 1u) * 8) =
                make_uint2(o[0] | (o[1] << 16), o[2] | (o[3] << 16));
        }
    }
}

__global__ void __launch_bounds__(256)
unpack_kernel(const uint8_t* __restrict__ blob, uint64_t table_off, int TK,
              uint16_t* __restrict__ What, int64_t ldw) {
    const int t = blockIdx.x;
    const TileDesc d = reinterpret_cast<const TileDesc*>(blob + table_off)[t];
    const int tn = t / TK, tk = t - tn * TK;
    uint16_t* wt = What + int64_t(tn) * kTile * ldw + int64_t(tk) * kTile;
    const uint8_t* pay = blob + uint64_t(d.payload_off16) * 16;
    if (d.kind >= PATCH_TILE_DENSE_Q4) {
        unpack_q4_tile(d, blob, wt, ldw);
    } else if (d.kind == PATCH_TILE_DENSE) {
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const uint32_t idx = it * 256 + threadIdx.x, r = idx >> 4, c = idx & 15u;
            const uint4 v = *reinterpret_cast<const uint4*>(pay + (c >> 3) * kAtomBytes + atom_chunk_offset(r, c & 7u));
            *reinterpret_cast<uint4*>(wt + int64_t(r) * ldw + c * 8) = v;
        }
    } else {
        const uint8_t* meta = blob + uint64_t(d.meta_off16) * 16;
#pragma unroll
        for (int it = 0; it < 4; ++it) {
            const uint32_t idx = it * 256 + threadIdx.x, r = idx >> 3, u = idx & 7u;
            const uint4 v = *reinterpret_cast<const uint4*>(pay + atom_chunk_offset(r, u));
            const uint32_t L = (r & ~15u) + 8u * (u & 1u) + (r & 7u), j = u >> 1, hi = (r >> 3) & 1u;
            const uint32_t code = *reinterpret_cast<const uint16_t*>(meta + L * 16 + j * 4 + hi * 2);
            const uint32_t in[4] = {v.x, v.y, v.z, v.w};
            uint32_t out[8];
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const uint32_t nib = (code >> (4 * g)) & 0xFu, i0 = nib & 3u, i1 = nib >> 2;
                uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
                for (int j2 = 0; j2 < 4; ++j2) {
                    if (uint32_t(j2) == i0) w[j2] = in[g] & 0xFFFFu;
                    if (uint32_t(j2) == i1) w[j2] = in[g] >> 16;
                }
                out[2 * g] = w[0] | (w[1] << 16);
                out[2 * g + 1] = w[2] | (w[3] << 16);
            }
            uint16_t* dst = wt + int64_t(r) * ldw + u * 16;
            *reinterpret_cast<uint4*>(dst) = make_uint4(out[0], out[1], out[2], out[3]);
            *reinterpret_cast<uint4*>(dst + 8) = make_uint4(out[4], out[5], out[6], out[7]);
        }
    }
}

// Layout of the bf16 blob that holds the dequantised values of an all-4-bit weight, and the expansion itself.
void q4_expanded_layout(const patch_layout_t* L, patch_layout_t* out) {
    *out = *L;
    out->n_dense = L->n_dense_q4;
    out->n_sparse = L->n_sparse_q4;
    out->n_dense_q4 = 0;
    out->n_sparse_q4 = 0;
    out->payload_bytes = uint64_t(kDenseBytes) * out->n_dense + uint64_t(kSparseBytes) * out->n_sparse;
    out->total_bytes = out->payload_off + out->payload_bytes;
}

int launch_expand_q4(const patch_layout_t* L, const uint8_t* packed, const patch_layout_t* out_layout, uint8_t* out,
                     int* status_dev, cudaStream_t stream) {
    const int64_t T = (L->N / kTile) * (L->K / kTile);
    // the padding behind the table (up to the first payload) is part of the blob
    if (cudaMemsetAsync(out + L->table_off + 16 * T, 0, L->payload_off - L->table_off - 16 * T, stream) != cudaSuccess)
        return PATCH_ERR_CUDA;
    expand_q4_kernel<<<unsigned(T), 256, 0, stream>>>(packed, L->table_off, uint32_t(L->payload_off), uint32_t(L->total_bytes / 16),
                                                      out, *out_layout, status_dev);
    return cudaGetLastError() == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

}  // namespace patch

using namespace patch;

extern "C" int patch_packed_size(int64_t N, int64_t K, int tile_n, int tile_k,
                                 const uint8_t* flags, patch_layout_t* out) {
    if (!flags || !out) return PATCH_ERR_NULL;
    if (tile_n != kTile || tile_k != kTile) return PATCH_ERR_TILE;
    if (N <= 0 || K <= 0 || N % kTile || K % kTile) return PATCH_ERR_SHAPE;
    const int64_t T = (N / kTile) * (K / kTile);
    int64_t n[4] = {0, 0, 0, 0};
    for (int64_t t = 0; t < T; ++t) {
        if (flags[t] > PATCH_TILE_SPARSE_2_4_Q4) return PATCH_ERR_FLAG;
        ++n[flags[t]];
    }
    patch_layout_t L;
    std::memset(&L, 0, sizeof L);
    L.magic = kMagic; L.version = kVersion;
    L.N = N; L.K = K; L.tile_n = kTile; L.tile_k = kTile;
    L.n_dense = n[PATCH_TILE_DENSE]; L.n_sparse = n[PATCH_TILE_SPARSE_2_4];
    L.n_dense_q4 = n[PATCH_TILE_DENSE_Q4]; L.n_sparse_q4 = n[PATCH_TILE_SPARSE_2_4_Q4];
    L.table_off = kHeaderBytes;
    L.payload_off = (kHeaderBytes + 16 * uint64_t(T) + 1023) / 1024 * 1024;
    L.payload_bytes = 0;
    for (uint32_t k = 0; k < 4; ++k) L.payload_bytes += uint64_t(tile_payload_bytes(k)) * uint64_t(n[k]);
    L.total_bytes = L.payload_off + L.payload_bytes;
    if (L.total_bytes / 16 > 0xFFFFFFF0ull) return PATCH_ERR_SHAPE;
    *out = L;
    return PATCH_OK;
}

static int pack_impl(const void* W_dev, int64_t ldw, const uint8_t* flags, const uint8_t* patterns_dev,
                     const patch_layout_t* L, void* packed_dev, size_t capacity, int* status_dev, void* stream) {
    if (!W_dev || !flags || !L || !packed_dev) return PATCH_ERR_NULL;
    int rc = validate_layout(L);
    if (rc) return rc;
    if (ldw < L->K || ldw % 8) return PATCH_ERR_SHAPE;
    if (!aligned16(W_dev) || !aligned16(packed_dev)) return PATCH_ERR_ALIGN;
    if (capacity < L->total_bytes) return PATCH_ERR_SIZE;
    const int64_t TK = L->K / kTile, T = (L->N / kTile) * TK;
    // header + tile table, built on the host from the flags
    std::vector<uint8_t> head(L->payload_off, 0);
    std::memcpy(head.data(), L, sizeof *L);
    TileDesc* table = reinterpret_cast<TileDesc*>(head.data() + L->table_off);
    uint64_t off = L->payload_off;
    int64_t n[4] = {0, 0, 0, 0};
    for (int64_t t = 0; t < T; ++t) {
        const uint32_t kind = flags[t];
        if (kind > PATCH_TILE_SPARSE_2_4_Q4) return PATCH_ERR_FLAG;
        TileDesc d = TileDesc{kind, uint32_t(off / 16), 0xFFFFFFFFu, 0};
        if (kind == PATCH_TILE_SPARSE_2_4) {
            d.meta_off16 = uint32_t((off + kAtomBytes) / 16);
        } else if (kind == PATCH_TILE_DENSE_Q4) {
            d.scales_off16 = uint32_t((off + kDenseQ4CodeBytes) / 16);
        } else if (kind == PATCH_TILE_SPARSE_2_4_Q4) {
            d.meta_off16 = uint32_t((off + kSparseQ4CodeBytes) / 16);
            d.scales_off16 = uint32_t((off + kSparseQ4CodeBytes + kMetaBytes) / 16);
        }
        table[t] = d;
        off += tile_payload_bytes(kind);
        ++n[kind];
    }
    if (n[0] != L->n_dense || n[1] != L->n_sparse || n[2] != L->n_dense_q4 || n[3] != L->n_sparse_q4)
        return PATCH_ERR_FORMAT;  // flags do not match the layout
    rc = check_device();
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // pageable source: the runtime stages it before returning, so `head` may die at scope exit
    if (cudaMemcpyAsync(packed_dev, head.data(), head.size(), cudaMemcpyHostToDevice, s) != cudaSuccess)
        return PATCH_ERR_CUDA;
    const DeviceFlags none = {nullptr, 0, 0, 0, 0};
    if (patterns_dev)
        pack_kernel<true, false><<<unsigned(T), 256, 0, s>>>(static_cast<const uint16_t*>(W_dev), ldw, int(TK),
                                                             static_cast<uint8_t*>(packed_dev), L->table_off, patterns_dev,
                                                             status_dev, none);
    else
        pack_kernel<false, false><<<unsigned(T), 256, 0, s>>>(static_cast<const uint16_t*>(W_dev), ldw, int(TK),
                                                              static_cast<uint8_t*>(packed_dev), L->table_off, nullptr,
                                                              nullptr, none);
    return cudaGetLastError() == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

extern "C" int patch_pack(const void* W_dev, int64_t ldw, const uint8_t* flags,
                          const patch_layout_t* L, void* packed_dev, size_t capacity, void* stream) {
    return pack_impl(W_dev, ldw, flags, nullptr, L, packed_dev, capacity, nullptr, stream);
}

extern "C" int patch_pack_patterns(const void* W_dev, int64_t ldw, const uint8_t* flags, const uint8_t* patterns_dev,
                                   const patch_layout_t* L, void* packed_dev, size_t capacity, int* status_dev,
                                   void* stream) {
    if (!patterns_dev) return PATCH_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(patterns_dev) & 3u) return PATCH_ERR_ALIGN;
    return pack_impl(W_dev, ldw, flags, patterns_dev, L, packed_dev, capacity, status_dev, stream);
}

extern "C" int patch_pack_dev(const void* W_dev, int64_t ldw, const uint8_t* flags_dev, const uint8_t* patterns_dev,
                              int64_t N, int64_t K, int tile_n, int tile_k, void* packed_dev, size_t capacity,
                              int* status_dev, void* stream) {
    if (!W_dev || !flags_dev || !packed_dev) return PATCH_ERR_NULL;
    if (tile_n != kTile || tile_k != kTile) return PATCH_ERR_TILE;
    if (N <= 0 || K <= 0 || N % kTile || K % kTile) return PATCH_ERR_SHAPE;
    if (ldw < K || ldw % 8) return PATCH_ERR_SHAPE;
    const int64_t TK = K / kTile, T = (N / kTile) * TK;
    if (T > 0x7FFFFFFF) return PATCH_ERR_SHAPE;
    if (!aligned16(W_dev) || !aligned16(packed_dev) || (patterns_dev && (reinterpret_cast<uintptr_t>(patterns_dev) & 3u)))
        return PATCH_ERR_ALIGN;
    const uint64_t payload_off = (kHeaderBytes + 16 * uint64_t(T) + 1023) / 1024 * 1024;
    if (capacity < payload_off + uint64_t(T) * kSparseQ4Bytes) return PATCH_ERR_SIZE;   // below the smallest possible blob
    int rc = check_device();
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* blob = static_cast<uint8_t*>(packed_dev);
    const DeviceFlags F = {flags_dev, T, N, K, uint64_t(capacity)};
    if (patterns_dev)
        pack_kernel<true, true><<<unsigned(T), 256, 0, s>>>(static_cast<const uint16_t*>(W_dev), ldw, int(TK), blob,
                                                            kHeaderBytes, patterns_dev, status_dev, F);
    else
        pack_kernel<false, true><<<unsigned(T), 256, 0, s>>>(static_cast<const uint16_t*>(W_dev), ldw, int(TK), blob,
                                                             kHeaderBytes, nullptr, status_dev, F);
    return cudaGetLastError() == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

extern "C" int patch_read_layout(const void* packed_dev, patch_layout_t* layout_out, void* stream) {
    if (!packed_dev || !layout_out) return PATCH_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    patch_layout_t L;
    if (cudaMemcpyAsync(&L, packed_dev, sizeof L, cudaMemcpyDeviceToHost, s) != cudaSuccess) return PATCH_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return PATCH_ERR_CUDA;
    const int rc = validate_layout(&L);
    if (rc) return rc;
    *layout_out = L;
    return PATCH_OK;
}

extern "C" int patch_unpack(const patch_layout_t* L, const void* packed_dev, void* What_dev,
                            int64_t ldw, void* stream) {
    if (!L || !packed_dev || !What_dev) return PATCH_ERR_NULL;
    int rc = validate_layout(L);
    if (rc) return rc;
    if (ldw < L->K || ldw % 8) return PATCH_ERR_SHAPE;
    if (!aligned16(What_dev) || !aligned16(packed_dev)) return PATCH_ERR_ALIGN;
    rc = check_device();
    if (rc) return rc;
    const int64_t TK = L->K / kTile, T = (L->N / kTile) * TK;
    unpack_kernel<<<unsigned(T), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const uint8_t*>(packed_dev), L->table_off, int(TK),
        static_cast<uint16_t*>(What_dev), ldw);
    return cudaGetLastError() == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}
