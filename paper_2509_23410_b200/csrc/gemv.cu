// Small-M (decode) variant of the hybrid tile matmul on the CUDA cores.
//
// The paper's deployment section names decode as the bottleneck of generation and split-K as
// the alternative schedule its inspector picks there (Appendix A).  For M <= 4 tokens the layer
// is a matrix-vector product bound by the bytes of the packed weight, so this kernel reads only
// the compressed payload, with coalesced 128-bit loads, and never expands a 2:4 tile in memory.
//
// Schedule: grid = (S, TN) with thread-block clusters of S CTAs along K.  CTA (s, tn) owns
// row-block tn (128 out-features) and the K-slice s of its tiles.  A warp reads 4 payload rows
// x 128 B per load instruction (512 contiguous bytes); lane l owns row 4*warp + l/8 (+32 per
// pass) and the 16-byte chunk l%8 of that row, so its slice of X stays in registers for all
// passes.  Per-lane fp32 partial sums are reduced over the 8 lanes of a row with warp shuffles,
// the S K-slices are then summed in fixed order through distributed shared memory, and the
// result is rounded to bf16 once.
#include <cooperative_groups.h>
#include "patch_internal.cuh"

namespace cg = cooperative_groups;

namespace patch {

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float bf_lo(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf_hi(uint32_t p) { return __uint_as_float(p & 0xFFFF0000u); }

__device__ __forceinline__ float dot8(const uint4& w, const uint4& x, float acc) {
    acc = fmaf(bf_lo(w.x), bf_lo(x.x), acc); acc = fmaf(bf_hi(w.x), bf_hi(x.x), acc);
    acc = fmaf(bf_lo(w.y), bf_lo(x.y), acc); acc = fmaf(bf_hi(w.y), bf_hi(x.y), acc);
    acc = fmaf(bf_lo(w.z), bf_lo(x.z), acc); acc = fmaf(bf_hi(w.z), bf_hi(x.z), acc);
    acc = fmaf(bf_lo(w.w), bf_lo(x.w), acc); acc = fmaf(bf_hi(w.w), bf_hi(x.w), acc);
    return acc;
}

// One group of four columns of a 2:4 tile: `v` holds the two kept values, `sel` the byte
// selector that gathers the two matching activations out of {x01, x23}.
__device__ __forceinline__ float dot_group(uint32_t v, uint32_t x01, uint32_t x23, uint32_t sel, float acc) {
    const uint32_t xp = __byte_perm(x01, x23, sel);
    acc = fmaf(bf_lo(v), bf_lo(xp), acc);
    return fmaf(bf_hi(v), bf_hi(xp), acc);
}

// One tile's worth of this lane's operands: 4 payload rows x one 16-byte chunk per K-half (dense: 8
// loads, 2:4: 4 loads + 4 metadata half-words), and the matching activations.
template <int M_MAX>
struct TileRegs {
    uint4 w[8];
    uint32_t code[4];
    uint4 x[2][M_MAX];     // dense: columns 64h + 8c .. +8 for h = 0, 1; 2:4: columns 16c .. 16c+15 as two vectors
    uint32_t kind;
};

template <int M_MAX>
__device__ __forceinline__ void load_tile(TileRegs<M_MAX>& t, const TileDesc& d, const uint8_t* __restrict__ blob,
                                          const __nv_bfloat16* __restrict__ X, int64_t ldx, int M, int tk,
                                          uint32_t row0, uint32_t c) {
    const uint8_t* pay = blob + uint64_t(d.payload_off16) * 16;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    t.kind = d.kind;
    if (d.kind == PATCH_TILE_DENSE) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
#pragma unroll
            for (int p = 0; p < 4; ++p)
                t.w[4 * h + p] = ldg_stream(pay + h * kAtomBytes + atom_chunk_offset(row0 + 32u * p, c));
#pragma unroll
            for (int m = 0; m < M_MAX; ++m)
                t.x[h][m] = m < M ? __ldg(reinterpret_cast<const uint4*>(X + int64_t(m) * ldx + int64_t(tk) * kTile + 64 * h + 8 * c))
                                  : zero4;
        }
    } else {
        const uint8_t* meta = pay + kAtomBytes;      // the metadata block follows the kept values
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const uint32_t r = row0 + 32u * p;
            t.w[p] = ldg_stream(pay + atom_chunk_offset(r, c));
            // metadata row L = 16q + 8h + i, word j; chunk c covers columns [16c, 16c+16): j = c/2, h = c%2
            const uint32_t L = (r & ~15u) + 8u * (c & 1u) + (r & 7u);
            t.code[p] = __ldg(reinterpret_cast<const uint16_t*>(meta + L * 16 + (c >> 1) * 4 + ((r >> 3) & 1u) * 2));
        }
#pragma unroll
        for (int m = 0; m < M_MAX; ++m) {
            const uint4* px = reinterpret_cast<const uint4*>(X + int64_t(m) * ldx + int64_t(tk) * kTile + 16 * c);
            t.x[0][m] = m < M ? __ldg(px) : zero4;
            t.x[1][m] = m < M ? __ldg(px + 1) : zero4;
        }
    }
}

template <int M_MAX>
__device__ __forceinline__ void fma_tile(const TileRegs<M_MAX>& t, float (&acc)[4][M_MAX]) {
    if (t.kind == PATCH_TILE_DENSE) {
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int p = 0; p < 4; ++p)
#pragma unroll
                for (int m = 0; m < M_MAX; ++m) acc[p][m] = dot8(t.w[4 * h + p], t.x[h][m], acc[p][m]);
    } else {
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            uint32_t sel[4];
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                const uint32_t nib = (t.code[p] >> (4 * g)) & 0xFu, i0 = nib & 3u, i1 = nib >> 2;
                sel[g] = (i0 * 0x22u + 0x10u) | ((i1 * 0x22u + 0x10u) << 8);
            }
#pragma unroll
            for (int m = 0; m < M_MAX; ++m) {
                float a = acc[p][m];
                a = dot_group(t.w[p].x, t.x[0][m].x, t.x[0][m].y, sel[0], a);
                a = dot_group(t.w[p].y, t.x[0][m].z, t.x[0][m].w, sel[1], a);
                a = dot_group(t.w[p].z, t.x[1][m].x, t.x[1][m].y, sel[2], a);
                a = dot_group(t.w[p].w, t.x[1][m].z, t.x[1][m].w, sel[3], a);
                acc[p][m] = a;
            }
        }
    }
}

template <int M_MAX>
__global__ void __launch_bounds__(256)
gemv_kernel(const __nv_bfloat16* __restrict__ X, int64_t ldx, int M,
            const uint8_t* __restrict__ blob, uint64_t table_off, uint32_t pay0_16, uint32_t end16, int TK,
            __nv_bfloat16* __restrict__ Y, int64_t ldy, int* status_dev) {
    cg::cluster_group cluster = cg::this_cluster();
    // programmatic dependent launch: let the next kernel start its prologue, then wait until the
    // previous kernel's results (X, and the last readers of Y) are complete
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int S = gridDim.x, s = blockIdx.x, tn = blockIdx.y;
    const int tk0 = int(int64_t(s) * TK / S), tk1 = int(int64_t(s + 1) * TK / S);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t c = lane & 7u;            // logical 16-byte chunk of the payload row
    const uint32_t row0 = 4u * warp + (lane >> 3);

    __shared__ float part[M_MAX][kTile];     // this CTA's K-slice partial sums
    __shared__ TileDesc descs[256];          // tile descriptors of the slice, staged 256 at a time

    float acc[4][M_MAX];
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int m = 0; m < M_MAX; ++m) acc[p][m] = 0.f;

    const TileDesc* table = reinterpret_cast<const TileDesc*>(blob + table_off) + int64_t(tn) * TK;
    // Register double buffer: the loads of tile i+1 are in flight while tile i is multiplied.
    TileRegs<M_MAX> cur, nxt;
    for (int base = tk0; base < tk1; base += 256) {
        const int n = tk1 - base < 256 ? tk1 - base : 256;
        __syncthreads();
        if (int(threadIdx.x) < n) {
            TileDesc d = table[base + threadIdx.x];
            sanitize_tile(d.kind, d.payload_off16, pay0_16, end16, status_dev);     // checked once, before any tile byte is read
            descs[threadIdx.x] = d;
        }
        __syncthreads();
        load_tile<M_MAX>(cur, descs[0], blob, X, ldx, M, base, row0, c);
        for (int i = 0; i < n; ++i) {
            if (i + 1 < n) load_tile<M_MAX>(nxt, descs[i + 1], blob, X, ldx, M, base + i + 1, row0, c);
            fma_tile<M_MAX>(cur, acc);
            if (i + 1 < n) cur = nxt;
        }
    }

    // reduce over the 8 lanes that share a row
#pragma unroll
    for (int p = 0; p < 4; ++p)
#pragma unroll
        for (int m = 0; m < M_MAX; ++m) {
            float a = acc[p][m];
            a += __shfl_xor_sync(0xFFFFFFFFu, a, 1);
            a += __shfl_xor_sync(0xFFFFFFFFu, a, 2);
            a += __shfl_xor_sync(0xFFFFFFFFu, a, 4);
            if (c == 0) part[m][row0 + 32u * p] = a;
        }
    cluster.sync();
    // sum the S K-slices in slice order; CTA s finishes an interleaved share of the outputs
    for (int idx = threadIdx.x + 256 * s; idx < M * kTile; idx += 256 * S) {
        const int m = idx >> 7, r = idx & 127;
        float a = 0.f;
        for (int q = 0; q < S; ++q) a += cluster.map_shared_rank(&part[0][0], q)[m * kTile + r];
        Y[int64_t(m) * ldy + int64_t(tn) * kTile + r] = __float2bfloat16_rn(a);
    }
    cluster.sync();  // keep shared memory alive until every peer has read it
}

// Split count: enough CTAs to fill the GPU about twice over, at most 8 (portable cluster size).
static int pick_splits(int TN, int TK) {
    int best = 1;
    for (int S = 1; S <= 8 && S <= TK; ++S)
        if (TN * S <= 2 * 148 || S == 1) best = S;
    return best;
}

template <int M_MAX>
static int launch_gemv_t(const __nv_bfloat16* X, int64_t ldx, int M, const patch_layout_t* L,
                         const uint8_t* packed, __nv_bfloat16* Y, int64_t ldy, int* status_dev, cudaStream_t stream) {
    const int TN = int(L->N / kTile), TK = int(L->K / kTile);
    const int S = pick_splits(TN, TK);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(S, TN, 1);
    cfg.blockDim = dim3(256, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = S;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    cudaError_t e = cudaLaunchKernelEx(&cfg, gemv_kernel<M_MAX>, X, ldx, M, packed, uint64_t(L->table_off),
                                       uint32_t(L->payload_off / 16), uint32_t(L->total_bytes / 16), TK, Y, ldy, status_dev);
    return e == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

int launch_gemv(const __nv_bfloat16* X, int64_t ldx, int M, const patch_layout_t* L,
                const uint8_t* packed, __nv_bfloat16* Y, int64_t ldy, int* status_dev,
                cudaStream_t stream) {
    if (M < 1 || M > 4) return PATCH_ERR_SHAPE;
    if (L->N / kTile > 65535) return PATCH_ERR_SHAPE;
    if (M == 1) return launch_gemv_t<1>(X, ldx, M, L, packed, Y, ldy, status_dev, stream);
    if (M == 2) return launch_gemv_t<2>(X, ldx, M, L, packed, Y, ldy, status_dev, stream);
    return launch_gemv_t<4>(X, ldx, M, L, packed, Y, ldy, status_dev, stream);
}

}  // namespace patch
