/*
 * CPU oracle for the tile-hybrid linear layer  Y = X * What^T  of PATCH.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, obviously-correct C.  Nothing in the product path
 * may call into this file; it shares no code, header or table with the CUDA library.
 *
 * What it computes, and the passage of the paper each step follows:
 *   - hard mask  M* = M*_tile + (1 - M*_tile) (.) M*_2:4   (Algorithm 1, last three lines; Eq. 4
 *     in its hard form).  M*_tile is 1 on tiles flagged dense; M*_2:4 keeps two of every four
 *     consecutive elements along K (Preliminaries, "Learnable 2:4 Mask": six candidate patterns
 *     per group of four).  The 2:4 mask itself is magnitude top-2 per group, the selection the
 *     workloads fix; ties go to the lower index.
 *   - pruned weight  What = W (.) M*  (last line of Algorithm 1), done as a select so
 *     that a pruned element is +0.
 *   - compression of the mixed matrix into kept values + metadata, per tile (Appendix A:
 *     the tile size fixes how the matrix is compressed and its metadata laid out);
 *     two metadata bits per kept value, the cost that reproduces the compression-ratio column
 *     of the 4-bit quantisation table.
 *   - 4-bit weight-only quantisation of the stored values of a tile (section "Combination with other
 *     compression methods", the 4-bit quantisation table).  The paper prints only the compression-ratio
 *     column -- 4 bits per stored value plus the 2 metadata bits per kept value, 16 / (4 - f) -- and no
 *     quantiser; the reading taken here: symmetric, round to nearest even, one bf16 scale per tile row
 *     (the 128 weights of a dense tile's row, the 64 kept values of a 2:4 tile's row),
 *         s = bf16(max|v| / 7),  q = clamp(rint(v / s), -7, 7)  (q = 0 where s = 0),  v^ = bf16(q * s),
 *     all in fp32 on bf16 inputs; the 2:4 selection is made first, on the unquantised weights.
 *   - the linear layer itself, on the same bf16-rounded inputs, accumulated in double (and in
 *     plain fp32 as a cross-check) in k order.
 *   - (last section of the file) the masks of the learning procedure: the Gumbel-softmax soft masks
 *     of Eq. 2-4 with the noise of Eq. 1 drawn from a counter-based generator, the per-matrix sums
 *     and the two regularisers of Eq. 5, the hard masks Algorithm 1 reads off the logits, and the
 *     compression with that given 2:4 mask instead of the magnitude rule.
 *
 * Pins: every function here is pinned by tests that do not call it to produce their expected
 * value (brute force over the six patterns, closed-form byte counts, numpy matmul, round trips,
 * hand-written fixtures; for the mask-learning part: scipy's softmax, closed forms, the
 * Gumbel-max property, the tau -> 0 limit that joins soft and hard masks).  No function is
 * "parity unpinned".
 *
 * Conventions: W is [N x K] row-major bf16 (uint16 bit patterns), N = out-features,
 * K = in-features; X is [M x K]; Y is [M x N].  flags[tn*TK + tk]: 0 = dense, 1 = 2:4,
 * 2 = dense with 4-bit values, 3 = 2:4 with 4-bit values.
 */
#include <stdint.h>
#include <stddef.h>
#include <string.h>
#include <stdlib.h>
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_MAGIC   0x48435450u /* "PTCH" little-endian */
#define ORACLE_VERSION 1u
#define KIND_DENSE  0u
#define KIND_SPARSE 1u
#define KIND_DENSE_Q4  2u     /* kind & 1: 2:4;  kind & 2: values stored as 4-bit codes + one scale per tile row */
#define KIND_SPARSE_Q4 3u

typedef struct {
    uint32_t magic, version;
    int64_t  N, K;
    int32_t  tile_n, tile_k;
    int64_t  n_dense, n_sparse;
    uint64_t table_off, payload_off, payload_bytes, total_bytes;
    int64_t  n_dense_q4, n_sparse_q4;
} oracle_layout_t;

/* ------------------------------------------------------------------------------------------- */
/* bf16 helpers (exact widening; round-to-nearest-even narrowing)                               */

static float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

static uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((u >> 16) | 0x0040u); /* NaN stays NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return (uint16_t)(u >> 16);
}

/* ------------------------------------------------------------------------------------------- */
/* 4-bit quantiser of one group of stored values (see the header): scale, codes, dequantised values. */

static uint16_t q4_scale(const uint16_t* v, int n) {
    float m = 0.0f;
    for (int i = 0; i < n; ++i) {
        float a = fabsf(bf16_to_f32(v[i]));
        if (a > m) m = a;
    }
    return f32_to_bf16_rne(m / 7.0f);
}
static int q4_code(uint16_t v, uint16_t scale) {            /* q in [-7, 7] */
    float s = bf16_to_f32(scale);
    if (s == 0.0f) return 0;
    float r = rintf(bf16_to_f32(v) / s);                    /* nearest, ties to even */
    if (r > 7.0f) r = 7.0f;
    if (r < -7.0f) r = -7.0f;
    return (int)r;
}
static uint16_t q4_value(int q, uint16_t scale) {           /* bf16(q * s): the product is exact in fp32 */
    return f32_to_bf16_rne((float)q * bf16_to_f32(scale));
}
/* exported for the tests: quantise n values -> scale, codes (q + 8 in 1..15), dequantised values */
int oracle_q4_group(const uint16_t* v, int n, uint16_t* scale, uint8_t* codes, uint16_t* deq) {
    if (!v || !scale || n <= 0) return -1;
    *scale = q4_scale(v, n);
    for (int i = 0; i < n; ++i) {
        int q = q4_code(v[i], *scale);
        if (codes) codes[i] = (uint8_t)(q + 8);
        if (deq) deq[i] = q4_value(q, *scale);
    }
    return 0;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------------------------------- */
/* 2:4 selection inside one group of four: keep the two largest |w|; equal magnitudes are       */
/* ordered by position, lower first.  Magnitude is the bf16 bit pattern without its sign bit,   */
/* which orders finite values exactly like |w| (and +0 == -0).                                  */

static void select_top2(const uint16_t w[4], int keep[4]) {
    for (int j = 0; j < 4; ++j) {
        uint32_t mj = w[j] & 0x7FFFu;
        int rank = 0; /* how many elements come before j in (magnitude desc, index asc) order */
        for (int l = 0; l < 4; ++l) {
            uint32_t ml = w[l] & 0x7FFFu;
            if (ml > mj || (ml == mj && l < j)) ++rank;
        }
        keep[j] = rank < 2;
    }
}

static int check_shape(int64_t N, int64_t K, int tile_n, int tile_k) {
    if (N <= 0 || K <= 0 || tile_n <= 0 || tile_k <= 0) return -2;
    if (tile_k % 4 != 0) return -3;
    if (N % tile_n != 0 || K % tile_k != 0) return -2;
    return 0;
}

/* Hard mask M* as bytes (1 = keep).  Algorithm 1: M* = M*_tile + (1 - M*_tile) (.) M*_2:4. */
int oracle_mask(const uint16_t* W, int64_t N, int64_t K, const uint8_t* flags,
                int tile_n, int tile_k, uint8_t* mask) {
    int rc = check_shape(N, K, tile_n, tile_k);
    if (rc) return rc;
    int64_t TK = K / tile_k;
    for (int64_t t = 0; t < (N / tile_n) * TK; ++t)
        if (flags[t] > 3) return -4;
    for (int64_t n = 0; n < N; ++n) {
        for (int64_t g = 0; g < K / 4; ++g) {
            int64_t k0 = 4 * g;
            int m_tile = (flags[(n / tile_n) * TK + k0 / tile_k] & 1u) == 0;   /* 1 = dense tile (bf16 or 4-bit) */
            int keep[4];
            select_top2(&W[n * K + k0], keep);
            for (int j = 0; j < 4; ++j)
                mask[n * K + k0 + j] = (uint8_t)(m_tile + (1 - m_tile) * keep[j]);
        }
    }
    return 0;
}

/* What = W (.) M*  as a select: kept elements verbatim, pruned elements +0. */
int oracle_prune(const uint16_t* W, int64_t N, int64_t K, const uint8_t* flags,
                 int tile_n, int tile_k, uint16_t* What) {
    uint8_t* mask = (uint8_t*)malloc((size_t)(N * K));
    if (!mask) return -6;
    int rc = oracle_mask(W, N, K, flags, tile_n, tile_k, mask);
    if (rc == 0)
        for (int64_t i = 0; i < N * K; ++i) What[i] = mask[i] ? W[i] : (uint16_t)0;
    /* tiles with 4-bit values: what the layer multiplies is the dequantised kept value; the group that shares a
     * scale is the tile row's stored values (all of them in a dense tile, the kept ones in a 2:4 tile) */
    if (rc == 0) {
        int64_t TK = K / tile_k;
        uint16_t* v = (uint16_t*)malloc((size_t)tile_k * 2);
        if (!v) { free(mask); return -6; }
        for (int64_t n = 0; n < N; ++n)
            for (int64_t tk = 0; tk < TK; ++tk) {
                if ((flags[(n / tile_n) * TK + tk] & 2u) == 0) continue;
                int cnt = 0;
                for (int c = 0; c < tile_k; ++c)
                    if (mask[n * K + tk * tile_k + c]) v[cnt++] = W[n * K + tk * tile_k + c];
                uint16_t s = q4_scale(v, cnt);
                for (int c = 0; c < tile_k; ++c)
                    if (mask[n * K + tk * tile_k + c])
                        What[n * K + tk * tile_k + c] = q4_value(q4_code(W[n * K + tk * tile_k + c], s), s);
            }
        free(v);
    }
    free(mask);
    return rc;
}

/* ------------------------------------------------------------------------------------------- */
static uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

/* Canonical packed blob:
 *   [ header 256 B | table: 16 B per tile, padded to 1024 B | payloads ]
 * Tile order t = tn*TK + tk.  Dense payload: tile_n rows x tile_k bf16, row-major.
 * 2:4 payload: vals[tile_n][tile_k/2] bf16 (the two kept elements of each group, in position
 * order; the block is padded to a multiple of 16 B) followed by meta[tile_n][words]
 * little-endian uint32, words = ceil(tile_k/32); the nibble of group g sits at bits
 * [4*(g%8), +4) of word g/8 and equals i0 | (i1 << 2) with i0 < i1 the kept positions.
 * Payloads are aligned to 1024 B for 128x128 tiles, 16 B otherwise.
 * Table entry: { u32 kind, u32 payload_off/16, u32 meta_off/16 (0xFFFFFFFF if dense), u32 0 },
 * offsets from the start of the blob. */

static uint64_t payload_align(int tile_n, int tile_k) {
    return (tile_n == 128 && tile_k == 128) ? 1024u : 16u;
}
static uint64_t dense_bytes(int tile_n, int tile_k) { return (uint64_t)tile_n * tile_k * 2; }
static uint64_t meta_words(int tile_k) { return (uint64_t)(tile_k + 31) / 32; }
/* kept values of a 2:4 tile, padded to 16 B so that the metadata offset is expressible */
static uint64_t vals_bytes(int tile_n, int tile_k) {
    return round_up((uint64_t)tile_n * (tile_k / 2) * 2, 16);
}
static uint64_t sparse_bytes(int tile_n, int tile_k) {
    return vals_bytes(tile_n, tile_k) + (uint64_t)tile_n * meta_words(tile_k) * 4;
}
/* 4-bit kinds: [codes: value c of row r in byte r * (vals / 2) + c / 2, even c in the low nibble, code = q + 8;
 * padded to 16 B | metadata as for the 2:4 kind (2:4 only) | scales: tile_n bf16, padded to 16 B].
 * Payloads of 128x128 tiles are aligned to 256 B (8 448 B and 6 400 B), 16 B otherwise. */
static uint64_t q4_codes_bytes(int tile_n, int vals_per_row) { return round_up((uint64_t)tile_n * vals_per_row / 2, 16); }
static uint64_t q4_scales_bytes(int tile_n) { return round_up((uint64_t)tile_n * 2, 16); }
static uint64_t dense_q4_bytes(int tile_n, int tile_k) { return q4_codes_bytes(tile_n, tile_k) + q4_scales_bytes(tile_n); }
static uint64_t sparse_q4_bytes(int tile_n, int tile_k) {
    return q4_codes_bytes(tile_n, tile_k / 2) + (uint64_t)tile_n * meta_words(tile_k) * 4 + q4_scales_bytes(tile_n);
}
static uint64_t q4_align(int tile_n, int tile_k) { return (tile_n == 128 && tile_k == 128) ? 256u : 16u; }
static uint64_t kind_bytes(uint32_t kind, int tile_n, int tile_k) {       /* aligned size of a payload */
    switch (kind) {
        case KIND_DENSE: return round_up(dense_bytes(tile_n, tile_k), payload_align(tile_n, tile_k));
        case KIND_SPARSE: return round_up(sparse_bytes(tile_n, tile_k), payload_align(tile_n, tile_k));
        case KIND_DENSE_Q4: return round_up(dense_q4_bytes(tile_n, tile_k), q4_align(tile_n, tile_k));
        default: return round_up(sparse_q4_bytes(tile_n, tile_k), q4_align(tile_n, tile_k));
    }
}

int oracle_packed_size(int64_t N, int64_t K, int tile_n, int tile_k, const uint8_t* flags,
                       oracle_layout_t* L) {
    int rc = check_shape(N, K, tile_n, tile_k);
    if (rc) return rc;
    int64_t T = (N / tile_n) * (K / tile_k);
    int64_t nd = 0, ns = 0, ndq = 0, nsq = 0;
    uint64_t bytes = 0;
    for (int64_t t = 0; t < T; ++t) {
        if (flags[t] == KIND_DENSE) ++nd;
        else if (flags[t] == KIND_SPARSE) ++ns;
        else if (flags[t] == KIND_DENSE_Q4) ++ndq;
        else if (flags[t] == KIND_SPARSE_Q4) ++nsq;
        else return -4;
        bytes += kind_bytes(flags[t], tile_n, tile_k);
    }
    memset(L, 0, sizeof *L);
    L->magic = ORACLE_MAGIC; L->version = ORACLE_VERSION;
    L->N = N; L->K = K; L->tile_n = tile_n; L->tile_k = tile_k;
    L->n_dense = nd; L->n_sparse = ns; L->n_dense_q4 = ndq; L->n_sparse_q4 = nsq;
    L->table_off = 256;
    L->payload_off = round_up(256 + 16 * (uint64_t)T, 1024);
    L->payload_bytes = bytes;
    L->total_bytes = L->payload_off + bytes;
    return 0;
}

static void write_header_and_table(const oracle_layout_t* L, const uint8_t* flags, uint8_t* blob) {
    memset(blob, 0, (size_t)L->payload_off);
    memcpy(blob, L, sizeof *L);
    int64_t T = (L->N / L->tile_n) * (L->K / L->tile_k);
    uint64_t off = L->payload_off;
    int tn_ = L->tile_n, tk_ = L->tile_k;
    uint32_t* table = (uint32_t*)(blob + L->table_off);
    for (int64_t t = 0; t < T; ++t) {
        /* { kind, payload / 16, metadata / 16 (0xFFFFFFFF if none), scales / 16 (0 if none) } */
        table[4 * t + 0] = flags[t];
        table[4 * t + 1] = (uint32_t)(off / 16);
        table[4 * t + 2] = 0xFFFFFFFFu;
        table[4 * t + 3] = 0;
        if (flags[t] == KIND_SPARSE) {
            table[4 * t + 2] = (uint32_t)((off + vals_bytes(tn_, tk_)) / 16);
        } else if (flags[t] == KIND_DENSE_Q4) {
            table[4 * t + 3] = (uint32_t)((off + q4_codes_bytes(tn_, tk_)) / 16);
        } else if (flags[t] == KIND_SPARSE_Q4) {
            uint64_t m = off + q4_codes_bytes(tn_, tk_ / 2);
            table[4 * t + 2] = (uint32_t)(m / 16);
            table[4 * t + 3] = (uint32_t)((m + (uint64_t)tn_ * meta_words(tk_) * 4) / 16);
        }
        off += kind_bytes(flags[t], tn_, tk_);
    }
}

/* S: the six 2:4 candidates ("Learnable 2:4 Mask": the matrix whose rows are the candidate masks).
 * The paper does not print the row order; rows are taken in lexicographic order of the kept positions. */
static const uint8_t S_24[6][4] = {
    {1, 1, 0, 0}, {1, 0, 1, 0}, {1, 0, 0, 1}, {0, 1, 1, 0}, {0, 1, 0, 1}, {0, 0, 1, 1}};

/* patterns == NULL: magnitude top-2 per group; otherwise group (n, g) keeps row patterns[n*K/4 + g] of S. */
static int pack_impl(const uint16_t* W, const uint8_t* flags, const uint8_t* patterns,
                     const oracle_layout_t* L, uint8_t* blob, uint64_t capacity) {
    if (!W || !flags || !L || !blob) return -1;
    if (L->magic != ORACLE_MAGIC || L->version != ORACLE_VERSION) return -7;
    if (capacity < L->total_bytes) return -6;
    int tn_ = L->tile_n, tk_ = L->tile_k;
    int64_t N = L->N, K = L->K, TN = N / tn_, TK = K / tk_;
    memset(blob, 0, (size_t)L->total_bytes);
    write_header_and_table(L, flags, blob);
    const uint32_t* table = (const uint32_t*)(blob + L->table_off);
    for (int64_t tn = 0; tn < TN; ++tn)
        for (int64_t tk = 0; tk < TK; ++tk) {
            int64_t t = tn * TK + tk;
            uint8_t* pay = blob + (uint64_t)table[4 * t + 1] * 16;
            uint32_t kind = table[4 * t + 0];
            uint16_t* rowbuf = NULL;     /* 4-bit kinds: the stored values of the tile, row by row, before quantisation */
            if (kind & 2u) {
                rowbuf = (uint16_t*)malloc((size_t)tn_ * tk_ * 2);
                if (!rowbuf) return -6;
            }
            if ((kind & 1u) == 0) {
                uint16_t* d = (kind & 2u) ? rowbuf : (uint16_t*)pay;
                for (int r = 0; r < tn_; ++r)
                    for (int c = 0; c < tk_; ++c)
                        d[r * tk_ + c] = W[(tn * tn_ + r) * K + tk * tk_ + c];
            } else {
                uint16_t* vals = (kind & 2u) ? rowbuf : (uint16_t*)pay;
                uint32_t* meta = (uint32_t*)(blob + (uint64_t)table[4 * t + 2] * 16);
                int words = (int)meta_words(tk_);
                for (int r = 0; r < tn_; ++r)
                    for (int g = 0; g < tk_ / 4; ++g) {
                        const uint16_t* w = &W[(tn * tn_ + r) * K + tk * tk_ + 4 * g];
                        int keep[4], pos[2], cnt = 0;
                        if (patterns) {
                            uint8_t c = patterns[(tn * tn_ + r) * (K / 4) + (tk * tk_) / 4 + g];
                            if (c > 5) return -4;
                            for (int j = 0; j < 4; ++j) keep[j] = S_24[c][j];
                        } else {
                            select_top2(w, keep);
                        }
                        for (int j = 0; j < 4; ++j) if (keep[j]) pos[cnt++] = j;
                        vals[r * (tk_ / 2) + 2 * g + 0] = w[pos[0]];
                        vals[r * (tk_ / 2) + 2 * g + 1] = w[pos[1]];
                        uint32_t nib = (uint32_t)pos[0] | ((uint32_t)pos[1] << 2);
                        meta[r * words + g / 8] |= nib << (4 * (g % 8));
                    }
            }
            if (kind & 2u) {
                /* quantise the stored values row by row: codes into the payload, one scale per row behind them */
                int n_vals = (kind & 1u) ? tk_ / 2 : tk_;
                uint16_t* scales = (uint16_t*)(blob + (uint64_t)table[4 * t + 3] * 16);
                for (int r = 0; r < tn_; ++r) {
                    const uint16_t* v = &rowbuf[r * n_vals];
                    uint16_t s = q4_scale(v, n_vals);
                    scales[r] = s;
                    for (int c = 0; c < n_vals; ++c) {
                        uint8_t code = (uint8_t)(q4_code(v[c], s) + 8);
                        pay[(r * n_vals + c) / 2] |= (uint8_t)(code << (4 * (c & 1)));
                    }
                }
                free(rowbuf);
            }
        }
    return 0;
}

int oracle_pack(const uint16_t* W, const uint8_t* flags, const oracle_layout_t* L,
                uint8_t* blob, uint64_t capacity) {
    return pack_impl(W, flags, NULL, L, blob, capacity);
}

/* The same compression with the 2:4 mask given (the per-group candidate that Algorithm 1 keeps at the end),
 * one candidate index per group of four; groups inside dense tiles ignore theirs. */
int oracle_pack_patterns(const uint16_t* W, const uint8_t* flags, const uint8_t* patterns,
                         const oracle_layout_t* L, uint8_t* blob, uint64_t capacity) {
    if (!patterns) return -1;
    return pack_impl(W, flags, patterns, L, blob, capacity);
}

/* Inverse of oracle_pack: canonical blob -> What [N x K]. */
int oracle_unpack(const uint8_t* blob, uint64_t blob_bytes, uint16_t* What) {
    if (!blob || !What) return -1;
    if (blob_bytes < sizeof(oracle_layout_t)) return -6;
    oracle_layout_t L;
    memcpy(&L, blob, sizeof L);
    if (L.magic != ORACLE_MAGIC || L.version != ORACLE_VERSION) return -7;
    if (blob_bytes < L.total_bytes) return -6;
    int tn_ = L.tile_n, tk_ = L.tile_k;
    int64_t K = L.K, TN = L.N / tn_, TK = K / tk_;
    const uint32_t* table = (const uint32_t*)(blob + L.table_off);
    for (int64_t tn = 0; tn < TN; ++tn)
        for (int64_t tk = 0; tk < TK; ++tk) {
            int64_t t = tn * TK + tk;
            const uint8_t* pay = blob + (uint64_t)table[4 * t + 1] * 16;
            if (table[4 * t + 0] == KIND_DENSE) {
                const uint16_t* d = (const uint16_t*)pay;
                for (int r = 0; r < tn_; ++r)
                    for (int c = 0; c < tk_; ++c)
                        What[(tn * tn_ + r) * K + tk * tk_ + c] = d[r * tk_ + c];
            } else if (table[4 * t + 0] == KIND_SPARSE) {
                const uint16_t* vals = (const uint16_t*)pay;
                const uint32_t* meta = (const uint32_t*)(blob + (uint64_t)table[4 * t + 2] * 16);
                int words = (int)meta_words(tk_);
                for (int r = 0; r < tn_; ++r)
                    for (int g = 0; g < tk_ / 4; ++g) {
                        uint16_t* w = &What[(tn * tn_ + r) * K + tk * tk_ + 4 * g];
                        uint32_t nib = (meta[r * words + g / 8] >> (4 * (g % 8))) & 0xFu;
                        int i0 = (int)(nib & 3u), i1 = (int)(nib >> 2);
                        if (i0 >= i1) return -7;
                        w[0] = w[1] = w[2] = w[3] = 0;
                        w[i0] = vals[r * (tk_ / 2) + 2 * g + 0];
                        w[i1] = vals[r * (tk_ / 2) + 2 * g + 1];
                    }
            } else if (table[4 * t + 0] == KIND_DENSE_Q4 || table[4 * t + 0] == KIND_SPARSE_Q4) {
                int sparse = table[4 * t + 0] == KIND_SPARSE_Q4;
                int n_vals = sparse ? tk_ / 2 : tk_;
                const uint16_t* scales = (const uint16_t*)(blob + (uint64_t)table[4 * t + 3] * 16);
                const uint32_t* meta = sparse ? (const uint32_t*)(blob + (uint64_t)table[4 * t + 2] * 16) : NULL;
                int words = (int)meta_words(tk_);
                for (int r = 0; r < tn_; ++r) {
                    uint16_t* wrow = &What[(tn * tn_ + r) * K + tk * tk_];
                    for (int c = 0; c < tk_; ++c) wrow[c] = 0;
                    for (int c = 0; c < n_vals; ++c) {
                        int code = (pay[(r * n_vals + c) / 2] >> (4 * (c & 1))) & 0xF;
                        if (code == 0) return -7;                       /* q + 8 lies in 1..15 */
                        uint16_t v = q4_value(code - 8, scales[r]);
                        if (!sparse) { wrow[c] = v; continue; }
                        int g = c / 2;
                        uint32_t nib = (meta[r * words + g / 8] >> (4 * (g % 8))) & 0xFu;
                        int i0 = (int)(nib & 3u), i1 = (int)(nib >> 2);
                        if (i0 >= i1) return -7;
                        wrow[4 * g + ((c & 1) ? i1 : i0)] = v;
                    }
                }
            } else return -7;
        }
    return 0;
}

/* ------------------------------------------------------------------------------------------- */
/* Device image (128x128 tiles only): a per-tile bijection of the canonical payload bytes.      */
/* Header and table are identical to the canonical blob.                                        */
/*                                                                                              */
/* Values are stored as "swizzled K-major atoms" of 128 rows x 64 bf16 (16 384 B): row r, 16-B  */
/* chunk c (8 elements) of the 128-B row lives at                                               */
/*      (r / 8) * 1024 + (r % 8) * 128 + ((c ^ (r % 8)) * 16).                                  */
/* A dense tile is two atoms (columns 0..63, then 64..127); a 2:4 tile is one atom holding its  */
/* 64 kept values per row.                                                                      */
/*                                                                                              */
/* Metadata (2 048 B) is stored as 128 rows of four uint32.  Row L = 16*q + 8*h + i (i < 8),    */
/* word j (the j-th run of 32 columns): low 16 bits = the four nibbles of tile row 16q+i for    */
/* columns [32j + 16h, 32j + 16h + 16), high 16 bits = the same for tile row 16q+8+i.           */

static uint64_t atom_offset(int r, int col) { /* col in [0,64): element column inside the atom */
    int chunk = col / 8, within = col % 8;
    return (uint64_t)(r / 8) * 1024 + (uint64_t)(r % 8) * 128 + (uint64_t)((chunk ^ (r % 8)) * 16)
           + (uint64_t)within * 2;
}

int oracle_device_image(const uint8_t* canon, uint64_t blob_bytes, uint8_t* image) {
    if (!canon || !image) return -1;
    if (blob_bytes < sizeof(oracle_layout_t)) return -6;
    oracle_layout_t L;
    memcpy(&L, canon, sizeof L);
    if (L.magic != ORACLE_MAGIC || L.version != ORACLE_VERSION) return -7;
    if (L.tile_n != 128 || L.tile_k != 128) return -3;
    if (blob_bytes < L.total_bytes) return -6;
    memcpy(image, canon, (size_t)L.payload_off);
    int64_t T = (L.N / 128) * (L.K / 128);
    const uint32_t* table = (const uint32_t*)(canon + L.table_off);
    for (int64_t t = 0; t < T; ++t) {
        uint64_t off = (uint64_t)table[4 * t + 1] * 16;
        if (table[4 * t + 0] == KIND_DENSE_Q4 || table[4 * t + 0] == KIND_SPARSE_Q4) {
            /* 4-bit kinds: scales are stored as they are; the metadata of the 2:4 kind takes the same order as
             * below.  Codes: the row's stored values (128, or the 64 kept ones) in order, eight to a 32-bit word,
             * inside a word the even values in nibbles 0..3 and the odd ones in nibbles 4..7 (value 8w + i in nibble
             * (i % 2) * 4 + i / 2 of word w); four words make a 16-byte unit, and unit j of tile row r lives at byte
             * (128 j + r) * 16.  (A choice of byte order only: the paper fixes none for 4-bit payloads.) */
            uint64_t size = kind_bytes(table[4 * t + 0], 128, 128);
            memcpy(image + off, canon + off, (size_t)size);
            int vals = table[4 * t + 0] == KIND_SPARSE_Q4 ? 64 : 128;
            for (int r = 0; r < 128; ++r)
                for (int w = 0; w < vals / 8; ++w) {
                    uint32_t word = 0;
                    for (int i = 0; i < 8; ++i) {
                        int c = 8 * w + i;                                   /* stored value c of row r */
                        uint8_t byte = canon[off + (uint64_t)r * (vals / 2) + (uint64_t)(c / 2)];
                        uint32_t nib = (c % 2) ? (uint32_t)(byte >> 4) : (uint32_t)(byte & 0xF);
                        word |= nib << (4 * ((i % 2) * 4 + i / 2));
                    }
                    memcpy(image + off + ((uint64_t)(w / 4) * 128 + r) * 16 + (uint64_t)(w % 4) * 4, &word, 4);
                }
            if (table[4 * t + 0] == KIND_SPARSE_Q4) {
                uint64_t moff = (uint64_t)table[4 * t + 2] * 16;
                const uint32_t* cm = (const uint32_t*)(canon + moff);
                for (int Lr = 0; Lr < 128; ++Lr) {
                    int q = Lr / 16, h = (Lr / 8) % 2, i = Lr % 8;
                    for (int j = 0; j < 4; ++j) {
                        uint32_t lo = (cm[(16 * q + i) * 4 + j] >> (16 * h)) & 0xFFFFu;
                        uint32_t hi = (cm[(16 * q + 8 + i) * 4 + j] >> (16 * h)) & 0xFFFFu;
                        uint32_t word = lo | (hi << 16);
                        memcpy(image + moff + (uint64_t)Lr * 16 + (uint64_t)j * 4, &word, 4);
                    }
                }
            }
        } else if (table[4 * t + 0] == KIND_DENSE) {
            const uint16_t* src = (const uint16_t*)(canon + off);
            for (int r = 0; r < 128; ++r)
                for (int c = 0; c < 128; ++c) {
                    uint64_t o = (uint64_t)(c / 64) * 16384 + atom_offset(r, c % 64);
                    memcpy(image + off + o, &src[r * 128 + c], 2);
                }
        } else {
            const uint16_t* src = (const uint16_t*)(canon + off);
            for (int r = 0; r < 128; ++r)
                for (int c = 0; c < 64; ++c)
                    memcpy(image + off + atom_offset(r, c), &src[r * 64 + c], 2);
            uint64_t moff = (uint64_t)table[4 * t + 2] * 16;
            const uint32_t* cm = (const uint32_t*)(canon + moff);
            for (int Lr = 0; Lr < 128; ++Lr) {
                int q = Lr / 16, h = (Lr / 8) % 2, i = Lr % 8;
                for (int j = 0; j < 4; ++j) {
                    uint32_t lo = (cm[(16 * q + i) * 4 + j] >> (16 * h)) & 0xFFFFu;
                    uint32_t hi = (cm[(16 * q + 8 + i) * 4 + j] >> (16 * h)) & 0xFFFFu;
                    uint32_t word = lo | (hi << 16);
                    memcpy(image + moff + (uint64_t)Lr * 16 + (uint64_t)j * 4, &word, 4);
                }
            }
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------------------------- */
/* The linear layer.  Y[m][n] = sum_k X[m][k] * What[n][k], k ascending.                        */

/* double accumulation, rounded once to fp32 (Y32) and from that, RNE, to bf16 (Y16, optional) */
int oracle_gemm_f64(const uint16_t* X, int64_t M, int64_t K, const uint16_t* What, int64_t N,
                    float* Y32, uint16_t* Y16) {
    if (!X || !What || !Y32) return -1;
    if (M < 0 || K <= 0 || N <= 0) return -2;
    int64_t MN = M * N;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < MN; ++i) {
        int64_t m = i / N, n = i % N;
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k)
            acc += (double)bf16_to_f32(X[m * K + k]) * (double)bf16_to_f32(What[n * K + k]);
        float y = (float)acc;
        Y32[i] = y;
        if (Y16) Y16[i] = f32_to_bf16_rne(y);
    }
    return 0;
}

/* plain fp32 accumulation in k order on the same bf16-rounded inputs */
int oracle_gemm_f32(const uint16_t* X, int64_t M, int64_t K, const uint16_t* What, int64_t N,
                    float* Y32) {
    if (!X || !What || !Y32) return -1;
    if (M < 0 || K <= 0 || N <= 0) return -2;
    int64_t MN = M * N;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < MN; ++i) {
        int64_t m = i / N, n = i % N;
        volatile float acc = 0.0f; /* volatile: forbid reassociation / wider intermediates */
        for (int64_t k = 0; k < K; ++k) {
            float p = bf16_to_f32(X[m * K + k]) * bf16_to_f32(What[n * K + k]);
            acc = acc + p;
        }
        Y32[i] = acc;
    }
    return 0;
}

/* Selected rows of Y only (for sampled parity at large M): rows[i] indexes X. */
int oracle_gemm_f64_rows(const uint16_t* X, int64_t K, const int64_t* rows, int64_t n_rows,
                         const uint16_t* What, int64_t N, float* Y32) {
    if (!X || !What || !Y32 || !rows) return -1;
    int64_t total = n_rows * N;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < total; ++i) {
        int64_t m = rows[i / N], n = i % N;
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k)
            acc += (double)bf16_to_f32(X[m * K + k]) * (double)bf16_to_f32(What[n * K + k]);
        Y32[i] = (float)acc;
    }
    return 0;
}

/* =========================================================================================== */
/* Mask learning: soft masks (Eq. 1-4), the two regularisers of the loss (Eq. 5) and the hard   */
/* mask read off the logits (Algorithm 1, the lines after the training loop).                   */
/*                                                                                             */
/* Layouts: P_tile [TN x TK] row-major, one logit per tile.  P_24 [6 x G] row-major with        */
/* G = N*K/4 and group index n*(K/4) + g, so row c holds the logit of candidate c for every     */
/* group ("P_2:4 in R^{6 x d1 d2 / 4}").                                                        */
/* =========================================================================================== */
#include <math.h>

/* Counter-based uniform in (0, 1).  One 64-bit splitmix64-style mix of (seed, stream, idx / 2) serves two
 * consecutive counters: the even one takes its top 23 bits, the odd one bits 9..31.  The 23 bits are
 * centred in their cell, so 0 and 1 never occur and the value is exact in fp32.
 * stream 0 = tile classes (idx = 2*t + class), stream 1 = 2:4 candidates (idx = c*G + group). */
double oracle_uniform(uint64_t seed, uint64_t stream, uint64_t idx) {
    uint64_t x = seed + 0x9E3779B97F4A7C15ull * (idx / 2 + 1) + 0xD1B54A32D192ED03ull * stream;
    x ^= x >> 30; x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27; x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    uint64_t bits = (idx & 1) ? (x >> 9) & 0x7FFFFFull : x >> 41;
    return ((double)bits + 0.5) / 8388608.0;
}

/* Gumbel noise z = -log(-log(u))  (Eq. 1). */
double oracle_gumbel(uint64_t seed, uint64_t stream, uint64_t idx) {
    return -log(-log(oracle_uniform(seed, stream, idx)));
}

/* GS(p; tau, kappa)_k = exp((kappa p_k + z_k)/tau) / sum_j exp((kappa p_j + z_j)/tau)  (Eq. 1 with the
 * scaling factor kappa on the logits).  The largest exponent is subtracted from all of them first, which
 * leaves the quotient unchanged and keeps exp() in range. */
static void gumbel_softmax(const double* p, const double* z, int n, double tau, double kappa, double* out) {
    double e[6], top = -INFINITY, sum = 0.0;
    for (int k = 0; k < n; ++k) { e[k] = (kappa * p[k] + z[k]) / tau; if (e[k] > top) top = e[k]; }
    for (int k = 0; k < n; ++k) { out[k] = exp(e[k] - top); sum += out[k]; }
    for (int k = 0; k < n; ++k) out[k] /= sum;
}

/* Soft mask  Mt = Mt_tile + (1 - Mt_tile) (.) Mt_2:4  (Eq. 4) with
 *   Mt_tile = GS([P_tile, 0])_0 broadcast over the tile (Eq. 3),
 *   Mt_2:4  = GS(P_2:4) x S per group of four (Eq. 2),
 * the masked weight Mt (.) W (double, and rounded once to bf16), and the four sums Eq. 5 needs from one
 * matrix:  sums = { sum Mt, ||W||_0, ||Mt (.) W||_2^2, ||W||_2^2 }.
 * use_noise == 0 drops z (all zeros).  Mt, Wt16 may be NULL. */
int oracle_soft_mask(const uint16_t* W, int64_t N, int64_t K, const float* P_tile, const float* P24,
                     int tile_n, int tile_k, double tau, double kappa, uint64_t seed, int use_noise,
                     double* Mt, uint16_t* Wt16, double* sums) {
    int rc = check_shape(N, K, tile_n, tile_k);
    if (rc) return rc;
    if (!W || !P_tile || !P24 || !sums) return -1;
    if (!(tau > 0.0)) return -2;
    int64_t TK = K / tile_k, G = N * (K / 4);
    double s_m = 0.0, s_nz = 0.0, s_mw2 = 0.0, s_w2 = 0.0;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t g = 0; g < K / 4; ++g) {
            int64_t t = (n / tile_n) * TK + (4 * g) / tile_k, grp = n * (K / 4) + g;
            double p2[2] = {(double)P_tile[t], 0.0}, z2[2] = {0.0, 0.0}, gs2[2];
            double p6[6], z6[6], gs6[6];
            for (int c = 0; c < 6; ++c) { p6[c] = (double)P24[c * G + grp]; z6[c] = 0.0; }
            if (use_noise) {
                for (int c = 0; c < 2; ++c) z2[c] = oracle_gumbel(seed, 0, 2 * (uint64_t)t + c);
                for (int c = 0; c < 6; ++c) z6[c] = oracle_gumbel(seed, 1, (uint64_t)c * G + grp);
            }
            gumbel_softmax(p2, z2, 2, tau, kappa, gs2);
            gumbel_softmax(p6, z6, 6, tau, kappa, gs6);
            for (int j = 0; j < 4; ++j) {
                double m24 = 0.0;
                for (int c = 0; c < 6; ++c) m24 += gs6[c] * S_24[c][j];
                double m = gs2[0] + (1.0 - gs2[0]) * m24;
                double w = (double)bf16_to_f32(W[n * K + 4 * g + j]), mw = m * w;
                if (Mt) Mt[n * K + 4 * g + j] = m;
                if (Wt16) Wt16[n * K + 4 * g + j] = f32_to_bf16_rne((float)mw);
                s_m += m; s_nz += (w != 0.0); s_mw2 += mw * mw; s_w2 += w * w;
            }
        }
    sums[0] = s_m; sums[1] = s_nz; sums[2] = s_mw2; sums[3] = s_w2;
    return 0;
}

/* The two regularisers of Eq. 5 over matrices i = 0..n-1, from their per-matrix sums:
 *   lambda1 * | sum_i sum(Mt_i) / sum_i ||W_i||_0 - rho |  -  lambda2 * sum_i ||Mt_i (.) W_i||^2 / sum_i ||W_i||^2 */
double oracle_regularizers(const double* sums, int n, double rho, double lambda1, double lambda2) {
    double a = 0, b = 0, c = 0, d = 0;
    for (int i = 0; i < n; ++i) { a += sums[4 * i]; b += sums[4 * i + 1]; c += sums[4 * i + 2]; d += sums[4 * i + 3]; }
    return lambda1 * fabs(a / b - rho) - lambda2 * (c / d);
}

/* Hard masks from the logits (Algorithm 1): tile t is dense iff P_tile[t] > 0 (flag 0), else 2:4 (flag 1);
 * every group takes the candidate with the largest logit (the algorithm's best-mask selection), the first of equals. */
int oracle_hard_mask(const float* P_tile, const float* P24, int64_t N, int64_t K, int tile_n, int tile_k,
                     uint8_t* flags, uint8_t* patterns) {
    int rc = check_shape(N, K, tile_n, tile_k);
    if (rc) return rc;
    if (!P_tile || !P24 || !flags || !patterns) return -1;
    int64_t T = (N / tile_n) * (K / tile_k), G = N * (K / 4);
    for (int64_t t = 0; t < T; ++t) flags[t] = P_tile[t] > 0.0f ? KIND_DENSE : KIND_SPARSE;
    for (int64_t grp = 0; grp < G; ++grp) {
        int best = 0;
        for (int c = 1; c < 6; ++c)
            if (P24[c * G + grp] > P24[best * G + grp]) best = c;
        patterns[grp] = (uint8_t)best;
    }
    return 0;
}

/* M* = M*_tile + (1 - M*_tile) (.) M*_2:4 with the 2:4 part given by candidate indices. */
int oracle_mask_patterns(int64_t N, int64_t K, const uint8_t* flags, const uint8_t* patterns,
                         int tile_n, int tile_k, uint8_t* mask) {
    int rc = check_shape(N, K, tile_n, tile_k);
    if (rc) return rc;
    int64_t TK = K / tile_k;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t g = 0; g < K / 4; ++g) {
            uint8_t c = patterns[n * (K / 4) + g];
            if (c > 5) return -4;
            int m_tile = flags[(n / tile_n) * TK + (4 * g) / tile_k] == KIND_DENSE;
            for (int j = 0; j < 4; ++j)
                mask[n * K + 4 * g + j] = (uint8_t)(m_tile + (1 - m_tile) * S_24[c][j]);
        }
    return 0;
}

/* Coefficients with which one element's soft-mask value enters the gradient of the two regularisers of
 * Eq. 5 (pooled sums a = sum Mt, b = sum ||W||_0, d = sum ||W||^2 over all matrices):
 *   d/dMt_e [ lambda1 |a/b - rho| ]        = lambda1 sign(a/b - rho) / b         =: c1
 *   d/dMt_e [ -lambda2 sum (Mt W)^2 / d ]  = -(2 lambda2 / d) Mt_e W_e^2         =: -c2 Mt_e W_e^2 */
void oracle_regularizer_coefficients(const double* sums, int n, double rho, double lambda1, double lambda2,
                                     double* c1, double* c2) {
    double a = 0, b = 0, d = 0;
    for (int i = 0; i < n; ++i) { a += sums[4 * i]; b += sums[4 * i + 1]; d += sums[4 * i + 3]; }
    double dev = a / b - rho;
    *c1 = lambda1 * (dev > 0 ? 1.0 : dev < 0 ? -1.0 : 0.0) / b;
    *c2 = 2.0 * lambda2 / d;
}

/* Gradient with respect to the logits (the logit update step of Algorithm 1) of
 *   F = sum_e Gw_e Mt_e W_e  +  c1 sum_e Mt_e  -  (c2 / 2) sum_e (Mt_e W_e)^2
 * for fixed noise, where Gw = dL_LM / d(Mt (.) W) is the gradient the language-model loss hands back for
 * the masked weight.  Chain rule through Eq. 4, Eq. 2 / Eq. 3 and the softmax of Eq. 1:
 *   gM_e   = Gw_e W_e + c1 - c2 Mt_e W_e^2
 *   h_c    = (1 - Mt_tile) sum_j S[c][j] gM_j                      (per group)
 *   gP24_c = (kappa / tau) GS_c (h_c - sum_k GS_k h_k)
 *   gP_tile = (kappa / tau) Mt_tile (1 - Mt_tile) sum_{e in tile} gM_e (1 - Mt_2:4,e)
 * gP_tile [TN x TK], gP24 [6 x G], both double. */
int oracle_soft_mask_backward(const uint16_t* W, int64_t N, int64_t K, const float* P_tile, const float* P24,
                              int tile_n, int tile_k, double tau, double kappa, uint64_t seed, int use_noise,
                              const float* Gw, double c1, double c2, double* gP_tile, double* gP24) {
    int rc = check_shape(N, K, tile_n, tile_k);
    if (rc) return rc;
    if (!W || !P_tile || !P24 || !Gw || !gP_tile || !gP24) return -1;
    if (!(tau > 0.0)) return -2;
    int64_t TK = K / tile_k, T = (N / tile_n) * TK, G = N * (K / 4);
    for (int64_t t = 0; t < T; ++t) gP_tile[t] = 0.0;
    for (int64_t n = 0; n < N; ++n)
        for (int64_t g = 0; g < K / 4; ++g) {
            int64_t t = (n / tile_n) * TK + (4 * g) / tile_k, grp = n * (K / 4) + g;
            double p2[2] = {(double)P_tile[t], 0.0}, z2[2] = {0.0, 0.0}, gs2[2];
            double p6[6], z6[6], gs6[6], m24[4], gM[4], h[6], hbar = 0.0;
            for (int c = 0; c < 6; ++c) { p6[c] = (double)P24[c * G + grp]; z6[c] = 0.0; }
            if (use_noise) {
                for (int c = 0; c < 2; ++c) z2[c] = oracle_gumbel(seed, 0, 2 * (uint64_t)t + c);
                for (int c = 0; c < 6; ++c) z6[c] = oracle_gumbel(seed, 1, (uint64_t)c * G + grp);
            }
            gumbel_softmax(p2, z2, 2, tau, kappa, gs2);
            gumbel_softmax(p6, z6, 6, tau, kappa, gs6);
            double mt = gs2[0];
            for (int j = 0; j < 4; ++j) {
                m24[j] = 0.0;
                for (int c = 0; c < 6; ++c) m24[j] += gs6[c] * S_24[c][j];
                double m = mt + (1.0 - mt) * m24[j];
                double w = (double)bf16_to_f32(W[n * K + 4 * g + j]);
                gM[j] = (double)Gw[n * K + 4 * g + j] * w + c1 - c2 * m * w * w;
                gP_tile[t] += gM[j] * (1.0 - m24[j]);
            }
            for (int c = 0; c < 6; ++c) {
                h[c] = 0.0;
                for (int j = 0; j < 4; ++j) h[c] += S_24[c][j] * gM[j];
                h[c] *= 1.0 - mt;
                hbar += gs6[c] * h[c];
            }
            for (int c = 0; c < 6; ++c) gP24[c * G + grp] = kappa / tau * gs6[c] * (h[c] - hbar);
        }
    for (int64_t t = 0; t < T; ++t) {
        double p2[2] = {(double)P_tile[t], 0.0}, z2[2] = {0.0, 0.0}, gs2[2];
        if (use_noise)
            for (int c = 0; c < 2; ++c) z2[c] = oracle_gumbel(seed, 0, 2 * (uint64_t)t + c);
        gumbel_softmax(p2, z2, 2, tau, kappa, gs2);
        gP_tile[t] *= kappa / tau * gs2[0] * (1.0 - gs2[0]);
    }
    return 0;
}
