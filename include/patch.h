/*
 * patch.h -- C ABI of the B200 (sm_100a) tile-hybrid linear layer  Y = X * What^T.
 *
 * The weight W [N x K] (N = out-features, K = in-features, row-major bf16) is cut into
 * 128 x 128 tiles; a per-tile flag says whether the tile is stored dense or 2:4-sparse
 * (two kept values of every four consecutive elements along K, plus two position bits per
 * kept value).  This is the deployment format of PATCH (arXiv 2509.23410): the hard mask
 * M* = M*_tile + (1 - M*_tile) (.) M*_2:4 of Algorithm 1 applied to W, compressed per tile
 * (deployment section, Appendix A), and the matmul that mixes dense and 2:4 tiles inside one
 * multiplication.
 *
 * General rules
 *   - Every function returns a status (PATCH_OK = 0, errors negative).  Nothing throws,
 *     prints or exits.  All argument validation happens on the host before any launch.
 *   - Pointers named *_dev are device pointers, *_host are host pointers.  The library
 *     allocates no device memory; every buffer is the caller's.  What it remembers between
 *     calls is per device and read-mostly: the SM count and which kernels already had their
 *     shared-memory limit raised there (plus patch_gemm_noalloc's scratch array, see there).
 *     No environment variable changes its behaviour.
 *   - Entry points may be called from several host threads (on different streams or devices);
 *     calls that share a workspace must be ordered on one stream.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls enqueue work
 *     and return; patch_pack, patch_gemm_host and the patch_gemm_host_batch pair are the exceptions noted below.
 *   - Supported: tile_n = tile_k = 128, N % 128 == 0, K % 128 == 0, device pointers 16-byte
 *     aligned, leading dimensions multiples of 8 elements.  Device must be sm_100
 *     (PATCH_ERR_ARCH otherwise; there is no fallback path).
 */
#ifndef PATCH_B200_H_
#define PATCH_B200_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Tile kinds.  Bit 0 is 1 - M*_tile of Algorithm 1 (the paper's tile mask is 1 = dense).  Bit 1 selects the
 * 4-bit payload of the section "Combination with other compression methods" (the 4-bit weight-only
 * quantisation table): the tile's stored values -- all 128 of a row in a dense tile, the 64 kept ones in a 2:4
 * tile -- are 4-bit codes with one bf16 scale per tile row.  The paper prints the compression ratio of this
 * combination, 16 / (4 - f) (four bits per stored value, two metadata bits per kept value), and no quantiser;
 * this library's reading is symmetric round-to-nearest-even,
 *     s = bf16(max|v| / 7),  q = clamp(rint(v / s), -7, 7)  (0 where s = 0),  v^ = bf16(q * s),
 * evaluated in fp32 on the bf16 values, the 2:4 selection made first on the unquantised weights.  The layer
 * then multiplies by the dequantised values v^. */
enum { PATCH_TILE_DENSE = 0, PATCH_TILE_SPARSE_2_4 = 1, PATCH_TILE_DENSE_Q4 = 2, PATCH_TILE_SPARSE_2_4_Q4 = 3 };

enum {
    PATCH_OK = 0,
    PATCH_ERR_NULL = -1,    /* a required pointer is NULL */
    PATCH_ERR_SHAPE = -2,   /* N, K, M or a leading dimension is not supported */
    PATCH_ERR_TILE = -3,    /* tile shape other than 128 x 128 */
    PATCH_ERR_FLAG = -4,    /* a tile flag is neither DENSE nor SPARSE_2_4 */
    PATCH_ERR_ALIGN = -5,   /* a device pointer or row pitch is not 16-byte aligned */
    PATCH_ERR_SIZE = -6,    /* a buffer (packed blob, workspace) is too small */
    PATCH_ERR_FORMAT = -7,  /* layout magic / version / offsets are inconsistent */
    PATCH_ERR_ARCH = -8,    /* current device is not sm_100 */
    PATCH_ERR_CUDA = -9,    /* a CUDA runtime call failed */
    PATCH_ERR_TIMEOUT = -10 /* a bounded device-side wait expired (reported through status_dev) */
};

/* Kernel choice for patch_gemm_ex (low bits), optionally OR-ed with PATCH_GEMM_WEIGHTS_STATIC. */
enum { PATCH_VARIANT_AUTO = 0, PATCH_VARIANT_GEMV = 1, PATCH_VARIANT_MMA = 2, PATCH_VARIANT_PAIR = 3 };
/*
 * Launch promises.  Every GEMM kernel is launched with programmatic dependent launch and lets its
 * successor become resident as soon as it has started itself; each kernel orders itself against
 * what came before with a device-side wait.  A promise lets it do part of its work before that wait.
 * Since the kernels before it may have started early in the same way, a GEMM can be running at the
 * same time as ANY of the GEMMs of this library that were enqueued directly before it, one after the
 * other, on the same stream -- however those were launched.  Call that run of consecutive GEMM calls,
 * back to the nearest operation that is not one of this library's GEMMs (a copy, a memset, any other
 * kernel: those complete before the next kernel starts), the GEMM's "overlap window".
 *
 * PATCH_GEMM_WEIGHTS_STATIC: no operation in the overlap window writes the packed weight (the serving
 *   case: weights are packed once, offline).  The kernel then requests weight tiles before its wait.
 * PATCH_GEMM_INPUT_STATIC (only honoured together with the first): no operation in the overlap window
 *   writes X either (e.g. q, k and v projections enqueued one after the other behind the kernel that
 *   produced their common X; not a GEMM whose X is the Y of a GEMM enqueued directly before it).
 *   Activations are then fetched without waiting too.
 * PATCH_GEMM_OUTPUT_STATIC (only honoured together with the first two, and for M <= 64): no operation in the
 *   overlap window reads or writes Y either (q, k and v projections writing three buffers of their own; not two
 *   calls that write the same Y with only GEMM calls of this library between them).  The CTAs of the kernel
 *   then store Y and leave as soon as they are done, instead of each holding its SM until the preceding
 *   kernels have completed; one cluster of every launch still waits.
 * Without the third promise, writes to Y wait for everything before them; writes to the workspace always do.
 * With or without it no kernel completes before its predecessors, so stream order as seen from later
 * operations is unchanged.
 *
 * With BOTH promises a GEMM of M <= 64 tokens runs on a schedule made for streams of independent
 * GEMMs: one CTA per row-block (a small cluster splitting K where row-blocks are few), so that several
 * consecutive GEMMs are resident on the GPU at once.  With the weights promise alone it runs on the same
 * row-block schedule with larger clusters (at least 128 CTAs: it streams alone once its predecessor is
 * done); without any promise it runs stream-K over all SMs.  For M > 64 both promises let the kernel
 * start on the SMs that the tail of the previous kernel leaves idle.  All schedules are deterministic;
 * their results may differ in the last bit (different fp32 summation order).
 */
enum { PATCH_GEMM_WEIGHTS_STATIC = 0x100 };
enum { PATCH_GEMM_INPUT_STATIC = 0x200 };
enum { PATCH_GEMM_OUTPUT_STATIC = 0x400 };

/*
 * Description of a packed blob.  Plain host struct, caller-owned, filled by patch_packed_size.
 * The blob in device memory is position independent (offsets only):
 *   [ header 256 B (a copy of this struct, zero padded)
 *   | tile table: 16 B per tile in (tn, tk) row-major order, zero padded to a multiple of 1024 B
 *   | payloads: 32 768 B per dense tile, 18 432 B per 2:4 tile (offsets multiples of 1024 while only these two
 *     kinds occur), 8 448 B / 6 400 B per dense / 2:4 tile with 4-bit values (offsets multiples of 256) ]
 * Table entry: { u32 kind, u32 payload_off / 16, u32 meta_off / 16 (0xFFFFFFFF if the kind has no metadata),
 * u32 scales_off / 16 (0 if the kind has no scales) }, offsets counted from the start of the blob.
 *
 * Payload bytes (the "device image"):
 *   values are stored in 16 384-byte atoms of 128 rows x 64 bf16; inside an atom the 16-byte
 *   chunk c (8 elements) of row r lives at (r/8)*1024 + (r%8)*128 + ((c ^ (r%8))*16), i.e. the
 *   128-byte-swizzled K-major layout the tensor core reads from shared memory, so a linear
 *   copy of the payload is ready to multiply.  A dense tile is two atoms (columns 0..63, then
 *   64..127).  A 2:4 tile is one atom holding the 64 kept values of each row (in position
 *   order), followed by 2 048 B of metadata: 128 rows x four u32; row L = 16q + 8h + i
 *   (i < 8), word j: low 16 bits = the four 4-bit position codes (i0 | i1 << 2, i0 < i1) of
 *   tile row 16q+i for columns [32j + 16h, 32j + 16h + 16), high 16 bits = the same for tile
 *   row 16q+8+i.
 *   4-bit kinds: [ codes: value c of tile row r in byte r * (V / 2) + c / 2, even c in the low nibble, code = q + 8
 *   (1..15), V = 128 (dense) or 64 (2:4: the kept values in position order) | 2:4 only: 2 048 B of metadata in
 *   the order above | scales: 128 bf16, one per tile row ].
 */
typedef struct patch_layout_t {
    uint32_t magic;          /* 0x48435450 */
    uint32_t version;        /* 1 */
    int64_t  N, K;
    int32_t  tile_n, tile_k;
    int64_t  n_dense, n_sparse;
    uint64_t table_off;      /* 256 */
    uint64_t payload_off;    /* first payload byte */
    uint64_t payload_bytes;  /* 32768 * n_dense + 18432 * n_sparse */
    uint64_t total_bytes;    /* payload_off + payload_bytes = size of the blob */
    int64_t  n_dense_q4, n_sparse_q4;   /* tiles of the 4-bit kinds (payload_bytes includes 8448 / 6400 B for each) */
} patch_layout_t;

/*
 * Size and layout of the packed blob for a weight of N x K with the given tile flags.
 * (Appendix A: the tile size fixes the compressed format; here it is 128 x 128.)
 *   tile_flags_host  [N/128 x K/128] row-major bytes, one of the four tile kinds
 *   layout_out       filled on success
 * Host only; touches no device.
 */
int patch_packed_size(int64_t N, int64_t K, int tile_n, int tile_k,
                      const uint8_t* tile_flags_host, patch_layout_t* layout_out);

/*
 * Compress W into the packed blob (the paper's `compress` step of the conversion pseudocode,
 * Appendix A; mask semantics of Algorithm 1's last four lines).
 * In every 2:4 tile, each group of four consecutive elements along K keeps its two largest
 * magnitudes (equal magnitudes: lower index first; magnitude = bit pattern without sign);
 * dense tiles are copied.  A weight that is already 2:4 inside those tiles is packed losslessly.
 * Tiles of the 4-bit kinds are quantised as described at the tile kinds (by the same kernel).
 *   W_dev            bf16 [N x ldw], ldw >= K elements, ldw % 8 == 0
 *   tile_flags_host  as for patch_packed_size; must be the flags `layout` was computed from
 *   packed_dev       destination, packed_capacity >= layout->total_bytes, 16-byte aligned
 * Copies header and tile table host->device on `stream` (the host staging buffer is consumed
 * before the call returns), then launches one kernel.  Every byte of the blob is written.
 */
int patch_pack(const void* W_dev, int64_t ldw, const uint8_t* tile_flags_host,
               const patch_layout_t* layout, void* packed_dev, size_t packed_capacity,
               void* stream);

/*
 * Inverse of patch_pack: writes What = W (.) M* (pruned elements are +0) as bf16 [N x ldw]; for tiles of the
 * 4-bit kinds the dequantised values, i.e. exactly the matrix the layer multiplies by.
 */
int patch_unpack(const patch_layout_t* layout, const void* packed_dev, void* What_dev,
                 int64_t ldw, void* stream);

/*
 * Scratch memory patch_gemm needs for `M` tokens (may be 0 bytes).  The scratch holds fp32
 * split-K partial sums and arrival counters of the small-M schedules (split-K is the schedule
 * Appendix A names for decode).
 */
int patch_gemm_workspace_size(const patch_layout_t* layout, int64_t M, size_t* bytes_out);

/*
 * Zero a workspace once after allocating it (arrival counters and partial-sum flags must start at
 * zero; every successful patch_gemm leaves them zero again).  Zero it again after a call that
 * reported PATCH_ERR_TIMEOUT.  A workspace of patch_gemm_workspace_size(layout, 64) bytes serves
 * calls of every M in any order, and calls on different layouts with N <= 131072 may share it.
 */
int patch_workspace_init(void* workspace_dev, size_t workspace_bytes, void* stream);

/*
 * Y = X * What^T with fp32 accumulation and bf16 (round-to-nearest-even) output: the hybrid
 * dense / 2:4 tile matmul of Appendix A.  One kernel launch; no host synchronisation, no
 * allocation, no host<->device copy.
 *   X_dev   bf16 [M x ldx], ldx >= K, ldx % 8 == 0
 *   Y_dev   bf16 [M x ldy], ldy >= N, ldy % 8 == 0
 *   workspace_dev / workspace_bytes   at least patch_gemm_workspace_size(layout, M) bytes,
 *           256-byte aligned, initialised once with patch_workspace_init; may be NULL if 0
 *   status_dev   optional device int, must be zero before the call; receives the first device-side
 *           error: PATCH_ERR_TIMEOUT if a bounded wait expired (the kernel then stops early), or
 *           PATCH_ERR_FORMAT if an entry of the blob's tile table is not a dense or 2:4 tile lying
 *           inside the blob (every entry is checked before a byte of its tile is requested; the
 *           kernel reads the blob's first payload in its place, so nothing is read out of range).
 *           In both cases Y is undefined.  NULL = not reported.
 * M == 0 returns PATCH_OK without launching.  Calls sharing a workspace must be ordered on
 * one stream.
 * Weights with 4-bit tiles: served if every tile is of a 4-bit kind, by a dequantising kernel of its own made
 * for M <= 16 tokens (the decode case, where the bytes of the weight are what the layer costs); no workspace.
 * 17 to 64 tokens are multiplied sixteen at a time, one launch after the other.  Beyond 64 tokens the call first
 * rewrites the weight as the bf16 blob of its dequantised values -- into the workspace, which must then hold
 * patch_gemm_workspace_size(layout, M) bytes (32 MiB plus the size of that blob; no initialisation needed: the
 * blob starts 32 MiB into the workspace, past every word that other calls keep zero there, so the workspace may be
 * shared with them as before) -- and runs the large-M schedule on it: the dequantisation is paid once per call.  Weights that mix bf16 and 4-bit tiles
 * return PATCH_ERR_SHAPE -- as do
 * PATCH_VARIANT_GEMV / PATCH_VARIANT_PAIR, patch_gemm_gated and patch_gemm_noalloc for such weights (the host
 * entry points follow patch_gemm).  All pack entry points serve the four kinds (with a given 2:4 mask, the mask
 * is applied first, then the kept values are quantised).
 * The launch promises mean the same as for bf16 tiles; launches with different promises may split K
 * differently and then differ in the last bit.
 */
int patch_gemm(const void* X_dev, int64_t ldx, int64_t M,
               const patch_layout_t* layout, const void* packed_dev,
               void* Y_dev, int64_t ldy,
               void* workspace_dev, size_t workspace_bytes, int* status_dev, void* stream);

/* patch_gemm with an explicit kernel choice and options.
 *   PATCH_VARIANT_GEMV  CUDA-core decode kernel, M <= 4 only (PATCH_ERR_SHAPE otherwise)
 *   PATCH_VARIANT_MMA   tcgen05 tensor-core kernel, any M
 *   PATCH_VARIANT_PAIR  the CTA-pair (cta_group::2) large-M kernels, M > 64 (PATCH_ERR_SHAPE otherwise).  AUTO
 *                       picks the pair schedule for weights whose tiles are all of one kind wherever every CTA
 *                       pair gets a tile of a useful width; for weights that mix kinds it is slower than the
 *                       one-CTA schedule and runs only when asked for
 *   | PATCH_GEMM_WEIGHTS_STATIC | PATCH_GEMM_INPUT_STATIC | PATCH_GEMM_OUTPUT_STATIC  see above */
int patch_gemm_ex(const void* X_dev, int64_t ldx, int64_t M,
                  const patch_layout_t* layout, const void* packed_dev,
                  void* Y_dev, int64_t ldy,
                  void* workspace_dev, size_t workspace_bytes, int* status_dev, void* stream,
                  int variant);

/*
 * Gated product of the MLP's gate and up projections in one launch (a first step of the
 * block-level fusion that follows the per-matrix matmul; the paper treats the MLP's up, gate and
 * down matrices separately, and in the LLaMA models it measures the MLP computes
 * down(silu(gate x) * up x)):
 *     Y[m][128 j + r] = silu(G[m][128 j + r]) * U[m][128 j + r],   silu(x) = x / (1 + exp(-x)),
 * where G = X Wgate^T and U = X Wup^T come from ONE packed weight that stacks the two matrices
 * with their 128-row blocks interleaved: row-block 2j of the packed matrix is row-block j of
 * Wgate, row-block 2j + 1 is row-block j of Wup (each keeps its own tile flags).  fp32
 * accumulation, the product evaluated in fp32 on the accumulators, one bf16 rounding.
 *   layout->N  must be a multiple of 256; Y_dev is bf16 [M x ldy], ldy >= N / 2, ldy % 8 == 0.
 *   workspace_dev / workspace_bytes   optional.  With M <= 16 and at least
 *           patch_gemm_gated_workspace_size(layout, M) bytes (256-byte aligned, zeroed once with
 *           patch_workspace_init, left zero by every call, shareable with patch_gemm calls) the
 *           small-M stream-K schedule is used: the finisher of a gate row-block publishes its
 *           fp32 values, the finisher of the matching up row-block multiplies.  Otherwise (or for
 *           larger M) the large-M schedule runs, whose CTA holds both accumulators.
 *   flags   0 or PATCH_GEMM_WEIGHTS_STATIC [| PATCH_GEMM_INPUT_STATIC], as for patch_gemm_ex.
 *           With the weights promise and M <= 16 the call needs no workspace at all: a cluster of CTAs owns a
 *           (gate, up) pair of row-blocks, holds both accumulators and applies the product itself -- few CTAs
 *           per launch with both promises, at least 128 with the weights promise alone (the gated product of
 *           a decoder block reads what the projection before it wrote).
 * Other arguments and error behaviour as patch_gemm.
 */
int patch_gemm_gated_workspace_size(const patch_layout_t* layout, int64_t M, size_t* bytes_out);
int patch_gemm_gated(const void* X_dev, int64_t ldx, int64_t M,
                     const patch_layout_t* layout, const void* packed_dev,
                     void* Y_dev, int64_t ldy,
                     void* workspace_dev, size_t workspace_bytes, int* status_dev, void* stream, int flags);

/*
 * End-to-end form with HOST activations and results: copies X host->device into
 * X_stage_dev, runs patch_gemm, copies Y device->host and synchronises `stream`.
 *   X_host  bf16 [M x K] contiguous; Y_host bf16 [M x N] contiguous (pinned memory advised)
 *   X_stage_dev / Y_stage_dev   device staging buffers of M*K and M*N bf16
 * The packed weight stays resident on the device.
 */
int patch_gemm_host(const void* X_host, int64_t M, const patch_layout_t* layout,
                    const void* packed_dev, void* Y_host,
                    void* X_stage_dev, void* Y_stage_dev,
                    void* workspace_dev, size_t workspace_bytes, void* stream);

/*
 * The same for a whole step of GEMMs with ONE synchronisation: all activations are copied to
 * the device first, then all GEMMs are launched back to back, then all results are copied
 * back, then `stream` is synchronised.  Because every copy of an X precedes every launch, the
 * launches carry PATCH_GEMM_INPUT_STATIC whenever `weights_static` is non-zero (the caller's
 * promise that no packed weight is written on this stream meanwhile).  Jobs are independent:
 * no job's X_stage_dev, Y_stage_dev or Y_host may alias another's; jobs may share a workspace.
 * Copies of consecutive jobs whose host buffers AND staging buffers are both adjacent in memory
 * (job i+1's begin where job i's end) are issued as one copy, so a step whose activations live
 * in one pinned arena, staged in one device arena in the same order, costs one transfer each way.
 */
typedef struct {
    const void* X_host;             /* bf16 [M x K] contiguous */
    int64_t M;
    const patch_layout_t* layout;
    const void* packed_dev;
    void* Y_host;                   /* bf16 [M x N] contiguous */
    void* X_stage_dev;              /* M*K bf16 */
    void* Y_stage_dev;              /* M*N bf16 */
    void* workspace_dev;
    size_t workspace_bytes;
} patch_host_job_t;
int patch_gemm_host_batch(const patch_host_job_t* jobs, int n_jobs, int weights_static, void* stream);

/*
 * The same step with the transfers overlapped with the GEMMs.  The jobs are cut into `n_chunks`
 * runs of consecutive jobs (by bytes moved); run c's activations are copied on `copy_in_stream`,
 * its GEMMs run on `stream` once they have landed, its results are copied back on
 * `copy_out_stream` once they are computed -- so run c+1's copy in, run c's GEMMs and run c-1's
 * copy out proceed at the same time (PCIe is full duplex).  The three streams must be distinct
 * and are all synchronised before the call returns (also when it returns an error after having
 * enqueued part of the work).  2 * n_chunks events are created and destroyed inside the call;
 * 1 <= n_chunks <= 64 (clamped to n_jobs).  Everything else as for patch_gemm_host_batch.
 */
int patch_gemm_host_batch_pipelined(const patch_host_job_t* jobs, int n_jobs, int weights_static, int n_chunks,
                                    void* stream, void* copy_in_stream, void* copy_out_stream);

/*
 * patch_gemm for callers that cannot allocate device memory.  (The paper has no counterpart;
 * this is a convenience of this library.)
 *
 * Some callers of a GEMM run where cudaMalloc is off limits: inside a framework's capture or
 * replay phase, under a memory pool that must not be disturbed, in a plug-in that is handed
 * pointers and a stream and nothing else, or late in a process whose memory is fully committed.
 * They cannot provide the workspace patch_gemm needs for its split-K partial sums.  This entry
 * point keeps that scratch in a fixed array inside the library image instead (about 3.2 MB,
 * held on every GPU that loads the library until the process exits) and calls no cudaMalloc,
 * cudaFree or any allocating routine.
 *
 *   Arguments as for patch_gemm, without workspace and status.  Result and rounding are those
 *   of patch_gemm (same kernel, same summation order).  There is no status word: a bounded
 *   device-side wait that expires (PATCH_ERR_TIMEOUT in patch_gemm) is NOT reported here and
 *   leaves Y undefined; a caller that needs to know uses patch_gemm.
 *   Limits: M <= 16 tokens and N <= 131072; beyond them the call returns PATCH_ERR_SIZE and
 *   launches nothing (use patch_gemm with a caller-owned workspace instead).
 *   The first call on each device looks up the array's device address; make that first call
 *   with the device current and before any stream capture.  Every call enqueues a memset of
 *   the whole scratch array followed by the kernel: the array must start empty, also after a
 *   call that was cut short or that raced with another one.
 *   All calls on a device share the one array, which keeps the last call's contents: calls that
 *   may overlap on the GPU (different streams) race with each other -- issue them on one stream
 *   or order them with events.
 */
int patch_gemm_noalloc(const void* X_dev, int64_t ldx, int64_t M,
                       const patch_layout_t* layout, const void* packed_dev,
                       void* Y_dev, int64_t ldy, void* stream);

/* =========================================================================================
 * Mask learning (the training side of Algorithm 1): soft masks, regulariser sums, hard masks.
 *
 * Logit layouts (fp32, device): P_tile [N/128 x K/128] row-major, one logit per tile;
 * P_24 [6 x G] row-major with G = N*K/4 and group index n*(K/4) + g, i.e. row c holds the
 * logit of candidate c for every group of four ("P_2:4 in R^{6 x d1 d2 / 4}").  The six
 * candidates (the rows of the matrix S of the 2:4 paragraph) are taken in lexicographic
 * order of the kept positions: 0:(0,1) 1:(0,2) 2:(0,3) 3:(1,2) 4:(1,3) 5:(2,3).
 * ========================================================================================= */

/* patch_soft_mask flag: drop the Gumbel noise (z = 0), e.g. for evaluation. */
enum { PATCH_MASK_NO_NOISE = 1 };

/*
 * Hard masks read off the logits (Algorithm 1, the lines after the loop):
 *   tile_flags_dev[t] = PATCH_TILE_DENSE if P_tile[t] > 0 else PATCH_TILE_SPARSE_2_4
 *                       (a positive tile logit means dense; 0 and NaN are not positive);
 *   patterns_dev[grp] = index of the largest of the group's six logits, the first of equals
 *                       (the candidate Algorithm 1 keeps for deployment).
 *   tile_flags_dev  u8 [N/128 x K/128];  patterns_dev  u8 [N x K/4], 16-byte aligned.
 * One kernel, no host synchronisation.  The flags must be copied to the host by the caller
 * before patch_packed_size / patch_pack_patterns, which take them as host arrays.
 */
int patch_hard_mask(const float* P_tile_dev, const float* P24_dev, int64_t N, int64_t K,
                    int tile_n, int tile_k, uint8_t* tile_flags_dev, uint8_t* patterns_dev,
                    void* stream);

/*
 * patch_pack with the 2:4 mask given instead of chosen by magnitude (the deployment input of
 * a learned or otherwise precomputed mask): in every 2:4 tile, group (n, g) keeps the two
 * positions of candidate patterns_dev[n*(K/4) + g]; groups inside dense tiles ignore theirs.
 * In a 2:4 tile of the 4-bit kind the kept values are then quantised (the "PATCH + 4-bit" combination of
 * the paper's quantisation table with PATCH's own, learned masks).
 *   patterns_dev  u8 [N x K/4] device, 4-byte aligned, values 0..5
 *   status_dev    optional device int (caller zeroes it): set to PATCH_ERR_FLAG if a 2:4 tile
 *                 holds an index above 5 (that group is then packed as candidate 0)
 * Everything else as for patch_pack.
 */
int patch_pack_patterns(const void* W_dev, int64_t ldw, const uint8_t* tile_flags_host,
                        const uint8_t* patterns_dev, const patch_layout_t* layout, void* packed_dev,
                        size_t packed_capacity, int* status_dev, void* stream);

/*
 * patch_pack / patch_pack_patterns with the tile flags in DEVICE memory (e.g. as written by
 * patch_hard_mask) and no host work at all: every CTA of the pack kernel derives its tile's offset
 * from the flags (sum of the payload sizes before it) and writes its table entry; CTA 0 writes the
 * header.  The blob is byte for byte the one patch_pack writes for the same flags.
 *   tile_flags_dev  u8 [N/128 x K/128] device
 *   patterns_dev    NULL (magnitude top-2, as patch_pack) or u8 [N x K/4] device (as patch_pack_patterns)
 *   packed_capacity must hold the blob the flags imply; N/128 * K/128 * 32768 + table always does.
 *                   The host checks only the smallest possible size (all tiles 2:4 with 4-bit values).
 *   status_dev      optional device int (caller zeroes it): PATCH_ERR_SIZE if the blob did not fit
 *                   (then nothing but a header without magic number is written), PATCH_ERR_FLAG for
 *                   a flag above 3 (packed as dense) or a candidate index above 5.
 * Every CTA reads the whole flag array (one byte per tile, from L2), so the extra work grows with the
 * square of the tile count: negligible for the tens of thousands of tiles of an LLM weight.
 * Enqueues one kernel; no copy, no synchronisation.  The host-side layout that patch_gemm
 * needs comes from patch_packed_size when the flags are also known on the host, else from
 * patch_read_layout.
 */
int patch_pack_dev(const void* W_dev, int64_t ldw, const uint8_t* tile_flags_dev, const uint8_t* patterns_dev,
                   int64_t N, int64_t K, int tile_n, int tile_k, void* packed_dev, size_t packed_capacity,
                   int* status_dev, void* stream);

/*
 * Reads the header of a packed blob back into a host layout struct and validates it
 * (PATCH_ERR_FORMAT if it is not a valid header, e.g. after a patch_pack_dev that did not fit).
 * Copies 80 bytes device->host on `stream` and synchronises it.
 */
int patch_read_layout(const void* packed_dev, patch_layout_t* layout_out, void* stream);

/* Scratch bytes of patch_soft_mask: four doubles per tile. */
int patch_soft_mask_workspace_size(int64_t N, int64_t K, int tile_n, int tile_k, size_t* bytes_out);

/*
 * One training-forward evaluation of the soft mask of a matrix and of everything Eq. 5 needs from it:
 *   Mt_tile = GS([P_tile, 0]; tau, kappa)_0, one value per tile                     (Eq. 3)
 *   Mt_2:4  = GS(P_2:4; tau, kappa) x S, four values per group                     (Eq. 2)
 *   Mt      = Mt_tile + (1 - Mt_tile) (.) Mt_2:4                                    (Eq. 4)
 *   Wt_dev  = Mt (.) W, rounded once to bf16 [N x ldo] -- the weight the language-model loss runs on
 *   sums_dev[4] = { sum Mt, ||W||_0, ||Mt (.) W||_2^2 (before rounding), ||W||_2^2 }, doubles
 * with GS(p)_k = exp((kappa p_k + z_k)/tau) / sum_j exp((kappa p_j + z_j)/tau), z = -log(-log(u)) (Eq. 1).
 * The noise is drawn on the device from a counter-based generator keyed by `seed`, so that a
 * call is reproducible and needs no noise buffers: u = (b + 0.5) / 2^23 with b 23 bits of
 * x = mix(seed + 0x9E3779B97F4A7C15 * (i/2 + 1) + 0xD1B54A32D192ED03 * stream), mix = the
 * splitmix64 finaliser (x ^= x >> 30, *= 0xBF58476D1CE4E5B9, ^= x >> 27, *= 0x94D049BB133111EB,
 * ^= x >> 31); even counters i take b = x >> 41, odd ones b = (x >> 9) & 0x7FFFFF; stream 0,
 * i = 2 t + class for the tiles (class 0 = dense); stream 1, i = c G + group for the candidates.
 *   tau > 0, kappa finite; flags = 0 or PATCH_MASK_NO_NOISE
 *   Mt_dev        optional fp32 [N x ldm] (ldm % 4 == 0): the soft mask itself, e.g. for a backward pass
 *   workspace_dev at least patch_soft_mask_workspace_size bytes, 8-byte aligned; no initialisation needed
 * Arithmetic is fp32 (sums: fp32 within a thread's 64 elements, double above that, in a fixed
 * order: the result does not depend on scheduling).  Two kernels, no host synchronisation.
 */
int patch_soft_mask(const void* W_dev, int64_t ldw, const float* P_tile_dev, const float* P24_dev,
                    int64_t N, int64_t K, int tile_n, int tile_k, float tau, float kappa, uint64_t seed,
                    int flags, void* Wt_dev, int64_t ldo, float* Mt_dev, int64_t ldm, double* sums_dev,
                    void* workspace_dev, size_t workspace_bytes, void* stream);

/*
 * The two regularisers of Eq. 5 from the sums of n matrices (host arrays, [n x 4] as written by
 * patch_soft_mask): lambda1 * | sum_i sum(Mt_i) / sum_i ||W_i||_0 - rho | - lambda2 * sum_i ||Mt_i (.) W_i||^2 / sum_i ||W_i||^2.
 * Host only.
 */
int patch_mask_regularizers(const double* sums_host, int n, double rho, double lambda1, double lambda2,
                            double* out_host);

/*
 * Coefficients with which one element's soft-mask value enters the gradient of the regularisers of
 * Eq. 5, from the pooled sums of n matrices (host arrays as for patch_mask_regularizers):
 *   *c1_host = lambda1 * sign(sum Mt / sum ||W||_0 - rho) / sum ||W||_0
 *   *c2_host = 2 * lambda2 / sum ||W||^2
 * so that d(regularisers)/dMt_e = c1 - c2 * Mt_e * W_e^2.  Host only.
 */
int patch_mask_regularizer_coefficients(const double* sums_host, int n, double rho, double lambda1,
                                        double lambda2, double* c1_host, double* c2_host);

/*
 * Backward of patch_soft_mask (the logit update step of Algorithm 1): gradient with
 * respect to the logits of
 *   F = sum_e Gw_e Mt_e W_e + c1 sum_e Mt_e - (c2 / 2) sum_e (Mt_e W_e)^2,
 * where Gw = dL_LM / d(Mt (.) W) is the gradient the language-model loss returns for the masked weight
 * and c1, c2 come from patch_mask_regularizer_coefficients.  The forward is recomputed on the fly with
 * the same (seed, flags), so nothing has to be kept from the forward call:
 *   gM_e = Gw_e W_e + c1 - c2 Mt_e W_e^2;   h_c = (1 - Mt_tile) sum_j S[c][j] gM_j   (per group)
 *   gP24_dev[c][grp] = (kappa / tau) GS_c (h_c - sum_k GS_k h_k)
 *   gP_tile_dev[t]   = (kappa / tau) Mt_tile (1 - Mt_tile) sum_{e in tile t} gM_e (1 - Mt_2:4,e)
 *   Gw_dev  bf16 [N x ldg];  gP_tile_dev fp32 [N/128 x K/128];  gP24_dev fp32 [6 x G], 16-byte aligned.
 * Every output element is written (no accumulation into the buffers).  fp32 arithmetic, the tile sum in
 * a fixed order.  One kernel, no workspace, no host synchronisation.
 */
int patch_soft_mask_backward(const void* W_dev, int64_t ldw, const float* P_tile_dev, const float* P24_dev,
                             int64_t N, int64_t K, int tile_n, int tile_k, float tau, float kappa,
                             uint64_t seed, int flags, const void* Gw_dev, int64_t ldg, double c1, double c2,
                             float* gP_tile_dev, float* gP24_dev, void* stream);

/* Human-readable text for a status code (static storage). */
const char* patch_strerror(int status);

/* Library version (1). */
int patch_version(void);

#ifdef __cplusplus
}
#endif
#endif /* PATCH_B200_H_ */
