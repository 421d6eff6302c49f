// C-ABI entry points of the matmul: argument validation and kernel choice.
#include "sm100_ptx.cuh"

using namespace patch;

static int check_gemm_args(const void* X, int64_t ldx, int64_t M, const patch_layout_t* L, const void* packed,
                           const void* Y, int64_t ldy) {
    if (!L) return PATCH_ERR_NULL;
    int rc = validate_layout(L);
    if (rc) return rc;
    if (M < 0) return PATCH_ERR_SHAPE;
    if (M == 0) return PATCH_OK;
    if (!X || !packed || !Y) return PATCH_ERR_NULL;
    if (ldx < L->K || ldy < L->N || ldx % 8 || ldy % 8) return PATCH_ERR_SHAPE;
    if (!aligned16(X) || !aligned16(Y) || !aligned16(packed)) return PATCH_ERR_ALIGN;
    return PATCH_OK;
}

extern "C" int patch_gemm_workspace_size(const patch_layout_t* L, int64_t M, size_t* bytes_out) {
    if (!L || !bytes_out) return PATCH_ERR_NULL;
    int rc = validate_layout(L);
    if (rc) return rc;
    if (M < 0) return PATCH_ERR_SHAPE;
    if (has_q4_tiles(L)) {
        // 4-bit tiles: nothing for the decode kernel; beyond 64 tokens, room for the weight's bf16 image
        *bytes_out = 0;
        if (M > 64 && !L->n_dense && !L->n_sparse) {
            patch_layout_t E;
            q4_expanded_layout(L, &E);
            *bytes_out = kQ4ExpandOffset + size_t(E.total_bytes);
        }
        return PATCH_OK;
    }
    *bytes_out = decode_workspace_bytes(L, M);
    return PATCH_OK;
}

extern "C" int patch_workspace_init(void* workspace_dev, size_t bytes, void* stream) {
    if (bytes == 0) return PATCH_OK;
    if (!workspace_dev) return PATCH_ERR_NULL;
    return cudaMemsetAsync(workspace_dev, 0, bytes, static_cast<cudaStream_t>(stream)) == cudaSuccess
               ? PATCH_OK : PATCH_ERR_CUDA;
}

extern "C" int patch_gemm_ex(const void* X_dev, int64_t ldx, int64_t M, const patch_layout_t* L,
                             const void* packed_dev, void* Y_dev, int64_t ldy, void* workspace_dev,
                             size_t workspace_bytes, int* status_dev, void* stream, int variant) {
    int rc = check_gemm_args(X_dev, ldx, M, L, packed_dev, Y_dev, ldy);
    if (rc) return rc;
    if (M == 0) return PATCH_OK;
    const bool wstatic = (variant & PATCH_GEMM_WEIGHTS_STATIC) != 0;
    const bool xstatic = (variant & PATCH_GEMM_INPUT_STATIC) != 0;
    const bool ystatic = wstatic && xstatic && (variant & PATCH_GEMM_OUTPUT_STATIC) != 0;
    variant &= ~(PATCH_GEMM_WEIGHTS_STATIC | PATCH_GEMM_INPUT_STATIC | PATCH_GEMM_OUTPUT_STATIC);
    if (variant != PATCH_VARIANT_AUTO && variant != PATCH_VARIANT_GEMV && variant != PATCH_VARIANT_MMA &&
        variant != PATCH_VARIANT_PAIR)
        return PATCH_ERR_SHAPE;
    if (variant == PATCH_VARIANT_GEMV && M > 4) return PATCH_ERR_SHAPE;
    if (variant == PATCH_VARIANT_PAIR && M <= 64) return PATCH_ERR_SHAPE;
    if (has_q4_tiles(L)) {
        // 4-bit tiles: the dequantising decode kernel, for weights made of such tiles only
        if (L->n_dense || L->n_sparse || variant == PATCH_VARIANT_GEMV || variant == PATCH_VARIANT_PAIR) return PATCH_ERR_SHAPE;
        rc = check_device();
        if (rc) return rc;
        if (M > 64) {
            // many tokens: the weight is rewritten once as the bf16 blob of its dequantised values (in the
            // workspace), and the large-M schedule multiplies by that -- the same values, so the same result as
            // the decode kernel's definition; the blob was just written, so no promise is passed on
            patch_layout_t E;
            q4_expanded_layout(L, &E);
            if (!workspace_dev) return PATCH_ERR_NULL;
            if (workspace_bytes < kQ4ExpandOffset + E.total_bytes) return PATCH_ERR_SIZE;
            if (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) return PATCH_ERR_ALIGN;
            cudaStream_t s4 = static_cast<cudaStream_t>(stream);
            uint8_t* image = static_cast<uint8_t*>(workspace_dev) + kQ4ExpandOffset;     // the words other calls keep zero stay untouched
            rc = launch_expand_q4(L, static_cast<const uint8_t*>(packed_dev), &E, image, status_dev, s4);
            if (rc) return rc;
            return launch_prefill(static_cast<const __nv_bfloat16*>(X_dev), ldx, M, &E, image,
                                  static_cast<__nv_bfloat16*>(Y_dev), ldy, status_dev, s4, false, false);
        }
        // 17 .. 64 tokens: sixteen at a time, one launch each, under the caller's promises (a later launch
        // may not assume more than the first: it can start while the kernels before this call still run)
        for (int64_t m0 = 0; m0 < M; m0 += 16) {
            rc = launch_decode_q4(static_cast<const __nv_bfloat16*>(X_dev) + m0 * ldx, ldx, M - m0 < 16 ? M - m0 : 16, L,
                                  static_cast<const uint8_t*>(packed_dev), static_cast<__nv_bfloat16*>(Y_dev) + m0 * ldy, ldy,
                                  status_dev, static_cast<cudaStream_t>(stream), wstatic, xstatic, ystatic);
            if (rc) return rc;
        }
        return PATCH_OK;
    }
    const size_t need = decode_workspace_bytes(L, M);
    if (need > 0) {
        if (!workspace_dev) return PATCH_ERR_NULL;
        if (workspace_bytes < need) return PATCH_ERR_SIZE;
        if (reinterpret_cast<uintptr_t>(workspace_dev) & 255u) return PATCH_ERR_ALIGN;
    }
    rc = check_device();
    if (rc) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const __nv_bfloat16* X = static_cast<const __nv_bfloat16*>(X_dev);
    __nv_bfloat16* Y = static_cast<__nv_bfloat16*>(Y_dev);
    const uint8_t* packed = static_cast<const uint8_t*>(packed_dev);
    if (variant == PATCH_VARIANT_GEMV) return launch_gemv(X, ldx, int(M), L, packed, Y, ldy, status_dev, s);
    if (M <= 64) return launch_decode(X, ldx, M, L, packed, Y, ldy, workspace_dev, status_dev, s, wstatic, xstatic, ystatic);
    return launch_prefill(X, ldx, M, L, packed, Y, ldy, status_dev, s, wstatic && xstatic, variant == PATCH_VARIANT_PAIR);
}

extern "C" int patch_gemm(const void* X_dev, int64_t ldx, int64_t M, const patch_layout_t* L,
                          const void* packed_dev, void* Y_dev, int64_t ldy, void* workspace_dev,
                          size_t workspace_bytes, int* status_dev, void* stream) {
    return patch_gemm_ex(X_dev, ldx, M, L, packed_dev, Y_dev, ldy, workspace_dev, workspace_bytes, status_dev,
                         stream, PATCH_VARIANT_AUTO);
}

extern "C" int patch_gemm_gated_workspace_size(const patch_layout_t* L, int64_t M, size_t* bytes_out) {
    if (!L || !bytes_out) return PATCH_ERR_NULL;
    int rc = validate_layout(L);
    if (rc) return rc;
    if (L->N % (2 * kTile) || M < 0) return PATCH_ERR_SHAPE;
    if (has_q4_tiles(L)) return PATCH_ERR_SHAPE;
    *bytes_out = decode_gated_workspace_bytes(L, M);
    return PATCH_OK;
}

extern "C" int patch_gemm_gated(const void* X_dev, int64_t ldx, int64_t M, const patch_layout_t* L,
                                const void* packed_dev, void* Y_dev, int64_t ldy, void* workspace_dev,
                                size_t workspace_bytes, int* status_dev, void* stream, int flags) {
    if (!L) return PATCH_ERR_NULL;
    int rc = validate_layout(L);
    if (rc) return rc;
    if (L->N % (2 * kTile)) return PATCH_ERR_SHAPE;      // whole (gate, up) pairs of row-blocks
    if (M < 0 || has_q4_tiles(L)) return PATCH_ERR_SHAPE;
    if (flags & ~(PATCH_GEMM_WEIGHTS_STATIC | PATCH_GEMM_INPUT_STATIC | PATCH_GEMM_OUTPUT_STATIC)) return PATCH_ERR_SHAPE;
    if (M == 0) return PATCH_OK;
    if (!X_dev || !packed_dev || !Y_dev) return PATCH_ERR_NULL;
    if (ldx < L->K || ldy < L->N / 2 || ldx % 8 || ldy % 8) return PATCH_ERR_SHAPE;
    if (!aligned16(X_dev) || !aligned16(Y_dev) || !aligned16(packed_dev)) return PATCH_ERR_ALIGN;
    rc = check_device();
    if (rc) return rc;
    const __nv_bfloat16* X = static_cast<const __nv_bfloat16*>(X_dev);
    __nv_bfloat16* Y = static_cast<__nv_bfloat16*>(Y_dev);
    const uint8_t* packed = static_cast<const uint8_t*>(packed_dev);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // small M on static weights: one cluster per (gate, up) pair of row-blocks, no workspace -- few CTAs if the launch
    // was also declared independent of its predecessor, at least 128 if it has to wait for it
    if (M <= 16 && (flags & PATCH_GEMM_WEIGHTS_STATIC)) {
        CUtensorMap map;
        rc = make_x_tensor_map(&map, X, ldx, M, L->K, 16);
        if (rc) return rc;
        return launch_decode_cluster_gated(map, L, packed, int(M), Y, ldy, status_dev, s, (flags & PATCH_GEMM_INPUT_STATIC) != 0);
    }
    // small M with a workspace: the stream-K schedule; otherwise the two-row-block schedule, which needs none
    const size_t need = decode_gated_workspace_bytes(L, M);
    if (need > 0 && workspace_dev && workspace_bytes >= need && !(reinterpret_cast<uintptr_t>(workspace_dev) & 255u))
        return launch_decode_gated(X, ldx, M, L, packed, Y, ldy, workspace_dev, status_dev, s,
                                   (flags & PATCH_GEMM_WEIGHTS_STATIC) != 0, (flags & PATCH_GEMM_INPUT_STATIC) != 0);
    return launch_prefill_gated(X, ldx, M, L, packed, Y, ldy, status_dev, s,
                                (flags & PATCH_GEMM_WEIGHTS_STATIC) && (flags & PATCH_GEMM_INPUT_STATIC));
}

extern "C" int patch_gemm_host(const void* X_host, int64_t M, const patch_layout_t* L, const void* packed_dev,
                               void* Y_host, void* X_stage_dev, void* Y_stage_dev, void* workspace_dev,
                               size_t workspace_bytes, void* stream) {
    if (!L) return PATCH_ERR_NULL;
    int rc = validate_layout(L);
    if (rc) return rc;
    if (M < 0) return PATCH_ERR_SHAPE;
    if (M == 0) return PATCH_OK;
    if (!X_host || !Y_host || !X_stage_dev || !Y_stage_dev) return PATCH_ERR_NULL;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(X_stage_dev, X_host, size_t(M) * L->K * 2, cudaMemcpyHostToDevice, s) != cudaSuccess)
        return PATCH_ERR_CUDA;
    rc = patch_gemm(X_stage_dev, L->K, M, L, packed_dev, Y_stage_dev, L->N, workspace_dev, workspace_bytes,
                    nullptr, stream);
    if (rc) return rc;
    if (cudaMemcpyAsync(Y_host, Y_stage_dev, size_t(M) * L->N * 2, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return PATCH_ERR_CUDA;
    return cudaStreamSynchronize(s) == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

// Validation shared by the batched host entry points: everything is checked before anything is enqueued.
static int check_host_jobs(const patch_host_job_t* jobs, int n_jobs) {
    if (n_jobs < 0) return PATCH_ERR_SHAPE;
    if (n_jobs == 0) return PATCH_OK;
    if (!jobs) return PATCH_ERR_NULL;
    for (int i = 0; i < n_jobs; ++i) {
        const patch_host_job_t& j = jobs[i];
        if (!j.layout) return PATCH_ERR_NULL;
        int rc = validate_layout(j.layout);
        if (rc) return rc;
        if (j.M < 0) return PATCH_ERR_SHAPE;
        if (j.M > 0 && (!j.X_host || !j.Y_host || !j.X_stage_dev || !j.Y_stage_dev || !j.packed_dev)) return PATCH_ERR_NULL;
    }
    return PATCH_OK;
}

// Copies of jobs [first, last) in one direction.  Consecutive jobs whose host buffers and staging buffers are
// both adjacent in memory are issued as one copy: a step whose activations live in one host arena costs one
// transfer each way.
static bool copy_jobs(const patch_host_job_t* jobs, int first, int last, bool inbound, cudaStream_t s) {
    const char* run_host = nullptr; const char* run_dev = nullptr; size_t run_bytes = 0;
    auto flush = [&]() -> bool {
        if (!run_bytes) return true;
        const cudaError_t e = inbound
            ? cudaMemcpyAsync(const_cast<char*>(run_dev), run_host, run_bytes, cudaMemcpyHostToDevice, s)
            : cudaMemcpyAsync(const_cast<char*>(run_host), run_dev, run_bytes, cudaMemcpyDeviceToHost, s);
        run_bytes = 0;
        return e == cudaSuccess;
    };
    for (int i = first; i < last; ++i) {
        const patch_host_job_t& j = jobs[i];
        if (!j.M) continue;
        const char* h = static_cast<const char*>(inbound ? j.X_host : j.Y_host);
        const char* d = static_cast<const char*>(inbound ? j.X_stage_dev : j.Y_stage_dev);
        const size_t bytes = size_t(j.M) * size_t(inbound ? j.layout->K : j.layout->N) * 2;
        if (run_bytes && h == run_host + run_bytes && d == run_dev + run_bytes) { run_bytes += bytes; continue; }
        if (!flush()) return false;
        run_host = h; run_dev = d; run_bytes = bytes;
    }
    return flush();
}

static int launch_jobs(const patch_host_job_t* jobs, int first, int last, int flags, void* stream) {
    for (int i = first; i < last; ++i) {
        const patch_host_job_t& j = jobs[i];
        int rc = patch_gemm_ex(j.X_stage_dev, j.layout->K, j.M, j.layout, j.packed_dev, j.Y_stage_dev, j.layout->N,
                               j.workspace_dev, j.workspace_bytes, nullptr, stream, PATCH_VARIANT_AUTO | flags);
        if (rc) return rc;
    }
    return PATCH_OK;
}

extern "C" int patch_gemm_host_batch(const patch_host_job_t* jobs, int n_jobs, int weights_static, void* stream) {
    int rc = check_host_jobs(jobs, n_jobs);
    if (rc || n_jobs == 0) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!copy_jobs(jobs, 0, n_jobs, true, s)) return PATCH_ERR_CUDA;
    // with two or more jobs the operation before any launch is another launch or the copy of a different X
    const int flags = weights_static ? (PATCH_GEMM_WEIGHTS_STATIC | (n_jobs >= 2 ? PATCH_GEMM_INPUT_STATIC : 0)) : 0;
    rc = launch_jobs(jobs, 0, n_jobs, flags, stream);
    if (rc) return rc;
    if (!copy_jobs(jobs, 0, n_jobs, false, s)) return PATCH_ERR_CUDA;
    return cudaStreamSynchronize(s) == cudaSuccess ? PATCH_OK : PATCH_ERR_CUDA;
}

extern "C" int patch_gemm_host_batch_pipelined(const patch_host_job_t* jobs, int n_jobs, int weights_static, int n_chunks,
                                               void* stream, void* copy_in_stream, void* copy_out_stream) {
    int rc = check_host_jobs(jobs, n_jobs);
    if (rc || n_jobs == 0) return rc;
    if (n_chunks < 1 || n_chunks > 64) return PATCH_ERR_SHAPE;
    cudaStream_t s = static_cast<cudaStream_t>(stream), sin = static_cast<cudaStream_t>(copy_in_stream),
                 sout = static_cast<cudaStream_t>(copy_out_stream);
    if (s == sin || s == sout || sin == sout) return PATCH_ERR_SHAPE;      // three distinct streams
    if (n_chunks > n_jobs) n_chunks = n_jobs;
    // chunk boundaries by output bytes, so that the last copy out (the only one nothing overlaps) is short
    int bound[65];
    {
        double total = 0, acc = 0;
        for (int i = 0; i < n_jobs; ++i) total += double(jobs[i].M) * double(jobs[i].layout->N + jobs[i].layout->K);
        int c = 0;
        bound[0] = 0;
        for (int i = 0; i < n_jobs && c + 1 < n_chunks; ++i) {
            acc += double(jobs[i].M) * double(jobs[i].layout->N + jobs[i].layout->K);
            if (acc >= total * (c + 1) / n_chunks && n_jobs - (i + 1) >= n_chunks - (c + 1)) bound[++c] = i + 1;
        }
        while (c + 1 < n_chunks) { bound[c + 1] = bound[c] + 1; ++c; }
        bound[n_chunks] = n_jobs;
    }
    cudaEvent_t landed[64], done[64];
    int n_events = 0;
    auto cleanup = [&]() { for (int i = 0; i < n_events; ++i) { cudaEventDestroy(landed[i]); cudaEventDestroy(done[i]); } };
    for (; n_events < n_chunks; ++n_events)
        if (cudaEventCreateWithFlags(&landed[n_events], cudaEventDisableTiming) != cudaSuccess ||
            cudaEventCreateWithFlags(&done[n_events], cudaEventDisableTiming) != cudaSuccess) {
            cleanup();
            return PATCH_ERR_CUDA;
        }
    // every X is on the device before the GEMM that reads it (event), and is written by a copy on another stream;
    // a Y is written by its own GEMM only and read by a copy that waits for the whole run (event)
    const int flags = weights_static ? (PATCH_GEMM_WEIGHTS_STATIC | PATCH_GEMM_INPUT_STATIC | PATCH_GEMM_OUTPUT_STATIC) : 0;
    rc = PATCH_OK;
    bool ok = true;
    for (int c = 0; c < n_chunks && ok && !rc; ++c) {
        ok = copy_jobs(jobs, bound[c], bound[c + 1], true, sin) && cudaEventRecord(landed[c], sin) == cudaSuccess &&
             cudaStreamWaitEvent(s, landed[c], 0) == cudaSuccess;
        if (!ok) break;
        rc = launch_jobs(jobs, bound[c], bound[c + 1], flags, stream);
        if (rc) break;
        ok = cudaEventRecord(done[c], s) == cudaSuccess && cudaStreamWaitEvent(sout, done[c], 0) == cudaSuccess &&
             copy_jobs(jobs, bound[c], bound[c + 1], false, sout);
    }
    // whatever was enqueued is waited for, also on failure: the caller's buffers are then quiescent
    const bool synced = cudaStreamSynchronize(sin) == cudaSuccess && cudaStreamSynchronize(s) == cudaSuccess &&
                        cudaStreamSynchronize(sout) == cudaSuccess;
    cleanup();
    if (rc) return rc;
    return ok && synced ? PATCH_OK : PATCH_ERR_CUDA;
}

extern "C" const char* patch_strerror(int status) {
    switch (status) {
        case PATCH_OK: return "ok";
        case PATCH_ERR_NULL: return "a required pointer is NULL";
        case PATCH_ERR_SHAPE: return "unsupported shape or leading dimension";
        case PATCH_ERR_TILE: return "tile shape must be 128 x 128";
        case PATCH_ERR_FLAG: return "tile flag is neither dense nor 2:4";
        case PATCH_ERR_ALIGN: return "pointer or pitch is not sufficiently aligned";
        case PATCH_ERR_SIZE: return "buffer too small";
        case PATCH_ERR_FORMAT: return "inconsistent packed layout";
        case PATCH_ERR_ARCH: return "device is not sm_100";
        case PATCH_ERR_CUDA: return "CUDA runtime error";
        case PATCH_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

extern "C" int patch_version(void) { return 1; }
