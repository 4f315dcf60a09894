// C ABI entry points: argument validation, host-side planning (block counts, split-K chunks, tensor
// maps) and kernel launches.  Everything a kernel needs to know about the batch is computed
// here from the caller's host arrays and passed by value, so no call waits for the device.
#include <stdarg.h>
#include <stdlib.h>

#include <new>

#include "dodo_internal.cuh"

int dodo_fail(dodo_ctx* ctx, int status, const char* fmt, ...) {
    if (ctx != nullptr) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof ctx->err, fmt, ap);
        va_end(ap);
    }
    return status;
}

int dodo_check_cuda(dodo_ctx* ctx, cudaError_t e, const char* what) {
    if (e == cudaSuccess) return DODO_OK;
    return dodo_fail(ctx, DODO_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

namespace {

bool valid_dtype(int dtype) { return dtype == DODO_F32 || dtype == DODO_BF16; }

// Offsets must start at 0 and never decrease.
bool valid_offsets(const int32_t* off, int B) {
    if (off == nullptr || off[0] != 0) return false;
    for (int b = 0; b < B; ++b)
        if (off[b + 1] < off[b]) return false;
    return true;
}

int check_score_args(dodo_ctx* ctx, const void* X, int dtype, int d, const void* w, const int32_t* seq_off,
                     int B, const float* scores) {
    if (B < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "B = %d is negative", B);
    if (!valid_dtype(dtype)) return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "dtype %d", dtype);
    if (d <= 0 || (static_cast<size_t>(d) * dodo_elem_bytes(dtype)) % 16 != 0)
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "d = %d: a row must be a positive multiple of 16 bytes", d);
    if (static_cast<size_t>(d) * dodo_elem_bytes(dtype) > 96 * 1024)
        return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "d = %d: weight vector exceeds 96 KB of shared memory", d);
    if (!valid_offsets(seq_off, B)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "seq_off must start at 0 and be non-decreasing");
    if (seq_off[B] > 0 && (X == nullptr || w == nullptr || scores == nullptr))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "X, w and scores must not be NULL");
    if (!dodo_aligned16(X) || !dodo_aligned16(w))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "X and w must be 16-byte aligned");
    return DODO_OK;
}

int check_select_args(dodo_ctx* ctx, const int32_t* seq_off, const int32_t* nug_off, int B, uint32_t flags,
                      const void* idx) {
    if (B < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "B = %d is negative", B);
    if (!valid_offsets(seq_off, B)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "seq_off must start at 0 and be non-decreasing");
    if (!valid_offsets(nug_off, B)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "nug_off must start at 0 and be non-decreasing");
    if (flags & ~static_cast<uint32_t>(DODO_FORCE_LAST)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "unknown flags 0x%x", flags);
    for (int b = 0; b < B; ++b) {
        const int n = seq_off[b + 1] - seq_off[b], k = nug_off[b + 1] - nug_off[b];
        if (k > n) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sequence %d: k = %d exceeds n = %d", b, k, n);
    }
    if (nug_off[B] > 0 && idx == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "idx must not be NULL");
    return DODO_OK;
}

void fill_score_group(ScoreSelectGroup& g, const int32_t* seq_off, const int32_t* nug_off, int b0, int nb,
                      int rpb = dodo_score_rows_per_block()) {
    g.nseq = nb;
    g.blk0[0] = 0;
    for (int i = 0; i < nb; ++i) {
        const int b = b0 + i;
        g.row0[i] = seq_off[b];
        g.n[i] = seq_off[b + 1] - seq_off[b];
        g.k[i] = nug_off ? nug_off[b + 1] - nug_off[b] : 0;
        g.idx0[i] = nug_off ? nug_off[b] : 0;
        g.blk0[i + 1] = g.blk0[i] + (g.n[i] + rpb - 1) / rpb;
    }
}

int score_impl(dodo_ctx* ctx, const void* X, int dtype, int d, const void* w, float bias,
               const int32_t* seq_off, const int32_t* nug_off, int B, bool fused, uint32_t flags,
               float* scores, int32_t* idx, void* stream) {
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int b0 = 0; b0 < B; b0 += DODO_GROUP) {
        ScoreSelectGroup g;
        fill_score_group(g, seq_off, nug_off, b0, B - b0 < DODO_GROUP ? B - b0 : DODO_GROUP);
        const int rc = dodo_launch_score(ctx, X, dtype, d, w, bias, g, fused ? 1 : 0, flags, scores, idx, ctx->tickets, nullptr, st);
        if (rc != DODO_OK) return rc;
    }
    return DODO_OK;
}

size_t attend_partial_rows_bound(const dodo_ctx* ctx) {
    // split-K only happens while (query tiles x heads) < target, and then the block count stays
    // below 2 x target; a block writes at most 8 partial rows
    return static_cast<size_t>(16) * static_cast<size_t>(ctx->attend_target_ctas);
}

}  // namespace

extern "C" {

int dodo_create(dodo_ctx** out, int device) {
    if (out == nullptr) return DODO_ERR_INVALID_ARG;
    *out = nullptr;
    dodo_ctx* ctx = new (std::nothrow) dodo_ctx();
    if (ctx == nullptr) return DODO_ERR_CUDA;
    memset(ctx, 0, sizeof *ctx);
    ctx->device = device;
    *out = ctx;  // handed back even on failure so the reason can be read; destroy it either way
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "cudaSetDevice");
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "cudaGetDeviceProperties");
    if (prop.major != 10)
        return dodo_fail(ctx, DODO_ERR_CUDA, "device %d is sm_%d%d; this library is built for sm_100a only", device,
                         prop.major, prop.minor);
    ctx->num_sms = prop.multiProcessorCount;
    ctx->max_smem_optin = static_cast<int>(prop.sharedMemPerBlockOptin);
    ctx->attend_target_ctas = 2 * ctx->num_sms;
    ctx->dense_min_tq = 32;
    ctx->dense_balance = 0;
    cudaDriverEntryPointQueryResult qres;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ctx->encode_tiled, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || ctx->encode_tiled == nullptr)
        return dodo_fail(ctx, DODO_ERR_CUDA, "cuTensorMapEncodeTiled is not available from this driver");
    e = cudaMalloc(&ctx->tickets, (DODO_NUM_TICKETS + 64 + DODO_FLAG_STRIDE * (1 + DODO_GROUP) + 256 * DODO_GROUP) * sizeof(int));
    if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "cudaMalloc(tickets)");
    ctx->dev_status = ctx->tickets + DODO_NUM_TICKETS;
    ctx->compress_state = ctx->tickets + DODO_NUM_TICKETS + 64;
    ctx->top_hist = ctx->compress_state + DODO_FLAG_STRIDE * (1 + DODO_GROUP);
    e = cudaMemset(ctx->tickets, 0, (DODO_NUM_TICKETS + 64 + DODO_FLAG_STRIDE * (1 + DODO_GROUP) + 256 * DODO_GROUP) * sizeof(int));
    if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "cudaMemset(tickets)");
    return DODO_OK;
}

int dodo_destroy(dodo_ctx* ctx) {
    if (ctx == nullptr) return DODO_OK;
    if (ctx->tickets != nullptr) cudaFree(ctx->tickets);
    delete ctx;
    return DODO_OK;
}

const char* dodo_last_error(const dodo_ctx* ctx) { return ctx ? ctx->err : "no context"; }

int dodo_reset(dodo_ctx* ctx, void* stream) {
    if (ctx == nullptr || ctx->tickets == nullptr) return DODO_ERR_INVALID_ARG;
    return dodo_check_cuda(ctx, cudaMemsetAsync(ctx->tickets, 0, (DODO_NUM_TICKETS + 64 + DODO_FLAG_STRIDE * (1 + DODO_GROUP) + 256 * DODO_GROUP) * sizeof(int),
                                                static_cast<cudaStream_t>(stream)), "reset");
}

int dodo_device_status(dodo_ctx* ctx, int* status) {
    if (ctx == nullptr || status == nullptr || ctx->dev_status == nullptr) return DODO_ERR_INVALID_ARG;
    return dodo_check_cuda(ctx, cudaMemcpy(status, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost),
                           "device status");
}

int dodo_cache_written(dodo_ctx* ctx) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    ctx->cache_clean = false;
    return DODO_OK;
}

int dodo_set_tuning(dodo_ctx* ctx, int knob, int value) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    if (knob == DODO_TUNE_ATTEND_TARGET_BLOCKS) {
        if (value < 1 || value > 4096) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "target blocks %d out of [1, 4096]", value);
        ctx->attend_target_ctas = value;
    } else if (knob == DODO_TUNE_DENSE_MIN_QUERIES) {
        if (value < 1) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "dense threshold %d must be positive", value);
        ctx->dense_min_tq = value;
    } else if (knob == DODO_TUNE_DENSE_BALANCE) {
        if (value < 0 || value > 3) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "dense balance mode %d (0 to 3)", value);
        ctx->dense_balance = value;
    } else {
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "unknown tuning knob %d", knob);
    }
    return DODO_OK;
}

int dodo_num_nuggets(int n, int r) {
    if (n < 0 || r < 1) return -1;
    return n / r + (n % r != 0 ? 1 : 0);
}

int dodo_score(dodo_ctx* ctx, const void* X, int dtype, int d, const void* w, float bias,
               const int32_t* seq_off, int B, float* scores, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    const int rc = check_score_args(ctx, X, dtype, d, w, seq_off, B, scores);
    if (rc != DODO_OK) return rc;
    return score_impl(ctx, X, dtype, d, w, bias, seq_off, nullptr, B, false, 0, scores, nullptr, stream);
}

int dodo_select(dodo_ctx* ctx, const float* scores, const int32_t* seq_off, const int32_t* nug_off,
                int B, uint32_t flags, int32_t* idx, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    const int rc = check_select_args(ctx, seq_off, nug_off, B, flags, idx);
    if (rc != DODO_OK) return rc;
    if (seq_off[B] > 0 && scores == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "scores must not be NULL");
    for (int b0 = 0; b0 < B; b0 += DODO_GROUP) {
        ScoreSelectGroup g;
        fill_score_group(g, seq_off, nug_off, b0, B - b0 < DODO_GROUP ? B - b0 : DODO_GROUP);
        const int r2 = dodo_launch_select(ctx, scores, g, flags, idx, false, static_cast<cudaStream_t>(stream));
        if (r2 != DODO_OK) return r2;
    }
    return DODO_OK;
}

size_t dodo_score_mlp_workspace_bytes(int rows, int dh) { return dodo_score_mlp_partial_bytes(rows, dh); }

int dodo_score_mlp(dodo_ctx* ctx, const void* X, int dtype, int d, const void* W1, const float* b1, const void* w2,
                   float b2, int dh, int act, const int32_t* seq_off, int B, float* scores, void* workspace,
                   size_t workspace_bytes, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    if (B < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "B = %d is negative", B);
    if (!valid_dtype(dtype)) return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "dtype %d", dtype);
    if (!valid_offsets(seq_off, B)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "seq_off must start at 0 and be non-decreasing");
    if (act < DODO_ACT_IDENTITY || act > DODO_ACT_GELU_TANH) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "activation %d", act);
    if (!dodo_score_mlp_supported(dtype, d, dh))
        return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "two-layer Scorer: bf16 with d a multiple of 64 and dh a multiple of 256 (got dtype %d, d %d, dh %d)", dtype, d, dh);
    const int rows = B > 0 ? seq_off[B] : 0;
    if (rows == 0) return DODO_OK;
    if (X == nullptr || W1 == nullptr || b1 == nullptr || w2 == nullptr || scores == nullptr)
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "X, W1, b1, w2 and scores must not be NULL");
    if (!dodo_aligned16(X) || !dodo_aligned16(W1)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "X and W1 must be 16-byte aligned");
    if (workspace == nullptr || !dodo_aligned16(workspace) || workspace_bytes < dodo_score_mlp_partial_bytes(rows, dh))
        return dodo_fail(ctx, DODO_ERR_CAPACITY, "workspace of %zu bytes is too small or misaligned (need %zu)", workspace_bytes,
                         dodo_score_mlp_partial_bytes(rows, dh));
    return dodo_launch_score_mlp(ctx, X, rows, d, W1, b1, w2, b2, dh, act, scores, static_cast<float*>(workspace), nullptr, 0, 0,
                                 nullptr, static_cast<cudaStream_t>(stream));
}

int dodo_score_mlp_select(dodo_ctx* ctx, const void* X, int dtype, int d, const void* W1, const float* b1, const void* w2,
                          float b2, int dh, int act, const int32_t* seq_off, const int32_t* nug_off, int B, uint32_t flags,
                          float* scores, int32_t* idx, void* workspace, size_t workspace_bytes, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    int rc = check_select_args(ctx, seq_off, nug_off, B, flags, idx);
    if (rc != DODO_OK) return rc;
    int max_n = 0;
    for (int b = 0; b < B; ++b) max_n = max_n > seq_off[b + 1] - seq_off[b] ? max_n : seq_off[b + 1] - seq_off[b];
    if (max_n > dodo_score_mlp_fused_max_tokens()) {
        // long sequences: the select's passes dominate, and a launch of its own gives it more threads per sequence
        rc = dodo_score_mlp(ctx, X, dtype, d, W1, b1, w2, b2, dh, act, seq_off, B, scores, workspace, workspace_bytes, stream);
        return rc != DODO_OK ? rc : dodo_select(ctx, scores, seq_off, nug_off, B, flags, idx, stream);
    }
    if (!valid_dtype(dtype)) return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "dtype %d", dtype);
    if (act < DODO_ACT_IDENTITY || act > DODO_ACT_GELU_TANH) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "activation %d", act);
    if (!dodo_score_mlp_supported(dtype, d, dh))
        return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "two-layer Scorer: bf16 with d a multiple of 64 and dh a multiple of 256 (got dtype %d, d %d, dh %d)", dtype, d, dh);
    const int rows = B > 0 ? seq_off[B] : 0;
    if (rows == 0) return DODO_OK;
    if (X == nullptr || W1 == nullptr || b1 == nullptr || w2 == nullptr || scores == nullptr)
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "X, W1, b1, w2 and scores must not be NULL");
    if (!dodo_aligned16(X) || !dodo_aligned16(W1)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "X and W1 must be 16-byte aligned");
    if (workspace == nullptr || !dodo_aligned16(workspace) || workspace_bytes < dodo_score_mlp_partial_bytes(rows, dh))
        return dodo_fail(ctx, DODO_ERR_CAPACITY, "workspace of %zu bytes is too small or misaligned (need %zu)", workspace_bytes,
                         dodo_score_mlp_partial_bytes(rows, dh));
    const int ngroups = (B + DODO_GROUP - 1) / DODO_GROUP;
    ScoreSelectGroup* groups = static_cast<ScoreSelectGroup*>(malloc(sizeof(ScoreSelectGroup) * static_cast<size_t>(ngroups)));
    if (groups == nullptr) return dodo_fail(ctx, DODO_ERR_CUDA, "out of host memory");
    for (int gi = 0; gi < ngroups; ++gi) {
        const int b0 = gi * DODO_GROUP;
        fill_score_group(groups[gi], seq_off, nug_off, b0, B - b0 < DODO_GROUP ? B - b0 : DODO_GROUP, dodo_score_mlp_reduce_rows());
    }
    rc = dodo_launch_score_mlp(ctx, X, rows, d, W1, b1, w2, b2, dh, act, scores, static_cast<float*>(workspace), groups, ngroups, flags,
                               idx, static_cast<cudaStream_t>(stream));
    free(groups);
    return rc;
}

int dodo_count_threshold(dodo_ctx* ctx, const float* scores, const int32_t* seq_off, int B, float lambda,
                         int32_t* counts, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    if (B < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "B = %d is negative", B);
    if (!valid_offsets(seq_off, B)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "seq_off must start at 0 and be non-decreasing");
    if (B > 0 && counts == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "counts must not be NULL");
    if (B > 0 && seq_off[B] > 0 && scores == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "scores must not be NULL");
    for (int b0 = 0; b0 < B; b0 += DODO_GROUP) {
        ThresholdGroup g;
        g.nseq = B - b0 < DODO_GROUP ? B - b0 : DODO_GROUP;
        for (int i = 0; i < g.nseq; ++i) {
            g.row0[i] = seq_off[b0 + i]; g.n[i] = seq_off[b0 + i + 1] - seq_off[b0 + i]; g.out0[i] = b0 + i; g.cap[i] = 0;
        }
        const int rc = dodo_launch_threshold(ctx, scores, g, lambda, false, counts, static_cast<cudaStream_t>(stream));
        if (rc != DODO_OK) return rc;
    }
    return DODO_OK;
}

int dodo_select_threshold(dodo_ctx* ctx, const float* scores, const int32_t* seq_off, const int32_t* nug_off, int B,
                          float lambda, int32_t* idx, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    const int rc0 = check_select_args(ctx, seq_off, nug_off, B, 0, idx);
    if (rc0 != DODO_OK) return rc0;
    if (seq_off[B] > 0 && scores == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "scores must not be NULL");
    for (int b0 = 0; b0 < B; b0 += DODO_GROUP) {
        ThresholdGroup g;
        g.nseq = B - b0 < DODO_GROUP ? B - b0 : DODO_GROUP;
        for (int i = 0; i < g.nseq; ++i) {
            g.row0[i] = seq_off[b0 + i]; g.n[i] = seq_off[b0 + i + 1] - seq_off[b0 + i];
            g.out0[i] = nug_off[b0 + i]; g.cap[i] = nug_off[b0 + i + 1] - nug_off[b0 + i];
        }
        const int rc = dodo_launch_threshold(ctx, scores, g, lambda, true, idx, static_cast<cudaStream_t>(stream));
        if (rc != DODO_OK) return rc;
    }
    return DODO_OK;
}

int dodo_estimate_threshold(dodo_ctx* ctx, const float* sample, int m, int r, float* lambda, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    if (m <= 0 || r < 1) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sample of %d scores, ratio %d", m, r);
    if (sample == nullptr || lambda == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sample and lambda must not be NULL");
    const int k = static_cast<int>((static_cast<long long>(m) + r - 1) / r);
    return dodo_launch_estimate_threshold(ctx, sample, m, k, lambda, static_cast<cudaStream_t>(stream));
}

int dodo_score_select(dodo_ctx* ctx, const void* X, int dtype, int d, const void* w, float bias,
                      const int32_t* seq_off, const int32_t* nug_off, int B, uint32_t flags,
                      float* scores, int32_t* idx, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    int rc = check_score_args(ctx, X, dtype, d, w, seq_off, B, scores);
    if (rc != DODO_OK) return rc;
    rc = check_select_args(ctx, seq_off, nug_off, B, flags, idx);
    if (rc != DODO_OK) return rc;
    // Short sequences: one launch, the last score block of a sequence selects out of shared memory.  Long ones:
    // the select's passes over the scores dominate, and a launch of its own gives it twice the threads.
    int max_n = 0;
    for (int b = 0; b < B; ++b) max_n = max_n > seq_off[b + 1] - seq_off[b] ? max_n : seq_off[b + 1] - seq_off[b];
    if (max_n <= dodo_select_fused_max_tokens())
        return score_impl(ctx, X, dtype, d, w, bias, seq_off, nug_off, B, true, flags, scores, idx, stream);
    // group by group: the score launch also counts the scores' top key digits, the select launch behind it starts
    // from those counts (and clears them)
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    for (int b0 = 0; b0 < B; b0 += DODO_GROUP) {
        ScoreSelectGroup g;
        fill_score_group(g, seq_off, nug_off, b0, B - b0 < DODO_GROUP ? B - b0 : DODO_GROUP);
        rc = dodo_launch_score(ctx, X, dtype, d, w, bias, g, 2, 0, scores, nullptr, ctx->tickets, nullptr, st);
        if (rc != DODO_OK) return rc;
        rc = dodo_launch_select(ctx, scores, g, flags, idx, true, st);
        if (rc != DODO_OK) return rc;
    }
    return DODO_OK;
}

// Checks shared by the two gather entry points (everything but the K/V pointers).  row_bytes is set.
static int gather_check(dodo_ctx* ctx, int dtype, int H, int dh, const int32_t* seq_off, const int32_t* nug_off,
                        const int32_t* pos_base, int B, const int32_t* cache_off, const int32_t* cache_len,
                        size_t* row_bytes) {
    if (B < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "B = %d is negative", B);
    if (!valid_dtype(dtype)) return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "dtype %d", dtype);
    if (H <= 0 || dh <= 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "H = %d, dh = %d", H, dh);
    *row_bytes = static_cast<size_t>(H) * static_cast<size_t>(dh) * dodo_elem_bytes(dtype);
    if (*row_bytes % 16 != 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "a K/V row (%zu bytes) must be a multiple of 16 bytes", *row_bytes);
    if (!valid_offsets(seq_off, B) || !valid_offsets(nug_off, B) || !valid_offsets(cache_off, B))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "seq_off, nug_off and cache_off must start at 0 and be non-decreasing");
    if (pos_base == nullptr || cache_len == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "pos_base and cache_len must not be NULL");
    for (int b = 0; b < B; ++b) {
        const int k = nug_off[b + 1] - nug_off[b], cap = cache_off[b + 1] - cache_off[b];
        if (k > seq_off[b + 1] - seq_off[b]) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sequence %d: k = %d exceeds its tokens", b, k);
        if (cache_len[b] < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sequence %d: negative cache_len", b);
        if (cache_len[b] + k > cap)
            return dodo_fail(ctx, DODO_ERR_CAPACITY, "sequence %d: %d cached + %d new nuggets exceed its %d cache rows", b, cache_len[b], k, cap);
    }
    return DODO_OK;
}

static void gather_group(GatherGroup& g, int b0, int B, const int32_t* seq_off, const int32_t* nug_off,
                         const int32_t* pos_base, const int32_t* cache_off, const int32_t* cache_len) {
    g.nseq = B - b0 < DODO_GROUP ? B - b0 : DODO_GROUP;
    for (int i = 0; i < g.nseq; ++i) {
        const int b = b0 + i;
        g.idx0[i] = nug_off[b];
        g.src_row0[i] = seq_off[b];
        g.n[i] = seq_off[b + 1] - seq_off[b];
        g.dst_row0[i] = cache_off[b] + cache_len[b];
        g.pos_base[i] = pos_base[b];
    }
    g.idx0[g.nseq] = nug_off[b0 + g.nseq];
}

int dodo_gather_kv(dodo_ctx* ctx, const void* K, const void* V, int dtype, int H, int dh,
                   const int32_t* seq_off, const int32_t* idx, const int32_t* nug_off,
                   const int32_t* pos_base, int B, void* cacheK, void* cacheV, int32_t* cache_pos,
                   const int32_t* cache_off, int32_t* cache_len, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    size_t row_bytes = 0;
    const int rc0 = gather_check(ctx, dtype, H, dh, seq_off, nug_off, pos_base, B, cache_off, cache_len, &row_bytes);
    if (rc0 != DODO_OK) return rc0;
    if (nug_off[B] > 0) {
        if (K == nullptr || V == nullptr || idx == nullptr || cacheK == nullptr || cacheV == nullptr || cache_pos == nullptr)
            return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "K, V, idx, cacheK, cacheV and cache_pos must not be NULL");
        if (!dodo_aligned16(K) || !dodo_aligned16(V) || !dodo_aligned16(cacheK) || !dodo_aligned16(cacheV))
            return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "K, V, cacheK and cacheV must be 16-byte aligned");
    }
    for (int b0 = 0; b0 < B; b0 += DODO_GROUP) {
        GatherGroup g;
        gather_group(g, b0, B, seq_off, nug_off, pos_base, cache_off, cache_len);
        ctx->cache_clean = false;   // the next attend must not read cache rows ahead of its dependency wait
        const int rc = dodo_launch_gather(ctx, K, V, row_bytes, idx, g, cacheK, cacheV, cache_pos, ctx->dev_status,
                                          static_cast<cudaStream_t>(stream));
        if (rc != DODO_OK) return rc;
    }
    for (int b = 0; b < B; ++b) cache_len[b] += nug_off[b + 1] - nug_off[b];
    return DODO_OK;
}

int dodo_compress(dodo_ctx* ctx, const void* X, int dtype, int d, const void* w, float bias, const void* K, const void* V,
                  int H, int dh, const int32_t* seq_off, const int32_t* nug_off, const int32_t* pos_base, int B,
                  uint32_t flags, float* scores, int32_t* idx, void* cacheK, void* cacheV, int32_t* cache_pos,
                  const int32_t* cache_off, int32_t* cache_len, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    int rc = check_score_args(ctx, X, dtype, d, w, seq_off, B, scores);
    if (rc != DODO_OK) return rc;
    rc = check_select_args(ctx, seq_off, nug_off, B, flags, idx);
    if (rc != DODO_OK) return rc;
    size_t row_bytes = 0;
    rc = gather_check(ctx, dtype, H, dh, seq_off, nug_off, pos_base, B, cache_off, cache_len, &row_bytes);
    if (rc != DODO_OK) return rc;
    if (nug_off[B] > 0) {
        if (K == nullptr || V == nullptr || cacheK == nullptr || cacheV == nullptr || cache_pos == nullptr)
            return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "K, V, cacheK, cacheV and cache_pos must not be NULL");
        if (!dodo_aligned16(K) || !dodo_aligned16(V) || !dodo_aligned16(cacheK) || !dodo_aligned16(cacheV))
            return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "K, V, cacheK and cacheV must be 16-byte aligned");
    }
    int max_n = 0;
    for (int b = 0; b < B; ++b) max_n = max_n > seq_off[b + 1] - seq_off[b] ? max_n : seq_off[b + 1] - seq_off[b];
    // While the selection rides on the score launch (no sequence longer than that allows) and one kernel argument
    // holds the batch, the gather follows each sequence's selection instead of the whole score launch.
    if (B <= DODO_GROUP && max_n <= dodo_select_fused_max_tokens() && nug_off[B] > 0) {
        ScoreSelectGroup sg;
        fill_score_group(sg, seq_off, nug_off, 0, B);
        GatherGroup gg;
        gather_group(gg, 0, B, seq_off, nug_off, pos_base, cache_off, cache_len);
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        rc = dodo_launch_score(ctx, X, dtype, d, w, bias, sg, 1, flags, scores, idx, ctx->tickets,
                               ctx->compress_state + DODO_FLAG_STRIDE, st);
        if (rc != DODO_OK) return rc;
        ctx->cache_clean = false;   // the next attend must not read cache rows ahead of its dependency wait
        rc = dodo_launch_gather_flagged(ctx, K, V, row_bytes, idx, gg, cacheK, cacheV, cache_pos, ctx->compress_state,
                                        ctx->dev_status, st);
        if (rc != DODO_OK) return rc;
        for (int b = 0; b < B; ++b) cache_len[b] += nug_off[b + 1] - nug_off[b];
        return DODO_OK;
    }
    rc = dodo_score_select(ctx, X, dtype, d, w, bias, seq_off, nug_off, B, flags, scores, idx, stream);
    if (rc != DODO_OK) return rc;
    return dodo_gather_kv(ctx, K, V, dtype, H, dh, seq_off, idx, nug_off, pos_base, B, cacheK, cacheV, cache_pos, cache_off,
                          cache_len, stream);
}

int dodo_gather_kv_layers(dodo_ctx* ctx, int L, const void* const* K, const void* const* V, int dtype, int H, int dh,
                          const int32_t* seq_off, const int32_t* idx, const int32_t* nug_off,
                          const int32_t* pos_base, int B, void* const* cacheK, void* const* cacheV,
                          int32_t* cache_pos, const int32_t* cache_off, int32_t* cache_len, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    if (L < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "L = %d is negative", L);
    size_t row_bytes = 0;
    const int rc0 = gather_check(ctx, dtype, H, dh, seq_off, nug_off, pos_base, B, cache_off, cache_len, &row_bytes);
    if (rc0 != DODO_OK) return rc0;
    if (L == 0) return DODO_OK;   // no layer: nothing is appended, cache_len stays
    if (nug_off[B] > 0) {
        if (K == nullptr || V == nullptr || cacheK == nullptr || cacheV == nullptr || idx == nullptr || cache_pos == nullptr)
            return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "K, V, cacheK, cacheV, idx and cache_pos must not be NULL");
        for (int l = 0; l < L; ++l) {
            if (K[l] == nullptr || V[l] == nullptr || cacheK[l] == nullptr || cacheV[l] == nullptr)
                return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "layer %d: K, V, cacheK and cacheV must not be NULL", l);
            if (!dodo_aligned16(K[l]) || !dodo_aligned16(V[l]) || !dodo_aligned16(cacheK[l]) || !dodo_aligned16(cacheV[l]))
                return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "layer %d: K, V, cacheK and cacheV must be 16-byte aligned", l);
        }
        for (int b0 = 0; b0 < B; b0 += DODO_GROUP) {
            GatherGroup g;
            gather_group(g, b0, B, seq_off, nug_off, pos_base, cache_off, cache_len);
            for (int l0 = 0; l0 < L; l0 += DODO_LAYER_GROUP) {
                GatherLayers lay;
                lay.n = L - l0 < DODO_LAYER_GROUP ? L - l0 : DODO_LAYER_GROUP;
                lay.first = l0 == 0;
                for (int i = 0; i < DODO_LAYER_GROUP; ++i) {
                    const bool live = i < lay.n;
                    lay.K[i] = live ? static_cast<const unsigned char*>(K[l0 + i]) : nullptr;
                    lay.V[i] = live ? static_cast<const unsigned char*>(V[l0 + i]) : nullptr;
                    lay.cacheK[i] = live ? static_cast<unsigned char*>(cacheK[l0 + i]) : nullptr;
                    lay.cacheV[i] = live ? static_cast<unsigned char*>(cacheV[l0 + i]) : nullptr;
                }
                ctx->cache_clean = false;
                const int rc = dodo_launch_gather_layers(ctx, lay, row_bytes, idx, g, cache_pos, ctx->dev_status,
                                                         static_cast<cudaStream_t>(stream));
                if (rc != DODO_OK) return rc;
            }
        }
    }
    for (int b = 0; b < B; ++b) cache_len[b] += nug_off[b + 1] - nug_off[b];
    return DODO_OK;
}

int dodo_pool_kv(dodo_ctx* ctx, const void* K, const void* V, int dtype, int H, int dh, const int32_t* seq_off, int r,
                 const int32_t* pos_base, int B, void* cacheK, void* cacheV, int32_t* cache_pos, const int32_t* cache_off,
                 int32_t* cache_len, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    if (B < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "B = %d is negative", B);
    if (r < 1) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "ratio %d must be at least 1", r);
    if (!valid_dtype(dtype)) return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "dtype %d", dtype);
    if (H <= 0 || dh <= 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "H = %d, dh = %d", H, dh);
    const size_t row_bytes = static_cast<size_t>(H) * static_cast<size_t>(dh) * dodo_elem_bytes(dtype);
    if (row_bytes % 16 != 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "a K/V row (%zu bytes) must be a multiple of 16 bytes", row_bytes);
    if (!valid_offsets(seq_off, B) || !valid_offsets(cache_off, B))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "seq_off and cache_off must start at 0 and be non-decreasing");
    if (pos_base == nullptr || cache_len == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "pos_base and cache_len must not be NULL");
    int total = 0;
    for (int b = 0; b < B; ++b) {
        const int k = dodo_num_nuggets(seq_off[b + 1] - seq_off[b], r), cap = cache_off[b + 1] - cache_off[b];
        if (cache_len[b] < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sequence %d: negative cache_len", b);
        if (cache_len[b] + k > cap)
            return dodo_fail(ctx, DODO_ERR_CAPACITY, "sequence %d: %d cached + %d pooled rows exceed its %d cache rows", b, cache_len[b], k, cap);
        total += k;
    }
    if (total > 0) {
        if (K == nullptr || V == nullptr || cacheK == nullptr || cacheV == nullptr || cache_pos == nullptr)
            return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "K, V, cacheK, cacheV and cache_pos must not be NULL");
        if (!dodo_aligned16(K) || !dodo_aligned16(V) || !dodo_aligned16(cacheK) || !dodo_aligned16(cacheV))
            return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "K, V, cacheK and cacheV must be 16-byte aligned");
    }
    for (int b0 = 0; b0 < B; b0 += DODO_GROUP) {
        PoolGroup g;
        g.nseq = B - b0 < DODO_GROUP ? B - b0 : DODO_GROUP;
        g.out0[0] = 0;
        for (int i = 0; i < DODO_GROUP; ++i) {
            const bool live = i < g.nseq;
            const int b = b0 + i;
            g.src_row0[i] = live ? seq_off[b] : 0;
            g.n[i] = live ? seq_off[b + 1] - seq_off[b] : 0;
            g.dst_row0[i] = live ? cache_off[b] + cache_len[b] : 0;
            g.pos_base[i] = live ? pos_base[b] : 0;
            g.out0[i + 1] = g.out0[i] + (live ? dodo_num_nuggets(g.n[i], r) : 0);
        }
        ctx->cache_clean = false;   // the next attend must not read cache rows ahead of its dependency wait
        const int rc = dodo_launch_pool(ctx, K, V, dtype, row_bytes, r, g, cacheK, cacheV, cache_pos, static_cast<cudaStream_t>(stream));
        if (rc != DODO_OK) return rc;
    }
    for (int b = 0; b < B; ++b) cache_len[b] += dodo_num_nuggets(seq_off[b + 1] - seq_off[b], r);
    return DODO_OK;
}

size_t dodo_attend_workspace_bytes(const dodo_ctx* ctx, int dh) {
    if (ctx == nullptr || dh <= 0) return 0;
    // split partial rows of the streaming kernel, or the cut units of the tensor-core kernel
    const size_t stream_bytes = attend_partial_rows_bound(ctx) * static_cast<size_t>(dh + 2) * sizeof(float);
    const size_t dense_bytes = dodo_dense_workspace_bytes(ctx->num_sms);
    return stream_bytes > dense_bytes ? stream_bytes : dense_bytes;
}

int dodo_attend(dodo_ctx* ctx, const void* Q, const int32_t* q_off, const int32_t* q_pos0,
                int dtype, int H, int dh, float sm_scale,
                const void* cacheK, const void* cacheV, const int32_t* cache_pos,
                const int32_t* cache_off, const int32_t* cache_len,
                const void* locK, const void* locV, const int32_t* loc_off,
                const int32_t* loc_len, const int32_t* loc_pos0, int loc_rows, int B,
                void* O, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    if (B < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "B = %d is negative", B);
    if (!valid_dtype(dtype)) return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "dtype %d", dtype);
    if (dh != 64 && dh != 128) return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "head size %d (supported: 64, 128)", dh);
    if (H <= 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "H = %d", H);
    if (!valid_offsets(q_off, B)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "q_off must start at 0 and be non-decreasing");
    if (B > 0 && q_pos0 == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "q_pos0 must not be NULL");
    if (q_off[B] == 0) return DODO_OK;
    if (Q == nullptr || O == nullptr || !dodo_aligned16(Q) || !dodo_aligned16(O))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "Q and O must be non-NULL and 16-byte aligned");

    // key segments
    bool any_cache = false, any_local = false;
    if (cache_len != nullptr) {
        if (!valid_offsets(cache_off, B)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "cache_off must start at 0 and be non-decreasing");
        for (int b = 0; b < B; ++b) {
            if (cache_len[b] < 0 || cache_len[b] > cache_off[b + 1] - cache_off[b])
                return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sequence %d: cache_len %d outside its region", b, cache_len[b]);
            any_cache = any_cache || cache_len[b] > 0;
        }
    }
    if (loc_len != nullptr) {
        for (int b = 0; b < B; ++b) {
            if (loc_len[b] < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sequence %d: negative loc_len", b);
            if (loc_len[b] > 0) {
                if (loc_off == nullptr || loc_pos0 == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "loc_off and loc_pos0 must not be NULL");
                if (loc_off[b] < 0 || static_cast<int64_t>(loc_off[b]) + loc_len[b] > loc_rows)
                    return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sequence %d: local rows [%d, %d) outside loc_rows = %d", b, loc_off[b], loc_off[b] + loc_len[b], loc_rows);
                any_local = true;
            }
        }
    }
    if (any_cache && (cacheK == nullptr || cacheV == nullptr || cache_pos == nullptr || !dodo_aligned16(cacheK) || !dodo_aligned16(cacheV)))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "cacheK, cacheV, cache_pos must be non-NULL, K/V 16-byte aligned");
    if (any_local && (locK == nullptr || locV == nullptr || !dodo_aligned16(locK) || !dodo_aligned16(locV)))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "locK and locV must be non-NULL and 16-byte aligned");

    // ---- plan (query tile, split-K chunks), descriptors, launches -----------------------------
    AttendShape shp = {q_off, q_pos0, cache_off, cache_len, loc_off, loc_len, loc_pos0, B, H, dh, dtype};
    AttendPlan plan;
    AttendTotals tot;
    dodo_attend_plan_begin(shp, ctx->attend_target_ctas, plan, tot);
    plan.cluster_cap = dodo_attend_cluster_cap(ctx, dtype, dh, plan.qt);
    // shape rule: blocks of many bf16 queries at head size 128 are a contraction -> tensor cores
    int max_tq = 0;
    for (int b = 0; b < B; ++b) max_tq = max_tq > q_off[b + 1] - q_off[b] ? max_tq : q_off[b + 1] - q_off[b];
    // (the tensor-core kernel takes row maxima before scaling, which needs a positive scale)
    const bool dense = dtype == DODO_BF16 && dh == 128 && max_tq >= ctx->dense_min_tq && sm_scale > 0.f;
    const AttendMaps maps = {any_cache ? cacheK : nullptr, any_cache ? cacheV : nullptr,
                             any_local ? locK : nullptr, any_local ? locV : nullptr};
    DenseMaps dmaps;
    int rc = DODO_OK;
    if (dense) {
        plan.qt = dodo_dense_tile_queries();
        tot.split = false;
        rc = dodo_dense_encode_maps(ctx, shp, Q, q_off[B], cacheK, cacheV, any_cache ? cache_off[B] : 0, dodo_dense_tile_keys(),
                                    locK, locV, any_local ? loc_rows : 0, dmaps);
    }
    if (rc != DODO_OK) return rc;

    // first pass over all launch groups: sizes, so that capacity errors come before any launch
    const int ngroups = (B + DODO_GROUP - 1) / DODO_GROUP;
    AttendGroup one;
    AttendGroup* groups = &one;
    if (ngroups > 1) {
        groups = static_cast<AttendGroup*>(malloc(sizeof(AttendGroup) * static_cast<size_t>(ngroups)));
        if (groups == nullptr) return dodo_fail(ctx, DODO_ERR_CUDA, "out of host memory");
    }
    for (int gi = 0; gi < ngroups; ++gi) {
        const int b0 = gi * DODO_GROUP;
        dodo_attend_plan_group(shp, plan, tot, b0, B - b0 < DODO_GROUP ? B - b0 : DODO_GROUP, groups[gi]);
    }
    rc = DODO_OK;
    const size_t part_rows_cap = workspace_bytes / (static_cast<size_t>(dh + 2) * sizeof(float));
    if (tot.part_rows > 0) {
        if (workspace == nullptr || !dodo_aligned16(workspace) || static_cast<size_t>(tot.part_rows) > part_rows_cap)
            rc = dodo_fail(ctx, DODO_ERR_CAPACITY, "workspace of %zu bytes is too small or misaligned (need %zu)", workspace_bytes,
                           static_cast<size_t>(tot.part_rows) * (dh + 2) * sizeof(float));
        else if (tot.tick_rows > DODO_NUM_TICKETS)
            rc = dodo_fail(ctx, DODO_ERR_CAPACITY, "too many split units (%lld)", static_cast<long long>(tot.tick_rows));
    }
    // A streaming launch may read cache rows ahead of its dependency wait only when nothing this context
    // launched since its last attend has written a cache -- and, under stream capture, only when that attend
    // belongs to the same capture: a graph must not bake in what happened to precede its recording.
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaStreamCaptureStatus cap_status = cudaStreamCaptureStatusNone;
    unsigned long long cap_id = 0;
    if (cudaStreamGetCaptureInfo(st, &cap_status, &cap_id) != cudaSuccess) {
        (void)cudaGetLastError();
        cap_status = cudaStreamCaptureStatusNone;
    }
    if (cap_status != cudaStreamCaptureStatusActive) cap_id = 0;
    for (int gi = 0; gi < ngroups && rc == DODO_OK; ++gi) {
        const bool early = ctx->cache_clean && ctx->clean_capture_id == cap_id;
        rc = dense ? dodo_launch_attend_dense(ctx, H, sm_scale, groups[gi], dmaps, cache_pos, O, lse, workspace, workspace_bytes,
                                              ctx->tickets, ctx->dev_status, nullptr, st)
                   : dodo_launch_attend(ctx, dtype, H, dh, sm_scale, plan, groups[gi], Q, maps, cache_pos, O, lse,
                                        static_cast<float*>(workspace), ctx->tickets, early, st);
        if (rc == DODO_OK) {   // an attend never writes a cache
            ctx->cache_clean = true;
            ctx->clean_capture_id = cap_id;
        }
    }
    if (groups != &one) free(groups);
    return rc;
}

int dodo_attend_indexed(dodo_ctx* ctx, const void* Q, const int32_t* q_off, const int32_t* q_pos0, int dtype, int H, int dh,
                        float sm_scale, const void* K, const void* V, const int32_t* seq_off, const int32_t* idx,
                        const int32_t* nug_off, const int32_t* pos_base, const void* locK, const void* locV,
                        const int32_t* loc_off, const int32_t* loc_len, const int32_t* loc_pos0, int loc_rows, int B,
                        void* O, float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    if (B < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "B = %d is negative", B);
    if (!valid_dtype(dtype)) return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "dtype %d", dtype);
    if (dtype != DODO_BF16 || dh != 128 || !(sm_scale > 0.f))
        return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "indexed attention runs on the tensor-core kernel only: bf16, head size 128, positive scale "
                         "(got dtype %d, head size %d, scale %g); gather into a cache and use dodo_attend otherwise", dtype, dh, sm_scale);
    if (H <= 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "H = %d", H);
    if (!valid_offsets(q_off, B)) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "q_off must start at 0 and be non-decreasing");
    if (B > 0 && q_pos0 == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "q_pos0 must not be NULL");
    if (q_off[B] == 0) return DODO_OK;
    if (Q == nullptr || O == nullptr || !dodo_aligned16(Q) || !dodo_aligned16(O))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "Q and O must be non-NULL and 16-byte aligned");
    if (!valid_offsets(seq_off, B) || !valid_offsets(nug_off, B))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "seq_off and nug_off must start at 0 and be non-decreasing");
    if (pos_base == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "pos_base must not be NULL");
    bool any_sel = false, any_local = false;
    for (int b = 0; b < B; ++b) {
        const int n = seq_off[b + 1] - seq_off[b], k = nug_off[b + 1] - nug_off[b];
        if (k > n) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sequence %d: k = %d exceeds n = %d", b, k, n);
        any_sel = any_sel || k > 0;
    }
    if (loc_len != nullptr) {
        for (int b = 0; b < B; ++b) {
            if (loc_len[b] < 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sequence %d: negative loc_len", b);
            if (loc_len[b] > 0) {
                if (loc_off == nullptr || loc_pos0 == nullptr) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "loc_off and loc_pos0 must not be NULL");
                if (loc_off[b] < 0 || static_cast<int64_t>(loc_off[b]) + loc_len[b] > loc_rows)
                    return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "sequence %d: local rows [%d, %d) outside loc_rows = %d", b, loc_off[b], loc_off[b] + loc_len[b], loc_rows);
                any_local = true;
            }
        }
    }
    if (any_sel && (K == nullptr || V == nullptr || idx == nullptr || !dodo_aligned16(K) || !dodo_aligned16(V)))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "K, V and idx must be non-NULL, K and V 16-byte aligned");
    if (any_local && (locK == nullptr || locV == nullptr || !dodo_aligned16(locK) || !dodo_aligned16(locV)))
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "locK and locV must be non-NULL and 16-byte aligned");

    // the selection plays the cache's part: sequence b's "cache rows" are its slots [nug_off[b], nug_off[b+1]) of idx
    int32_t* k_len = static_cast<int32_t*>(malloc(sizeof(int32_t) * static_cast<size_t>(B > 0 ? B : 1)));
    if (k_len == nullptr) return dodo_fail(ctx, DODO_ERR_CUDA, "out of host memory");
    for (int b = 0; b < B; ++b) k_len[b] = nug_off[b + 1] - nug_off[b];
    AttendShape shp = {q_off, q_pos0, nug_off, k_len, loc_off, loc_len, loc_pos0, B, H, dh, dtype};
    AttendPlan plan;
    AttendTotals tot;
    dodo_attend_plan_begin(shp, ctx->attend_target_ctas, plan, tot);
    plan.qt = dodo_dense_tile_queries();
    tot.split = false;
    DenseMaps dmaps;
    int rc = dodo_dense_encode_maps(ctx, shp, Q, q_off[B], K, V, any_sel ? seq_off[B] : 0, 1, locK, locV,
                                    any_local ? loc_rows : 0, dmaps);
    for (int b0 = 0; b0 < B && rc == DODO_OK; b0 += DODO_GROUP) {
        const int nb = B - b0 < DODO_GROUP ? B - b0 : DODO_GROUP;
        AttendGroup grp;
        dodo_attend_plan_group(shp, plan, tot, b0, nb, grp);
        DenseGather gat;
        memset(&gat, 0, sizeof gat);
        for (int i = 0; i < nb; ++i) {
            gat.row0[i] = seq_off[b0 + i];
            gat.n[i] = seq_off[b0 + i + 1] - seq_off[b0 + i];
            gat.pos_base[i] = pos_base[b0 + i];
        }
        rc = dodo_launch_attend_dense(ctx, H, sm_scale, grp, dmaps, idx, O, lse, workspace, workspace_bytes, ctx->tickets,
                                      ctx->dev_status, &gat, static_cast<cudaStream_t>(stream));
    }
    free(k_len);
    return rc;
}

}  // extern "C"
