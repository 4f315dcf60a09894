// Host-buffer form of the path for one layer: upload a batch's context (X, w), the local /
// decoded K/V rows and the decode queries from host memory, compress (fused score + TopK, gather),
// run every decode step's attention with a sliding local window, and download the outputs.  All
// copies and launches are asynchronous on the caller's stream; device memory comes from an arena
// the caller provides (size from dodo_host_arena_bytes).  This is what an application that keeps its
// tensors on the host calls; it adds nothing to the arithmetic of the device-pointer entry points.
// The context's K/V rows are only ever needed where a nugget was selected (Eq. 5), so when the
// host K and V are pinned and visible to the device the gather kernel reads just those rows
// straight out of host memory, a fraction 1/r of the bytes; pageable K/V are uploaded whole first.
#include <stdlib.h>

#include "dodo_internal.cuh"

namespace {

struct Arena {
    unsigned char* base;
    size_t used, cap;
    void* take(size_t bytes) {
        const size_t at = (used + 255) & ~static_cast<size_t>(255);
        used = at + bytes;
        return used <= cap ? base + at : nullptr;
    }
};

struct Sizes {
    size_t X, w, KV, loc, Q, scores, idx, cache, cpos, ws;
};

Sizes sizes_of(const dodo_ctx* ctx, int dtype, int d, int H, int dh, int N, int Kt, int B, int loc_cap, int steps) {
    const size_t e = dodo_elem_bytes(dtype), row = static_cast<size_t>(H) * dh * e;
    Sizes s;
    s.X = static_cast<size_t>(N) * d * e;
    s.w = static_cast<size_t>(d) * e;
    s.KV = static_cast<size_t>(N) * row;
    s.loc = static_cast<size_t>(B) * loc_cap * row;
    s.Q = static_cast<size_t>(steps) * B * row;
    s.scores = static_cast<size_t>(N) * sizeof(float);
    s.idx = static_cast<size_t>(Kt > 0 ? Kt : 1) * sizeof(int32_t);
    s.cache = static_cast<size_t>(Kt > 0 ? Kt : 1) * row;
    s.cpos = static_cast<size_t>(Kt > 0 ? Kt : 1) * sizeof(int32_t);
    s.ws = dodo_attend_workspace_bytes(ctx, dh);
    return s;
}

// The address at which the device sees a pinned, mapped host buffer; NULL for pageable memory.
const void* device_alias(const void* host) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, host) != cudaSuccess) {
        (void)cudaGetLastError();   // an unknown pointer is not an error here: it is simply copied
        return nullptr;
    }
    if (at.type != cudaMemoryTypeHost || at.devicePointer == nullptr) return nullptr;
    return (reinterpret_cast<uintptr_t>(at.devicePointer) & 15u) == 0 ? at.devicePointer : nullptr;
}

}  // namespace

extern "C" {

size_t dodo_host_arena_bytes(const dodo_ctx* ctx, int dtype, int d, int H, int dh, int total_tokens, int total_nuggets,
                             int B, int local, int steps) {
    if (ctx == nullptr || d <= 0 || H <= 0 || dh <= 0 || total_tokens < 0 || total_nuggets < 0 || B < 0 || local < 0 ||
        steps < 0)
        return 0;
    const Sizes s = sizes_of(ctx, dtype, d, H, dh, total_tokens, total_nuggets, B, local + steps, steps);
    // X w K V locK locV Q O scores idx cacheK cacheV cache_pos workspace, each rounded up to 256 bytes
    const size_t parts[] = {s.X, s.w, s.KV, s.KV, s.loc, s.loc, s.Q, s.Q, s.scores, s.idx, s.cache, s.cache, s.cpos, s.ws};
    size_t total = 0;
    for (size_t p : parts) total += (p + 255) & ~static_cast<size_t>(255);
    return total + 256;
}

int dodo_compress_decode_host(dodo_ctx* ctx, const void* hX, const void* hw, const void* hK, const void* hV, int dtype,
                              int d, int H, int dh, const int32_t* seq_off, const int32_t* nug_off, int B,
                              const void* hLocK, const void* hLocV, int local, const void* hQ, int steps,
                              float sm_scale, void* hO, void* arena, size_t arena_bytes, void* stream) {
    if (ctx == nullptr) return DODO_ERR_INVALID_ARG;
    if (B <= 0 || B > DODO_GROUP) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "B = %d: 1..%d sequences per call", B, DODO_GROUP);
    if (seq_off == nullptr || nug_off == nullptr || seq_off[0] != 0 || nug_off[0] != 0)
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "seq_off and nug_off must start at 0");
    if (local < 1 || steps < 1) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "local = %d and steps = %d must be positive", local, steps);
    if (hX == nullptr || hw == nullptr || hK == nullptr || hV == nullptr || hLocK == nullptr || hLocV == nullptr ||
        hQ == nullptr || hO == nullptr || arena == nullptr)
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "host buffers and the arena must not be NULL");
    if (dtype != DODO_F32 && dtype != DODO_BF16) return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "dtype %d", dtype);
    const int N = seq_off[B], Kt = nug_off[B], loc_cap = local + steps;
    const Sizes s = sizes_of(ctx, dtype, d, H, dh, N, Kt, B, loc_cap, steps);
    Arena a = {static_cast<unsigned char*>(arena), 0, arena_bytes};
    if ((reinterpret_cast<uintptr_t>(arena) & 255u) != 0) return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "the arena must be 256-byte aligned");
    void* dX = a.take(s.X); void* dw = a.take(s.w); void* dK = a.take(s.KV); void* dV = a.take(s.KV);
    void* dLK = a.take(s.loc); void* dLV = a.take(s.loc); void* dQ = a.take(s.Q); void* dO = a.take(s.Q);
    float* dS = static_cast<float*>(a.take(s.scores));
    int32_t* dIdx = static_cast<int32_t*>(a.take(s.idx));
    void* dCK = a.take(s.cache); void* dCV = a.take(s.cache);
    int32_t* dCP = static_cast<int32_t*>(a.take(s.cpos));
    void* dWs = a.take(s.ws);
    if (dWs == nullptr)
        return dodo_fail(ctx, DODO_ERR_CAPACITY, "arena of %zu bytes is too small (need %zu)", arena_bytes,
                         dodo_host_arena_bytes(ctx, dtype, d, H, dh, N, Kt, B, local, steps));

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // K and V of the context: read in place by the gather when the device can see them, else uploaded
    const void* zK = device_alias(hK);
    const void* zV = device_alias(hV);
    const bool in_place = zK != nullptr && zV != nullptr;
    const void* srcK = in_place ? zK : dK;
    const void* srcV = in_place ? zV : dV;
    const struct { void* dst; const void* src; size_t n; } up[] = {
        {dX, hX, s.X}, {dw, hw, s.w}, {dK, hK, in_place ? 0 : s.KV}, {dV, hV, in_place ? 0 : s.KV},
        {dLK, hLocK, s.loc}, {dLV, hLocV, s.loc}, {dQ, hQ, s.Q}};
    for (const auto& c : up) {
        if (c.n == 0) continue;
        const cudaError_t e = cudaMemcpyAsync(c.dst, c.src, c.n, cudaMemcpyHostToDevice, st);
        if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "host-to-device copy");
    }
    int rc = dodo_score_select(ctx, dX, dtype, d, dw, 0.f, seq_off, nug_off, B, 0, dS, dIdx, stream);
    if (rc != DODO_OK) return rc;
    int32_t cache_len[DODO_GROUP], pos_base[DODO_GROUP], q_off[DODO_GROUP + 1], q_pos0[DODO_GROUP], loc_off[DODO_GROUP],
        loc_len[DODO_GROUP], loc_pos0[DODO_GROUP];
    for (int b = 0; b < B; ++b) { cache_len[b] = 0; pos_base[b] = 0; }
    rc = dodo_gather_kv(ctx, srcK, srcV, dtype, H, dh, seq_off, dIdx, nug_off, pos_base, B, dCK, dCV, dCP, nug_off, cache_len, stream);
    if (rc != DODO_OK) return rc;
    const size_t step_bytes = static_cast<size_t>(B) * H * dh * dodo_elem_bytes(dtype);
    for (int b = 0; b <= B; ++b) q_off[b] = b;
    for (int t = 0; t < steps; ++t) {
        // the `local` most recent positions, the decoded token itself last
        for (int b = 0; b < B; ++b) {
            const int n = seq_off[b + 1] - seq_off[b];
            loc_off[b] = b * loc_cap + t + 1;
            loc_len[b] = local;
            loc_pos0[b] = n + t + 1;
            q_pos0[b] = n + local + t;
        }
        rc = dodo_attend(ctx, static_cast<unsigned char*>(dQ) + t * step_bytes, q_off, q_pos0, dtype, H, dh, sm_scale, dCK,
                         dCV, dCP, nug_off, cache_len, dLK, dLV, loc_off, loc_len, loc_pos0, B * loc_cap, B,
                         static_cast<unsigned char*>(dO) + t * step_bytes, nullptr, dWs, s.ws, stream);
        if (rc != DODO_OK) return rc;
    }
    return dodo_check_cuda(ctx, cudaMemcpyAsync(hO, dO, s.Q, cudaMemcpyDeviceToHost, st), "device-to-host copy");
}

}  // extern "C"
