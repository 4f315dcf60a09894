// Threshold selection (Eq. 8): token i becomes a nugget iff its score is strictly above Lambda.  The
// number of nuggets is data-dependent, so the work comes in two launches with the caller's read of
// the counts between them: count per sequence, then an ordered compaction into the slots the
// caller laid out from the counts.  One thread block per sequence; scores are 4 bytes per token, so
// both launches are latency-bound and cheap beside the scoring pass that produced them.
#include "dodo_internal.cuh"

namespace {

constexpr int kThreads = 1024;

__global__ void __launch_bounds__(kThreads, 1)
threshold_count_kernel(const float* __restrict__ scores, const __grid_constant__ ThresholdGroup g, float lambda,
                       int32_t* __restrict__ counts) {
    __shared__ int warp_sum[kThreads / 32];
    const int b = blockIdx.x, tid = threadIdx.x;
    const float* s = scores + g.row0[b];
    const int n = g.n[b];
    int c = 0;
    for (int i = tid; i < n; i += kThreads) c += __ldcg(s + i) > lambda ? 1 : 0;   // IEEE: NaN is never above
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if ((tid & 31) == 0) warp_sum[tid >> 5] = c;
    __syncthreads();
    if (tid < 32) {
        int t = warp_sum[tid];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (tid == 0) counts[g.out0[b]] = t;
    }
}

// Positions above Lambda, ascending, into idx[idx0 .. idx0 + cap); anything beyond cap is dropped.
__global__ void __launch_bounds__(kThreads, 1)
threshold_select_kernel(const float* __restrict__ scores, const __grid_constant__ ThresholdGroup g, float lambda,
                        int32_t* __restrict__ idx) {
    __shared__ int warp_cnt[2][kThreads / 32];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* s = scores + g.row0[b];
    const int n = g.n[b], cap = g.cap[b];
    int32_t* out = idx + g.out0[b];
    int run = 0, buf = 0;
    for (int base = 0; base < n; base += kThreads, buf ^= 1) {
        const int i = base + tid;
        const bool keep = i < n && __ldcg(s + i) > lambda;
        const uint32_t m = __ballot_sync(0xffffffffu, keep);
        if (lane == 0) warp_cnt[buf][warp] = __popc(m);
        __syncthreads();
        // every warp scans the 32 warp counts itself: lane L holds warp L's count
        const int mine = warp_cnt[buf][lane];
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const int before = __shfl_sync(0xffffffffu, incl - mine, warp);
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        const int slot = run + before + __popc(m & ((1u << lane) - 1u));
        if (keep && slot < cap) out[slot] = i;
        run += total;
    }
}

}  // namespace

int dodo_launch_threshold(dodo_ctx* ctx, const float* scores, const ThresholdGroup& g, float lambda, bool select,
                          int32_t* out, cudaStream_t st) {
    if (g.nseq == 0) return DODO_OK;
    if (select) threshold_select_kernel<<<g.nseq, kThreads, 0, st>>>(scores, g, lambda, out);
    else threshold_count_kernel<<<g.nseq, kThreads, 0, st>>>(scores, g, lambda, out);
    return dodo_check_cuda(ctx, cudaGetLastError(), select ? "threshold select launch" : "threshold count launch");
}
