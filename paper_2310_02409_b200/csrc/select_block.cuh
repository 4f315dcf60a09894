// TopK selection by a team of warps of one thread block (Eq. 14): order-preserving keys, radix select of the k-th
// largest, position-ordered compaction.  Shared by the kernels that end in a selection: the fused linear Scorer, the
// select launches and the two-layer Scorer's reduction.
#pragma once

#include "dodo_internal.cuh"

namespace dodo_sel {

// Monotone map float -> uint32: larger score <=> larger key.  -0 maps with +0; every NaN maps to 0,
// below -inf.
__device__ __forceinline__ uint32_t score_key(float f) {
    uint32_t u = __float_as_uint(f);
    if ((u & 0x7fffffffu) > 0x7f800000u) return 0u;
    if (u == 0x80000000u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kHistCopies = 8;    // private histograms: warp w counts into copy w % kHistCopies

struct __align__(16) SelectSmem {
    int hist[kHistCopies][256];
    int tot[256];
    int warp_gt[32];
    int warp_eq[32];
};

// A selection is run by a *team*: the first nt threads of the block (a multiple of 32, at least 256), which meet
// at named barrier 1; the other threads of the block have left.  Every instruction of a phase costs one issue
// slot per warp, so a short sequence is selected faster by few warps: about eight keys per thread.
__device__ __forceinline__ void team_sync(int nt) { asm volatile("bar.sync 1, %0;" ::"r"(nt) : "memory"); }
__host__ __device__ inline int select_team_threads(int n, int block_threads) {
    const int want = n <= 1024 ? 256 : n <= 4096 ? 512 : 1024;
    return want < block_threads ? want : block_threads;
}

// The k-th largest key among key_at(0..n) (1 <= k <= n) by a team: four 8-bit radix passes.  *need_eq = how
// many keys equal to it belong to the k largest.  Scores cluster in a few exponent bins, so one histogram per
// block would serialise its atomics on a handful of words: warps count into private copies, 256 threads add
// the copies up (and clear them for the next pass), then every warp finds the digit by itself from the totals
// (a scan over its lanes), so nothing has to be published: two team barriers per pass.  Called by all threads
// of the team, which have passed a team barrier since the keys were put in place.
template <typename KeyAt>
__device__ uint32_t block_kth_key(KeyAt key_at, int n, int k, SelectSmem& sm, int* need_eq, int nt) {
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5;
    for (int b = tid; b < kHistCopies * 256; b += nt) (&sm.hist[0][0])[b] = 0;
    team_sync(nt);
    int* hist = sm.hist[warp % kHistCopies];
    uint32_t prefix = 0, mask = 0;
    int remaining = k;
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
        // four keys per thread and step, all four loads before the first atomic (keys that are not cached in
        // shared memory come from L2)
        for (int base = 0; base < n; base += 4 * nt) {
            uint32_t key[4];
            bool in[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = base + u * nt + tid;
                in[u] = i < n;
                key[u] = in[u] ? key_at(i) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (in[u] && (key[u] & mask) == prefix) atomicAdd(&hist[(key[u] >> shift) & 255u], 1);
        }
        team_sync(nt);
        if (tid < 256) {
            int sum = 0;
#pragma unroll
            for (int c = 0; c < kHistCopies; ++c) { sum += sm.hist[c][tid]; sm.hist[c][tid] = 0; }
            sm.tot[tid] = sum;
        }
        team_sync(nt);
        // lane L owns bins 255-8L .. 248-8L (descending): where does the running count reach `remaining`?
        int local[8], sum = 0;
        {
            const int4 lo = *reinterpret_cast<const int4*>(sm.tot + 248 - 8 * lane);       // bins 248-8L .. 251-8L
            const int4 hi = *reinterpret_cast<const int4*>(sm.tot + 252 - 8 * lane);       // bins 252-8L .. 255-8L
            local[0] = hi.w; local[1] = hi.z; local[2] = hi.y; local[3] = hi.x;
            local[4] = lo.w; local[5] = lo.z; local[6] = lo.y; local[7] = lo.x;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) sum += local[j];
        int incl = sum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        const int excl = incl - sum;
        const bool mine = excl < remaining && remaining <= incl;     // exactly one lane (1 <= remaining <= total)
        int bin = 0, rem = 0;
        if (mine) {
            int run = excl;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (run < remaining && remaining <= run + local[j]) { bin = 255 - 8 * lane - j; rem = remaining - run; }
                run += local[j];
            }
        }
        const int src = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
        bin = __shfl_sync(0xffffffffu, bin, src);
        remaining = __shfl_sync(0xffffffffu, rem, src);
        prefix |= static_cast<uint32_t>(bin) << shift;
        mask |= 255u << shift;
        // (the totals are next written after the next pass's first barrier, which every warp reaches after this scan)
    }
    *need_eq = remaining;
    return prefix;
}

// TopK of one sequence by a team of nt threads (see team_sync).  `s` are n scores in global memory, visible to
// this block; `keys` is shared memory for key_cap keys (longer sequences re-read their scores from L2 in every
// pass).  Writes k ascending positions to `out`.
static __device__ void block_select(const float* __restrict__ s, int n, int k, uint32_t flags,
                             int32_t* __restrict__ out, SelectSmem& sm, uint32_t* keys, int key_cap, int nt) {
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, nwarp = nt >> 5;
    if (k <= 0) return;
    if (flags & DODO_FORCE_LAST) {
        if (tid == 0) out[k - 1] = n - 1;
        n -= 1;
        k -= 1;
        if (k <= 0) return;
    }
    const bool cached = n <= key_cap;
    if (cached) {
        for (int i = tid; i < n; i += nt) keys[i] = score_key(__ldcg(s + i));
    }
    team_sync(nt);
    auto key_at = [&](int i) -> uint32_t { return cached ? keys[i] : score_key(__ldcg(s + i)); };

    int need_eq;   // how many keys equal to T are kept (the lowest positions)
    const uint32_t T = block_kth_key(key_at, n, k, sm, &need_eq, nt);

    // ---- position-ordered compaction -------------------------------------------------------
    // Warp w owns the contiguous positions [w*seg, (w+1)*seg): it counts its keys above and equal to T, the
    // warp counts are scanned once, and a second walk over the same positions writes the kept ones.  One
    // team barrier in all.
    const int seg = (((n + nwarp - 1) / nwarp) + 31) & ~31;
    const int p0 = min(n, warp * seg), p1 = min(n, p0 + seg);
    int n_gt = 0, n_eq = 0;
    for (int base = p0; base < p1; base += 32) {
        const int i = base + lane;
        const uint32_t key = i < p1 ? key_at(i) : 0u;
        n_gt += __popc(__ballot_sync(0xffffffffu, i < p1 && key > T));
        n_eq += __popc(__ballot_sync(0xffffffffu, i < p1 && key == T));
    }
    if (lane == 0) { sm.warp_gt[warp] = n_gt; sm.warp_eq[warp] = n_eq; }
    team_sync(nt);
    // every warp scans the warp counts itself: lane L holds warp L's counts
    const int g_mine = lane < nwarp ? sm.warp_gt[lane] : 0, e_mine = lane < nwarp ? sm.warp_eq[lane] : 0;
    int g_incl = g_mine, e_incl = e_mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int gv = __shfl_up_sync(0xffffffffu, g_incl, o), ev = __shfl_up_sync(0xffffffffu, e_incl, o);
        if (lane >= o) { g_incl += gv; e_incl += ev; }
    }
    int gt_run = __shfl_sync(0xffffffffu, g_incl - g_mine, warp);   // keys above / equal to T before this warp's positions
    int eq_run = __shfl_sync(0xffffffffu, e_incl - e_mine, warp);
    const uint32_t lt = (1u << lane) - 1u;
    for (int base = p0; base < p1; base += 32) {
        const int i = base + lane;
        const uint32_t key = i < p1 ? key_at(i) : 0u;
        const bool gt = i < p1 && key > T;
        const bool eq = i < p1 && key == T;
        const uint32_t gt_m = __ballot_sync(0xffffffffu, gt);
        const uint32_t eq_m = __ballot_sync(0xffffffffu, eq);
        const int gt_before = gt_run + __popc(gt_m & lt);
        const int eq_before = eq_run + __popc(eq_m & lt);
        if (gt || (eq && eq_before < need_eq)) out[gt_before + min(eq_before, need_eq)] = i;
        gt_run += __popc(gt_m);
        eq_run += __popc(eq_m);
    }
}

}  // namespace dodo_sel
