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

constexpr int kRegKeys = 8;       // keys per thread: of the register form, and per tile of the streaming form
constexpr int kRankMax = 512;     // at most this many candidates are ranked against each other directly

struct __align__(16) SelectSmem {
    int hist[kHistCopies][256];
    int tot[256];
    int warp_gt[32];
    int warp_eq[32];
    uint32_t cand[kRankMax];      // short sequences: the keys still in the race
    int ncand;
    uint32_t kth;                 // ... and what ranking them found
    int need_eq;
};

// A selection is run by a *team*: the first nt threads of the block (a multiple of 32, at least 256), which meet
// at named barrier 1; the other threads of the block have left.  Every instruction of a phase costs one issue
// slot per warp, so a short sequence is selected faster by few warps: about eight keys per thread.
__device__ __forceinline__ void team_sync(int nt) { asm volatile("bar.sync 1, %0;" ::"r"(nt) : "memory"); }
__host__ __device__ inline int select_team_threads(int n, int block_threads) {
    const int want = n <= 1024 ? 256 : n <= 4096 ? 512 : 1024;
    return want < block_threads ? want : block_threads;
}

// Every lane of a warp, from the 256 bin totals in shared memory: the bin (digit) in which the running count, taken
// from the highest bin down, reaches `remaining` (1 <= remaining <= sum of the totals), how many of that bin's keys
// are still wanted, and how many keys the bin holds.  Lane L owns bins 255-8L .. 248-8L.
__device__ __forceinline__ void find_bin(const int* tot, int lane, int remaining, int* bin_out, int* rem_out, int* cnt_out) {
    int local[8], sum = 0;
    {
        const int4 lo = *reinterpret_cast<const int4*>(tot + 248 - 8 * lane);       // bins 248-8L .. 251-8L
        const int4 hi = *reinterpret_cast<const int4*>(tot + 252 - 8 * lane);       // bins 252-8L .. 255-8L
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
    const bool mine = excl < remaining && remaining <= incl;     // exactly one lane
    int bin = 0, rem = 0, cnt = 0;
    if (mine) {
        int run = excl;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (run < remaining && remaining <= run + local[j]) { bin = 255 - 8 * lane - j; rem = remaining - run; cnt = local[j]; }
            run += local[j];
        }
    }
    const int src = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
    *bin_out = __shfl_sync(0xffffffffu, bin, src);
    *rem_out = __shfl_sync(0xffffffffu, rem, src);
    *cnt_out = __shfl_sync(0xffffffffu, cnt, src);
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
        int bin, cnt;
        find_bin(sm.tot, lane, remaining, &bin, &remaining, &cnt);
        prefix |= static_cast<uint32_t>(bin) << shift;
        mask |= 255u << shift;
        // (the totals are next written after the next pass's first barrier, which every warp reaches after this scan)
    }
    *need_eq = remaining;
    return prefix;
}

// TopK of a sequence whose keys fit the team's registers (n + 3 <= KPT * nt at most, KPT keys per thread, a
// multiple of 4): thread t holds the keys of KPT consecutive positions.  Radix passes as in block_kth_key narrow the race down, but only until at most
// kRankMax keys are left in it: those are gathered in shared memory and each is ranked against all the others
// (one thread per candidate, broadcast reads), which yields the k-th largest key and the number of its equals to
// keep at once -- with scores of a few thousand tokens that is after one or two passes instead of four.  The first
// pass can come for nothing: `top_hist`, when given, holds the counts of the keys' top digits (256 ints in global
// memory, every score of the sequence counted once; kernels that produce the scores count them on the way).
// Compaction is positional by construction: counts of kept keys are scanned over threads in position order.
template <int KPT>
static __device__ void block_select_small(const float* __restrict__ s, int n, int k, uint32_t flags,
                                          int32_t* __restrict__ out, SelectSmem& sm, int nt, const int* top_hist) {
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, nwarp = nt >> 5;
    if (k <= 0) return;
    const int n_all = n;
    if (flags & DODO_FORCE_LAST) {
        if (tid == 0) out[k - 1] = n - 1;
        n -= 1;
        k -= 1;
        if (k <= 0) return;
    }
    // Thread t holds positions [KPT t - a, KPT t - a + KPT), a = elements by which `s` lies behind a 16-byte boundary, so that
    // a thread's keys are two aligned 16-byte loads (the threads at the sequence's two ends load element by element).
    const int a = static_cast<int>((reinterpret_cast<uintptr_t>(s) >> 2) & 3u);
    const int p0 = tid * KPT - a;
    const int e_lo = max(0, -p0), e_hi = min(KPT, n - p0);   // this thread's valid slots: [e_lo, e_hi)
    uint32_t key[KPT];
    if (e_lo == 0 && e_hi == KPT) {
#pragma unroll
        for (int q = 0; q < KPT / 4; ++q) {
            const float4 f = __ldcg(reinterpret_cast<const float4*>(s + p0 + 4 * q));
            key[4 * q] = score_key(f.x); key[4 * q + 1] = score_key(f.y); key[4 * q + 2] = score_key(f.z); key[4 * q + 3] = score_key(f.w);
        }
    } else {
#pragma unroll
        for (int e = 0; e < KPT; ++e) key[e] = (e >= e_lo && e < e_hi) ? score_key(__ldcg(s + p0 + e)) : 0u;
    }
    for (int b = tid; b < kHistCopies * 256; b += nt) (&sm.hist[0][0])[b] = 0;
    if (tid == 0) sm.ncand = 0;
    bool have_top = top_hist != nullptr;
    if (have_top && tid < 256) {
        int c = __ldcg(top_hist + tid);
        // the forced last token is not in the race
        if ((flags & DODO_FORCE_LAST) && static_cast<int>(score_key(__ldcg(s + n_all - 1)) >> 24) == tid) c -= 1;
        sm.tot[tid] = c;
    }
    team_sync(nt);

    int* hist = sm.hist[warp % kHistCopies];
    uint32_t prefix = 0, mask = 0;
    int remaining = k, m = n;   // m keys match the prefix; the `remaining`-th largest of them is wanted
    int shift = 24;
    while (m > kRankMax && shift >= 0) {
        if (!have_top) {
#pragma unroll
            for (int e = 0; e < KPT; ++e)
                if (e >= e_lo && e < e_hi && (key[e] & mask) == prefix) atomicAdd(&hist[(key[e] >> shift) & 255u], 1);
            team_sync(nt);
            if (tid < 256) {
                int sum = 0;
#pragma unroll
                for (int c = 0; c < kHistCopies; ++c) { sum += sm.hist[c][tid]; sm.hist[c][tid] = 0; }
                sm.tot[tid] = sum;
            }
            team_sync(nt);
        }
        have_top = false;
        int bin;
        find_bin(sm.tot, lane, remaining, &bin, &remaining, &m);
        prefix |= static_cast<uint32_t>(bin) << shift;
        mask |= 255u << shift;
        shift -= 8;
    }

    uint32_t T = prefix;
    int need_eq = remaining;   // (all 32 bits fixed: the keys left are all equal)
    if (m <= kRankMax) {
#pragma unroll
        for (int e = 0; e < KPT; ++e)
            if (e >= e_lo && e < e_hi && (key[e] & mask) == prefix) sm.cand[atomicAdd(&sm.ncand, 1)] = key[e];
        team_sync(nt);
        for (int c = tid; c < m; c += nt) {
            const uint32_t mine = sm.cand[c];
            int gt = 0, eq = 0;
            for (int j = 0; j < m; ++j) {
                const uint32_t other = sm.cand[j];
                gt += other > mine ? 1 : 0;
                eq += other == mine ? 1 : 0;
            }
            if (gt < remaining && remaining <= gt + eq) { sm.kth = mine; sm.need_eq = remaining - gt; }   // equal keys write the same
        }
        team_sync(nt);
        T = sm.kth;
        need_eq = sm.need_eq;
    }

    // ---- compaction in position order: counts above / equal to T, packed as (equal << 16 | above) -------------------
    int mine = 0;
#pragma unroll
    for (int e = 0; e < KPT; ++e)
        if (e >= e_lo && e < e_hi) mine += key[e] > T ? 1 : key[e] == T ? 0x10000 : 0;
    int incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) sm.warp_gt[warp] = incl;
    team_sync(nt);
    const int w_mine = lane < nwarp ? sm.warp_gt[lane] : 0;
    int w_incl = w_mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, w_incl, o);
        if (lane >= o) w_incl += v;
    }
    const int before = __shfl_sync(0xffffffffu, w_incl - w_mine, warp) + incl - mine;
    int gt_b = before & 0xffff, eq_b = before >> 16;
#pragma unroll
    for (int e = 0; e < KPT; ++e) {
        if (e >= e_lo && e < e_hi) {
            if (key[e] > T) {
                out[gt_b + min(eq_b, need_eq)] = p0 + e;
                ++gt_b;
            } else if (key[e] == T) {
                if (eq_b < need_eq) out[gt_b + eq_b] = p0 + e;
                ++eq_b;
            }
        }
    }
}

// TopK of a longer sequence by a team of nt threads, without room for its keys: the same steps as
// block_select_small, but every step streams the scores again from global memory (L2) in tiles of kRegKeys * nt
// consecutive positions, the next tile's loads in flight while this one is worked on.  A step over a tile is what
// block_select_small does with its registers; the compaction carries the counts of kept keys from tile to tile.
// Cost: one pass over the scores per radix pass that is still needed (usually one, the first being pre-counted),
// one to collect the candidates, one to write the result.
struct KeyTile {
    uint32_t key[kRegKeys];
    int p0, e_lo, e_hi;   // first position, valid slots [e_lo, e_hi)
};
__device__ __forceinline__ void load_key_tile(KeyTile& kt, const float* __restrict__ s, int n, int a, int tile, int nt) {
    kt.p0 = (tile * nt + static_cast<int>(threadIdx.x)) * kRegKeys - a;
    kt.e_lo = max(0, -kt.p0);
    kt.e_hi = min(kRegKeys, n - kt.p0);
    if (kt.e_lo == 0 && kt.e_hi == kRegKeys) {
        const float4 lo = __ldcg(reinterpret_cast<const float4*>(s + kt.p0));
        const float4 hi = __ldcg(reinterpret_cast<const float4*>(s + kt.p0 + 4));
        kt.key[0] = score_key(lo.x); kt.key[1] = score_key(lo.y); kt.key[2] = score_key(lo.z); kt.key[3] = score_key(lo.w);
        kt.key[4] = score_key(hi.x); kt.key[5] = score_key(hi.y); kt.key[6] = score_key(hi.z); kt.key[7] = score_key(hi.w);
    } else {
#pragma unroll
        for (int e = 0; e < kRegKeys; ++e) kt.key[e] = (e >= kt.e_lo && e < kt.e_hi) ? score_key(__ldcg(s + kt.p0 + e)) : 0u;
    }
}

// f(tile) for every tile of the sequence, each thread's keys of the next tile requested before f runs on this one.
template <typename F>
__device__ __forceinline__ void for_each_key_tile(const float* __restrict__ s, int n, int a, int ntiles, int nt, F f) {
    KeyTile cur, nxt;
    load_key_tile(cur, s, n, a, 0, nt);
    for (int t = 0; t < ntiles; ++t) {
        if (t + 1 < ntiles) load_key_tile(nxt, s, n, a, t + 1, nt);
        f(cur);
        if (t + 1 < ntiles) cur = nxt;
    }
}

static __device__ void block_select_stream(const float* __restrict__ s, int n, int k, uint32_t flags,
                                           int32_t* __restrict__ out, SelectSmem& sm, int nt, const int* top_hist) {
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, nwarp = nt >> 5;
    if (k <= 0) return;
    const int n_all = n;
    if (flags & DODO_FORCE_LAST) {
        if (tid == 0) out[k - 1] = n - 1;
        n -= 1;
        k -= 1;
        if (k <= 0) return;
    }
    const int a = static_cast<int>((reinterpret_cast<uintptr_t>(s) >> 2) & 3u);
    const int ntiles = (n + a + kRegKeys * nt - 1) / (kRegKeys * nt);
    for (int b = tid; b < kHistCopies * 256; b += nt) (&sm.hist[0][0])[b] = 0;
    if (tid == 0) sm.ncand = 0;
    bool have_top = top_hist != nullptr;
    if (have_top && tid < 256) {
        int c = __ldcg(top_hist + tid);
        if ((flags & DODO_FORCE_LAST) && static_cast<int>(score_key(__ldcg(s + n_all - 1)) >> 24) == tid) c -= 1;
        sm.tot[tid] = c;
    }
    team_sync(nt);

    int* hist = sm.hist[warp % kHistCopies];
    uint32_t prefix = 0, mask = 0;
    int remaining = k, m = n;
    int shift = 24;
    while (m > kRankMax && shift >= 0) {
        if (!have_top) {
            for_each_key_tile(s, n, a, ntiles, nt, [&](const KeyTile& kt) {
#pragma unroll
                for (int e = 0; e < kRegKeys; ++e)
                    if (e >= kt.e_lo && e < kt.e_hi && (kt.key[e] & mask) == prefix) atomicAdd(&hist[(kt.key[e] >> shift) & 255u], 1);
            });
            team_sync(nt);
            if (tid < 256) {
                int sum = 0;
#pragma unroll
                for (int c = 0; c < kHistCopies; ++c) { sum += sm.hist[c][tid]; sm.hist[c][tid] = 0; }
                sm.tot[tid] = sum;
            }
            team_sync(nt);
        }
        have_top = false;
        int bin;
        find_bin(sm.tot, lane, remaining, &bin, &remaining, &m);
        prefix |= static_cast<uint32_t>(bin) << shift;
        mask |= 255u << shift;
        shift -= 8;
    }

    uint32_t T = prefix;
    int need_eq = remaining;
    if (m <= kRankMax) {
        for_each_key_tile(s, n, a, ntiles, nt, [&](const KeyTile& kt) {
#pragma unroll
            for (int e = 0; e < kRegKeys; ++e)
                if (e >= kt.e_lo && e < kt.e_hi && (kt.key[e] & mask) == prefix) sm.cand[atomicAdd(&sm.ncand, 1)] = kt.key[e];
        });
        team_sync(nt);
        for (int c = tid; c < m; c += nt) {
            const uint32_t mine = sm.cand[c];
            int gt = 0, eq = 0;
            for (int j = 0; j < m; ++j) {
                const uint32_t other = sm.cand[j];
                gt += other > mine ? 1 : 0;
                eq += other == mine ? 1 : 0;
            }
            if (gt < remaining && remaining <= gt + eq) { sm.kth = mine; sm.need_eq = remaining - gt; }
        }
        team_sync(nt);
        T = sm.kth;
        need_eq = sm.need_eq;
    }

    // ---- compaction, tile by tile in position order; `base` = kept-key counts of the tiles before (equal << 16 | above)
    int base_gt = 0, base_eq = 0;
    for_each_key_tile(s, n, a, ntiles, nt, [&](const KeyTile& kt) {
        int mine = 0;
#pragma unroll
        for (int e = 0; e < kRegKeys; ++e)
            if (e >= kt.e_lo && e < kt.e_hi) mine += kt.key[e] > T ? 1 : kt.key[e] == T ? 0x10000 : 0;
        int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += v;
        }
        if (lane == 31) sm.warp_gt[warp] = incl;
        team_sync(nt);
        const int w_mine = lane < nwarp ? sm.warp_gt[lane] : 0;
        int w_incl = w_mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, w_incl, o);
            if (lane >= o) w_incl += v;
        }
        const int before = __shfl_sync(0xffffffffu, w_incl - w_mine, warp) + incl - mine;
        const int total = __shfl_sync(0xffffffffu, w_incl, nwarp - 1);
        int gt_b = base_gt + (before & 0xffff), eq_b = base_eq + (before >> 16);
#pragma unroll
        for (int e = 0; e < kRegKeys; ++e) {
            if (e >= kt.e_lo && e < kt.e_hi) {
                if (kt.key[e] > T) {
                    out[gt_b + min(eq_b, need_eq)] = kt.p0 + e;
                    ++gt_b;
                } else if (kt.key[e] == T) {
                    if (eq_b < need_eq) out[gt_b + eq_b] = kt.p0 + e;
                    ++eq_b;
                }
            }
        }
        base_gt += total & 0xffff;
        base_eq += total >> 16;
        team_sync(nt);   // the warp totals are read before the next tile writes them
    });
}

// TopK of one sequence by a team of nt threads (see team_sync).  `s` are n scores in global memory, visible to
// this block; `keys` is shared memory for key_cap keys.  Sequences of up to eight keys per thread keep their keys
// in registers (block_select_small), sequences longer than key_cap are streamed from L2 step by step (block_select_stream);
// in between the keys are parked in `keys`.  Writes k ascending positions to `out`.
static __device__ void block_select(const float* __restrict__ s, int n, int k, uint32_t flags,
                             int32_t* __restrict__ out, SelectSmem& sm, uint32_t* keys, int key_cap, int nt,
                             const int* top_hist = nullptr) {
    const int span = n + static_cast<int>((reinterpret_cast<uintptr_t>(s) >> 2) & 3u);
    if (span <= kRegKeys * nt) return block_select_small<kRegKeys>(s, n, k, flags, out, sm, nt, top_hist);
    // 16 keys per thread: 16,384 scores by one block of 1024 threads take 11.2 us against 13.0 us for a cluster of 8 at
    // k = n/10, but 25.6 us at k = n, where one SM writes every index -- the launcher sends a sequence here only when
    // it keeps at most a quarter of its tokens (32 keys per thread lose to the cluster outright: 20.5 against 14.0 us)
    if (span <= 2 * kRegKeys * nt && 4 * k <= n) return block_select_small<2 * kRegKeys>(s, n, k, flags, out, sm, nt, top_hist);
    if (n > key_cap) return block_select_stream(s, n, k, flags, out, sm, nt, top_hist);
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
