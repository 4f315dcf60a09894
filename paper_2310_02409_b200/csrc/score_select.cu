// Scorer GEMV (Eq. 6 / Eq. 15, linear form) and per-sequence TopK selection (Eq. 14), separately and
// fused in one launch.
//
// Score: HBM-bound.  Each warp streams two token rows with 16-byte loads, several in flight per
// lane, against the weight vector held in shared memory; fp32 accumulation, butterfly reduction.
//
// Select: radix select on order-preserving 32-bit keys (8-bit digits, private shared-memory histograms) finds
// the k-th largest key T; one position-ordered pass then keeps every key > T plus the first (k - #greater) keys
// == T, writing indices in ascending position.  Ties therefore go to the lower position by construction and the
// output needs no sort and no atomics.  Sequences of up to 8 keys per thread keep their keys in registers and stop
// the radix passes as soon as at most 512 keys are left in the race, which are then ranked against each other
// directly (select_block.cuh).
//
// Fused: score blocks of one sequence take a ticket when their scores are globally visible; the block holding the
// last ticket runs that sequence's selection out of L2.  No block ever waits.  The score blocks also count their
// scores' top key digits into a per-sequence histogram in global memory, so the selection's first radix pass is
// already done when it starts; and on request the selecting block raises a per-sequence flag behind its indices,
// for a gather that follows each sequence's selection instead of the whole launch (gather_flagged_kernel).
#include "dodo_internal.cuh"
#include "select_block.cuh"
#include "stream_rows.cuh"

namespace {

using namespace dodo_sel;

constexpr int kScoreThreads = 512;
constexpr int kRowsPerWarp = 2;
constexpr int kRowsPerBlock = (kScoreThreads / 32) * kRowsPerWarp;
constexpr int kSelectThreads = 1024;
constexpr int kFusedMaxTokens = 4096;   // fused kernel: longer sequences are selected by a launch of their own (more threads, or a cluster, per sequence)
constexpr int kSelectCluster = 8;     // most blocks (SMs) that share one long sequence
constexpr int kKeyCacheMax = 48 * 1024;  // select / estimate launches: keys of up to this many scores (192 KB)

template <typename T>
__global__ void __launch_bounds__(kScoreThreads, 2)
score_select_kernel(const T* __restrict__ X, const T* __restrict__ w, int d, float bias,
                    const __grid_constant__ ScoreSelectGroup g, int mode, uint32_t flags,
                    float* __restrict__ scores, int32_t* __restrict__ idx, int* __restrict__ tickets,
                    int* __restrict__ seq_flag, int* __restrict__ top_hist) {
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    __shared__ SelectSmem sel;
    __shared__ int is_last;
    uint4* sw = reinterpret_cast<uint4*>(dyn_smem);
    const int nvec = d / Vec16<T>::kElems;  // 16-byte chunks per row
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    dodo_grid_dependency_sync();   // nothing is read or written before everything earlier on the stream is complete
    for (int c = tid; c < nvec; c += kScoreThreads) sw[c] = reinterpret_cast<const uint4*>(w)[c];
    // mode 0: scores only; 1: the block that completes a sequence selects it (fused); 2: scores and, as in 1, the
    // counts of their top key digits, for a selection launched behind this kernel
    const bool fused = mode == 1, counting = mode != 0;
    int* digits = sel.hist[0];   // this block's counts of its scores' top key digits
    if (counting && tid < 256) digits[tid] = 0;

    // which sequence does this block serve?
    int lo = 0, hi = g.nseq;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (g.blk0[mid] <= static_cast<int>(blockIdx.x)) lo = mid; else hi = mid;
    }
    const int b = lo;
    const int n = g.n[b];
    const int lrow = (static_cast<int>(blockIdx.x) - g.blk0[b]) * kRowsPerBlock + warp * kRowsPerWarp;
    __syncthreads();

    if (lrow < n) {
        const bool two = lrow + 1 < n;
        const size_t r0 = static_cast<size_t>(g.row0[b]) + static_cast<size_t>(lrow);
        const uint4* x0 = reinterpret_cast<const uint4*>(X + r0 * static_cast<size_t>(d));
        const uint4* x1 = two ? x0 + nvec : x0;
        float acc0, acc1;
        dodo_rows::dot_two_rows<T>(x0, x1, sw, nvec, lane, acc0, acc1);
        if (lane == 0) {
            const float v0 = acc0 + bias, v1 = acc1 + bias;
            scores[r0] = v0;
            if (two) scores[r0 + 1] = v1;
            // the first radix pass of the selection is taken here, one count per score
            if (counting) {
                atomicAdd(&digits[score_key(v0) >> 24], 1);
                if (two) atomicAdd(&digits[score_key(v1) >> 24], 1);
            }
        }
    }
    if (!counting) return;

    // hand-over: add this block's digit counts to the sequence's (one atomic per digit that occurs, not per score: the
    // scores of a sequence share a handful of digits), make them and the scores visible, then take a ticket
    __syncthreads();
    if (tid < 256 && digits[tid] != 0) atomicAdd(&top_hist[b * 256 + tid], digits[tid]);
    if (!fused) return;
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int nblk = g.blk0[b + 1] - g.blk0[b];
        const int t = atomicAdd(&tickets[b], 1);
        is_last = (t == nblk - 1);
        if (is_last) tickets[b] = 0;  // leave the counter clean for the next launch
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const int team = select_team_threads(n, kScoreThreads);
    if (tid >= team) return;
    block_select(scores + g.row0[b], n, g.k[b], flags, idx + g.idx0[b], sel, nullptr, 0, team, top_hist + b * 256);
    if (tid < 256) top_hist[b * 256 + tid] = 0;   // clean for the next launch (each count was read, if at all, by this thread)
    // A gather launched behind this kernel with programmatic stream serialization may copy a sequence's rows as
    // soon as its indices are visible: raise the sequence's flag behind them.
    if (seq_flag != nullptr) {
        __threadfence();
        team_sync(team);
        if (tid == 0) st_release_gpu(seq_flag + b * DODO_FLAG_STRIDE, 1);
    }
}

// key_cap keys of dynamic shared memory per block
__global__ void __launch_bounds__(kSelectThreads, 1)
select_kernel(const float* __restrict__ scores, const __grid_constant__ ScoreSelectGroup g,
              uint32_t flags, int32_t* __restrict__ idx, int key_cap, int* __restrict__ top_hist) {
    __shared__ SelectSmem sel;
    extern __shared__ uint32_t dyn_keys[];
    const int b = blockIdx.x;
    const int team = select_team_threads(g.n[b], kSelectThreads);
    if (static_cast<int>(threadIdx.x) >= team) return;
    dodo_grid_dependency_sync();
    // top_hist, when given: the counts of the scores' top key digits, taken by the kernel that wrote the scores
    // (row g.blk0[b]: the sequence's number in that kernel's launch); read at most once, then cleared
    int* top = top_hist != nullptr ? top_hist + g.blk0[b] * 256 : nullptr;
    block_select(scores + g.row0[b], g.n[b], g.k[b], flags, idx + g.idx0[b], sel, dyn_keys, key_cap, team, top);
    if (top != nullptr && threadIdx.x < 256) top[threadIdx.x] = 0;
}

// Inverse of score_key for the keys of numbers (key 0, the NaN class, comes back as a NaN).
__device__ __forceinline__ float key_score(uint32_t key) {
    return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Lambda from m sampled scores (text after Eq. 8): the (k+1)-th largest, one thread block.
__global__ void __launch_bounds__(kSelectThreads, 1)
estimate_threshold_kernel(const float* __restrict__ sample, int m, int k, float* __restrict__ lambda, int key_cap) {
    __shared__ SelectSmem sel;
    extern __shared__ uint32_t dyn_keys[];
    const int tid = threadIdx.x;
    const int nt = select_team_threads(m, kSelectThreads);
    if (tid >= nt) return;
    dodo_grid_dependency_sync();
    if (k >= m) {   // every score has to pass
        if (tid == 0) *lambda = -INFINITY;
        return;
    }
    const bool cached = m <= key_cap;
    if (cached) {
        for (int i = tid; i < m; i += nt) dyn_keys[i] = score_key(__ldcg(sample + i));
    }
    team_sync(nt);
    auto key_at = [&](int i) -> uint32_t { return cached ? dyn_keys[i] : score_key(__ldcg(sample + i)); };
    int need_eq;
    const uint32_t key = block_kth_key(key_at, m, k + 1, sel, &need_eq, nt);
    if (tid == 0) *lambda = key_score(key);
}

// ---- selection by a thread-block cluster -------------------------------------------------------------
// Long sequences: the C blocks of a cluster take contiguous slices of one sequence (keys in their own shared
// memory), so that the radix passes and the compaction run on C SMs instead of one.  A pass builds C local
// histograms; after one cluster barrier every block adds up all C of them through distributed shared memory
// and finds the same bin by itself.  The histogram is double-buffered, so a pass needs one cluster barrier.
// Every block of a cluster executes the same sequence of cluster barriers (n, k and flags are per sequence).
struct ClusterSelectSmem {
    int hist[2][256];
    int tot[256];
    int warp_gt[32];
    int warp_eq[32];
    int count[2];      // this block's keys above / equal to the threshold key (read by the other blocks)
    int bin;
    int remaining;
};

// Sum over the blocks [0, count) of the cluster of the int each holds at `local`'s place in its shared memory
// (all loads issued before the first is used; the caller has passed a cluster barrier since those were written).
__device__ __forceinline__ int cluster_sum(const int* local, int count) {
    const uint32_t mine = static_cast<uint32_t>(__cvta_generic_to_shared(local));
    int v[kSelectCluster];
#pragma unroll
    for (int r = 0; r < kSelectCluster; ++r) {
        v[r] = 0;
        if (r < count) {
            uint32_t remote;
            asm("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(mine), "r"(r));
            asm volatile("ld.shared::cluster.s32 %0, [%1];" : "=r"(v[r]) : "r"(remote));
        }
    }
    int t = 0;
#pragma unroll
    for (int r = 0; r < kSelectCluster; ++r) t += v[r];
    return t;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}

// The k-th largest key (1 <= k <= total keys) among the keys of all C blocks, key_at(0..m) being this block's.
// Called by every thread of every block of the cluster, after a cluster barrier that all blocks have passed.
template <typename KeyAt>
__device__ uint32_t cluster_kth_key(KeyAt key_at, int m, int k, ClusterSelectSmem& sm, int C, int* need_eq,
                                    const int* top = nullptr, int top_skip = -1) {
    const int tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5;
    uint32_t prefix = 0, mask = 0;
    int remaining = k;
    int buf = 0;
    for (int shift = 24; shift >= 0; shift -= 8, buf ^= 1) {
        int* hist = sm.hist[buf];
        if (shift == 24 && top != nullptr) {
            // the first pass was taken by the kernel that wrote the scores: its counts of the top digits (256 ints in
            // global memory, every block reads them; one key, the forced last token's, may have to be taken out)
            if (tid < 256) sm.tot[tid] = __ldcg(top + tid) - (tid == top_skip ? 1 : 0);
            __syncthreads();
        } else {
        for (int b = tid; b < 256; b += nt) hist[b] = 0;
        __syncthreads();
        for (int base = 0; base < m; base += 4 * nt) {
            uint32_t key[4];
            bool in[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = base + u * nt + tid;
                in[u] = i < m;
                key[u] = in[u] ? key_at(i) : 0u;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (in[u] && (key[u] & mask) == prefix) atomicAdd(&hist[(key[u] >> shift) & 255u], 1);
        }
        __syncthreads();
        cluster_sync_all();   // all C histograms of this pass are complete and visible
        if (tid < 256) {
            sm.tot[tid] = cluster_sum(hist + tid, C);
        }
        __syncthreads();
        }
        if (warp == 0) {
            // lane L owns bins 255-8L .. 248-8L (descending); find where the running count reaches `remaining`
            int local[8], sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { local[j] = sm.tot[255 - 8 * lane - j]; sum += local[j]; }
            int incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += v;
            }
            const int excl = incl - sum;
            if (excl < remaining && remaining <= incl) {
                int run = excl;
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (run < remaining && remaining <= run + local[j]) {
                        sm.bin = 255 - 8 * lane - j;
                        sm.remaining = remaining - run;
                    }
                    run += local[j];
                }
            }
        }
        __syncthreads();
        prefix |= static_cast<uint32_t>(sm.bin) << shift;
        mask |= 255u << shift;
        remaining = sm.remaining;
        // (tot, bin and remaining are next written after two more block barriers; the histogram buffer of this
        // pass is next cleared two passes on, after a cluster barrier that every reader of it has passed)
    }
    *need_eq = remaining;
    return prefix;
}

// key_cap keys of dynamic shared memory per block; launched with clusters of C blocks, C blocks per sequence
__global__ void __launch_bounds__(kSelectThreads, 1)
cluster_select_kernel(const float* __restrict__ scores, const __grid_constant__ ScoreSelectGroup g,
                      uint32_t flags, int32_t* __restrict__ idx, int key_cap, int C, int* __restrict__ top_hist) {
    __shared__ ClusterSelectSmem sm;
    extern __shared__ uint32_t dyn_keys[];
    asm volatile("barrier.cluster.arrive.relaxed;" ::: "memory");   // "this block runs"; waited for below
    const int tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, nwarp = nt >> 5;
    const int b = static_cast<int>(blockIdx.x) / C, rank = static_cast<int>(blockIdx.x) % C;
    dodo_grid_dependency_sync();
    int* top = top_hist != nullptr ? top_hist + g.blk0[b] * 256 : nullptr;   // digit counts that came with the scores
    const float* s = scores + g.row0[b];
    int32_t* out = idx + g.idx0[b];
    int n = g.n[b], k = g.k[b];
    int top_skip = -1;
    if ((flags & DODO_FORCE_LAST) && k > 0) {
        if (rank == 0 && tid == 0) out[k - 1] = n - 1;
        if (top != nullptr) top_skip = static_cast<int>(score_key(__ldcg(s + n - 1)) >> 24);
        n -= 1;
        k -= 1;
    }
    // this block's slice of the positions (a multiple of 32 long, so that warps own aligned pieces)
    const int per = (((n + C - 1) / C) + 31) & ~31;
    const int q0 = min(n, rank * per), m = min(n, q0 + per) - q0;
    const bool cached = per <= key_cap;
    if (cached && k > 0) {
        for (int i = tid; i < m; i += nt) dyn_keys[i] = score_key(__ldcg(s + q0 + i));
    }
    __syncthreads();
    asm volatile("barrier.cluster.wait;" ::: "memory");   // every block of the cluster has started
    if (k <= 0) {                                          // (uniform over the cluster)
        if (top != nullptr && rank == 0 && tid < 256) top[tid] = 0;
        return;
    }
    auto key_at = [&](int i) -> uint32_t { return cached ? dyn_keys[i] : score_key(__ldcg(s + q0 + i)); };

    int need_eq;
    const uint32_t T = cluster_kth_key(key_at, m, k, sm, C, &need_eq, top, top_skip);
    // (every block has passed a cluster barrier since it read the counts: they are cleared for the next launch)
    if (top != nullptr && rank == 0 && tid < 256) top[tid] = 0;

    // position-ordered compaction: counts per warp segment, per block, then over the lower-ranked blocks
    const int seg = (((m + nwarp - 1) / nwarp) + 31) & ~31;
    const int p0 = min(m, warp * seg), p1 = min(m, p0 + seg);
    int n_gt = 0, n_eq = 0;
    for (int base = p0; base < p1; base += 32) {
        const int i = base + lane;
        const uint32_t key = i < p1 ? key_at(i) : 0u;
        n_gt += __popc(__ballot_sync(0xffffffffu, i < p1 && key > T));
        n_eq += __popc(__ballot_sync(0xffffffffu, i < p1 && key == T));
    }
    if (lane == 0) { sm.warp_gt[warp] = n_gt; sm.warp_eq[warp] = n_eq; }
    __syncthreads();
    const int g_mine = lane < nwarp ? sm.warp_gt[lane] : 0, e_mine = lane < nwarp ? sm.warp_eq[lane] : 0;
    int g_incl = g_mine, e_incl = e_mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int gv = __shfl_up_sync(0xffffffffu, g_incl, o), ev = __shfl_up_sync(0xffffffffu, e_incl, o);
        if (lane >= o) { g_incl += gv; e_incl += ev; }
    }
    if (tid == 31) { sm.count[0] = g_incl; sm.count[1] = e_incl; }   // lane 31 of warp 0 holds the block totals
    __syncthreads();
    cluster_sync_all();   // every block's totals are visible
    int gt_run = cluster_sum(&sm.count[0], rank), eq_run = cluster_sum(&sm.count[1], rank);   // lower-ranked blocks
    gt_run += __shfl_sync(0xffffffffu, g_incl - g_mine, warp);
    eq_run += __shfl_sync(0xffffffffu, e_incl - e_mine, warp);
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
        if (gt || (eq && eq_before < need_eq)) out[gt_before + min(eq_before, need_eq)] = q0 + i;
        gt_run += __popc(gt_m);
        eq_run += __popc(eq_m);
    }
    cluster_sync_all();   // no block leaves while another may still read its shared memory
}

// Lambda from m sampled scores by one cluster of C blocks.
__global__ void __launch_bounds__(kSelectThreads, 1)
cluster_estimate_kernel(const float* __restrict__ sample, int m, int k, float* __restrict__ lambda, int key_cap, int C) {
    __shared__ ClusterSelectSmem sm;
    extern __shared__ uint32_t dyn_keys[];
    asm volatile("barrier.cluster.arrive.relaxed;" ::: "memory");
    const int tid = threadIdx.x, nt = blockDim.x;
    const int rank = static_cast<int>(blockIdx.x) % C;
    dodo_grid_dependency_sync();
    const int per = (((m + C - 1) / C) + 31) & ~31;
    const int q0 = min(m, rank * per), mine = min(m, q0 + per) - q0;
    const bool cached = per <= key_cap;
    if (cached && k < m) {
        for (int i = tid; i < mine; i += nt) dyn_keys[i] = score_key(__ldcg(sample + q0 + i));
    }
    __syncthreads();
    asm volatile("barrier.cluster.wait;" ::: "memory");
    if (k >= m) {   // every score has to pass (uniform over the cluster)
        if (rank == 0 && tid == 0) *lambda = -INFINITY;
        return;
    }
    auto key_at = [&](int i) -> uint32_t { return cached ? dyn_keys[i] : score_key(__ldcg(sample + q0 + i)); };
    int need_eq;
    const uint32_t key = cluster_kth_key(key_at, mine, k + 1, sm, C, &need_eq);
    if (rank == 0 && tid == 0) *lambda = key_score(key);
    cluster_sync_all();   // no block leaves while another may still read its histograms
}

template <typename T>
int launch_score_t(dodo_ctx* ctx, const void* X, int d, const void* w, float bias,
                   const ScoreSelectGroup& g, int mode, uint32_t flags, float* scores, int32_t* idx,
                   int* tickets, int* seq_flag, cudaStream_t st) {
    const int nblocks = g.blk0[g.nseq];
    const size_t smem = static_cast<size_t>(d) * sizeof(T);
    auto kern = score_select_kernel<T>;
    if (smem > 24 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             static_cast<int>(smem));
        if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "score shared-memory attribute");
    }
    return dodo_check_cuda(ctx, dodo_launch_dependent(kern, dim3(nblocks), dim3(kScoreThreads), smem, st, static_cast<const T*>(X),
                                                      static_cast<const T*>(w), d, bias, g, mode, flags, scores, idx, tickets, seq_flag, ctx->top_hist),
                           "score launch");
}

}  // namespace

int dodo_score_rows_per_block() { return kRowsPerBlock; }
int dodo_select_fused_max_tokens() { return kFusedMaxTokens; }

// Keys of shared memory for a select / estimate launch whose longest input has max_n scores (0: none fit).
static int select_key_cap(dodo_ctx* ctx, int max_n) {
    if (!ctx->select_attr_set) {
        const int room = ctx->max_smem_optin - static_cast<int>(sizeof(SelectSmem)) - 4096;   // static shared memory of the kernels and slack
        int cap = kKeyCacheMax;
        if (room < cap * 4) cap = room > 0 ? room / 4 : 0;
        if (cap * 4 > 48 * 1024) {
            if (cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, cap * 4) != cudaSuccess ||
                cudaFuncSetAttribute(estimate_threshold_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, cap * 4) != cudaSuccess ||
                cudaFuncSetAttribute(cluster_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, cap * 4) != cudaSuccess ||
                cudaFuncSetAttribute(cluster_estimate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, cap * 4) != cudaSuccess) {
                (void)cudaGetLastError();
                cap = 48 * 1024 / 4;
            }
        }
        ctx->select_key_cap = cap;
        ctx->select_attr_set = true;
    }
    return max_n < ctx->select_key_cap ? (max_n > 0 ? max_n : 0) : ctx->select_key_cap;
}

// Blocks per sequence for inputs of up to max_n scores: one SM up to kClusterMin scores (the fixed cost of a pass
// -- barriers, the bin search -- outweighs the key work below that), then a cluster with about 2048 scores per block.
constexpr int kClusterMin = 8192;
static int select_cluster_size(int max_n) {
    if (max_n <= kClusterMin) return 1;
    const int c = (max_n + 2047) / 2048;
    return c < kSelectCluster ? c : kSelectCluster;
}

template <typename... Args>
static cudaError_t launch_cluster(void (*kern)(Args...), int blocks, int C, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(blocks));
    cfg.blockDim = dim3(kSelectThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(C);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

int dodo_launch_estimate_threshold(dodo_ctx* ctx, const float* sample, int m, int k, float* lambda, cudaStream_t st) {
    const int C = select_cluster_size(m);
    if (C > 1) {
        const int per = (((m + C - 1) / C) + 31) & ~31;
        const int key_cap = select_key_cap(ctx, per);
        return dodo_check_cuda(ctx, launch_cluster(cluster_estimate_kernel, C, C, static_cast<size_t>(key_cap) * 4, st,
                                                   sample, m, k, lambda, key_cap, C),
                               "threshold estimate launch");
    }
    const int key_cap = select_key_cap(ctx, m);
    return dodo_check_cuda(ctx, dodo_launch_dependent(estimate_threshold_kernel, dim3(1), dim3(kSelectThreads),
                                                      static_cast<size_t>(key_cap) * 4, st, sample, m, k, lambda, key_cap),
                           "threshold estimate launch");
}

int dodo_launch_score(dodo_ctx* ctx, const void* X, int dtype, int d, const void* w, float bias,
                      const ScoreSelectGroup& g, int mode, uint32_t flags, float* scores,
                      int32_t* idx, int* tickets, int* seq_flag, cudaStream_t st) {
    if (g.blk0[g.nseq] == 0) return DODO_OK;
    if (dtype == DODO_BF16)
        return launch_score_t<__nv_bfloat16>(ctx, X, d, w, bias, g, mode, flags, scores, idx, tickets, seq_flag, st);
    return launch_score_t<float>(ctx, X, d, w, bias, g, mode, flags, scores, idx, tickets, seq_flag, st);
}

// Clusters of C blocks of cluster_select_kernel that the device holds at once when the longest sequence has
// `longest` scores (occupancy calculator; cached for the usual case of at most 32 KB of keys per block).
static int select_clusters_resident(dodo_ctx* ctx, int C, int longest) {
    const int per = (((longest + C - 1) / C) + 31) & ~31;
    const size_t smem = static_cast<size_t>(select_key_cap(ctx, per)) * 4;
    const bool usual = smem <= 32 * 1024;
    if (usual && ctx->select_resident[C] > 0) return ctx->select_resident[C];
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(C * 64));
    cfg.blockDim = dim3(kSelectThreads);
    cfg.dynamicSmemBytes = usual ? 32 * 1024 : smem;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(C);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, cluster_select_kernel, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
    if (usual) ctx->select_resident[C] = n > 0 ? n : -1;
    return n;
}

// One launch per class of sequences: those of up to kClusterMin scores, one block each; the longer ones, one
// cluster each.
int dodo_launch_select(dodo_ctx* ctx, const float* scores, const ScoreSelectGroup& g, uint32_t flags,
                       int32_t* idx, bool counted, cudaStream_t st) {
    if (g.nseq == 0) return DODO_OK;
    ScoreSelectGroup part[2];   // [0] short, [1] long; the kernels read row0, n, k and idx0 only
    int max_n[2] = {0, 0};
    int nlong = 0, longest = 0;
    // a sequence of up to twice kClusterMin scores that keeps at most a quarter of them is still faster on one block
    // (16 keys per thread in registers); beyond that, or when most indices are written, a cluster
    auto is_long = [&](int i) { return g.n[i] > kClusterMin && !(g.n[i] <= 2 * kClusterMin && 4 * g.k[i] <= g.n[i]); };
    for (int i = 0; i < g.nseq; ++i)
        if (is_long(i)) { ++nlong; longest = g.n[i] > longest ? g.n[i] : longest; }
    // clusters only if all of them run at once (one block of this size per SM); else every sequence gets one block
    int C = nlong > 0 ? select_cluster_size(longest) : 1;
    while (C >= 2 && select_clusters_resident(ctx, C, longest) < nlong) --C;
    const bool clusters = C >= 2;
    part[0].nseq = part[1].nseq = 0;
    for (int i = 0; i < g.nseq; ++i) {
        const int c = (clusters && is_long(i)) ? 1 : 0;
        const int j = part[c].nseq++;
        part[c].row0[j] = g.row0[i];
        part[c].n[j] = g.n[i];
        part[c].k[j] = g.k[i];
        part[c].idx0[j] = g.idx0[i];
        part[c].blk0[j] = i;   // the sequence's number in the launch that wrote the scores (its row of digit counts)
        max_n[c] = g.n[i] > max_n[c] ? g.n[i] : max_n[c];
    }
    for (int c = 0; c < 2; ++c) {
        for (int j = part[c].nseq; j < DODO_GROUP; ++j) part[c].row0[j] = part[c].n[j] = part[c].k[j] = part[c].idx0[j] = 0;
        for (int j = part[c].nseq; j <= DODO_GROUP; ++j) part[c].blk0[j] = 0;
    }
    int* top_hist = counted ? ctx->top_hist : nullptr;
    if (part[0].nseq > 0) {
        const int key_cap = select_key_cap(ctx, max_n[0]);
        const int rc = dodo_check_cuda(ctx, dodo_launch_dependent(select_kernel, dim3(part[0].nseq), dim3(kSelectThreads),
                                                                  static_cast<size_t>(key_cap) * 4, st, scores, part[0], flags, idx, key_cap, top_hist),
                                       "select launch");
        if (rc != DODO_OK) return rc;
    }
    if (part[1].nseq > 0) {
        const int per = (((max_n[1] + C - 1) / C) + 31) & ~31;
        const int key_cap = select_key_cap(ctx, per);
        return dodo_check_cuda(ctx, launch_cluster(cluster_select_kernel, part[1].nseq * C, C, static_cast<size_t>(key_cap) * 4, st,
                                                   scores, part[1], flags, idx, key_cap, C, top_hist),
                               "select launch");
    }
    return DODO_OK;
}
