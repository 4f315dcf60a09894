// Nugget gather (Eq. 5): copy the selected tokens' K and V rows into the per-sequence nugget cache
// and record their absolute positions.  Pure HBM copy: one thread block per nugget moves its K row
// and its V row with 16-byte accesses, all loads of a pass issued before the first store.
// An index outside its sequence is never followed: the block sets DODO_DEV_BAD_INDEX in the status
// word and leaves that cache row and its position as they were.
#include "dodo_internal.cuh"
#include "stream_rows.cuh"

namespace {

constexpr int kGatherThreads = 128;
constexpr int kGatherBlocksPerSM = 12;   // 40 registers per thread: the 1640 blocks of a 8 x 205-nugget launch are one wave

__global__ void __launch_bounds__(kGatherThreads, kGatherBlocksPerSM)
gather_kernel(const unsigned char* __restrict__ K, const unsigned char* __restrict__ V, int row_vecs,
              const int32_t* __restrict__ idx, const __grid_constant__ GatherGroup g,
              unsigned char* __restrict__ cacheK, unsigned char* __restrict__ cacheV,
              int32_t* __restrict__ cache_pos, int* __restrict__ dev_status) {
    const int j = g.idx0[0] + static_cast<int>(blockIdx.x);  // nugget slot in idx
    int lo = 0, hi = g.nseq;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (g.idx0[mid] <= j) lo = mid; else hi = mid;
    }
    const int b = lo;
    dodo_grid_dependency_sync();   // the indices come from the kernel before
    const int token = __ldg(idx + j);
    if (static_cast<unsigned>(token) >= static_cast<unsigned>(g.n[b])) {
        if (threadIdx.x == 0) atomicOr(dev_status, DODO_DEV_BAD_INDEX);
        return;
    }
    const size_t row_bytes = static_cast<size_t>(row_vecs) * 16u;
    const size_t src = (static_cast<size_t>(g.src_row0[b]) + static_cast<size_t>(token)) * row_bytes;
    const int dst_row = g.dst_row0[b] + (j - g.idx0[b]);
    const size_t dst = static_cast<size_t>(dst_row) * row_bytes;
    const uint4* sk = reinterpret_cast<const uint4*>(K + src);
    const uint4* sv = reinterpret_cast<const uint4*>(V + src);
    uint4* dk = reinterpret_cast<uint4*>(cacheK + dst);
    uint4* dv = reinterpret_cast<uint4*>(cacheV + dst);
    if (threadIdx.x == 0) cache_pos[dst_row] = g.pos_base[b] + token;

    dodo_rows::copy_kv_row(sk, sv, dk, dv, row_vecs, static_cast<int>(threadIdx.x), kGatherThreads);
}

// The same copy behind a fused score + select launch (dodo_compress).  This kernel is launched with programmatic
// stream serialization, so its blocks become resident once every block of that launch has started, and instead
// of waiting for all of it they wait for their own sequence's flag, which the block that selected the sequence
// raises behind its indices (release / acquire): the copies of the sequences selected early run beside the scoring
// of the later ones, and only the last sequences' copies follow the last selection.  Every flag is raised by a
// block that is already running and waits for nothing, so the wait ends; it is bounded all the same (the block
// then sets DODO_DEV_WAIT_TIMEOUT and copies nothing).  Before a block leaves it still waits for the launch before
// it as a whole, so that whatever is ordered behind this kernel is ordered behind that launch too.
constexpr int kFlagPolls = 1 << 19;   // with the sleep between polls, about half a second

__global__ void __launch_bounds__(kGatherThreads, kGatherBlocksPerSM)
gather_flagged_kernel(const unsigned char* __restrict__ K, const unsigned char* __restrict__ V, int row_vecs,
                      const int32_t* idx, const __grid_constant__ GatherGroup g, unsigned char* __restrict__ cacheK,
                      unsigned char* __restrict__ cacheV, int32_t* __restrict__ cache_pos, int* state,
                      int* __restrict__ dev_status) {
    __shared__ int s_up;
    const int j = g.idx0[0] + static_cast<int>(blockIdx.x);  // nugget slot in idx
    int lo = 0, hi = g.nseq;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (g.idx0[mid] <= j) lo = mid; else hi = mid;
    }
    const int b = lo;
    int* left = state;
    const int* flag = state + DODO_FLAG_STRIDE * (1 + b);
    if (threadIdx.x == 0) {
        int up = 0;
        for (int it = 0; it < kFlagPolls && !up; ++it) {
            up = ld_acquire_gpu(flag);
            if (!up) __nanosleep(500);
        }
        s_up = up;
        if (!up) atomicOr(dev_status, DODO_DEV_WAIT_TIMEOUT);
    }
    __syncthreads();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // (the successor waits for this whole launch at its top)
    if (s_up) {
        const int token = __ldcg(idx + j);
        if (static_cast<unsigned>(token) >= static_cast<unsigned>(g.n[b])) {
            if (threadIdx.x == 0) atomicOr(dev_status, DODO_DEV_BAD_INDEX);
        } else {
            const size_t row_bytes = static_cast<size_t>(row_vecs) * 16u;
            const size_t src = (static_cast<size_t>(g.src_row0[b]) + static_cast<size_t>(token)) * row_bytes;
            const int dst_row = g.dst_row0[b] + (j - g.idx0[b]);
            const size_t dst = static_cast<size_t>(dst_row) * row_bytes;
            if (threadIdx.x == 0) cache_pos[dst_row] = g.pos_base[b] + token;
            dodo_rows::copy_kv_row(reinterpret_cast<const uint4*>(K + src), reinterpret_cast<const uint4*>(V + src),
                                   reinterpret_cast<uint4*>(cacheK + dst), reinterpret_cast<uint4*>(cacheV + dst), row_vecs,
                                   static_cast<int>(threadIdx.x), kGatherThreads);
        }
    }
    asm volatile("griddepcontrol.wait;" ::: "memory");   // the launch before this one is complete as a whole
    // the last block to leave puts the flags and the counter back to zero: every other block has read its flag
    __syncthreads();
    if (threadIdx.x == 0) {
        const int t = atomicAdd(left, 1);
        if (t == static_cast<int>(gridDim.x) - 1) {
            for (int i = 0; i < g.nseq; ++i) state[DODO_FLAG_STRIDE * (1 + i)] = 0;
            *left = 0;
        }
    }
}

// The same copy for several layers that share one selection (Sec. 2.1): blockIdx.y is the layer, the
// sequence search and the index are the same for all of them, positions are recorded once.
__global__ void __launch_bounds__(kGatherThreads, kGatherBlocksPerSM)
gather_layers_kernel(const __grid_constant__ GatherLayers lay, int row_vecs, const int32_t* __restrict__ idx,
                     const __grid_constant__ GatherGroup g, int32_t* __restrict__ cache_pos,
                     int* __restrict__ dev_status) {
    const int j = g.idx0[0] + static_cast<int>(blockIdx.x);
    const int l = static_cast<int>(blockIdx.y);
    int lo = 0, hi = g.nseq;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (g.idx0[mid] <= j) lo = mid; else hi = mid;
    }
    const int b = lo;
    dodo_grid_dependency_sync();
    const int token = __ldg(idx + j);
    if (static_cast<unsigned>(token) >= static_cast<unsigned>(g.n[b])) {
        if (threadIdx.x == 0) atomicOr(dev_status, DODO_DEV_BAD_INDEX);
        return;
    }
    const size_t row_bytes = static_cast<size_t>(row_vecs) * 16u;
    const size_t src = (static_cast<size_t>(g.src_row0[b]) + static_cast<size_t>(token)) * row_bytes;
    const int dst_row = g.dst_row0[b] + (j - g.idx0[b]);
    const size_t dst = static_cast<size_t>(dst_row) * row_bytes;
    const uint4* sk = reinterpret_cast<const uint4*>(lay.K[l] + src);
    const uint4* sv = reinterpret_cast<const uint4*>(lay.V[l] + src);
    uint4* dk = reinterpret_cast<uint4*>(lay.cacheK[l] + dst);
    uint4* dv = reinterpret_cast<uint4*>(lay.cacheV[l] + dst);
    if (l == 0 && lay.first && threadIdx.x == 0) cache_pos[dst_row] = g.pos_base[b] + token;

    dodo_rows::copy_kv_row(sk, sv, dk, dv, row_vecs, static_cast<int>(threadIdx.x), kGatherThreads);
}

}  // namespace

int dodo_launch_gather_layers(dodo_ctx* ctx, const GatherLayers& lay, size_t row_bytes, const int32_t* idx,
                              const GatherGroup& g, int32_t* cache_pos, int* dev_status, cudaStream_t st) {
    const int total = g.idx0[g.nseq] - g.idx0[0];
    if (total == 0 || lay.n == 0) return DODO_OK;
    return dodo_check_cuda(ctx, dodo_launch_dependent(gather_layers_kernel, dim3(static_cast<unsigned>(total), static_cast<unsigned>(lay.n)),
                                                      dim3(kGatherThreads), 0, st, lay, static_cast<int>(row_bytes / 16), idx, g, cache_pos,
                                                      dev_status),
                           "multi-layer gather launch");
}

int dodo_launch_gather_flagged(dodo_ctx* ctx, const void* K, const void* V, size_t row_bytes, const int32_t* idx,
                               const GatherGroup& g, void* cacheK, void* cacheV, int32_t* cache_pos, int* state,
                               int* dev_status, cudaStream_t st) {
    const int total = g.idx0[g.nseq] - g.idx0[0];
    if (total == 0) return DODO_OK;
    return dodo_check_cuda(ctx, dodo_launch_dependent(gather_flagged_kernel, dim3(static_cast<unsigned>(total)), dim3(kGatherThreads), 0,
                                                      st, static_cast<const unsigned char*>(K), static_cast<const unsigned char*>(V),
                                                      static_cast<int>(row_bytes / 16), idx, g, static_cast<unsigned char*>(cacheK),
                                                      static_cast<unsigned char*>(cacheV), cache_pos, state, dev_status),
                           "flagged gather launch");
}

int dodo_launch_gather(dodo_ctx* ctx, const void* K, const void* V, size_t row_bytes,
                       const int32_t* idx, const GatherGroup& g, void* cacheK, void* cacheV,
                       int32_t* cache_pos, int* dev_status, cudaStream_t st) {
    const int total = g.idx0[g.nseq] - g.idx0[0];
    if (total == 0) return DODO_OK;
    return dodo_check_cuda(ctx, dodo_launch_dependent(gather_kernel, dim3(static_cast<unsigned>(total)), dim3(kGatherThreads), 0, st,
                                                      static_cast<const unsigned char*>(K), static_cast<const unsigned char*>(V),
                                                      static_cast<int>(row_bytes / 16), idx, g, static_cast<unsigned char*>(cacheK),
                                                      static_cast<unsigned char*>(cacheV), cache_pos, dev_status),
                           "gather launch");
}
