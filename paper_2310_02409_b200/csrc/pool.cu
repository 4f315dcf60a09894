// Mean pooling of even chunks (Sec. 5.1): the comparison system the paper measures against cuts the text evenly
// into segments of r tokens and pools the states of each into one vector (the mean, in the paper's experiments).
// Here the K and V rows of every segment are averaged into one row of the same per-sequence cache the nugget
// gather fills, with the position of the segment's last token, so that the attend kernels serve it unchanged.
// HBM-bound: every K and V row is read once, one row in r written.  One thread block per pooled row; a thread
// owns 16-byte pieces of the row, sums the segment's rows in token order in fp32 (four rows' loads in flight),
// divides by the segment's length and rounds once to the storage type.
#include "dodo_internal.cuh"

namespace {

constexpr int kPoolThreads = 128;

template <typename T> struct Pack16;
template <> struct Pack16<float> {
    static __device__ __forceinline__ uint4 pack(const float* f) {
        return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
    }
};
template <> struct Pack16<__nv_bfloat16> {
    static __device__ __forceinline__ uint32_t two(float lo, float hi) {
        const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&v);
    }
    static __device__ __forceinline__ uint4 pack(const float* f) {
        return make_uint4(two(f[0], f[1]), two(f[2], f[3]), two(f[4], f[5]), two(f[6], f[7]));
    }
};

template <typename T>
__global__ void __launch_bounds__(kPoolThreads)
pool_kernel(const unsigned char* __restrict__ K, const unsigned char* __restrict__ V, int row_vecs, int r,
            const __grid_constant__ PoolGroup g, unsigned char* __restrict__ cacheK, unsigned char* __restrict__ cacheV,
            int32_t* __restrict__ cache_pos) {
    constexpr int E = Vec16<T>::kElems;
    const int j = static_cast<int>(blockIdx.x);          // pooled row of the launch group
    int lo = 0, hi = g.nseq;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (g.out0[mid] <= j) lo = mid; else hi = mid;
    }
    const int b = lo;
    const int seg = j - g.out0[b];
    const int first = seg * r;
    const int cnt = min(r, g.n[b] - first);               // the last segment of a sequence may be shorter
    const size_t row_bytes = static_cast<size_t>(row_vecs) * 16u;
    const unsigned char* sk = K + (static_cast<size_t>(g.src_row0[b]) + first) * row_bytes;
    const unsigned char* sv = V + (static_cast<size_t>(g.src_row0[b]) + first) * row_bytes;
    const int dst_row = g.dst_row0[b] + seg;
    dodo_grid_dependency_sync();
    if (threadIdx.x == 0) cache_pos[dst_row] = g.pos_base[b] + first + cnt - 1;
    const float inv_den = static_cast<float>(cnt);
    for (int c = threadIdx.x; c < row_vecs; c += kPoolThreads) {
        float ak[E], av[E];
#pragma unroll
        for (int e = 0; e < E; ++e) { ak[e] = 0.f; av[e] = 0.f; }
        for (int i0 = 0; i0 < cnt; i0 += 4) {
            uint4 k4[4], v4[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (i0 + u < cnt) {
                    k4[u] = ld_stream16(sk + static_cast<size_t>(i0 + u) * row_bytes + static_cast<size_t>(c) * 16u);
                    v4[u] = ld_stream16(sv + static_cast<size_t>(i0 + u) * row_bytes + static_cast<size_t>(c) * 16u);
                }
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (i0 + u < cnt) {
                    float fk[E], fv[E];
                    Vec16<T>::unpack(k4[u], fk);
                    Vec16<T>::unpack(v4[u], fv);
#pragma unroll
                    for (int e = 0; e < E; ++e) { ak[e] += fk[e]; av[e] += fv[e]; }
                }
            }
        }
#pragma unroll
        for (int e = 0; e < E; ++e) { ak[e] /= inv_den; av[e] /= inv_den; }
        *reinterpret_cast<uint4*>(cacheK + static_cast<size_t>(dst_row) * row_bytes + static_cast<size_t>(c) * 16u) = Pack16<T>::pack(ak);
        *reinterpret_cast<uint4*>(cacheV + static_cast<size_t>(dst_row) * row_bytes + static_cast<size_t>(c) * 16u) = Pack16<T>::pack(av);
    }
}

}  // namespace

int dodo_launch_pool(dodo_ctx* ctx, const void* K, const void* V, int dtype, size_t row_bytes, int r, const PoolGroup& g,
                     void* cacheK, void* cacheV, int32_t* cache_pos, cudaStream_t st) {
    const int total = g.out0[g.nseq];
    if (total == 0) return DODO_OK;
    const unsigned char* k = static_cast<const unsigned char*>(K);
    const unsigned char* v = static_cast<const unsigned char*>(V);
    unsigned char* ck = static_cast<unsigned char*>(cacheK);
    unsigned char* cv = static_cast<unsigned char*>(cacheV);
    const int row_vecs = static_cast<int>(row_bytes / 16);
    const cudaError_t e = dtype == DODO_BF16
        ? dodo_launch_dependent(pool_kernel<__nv_bfloat16>, dim3(static_cast<unsigned>(total)), dim3(kPoolThreads), 0, st, k, v, row_vecs, r, g, ck, cv, cache_pos)
        : dodo_launch_dependent(pool_kernel<float>, dim3(static_cast<unsigned>(total)), dim3(kPoolThreads), 0, st, k, v, row_vecs, r, g, ck, cv, cache_pos);
    return dodo_check_cuda(ctx, e, "pool launch");
}
