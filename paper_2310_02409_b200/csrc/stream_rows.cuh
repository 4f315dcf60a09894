// Row streaming shared by the kernels of the compression step: the Scorer's dot product of two token rows
// against the weight vector (Eq. 6 / Eq. 15) and the copy of one token's K and V rows (Eq. 5).  Kernels that
// produce the same quantity go through the same code, so their results agree bit for bit.
#pragma once

#include "dodo_internal.cuh"

namespace dodo_rows {

// One warp, two token rows of nvec 16-byte pieces each (x1 == x0 when there is only one row): fp32 dot
// products with the weight vector in shared memory, four loads per row in flight per lane, butterfly
// reduction.  Every lane returns both sums.
template <typename T>
__device__ __forceinline__ void dot_two_rows(const uint4* __restrict__ x0, const uint4* __restrict__ x1,
                                             const uint4* sw, int nvec, int lane, float& out0, float& out1) {
    constexpr int E = Vec16<T>::kElems;
    float acc0 = 0.f, acc1 = 0.f;
    int c = lane;
    for (; c + 96 < nvec; c += 128) {
        uint4 a[4], bb[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { a[u] = ld_stream16(x0 + c + 32 * u); bb[u] = ld_stream16(x1 + c + 32 * u); }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            float fw[E], fa[E], fb[E];
            Vec16<T>::unpack(sw[c + 32 * u], fw);
            Vec16<T>::unpack(a[u], fa);
            Vec16<T>::unpack(bb[u], fb);
#pragma unroll
            for (int e = 0; e < E; ++e) { acc0 = fmaf(fa[e], fw[e], acc0); acc1 = fmaf(fb[e], fw[e], acc1); }
        }
    }
    for (; c < nvec; c += 32) {
        float fw[E], fa[E], fb[E];
        Vec16<T>::unpack(sw[c], fw);
        Vec16<T>::unpack(ld_stream16(x0 + c), fa);
        Vec16<T>::unpack(ld_stream16(x1 + c), fb);
#pragma unroll
        for (int e = 0; e < E; ++e) { acc0 = fmaf(fa[e], fw[e], acc0); acc1 = fmaf(fb[e], fw[e], acc1); }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        acc0 += __shfl_xor_sync(0xffffffffu, acc0, o);
        acc1 += __shfl_xor_sync(0xffffffffu, acc1, o);
    }
    out0 = acc0;
    out1 = acc1;
}

constexpr int kCopyVecs = 4;   // 16-byte loads in flight per thread and per tensor

// A team of nt threads (this one is number t) copies one K row and one V row of row_vecs 16-byte pieces each;
// all loads of a pass are issued before its first store.
__device__ __forceinline__ void copy_kv_row(const uint4* __restrict__ sk, const uint4* __restrict__ sv,
                                            uint4* __restrict__ dk, uint4* __restrict__ dv, int row_vecs, int t, int nt) {
    for (int c0 = 0; c0 < row_vecs; c0 += nt * kCopyVecs) {
        uint4 a[kCopyVecs], bb[kCopyVecs];
#pragma unroll
        for (int u = 0; u < kCopyVecs; ++u) {
            const int c = c0 + u * nt + t;
            if (c < row_vecs) { a[u] = ld_stream16(sk + c); bb[u] = ld_stream16(sv + c); }
        }
#pragma unroll
        for (int u = 0; u < kCopyVecs; ++u) {
            const int c = c0 + u * nt + t;
            if (c < row_vecs) { dk[c] = a[u]; dv[c] = bb[u]; }
        }
    }
}

}  // namespace dodo_rows
