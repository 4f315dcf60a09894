// Attention of query tokens over [nugget cache ; local tokens] (Eq. 4, Eq. 9, Eq. 13, Eq. 16):
// persistent, warp-specialised flash-decode kernel, HBM-bound.
//
// Work is the list of (unit, key tile) pairs, a unit being (sequence, query tile of QT tokens, head)
// and a tile 16 KB of K plus 16 KB of V (64 keys at bf16/head 128).  The list is cut into equal
// contiguous ranges, one per thread block (one block per SM), so every SM pulls the same number of
// bytes whatever the batch looks like ("stream-K" over keys).
//
//   producer warp   one lane walks the block's range and issues TMA tensor copies (one box per full
//                   tile, 16-row boxes for a segment's ragged tail, so over-fetch stays < 16 rows)
//                   into a ring of shared-memory stages; full/empty mbarriers per stage.
//   consumer warps  four groups of four warps; each group takes every fourth tile of the current
//                   unit.  Inside a group lanes are bundled LPR = head_dim*elem/16 per key row (one
//                   16-byte chunk each): a dot product is a few FMAs plus a log2(LPR)-step
//                   butterfly.  The 128/LPR bundles are divided among the QT queries; bundles of one
//                   query take interleaved keys and keep private online-softmax states in fp32.
//
// At the end of a unit (or of the block's range) all bundles are merged in shared memory.  A unit
// that lies wholly inside one block's range is normalised and written at once.  A unit cut by a
// range boundary leaves an unnormalised partial (one of two slots per block) and takes a ticket; the
// block that takes the unit's last ticket merges the partials by log-sum-exp and writes O.  No block
// waits for another.  Every wait on a copy barrier is bounded; on time-out the kernel records a status
// word and carries on to its end (results of that launch are then invalid).
#include "dodo_internal.cuh"

namespace {

constexpr int kGroups = 4;                       // consumer warp groups
constexpr int kGroupThreads = 128;
constexpr int kConsumers = kGroups * kGroupThreads;
constexpr int kThreads = kConsumers + 32;        // + producer warp
constexpr int kBoxRows = 16;
constexpr int kTileBytes = 16 * 1024;            // one K (or V) tile
constexpr int kUnroll = 4;                       // keys a bundle processes together
constexpr int kKeysPerBundle = 8;                // keys of a tile that one bundle owns (decode)
constexpr int kMaxStages = 6;
constexpr float kNeg = -1.0e30f;                 // finite stand-in for -inf in running maxima
constexpr int kWaitPolls = 1 << 20;

template <typename T, int DH>
struct Cfg {
    static constexpr int E = 16 / sizeof(T);             // elements per lane
    static constexpr int LPR = DH / E;                   // lanes per key row
    static constexpr int NGW = kGroupThreads / LPR;      // bundles per warp group
    static constexpr int ROWB = DH * sizeof(T);          // bytes per key row of one head
    static constexpr int TK = kTileBytes / ROWB;         // keys per tile
    static constexpr int BOXB = kBoxRows * ROWB;
    static constexpr int RED = DH + 2;                   // floats per bundle in the merge buffer
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false when the barrier did not complete within the poll budget.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (int i = 0; i < kWaitPolls; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}
// Barrier among the consumer warps only (the producer warp never joins it).
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsumers) : "memory"); }

__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// Where a global tile index falls: sequence, unit inside the sequence, tile inside the unit.
struct UnitRef {
    int b, ul, t;
};
__device__ __forceinline__ UnitRef locate(const AttendGroup& g, long long tile) {
    int b = 0;  // independent compares: the parameter loads overlap instead of chaining
#pragma unroll 8
    for (int i = 1; i < DODO_GROUP; ++i) b += (i < g.nseq && g.tile0[i] <= tile) ? 1 : 0;
    const int rel = static_cast<int>(tile - g.tile0[b]);
    const int tiles = g.seq[b].tiles;
    UnitRef u;
    u.b = b;
    u.ul = rel / tiles;
    u.t = rel - u.ul * tiles;
    return u;
}
// First tile of block c's range when `total` tiles are dealt to `n` blocks.
__device__ __forceinline__ long long range_begin(long long total, int n, int c) { return total * c / n; }
// The block whose range holds tile `tile`.
__device__ __forceinline__ int block_of(long long total, int n, long long tile) {
    return static_cast<int>(((tile + 1) * n + total - 1) / total) - 1;
}

struct TileSrc {
    bool cache;   // nugget cache or local segment
    int row0;     // first global row
    int rows;     // rows that belong to the segment and can be visible (<= 0: nothing to do)
    int pos0;     // position of the tile's first row (local tiles)
};
template <int TK>
__device__ __forceinline__ TileSrc tile_src(const AttendSeq& sq, int t, int l_vis) {
    const int nt_c = (sq.c_len + TK - 1) / TK;
    TileSrc s;
    if (t < nt_c) {
        s.cache = true; s.row0 = sq.c_row0 + t * TK; s.rows = min(TK, sq.c_len - t * TK); s.pos0 = 0;
    } else {
        const int tl = t - nt_c;
        s.cache = false; s.row0 = sq.l_row0 + tl * TK; s.rows = min(TK, l_vis - tl * TK);
        s.pos0 = sq.l_pos0 + tl * TK;
    }
    return s;
}
// Local rows that at least one query of the tile [q_first, q_first + nq) can see.
__device__ __forceinline__ int local_visible(const AttendSeq& sq, int q_first, int nq) {
    return max(0, min(sq.l_len, sq.q_pos0 + q_first + nq - 1 - sq.l_pos0 + 1));
}

template <typename T, int DH, int QT>
__global__ void __launch_bounds__(kThreads, 1)
attend_kernel(const T* __restrict__ Q, const __grid_constant__ AttendMaps maps,
              const __grid_constant__ AttendGroup g, const int32_t* __restrict__ cache_pos, int H,
              float scale_log2, int nstage, T* __restrict__ O, float* __restrict__ lse,
              float* __restrict__ partials, int* __restrict__ tickets, int* __restrict__ dev_status) {
    using C = Cfg<T, DH>;
    constexpr int E = C::E, LPR = C::LPR, NGW = C::NGW, TK = C::TK, ROWB = C::ROWB, RED = C::RED;
    constexpr int G = NGW / QT;  // bundles (key subsets) per query inside a warp group
    static_assert(NGW % QT == 0 && G >= 1, "query tile does not divide the bundles");
    static_assert(TK % (G * kUnroll) == 0, "tile must split evenly over bundles and unroll");
    static_assert(TK / NGW == kKeysPerBundle, "tile geometry");
    constexpr int KPB = TK / G;  // keys of a tile that one bundle visits

    extern __shared__ unsigned char smem_raw[];
    unsigned char* stage_mem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~static_cast<uintptr_t>(1023u));
    float* red = reinterpret_cast<float*>(stage_mem + nstage * 2 * kTileBytes);  // [kGroups*NGW][RED]
    __shared__ __align__(8) uint64_t full_bar[kMaxStages];
    __shared__ __align__(8) uint64_t empty_bar[kMaxStages];
    __shared__ int s_flag;

    const int tid = threadIdx.x;
    const int nblk = static_cast<int>(gridDim.x), blk = static_cast<int>(blockIdx.x);
    const long long total = g.tile0[g.nseq];
    const long long g0 = range_begin(total, nblk, blk), g1 = range_begin(total, nblk, blk + 1);
    const int ntile = static_cast<int>(g1 - g0);

    if (tid == kConsumers) {
        for (int s = 0; s < nstage; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], kGroupThreads / 32); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();

    // =========================================== producer =====================================
    if (tid >= kConsumers) {
        if (tid != kConsumers || ntile == 0) return;
        UnitRef u = locate(g, g0);
        bool stuck = false;
        for (int it = 0; it < ntile; ++it) {
            const int st = it % nstage;
            const AttendSeq& sq = g.seq[u.b];
            const int h = u.ul % H, qtile = u.ul / H;
            const int nq = min(QT, sq.tq - qtile * QT);
            const TileSrc ts = tile_src<TK>(sq, u.t, local_visible(sq, qtile * QT, nq));
            if (it >= nstage && !mbar_wait(&empty_bar[st], static_cast<uint32_t>(it / nstage - 1) & 1u)) stuck = true;
            unsigned char* dk = stage_mem + st * 2 * kTileBytes;
            unsigned char* dv = dk + kTileBytes;
            const CUtensorMap* mk = ts.cache ? maps.cK : maps.lK;
            const CUtensorMap* mv = ts.cache ? maps.cV : maps.lV;
            if (ts.rows == TK) {
                mbar_expect_tx(&full_bar[st], static_cast<uint32_t>(2 * kTileBytes));
                tma_load_2d(dk, mk, h * DH, ts.row0, &full_bar[st]);
                tma_load_2d(dv, mv, h * DH, ts.row0, &full_bar[st]);
            } else {
                const int nbox = ts.rows > 0 ? (ts.rows + kBoxRows - 1) / kBoxRows : 0;
                mbar_expect_tx(&full_bar[st], static_cast<uint32_t>(nbox * C::BOXB * 2));
                for (int bx = 0; bx < nbox; ++bx) {
                    tma_load_2d(dk + bx * C::BOXB, mk + 1, h * DH, ts.row0 + bx * kBoxRows, &full_bar[st]);
                    tma_load_2d(dv + bx * C::BOXB, mv + 1, h * DH, ts.row0 + bx * kBoxRows, &full_bar[st]);
                }
            }
            // next tile of the list
            if (++u.t == sq.tiles) {
                u.t = 0;
                if (++u.ul == sq.units) {
                    u.ul = 0;
                    do { ++u.b; } while (u.b < g.nseq && g.seq[u.b].units == 0);
                }
            }
        }
        if (stuck) atomicExch(dev_status, DODO_DEV_WAIT_TIMEOUT);
        return;
    }

    // =========================================== consumers ====================================
    const int wg = tid / kGroupThreads;                 // warp group
    const int gt = tid % kGroupThreads;                 // thread inside the group
    const int bundle = gt / LPR, lig = gt % LPR;        // bundle inside the group, lane inside the bundle
    const int qs = bundle / G, kg = bundle % G;         // query slot, key subset
    const int bundle_all = wg * NGW + bundle;
    bool stuck = false;

    long long cur = g0;
    while (cur < g1) {
        const UnitRef u = locate(g, cur);
        const AttendSeq sq = g.seq[u.b];
        const int h = u.ul % H, qtile = u.ul / H;
        const int q_first = qtile * QT;
        const int nq = min(QT, sq.tq - q_first);
        const int l_vis = local_visible(sq, q_first, nq);
        const long long unit_begin = cur - u.t, unit_end = unit_begin + sq.tiles;
        const long long seg_end = unit_end < g1 ? unit_end : g1;

        // this bundle's query, pre-scaled so that softmax runs in base 2
        const bool q_live = qs < nq;
        const int my_qpos = q_live ? sq.q_pos0 + q_first + qs : static_cast<int>(0x80000000);
        float qf[E];
        {
            uint4 qv = make_uint4(0, 0, 0, 0);
            if (q_live) {
                const size_t qrow = static_cast<size_t>(sq.q_row0 + q_first + qs) * H + h;
                qv = *reinterpret_cast<const uint4*>(Q + qrow * DH + lig * E);
            }
            Vec16<T>::unpack(qv, qf);
#pragma unroll
            for (int e = 0; e < E; ++e) qf[e] *= scale_log2;
        }
        float m = kNeg, l = 0.f, acc[E];
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] = 0.f;

        // Every group waits for every tile in list order, although it computes only every fourth:
        // a parity wait cannot tell phase k from phase k-2 of a stage's barrier, and a group that
        // skipped tiles could otherwise run a whole lap ahead of the copies.
        for (long long j = cur; j < seg_end; ++j) {
            const int it = static_cast<int>(j - g0);
            const int st = it % nstage;
            const bool mine = static_cast<int>((j - cur) % kGroups) == wg;
            const TileSrc ts = tile_src<TK>(sq, static_cast<int>(j - unit_begin), l_vis);
            // positions of this bundle's keys, fetched ahead of use (the first two rounds while the
            // tile is still in flight)
            auto load_pos = [&](int r, int* out) {
#pragma unroll
                for (int q = 0; q < kUnroll; ++q) {
                    const int jj = r * G * kUnroll + kg + q * G;
                    out[q] = 0x7fffffff;
                    if (jj < ts.rows) out[q] = ts.cache ? __ldg(cache_pos + ts.row0 + jj) : ts.pos0 + jj;
                }
            };
            int kp_now[kUnroll], kp_next[kUnroll];
            if (mine) {
                load_pos(0, kp_now);
                load_pos(1, kp_next);
            }
            if (__any_sync(0xffffffffu, !mbar_wait(&full_bar[st], static_cast<uint32_t>(it / nstage) & 1u))) stuck = true;
            if (!mine) continue;
            const unsigned char* sK = stage_mem + st * 2 * kTileBytes;
            const unsigned char* sV = sK + kTileBytes;
#pragma unroll
            for (int r = 0; r < KPB / kUnroll; ++r) {
                if (r * G * kUnroll < ts.rows) {  // same decision for every bundle of the group
                    const int j0 = r * G * kUnroll + kg;
                    float s[kUnroll];
                    bool ok[kUnroll];
#pragma unroll
                    for (int q = 0; q < kUnroll; ++q) {
                        const int jj = j0 + q * G;
                        ok[q] = kp_now[q] <= my_qpos;
                        float kf[E];
                        Vec16<T>::unpack(*reinterpret_cast<const uint4*>(sK + jj * ROWB + lig * 16), kf);
                        float d = 0.f;
#pragma unroll
                        for (int e = 0; e < E; ++e) d = fmaf(qf[e], kf[e], d);
                        s[q] = d;
                    }
#pragma unroll
                    for (int o = LPR / 2; o > 0; o >>= 1) {
#pragma unroll
                        for (int q = 0; q < kUnroll; ++q) s[q] += __shfl_xor_sync(0xffffffffu, s[q], o);
                    }
                    float m_new = m;
#pragma unroll
                    for (int q = 0; q < kUnroll; ++q) {
                        s[q] = ok[q] ? s[q] : kNeg;
                        m_new = fmaxf(m_new, s[q]);
                    }
                    const float corr = exp2f(m - m_new);
                    m = m_new;
                    l *= corr;
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[e] *= corr;
#pragma unroll
                    for (int q = 0; q < kUnroll; ++q) {
                        if (ok[q]) {
                            const float p = exp2f(s[q] - m_new);
                            l += p;
                            float vf[E];
                            Vec16<T>::unpack(*reinterpret_cast<const uint4*>(sV + (j0 + q * G) * ROWB + lig * 16), vf);
#pragma unroll
                            for (int e = 0; e < E; ++e) acc[e] = fmaf(p, vf[e], acc[e]);
                        }
                    }
#pragma unroll
                    for (int q = 0; q < kUnroll; ++q) kp_now[q] = kp_next[q];
                    if (r + 2 < KPB / kUnroll) load_pos(r + 2, kp_next);
                }
            }
            __syncwarp();
            if ((tid & 31) == 0) mbar_arrive(&empty_bar[st]);  // this warp is done with the stage
        }

        // ---- merge all bundles of each query ---------------------------------------------------
#pragma unroll
        for (int e = 0; e < E; ++e) red[bundle_all * RED + lig * E + e] = acc[e];
        if (lig == 0) { red[bundle_all * RED + DH] = m; red[bundle_all * RED + DH + 1] = l; }
        consumer_sync();

        const bool whole = (cur == unit_begin) && (seg_end == unit_end);
        const int qrow0 = sq.q_row0 + q_first;
        // partial slot of this block: 0 for a unit that began in an earlier block, 1 otherwise
        float* my_part = partials + (static_cast<size_t>(blk) * 2 + (unit_begin < g0 ? 0 : 1)) * QT * RED;
        for (int i = tid; i < QT * DH; i += kConsumers) {
            const int q2 = i / DH, dim = i % DH;
            if (q2 >= nq) continue;
            float M = kNeg;
            for (int w2 = 0; w2 < kGroups; ++w2)
#pragma unroll
                for (int gg = 0; gg < G; ++gg) M = fmaxf(M, red[(w2 * NGW + q2 * G + gg) * RED + DH]);
            float L = 0.f, o = 0.f;
            for (int w2 = 0; w2 < kGroups; ++w2)
#pragma unroll
                for (int gg = 0; gg < G; ++gg) {
                    const float* rg = red + (w2 * NGW + q2 * G + gg) * RED;
                    const float wgt = exp2f(rg[DH] - M);
                    L = fmaf(rg[DH + 1], wgt, L);
                    o = fmaf(rg[dim], wgt, o);
                }
            if (whole) {
                const size_t orow = static_cast<size_t>(qrow0 + q2) * H + h;
                store_out(O + orow * DH + dim, L > 0.f ? o / L : 0.f);
                if (lse != nullptr && dim == 0)
                    lse[orow] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
            } else {
                float* pr = my_part + q2 * RED;
                pr[dim] = o;
                if (dim == 0) { pr[DH] = M; pr[DH + 1] = L; }
            }
        }
        if (!whole) {
            // ---- the unit is shared with neighbouring blocks: last one to arrive writes O ----------
            const int first_blk = block_of(total, nblk, unit_begin);
            const int last_blk = block_of(total, nblk, unit_end - 1);
            __threadfence();
            consumer_sync();
            if (tid == 0) {
                int* tk = tickets + sq.unit0 + u.ul;
                const int t = atomicAdd(tk, 1);
                s_flag = (t == last_blk - first_blk);
                if (s_flag) *tk = 0;  // leave the counter clean for the next launch
            }
            consumer_sync();
            if (s_flag) {
                __threadfence();
                for (int i = tid; i < QT * DH; i += kConsumers) {
                    const int q2 = i / DH, dim = i % DH;
                    if (q2 >= nq) continue;
                    float M = kNeg;
                    for (int c = first_blk; c <= last_blk; ++c) {
                        const float* pc = partials + ((static_cast<size_t>(c) * 2 + (c == first_blk ? 1 : 0)) * QT + q2) * RED;
                        M = fmaxf(M, __ldcg(pc + DH));
                    }
                    float L = 0.f, o = 0.f;
                    for (int c = first_blk; c <= last_blk; ++c) {
                        const float* pc = partials + ((static_cast<size_t>(c) * 2 + (c == first_blk ? 1 : 0)) * QT + q2) * RED;
                        const float wgt = exp2f(__ldcg(pc + DH) - M);
                        L = fmaf(__ldcg(pc + DH + 1), wgt, L);
                        o = fmaf(__ldcg(pc + dim), wgt, o);
                    }
                    const size_t orow = static_cast<size_t>(qrow0 + q2) * H + h;
                    store_out(O + orow * DH + dim, L > 0.f ? o / L : 0.f);
                    if (lse != nullptr && dim == 0)
                        lse[orow] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
                }
            }
        }
        consumer_sync();  // the merge buffer and s_flag are free again
        cur = seg_end;
    }
    if (stuck && (tid & 31) == 0) atomicExch(dev_status, DODO_DEV_WAIT_TIMEOUT);
}

template <typename T, int DH, int QT>
int launch_t(dodo_ctx* ctx, int H, float sm_scale, const AttendPlan& plan, const AttendGroup& g,
             const void* Q, const AttendMaps& maps, const int32_t* cache_pos, void* O, float* lse,
             float* partials, int* tickets, int* dev_status, cudaStream_t st) {
    using C = Cfg<T, DH>;
    const int nstage = plan.stages;
    const size_t smem = 1024 + static_cast<size_t>(nstage) * 2 * kTileBytes +
                        static_cast<size_t>(kGroups) * C::NGW * C::RED * sizeof(float);
    auto kern = attend_kernel<T, DH, QT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "attend shared-memory attribute");
    const float scale_log2 = sm_scale * 1.4426950408889634f;
    kern<<<g.nblocks, kThreads, smem, st>>>(static_cast<const T*>(Q), maps, g, cache_pos, H, scale_log2, nstage,
                                            static_cast<T*>(O), lse, partials, tickets, dev_status);
    return dodo_check_cuda(ctx, cudaGetLastError(), "attend launch");
}

template <typename T, int DH>
int launch_qt(dodo_ctx* ctx, int H, float sm_scale, const AttendPlan& plan, const AttendGroup& g,
              const void* Q, const AttendMaps& maps, const int32_t* cache_pos, void* O, float* lse,
              float* partials, int* tickets, int* dev_status, cudaStream_t st) {
    constexpr int NGW = Cfg<T, DH>::NGW;
    switch (plan.qt) {
        case 1: return launch_t<T, DH, 1>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
        case 2: return launch_t<T, DH, 2>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
        case 4: return launch_t<T, DH, 4>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
        case 8:
            if constexpr (NGW >= 8)
                return launch_t<T, DH, 8>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
            break;
        default: break;
    }
    return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "attend: query tile %d not built for this dtype/head size", plan.qt);
}

}  // namespace

int dodo_attend_tile_keys(int dtype, int dh) { return kTileBytes / (dh * static_cast<int>(dodo_elem_bytes(dtype))); }
int dodo_attend_box_rows() { return kBoxRows; }
int dodo_attend_max_qt(int dtype, int dh) {
    const int ngw = kGroupThreads / (dh * static_cast<int>(dodo_elem_bytes(dtype)) / 16);
    return ngw >= 8 ? 8 : ngw;
}
int dodo_attend_max_stages() { return kMaxStages; }

int dodo_launch_attend(dodo_ctx* ctx, int dtype, int H, int dh, float sm_scale, const AttendPlan& plan,
                       const AttendGroup& g, const void* Q, const AttendMaps& maps,
                       const int32_t* cache_pos, void* O, float* lse, float* partials, int* tickets,
                       int* dev_status, cudaStream_t st) {
    if (g.nblocks == 0) return DODO_OK;
    if (plan.stages < 1 || plan.stages > kMaxStages)
        return dodo_fail(ctx, DODO_ERR_INVALID_ARG, "attend: %d stages out of range", plan.stages);
    if (dtype == DODO_BF16 && dh == 128)
        return launch_qt<__nv_bfloat16, 128>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
    if (dtype == DODO_BF16 && dh == 64)
        return launch_qt<__nv_bfloat16, 64>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
    if (dtype == DODO_F32 && dh == 128)
        return launch_qt<float, 128>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
    if (dtype == DODO_F32 && dh == 64)
        return launch_qt<float, 64>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
    return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "attend: dtype %d with head size %d", dtype, dh);
}
