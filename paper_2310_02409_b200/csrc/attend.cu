// Attention of query tokens over [nugget cache ; local tokens] (Eq. 4, Eq. 9, Eq. 13, Eq. 16):
// split-K flash-decode kernel, HBM-bound.
//
// One thread block serves (sequence, query tile of QT tokens, head, key chunk).  K and V tiles of a
// chunk are fetched by TMA tensor copies (one box per full tile, 16-row boxes for a ragged tail so
// that over-fetch past a segment's end stays below 16 rows; one elected thread per stage, mbarrier
// completion) into a ring of shared-memory stages; for decode every tile of the chunk is in flight
// at once.  Lanes are grouped LPR = (head_dim * elem_bytes / 16) per key row: each lane owns 16 bytes
// of the row, a dot product is a handful of FMAs plus a log2(LPR)-step butterfly.  The 256/LPR lane
// groups of a block are divided among the QT queries; the groups of one query take interleaved keys and
// keep private online-softmax states (running max, sum, fp32 accumulator), merged once at the end.
// With several chunks per (query, head) each block writes an unnormalised partial and takes a
// ticket; the block with the last ticket merges all partials (log-sum-exp) and writes O.
#include "dodo_internal.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kBoxRows = 16;          // rows per TMA box: bounds over-fetch past a segment's end
constexpr int kTileBytes = 16 * 1024; // one K (or V) tile
constexpr int kUnroll = 4;            // keys per lane group processed together
constexpr int kMaxStages = 6;
constexpr float kNeg = -1.0e30f;      // finite stand-in for -inf in running maxima
constexpr int kWaitPolls = 1 << 20;   // bound on barrier polls before giving up

template <typename T, int DH>
struct Cfg {
    static constexpr int E = 16 / sizeof(T);          // elements per lane
    static constexpr int LPR = DH / E;                // lanes per key row
    static constexpr int NG = kThreads / LPR;         // lane groups per block
    static constexpr int ROWB = DH * sizeof(T);       // bytes per key row of one head
    static constexpr int TK = kTileBytes / ROWB;      // keys per tile
    static constexpr int NBOX = TK / kBoxRows;
    static constexpr int BOXB = kBoxRows * ROWB;
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

__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

struct TileInfo {
    bool cache;       // nugget cache or local segment
    int row0;         // first global row of the tile
    int rows;         // rows of the tile that belong to the segment
    int pos0;         // position of local row 0 of the tile (local tiles)
};

template <typename T, int DH, int QT>
__global__ void __launch_bounds__(kThreads)
attend_kernel(const T* __restrict__ Q, const __grid_constant__ AttendMaps maps,
              const __grid_constant__ AttendGroup g, const int32_t* __restrict__ cache_pos, int H,
              float scale_log2, int nstage, T* __restrict__ O, float* __restrict__ lse,
              float* __restrict__ partials, int* __restrict__ tickets, int* __restrict__ dev_status) {
    using C = Cfg<T, DH>;
    constexpr int E = C::E, LPR = C::LPR, NG = C::NG, TK = C::TK, ROWB = C::ROWB;
    constexpr int G = NG / QT;  // lane groups (key subsets) per query
    static_assert(NG % QT == 0 && G >= 1, "query tile does not divide the lane groups");
    static_assert(TK % (G * kUnroll) == 0, "tile must split evenly over groups and unroll");

    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~static_cast<uintptr_t>(1023u));
    unsigned char* stage_mem = smem;                                       // nstage * 2 * kTileBytes
    int* kpos = reinterpret_cast<int*>(stage_mem + nstage * 2 * kTileBytes);  // [nstage][TK]
    float* red = reinterpret_cast<float*>(kpos + nstage * TK);             // [NG][DH + 2]
    __shared__ __align__(8) uint64_t bars[kMaxStages];
    __shared__ int s_flag;

    const int tid = threadIdx.x;
    const int gid = tid / LPR, lig = tid % LPR;
    const int qs = gid / G, kg = gid % G;

    // ---- which (sequence, query tile, head, chunk) ------------------------------------------
    const int bid = static_cast<int>(blockIdx.x);
    int b;
    if (g.uniform_ctas > 0) {
        b = bid / g.uniform_ctas;
    } else {
        b = 0;  // independent compares: the loads of cta0[] overlap instead of chaining
#pragma unroll 8
        for (int i = 1; i < DODO_GROUP; ++i) b += (i < g.nseq && g.cta0[i] <= bid) ? 1 : 0;
    }
    const AttendSeq sq = g.seq[b];
    int r = bid - g.cta0[b];
    const int nchunk = sq.nchunk;
    const int chunk = r % nchunk; r /= nchunk;
    const int h = r % H;
    const int qtile = r / H;
    const int q_first = qtile * QT;
    const int nq = min(QT, sq.tq - q_first);
    const int qpos_last = sq.q_pos0 + q_first + nq - 1;
    const int c_len = sq.c_len;
    const int l_pos0 = sq.l_pos0;
    const int l_vis = max(0, min(sq.l_len, qpos_last - l_pos0 + 1));  // local rows some query can see
    const int nt_c = (c_len + TK - 1) / TK;
    const int nt_l = (l_vis + TK - 1) / TK;
    const int t_begin = chunk * sq.ctiles;
    const int t_end = min(nt_c + nt_l, t_begin + sq.ctiles);
    const int my_tiles = max(0, t_end - t_begin);
    const int c_row0 = sq.c_row0, l_row0 = sq.l_row0;

    auto tile_info = [&](int it) -> TileInfo {
        const int t = t_begin + it;
        TileInfo ti;
        if (t < nt_c) {
            ti.cache = true; ti.row0 = c_row0 + t * TK; ti.rows = min(TK, c_len - t * TK); ti.pos0 = 0;
        } else {
            const int tl = t - nt_c;
            ti.cache = false; ti.row0 = l_row0 + tl * TK; ti.rows = min(TK, l_vis - tl * TK);
            ti.pos0 = l_pos0 + tl * TK;
        }
        return ti;
    };
    // one elected thread: arm the stage's barrier and launch the tile's K and V boxes
    auto issue_tile = [&](int it) {
        const int st = it % nstage;
        const TileInfo ti = tile_info(it);
        unsigned char* dk = stage_mem + st * 2 * kTileBytes;
        unsigned char* dv = dk + kTileBytes;
        const CUtensorMap* mk = ti.cache ? maps.cK : maps.lK;
        const CUtensorMap* mv = ti.cache ? maps.cV : maps.lV;
        if (ti.rows == TK) {
            mbar_expect_tx(&bars[st], static_cast<uint32_t>(2 * kTileBytes));
            tma_load_2d(dk, mk, h * DH, ti.row0, &bars[st]);
            tma_load_2d(dv, mv, h * DH, ti.row0, &bars[st]);
        } else {
            const int nbox = (ti.rows + kBoxRows - 1) / kBoxRows;
            mbar_expect_tx(&bars[st], static_cast<uint32_t>(nbox * C::BOXB * 2));
            for (int bx = 0; bx < nbox; ++bx) {
                tma_load_2d(dk + bx * C::BOXB, mk + 1, h * DH, ti.row0 + bx * kBoxRows, &bars[st]);
                tma_load_2d(dv + bx * C::BOXB, mv + 1, h * DH, ti.row0 + bx * kBoxRows, &bars[st]);
            }
        }
    };
    // all threads: positions of the tile's keys (INT_MAX marks rows outside the segment)
    auto fill_pos = [&](int it) {
        const int st = it % nstage;
        const TileInfo ti = tile_info(it);
        for (int j = tid; j < TK; j += kThreads) {
            int p = 0x7fffffff;
            if (j < ti.rows) p = ti.cache ? __ldg(cache_pos + ti.row0 + j) : ti.pos0 + j;
            kpos[st * TK + j] = p;
        }
    };

    // Stage s belongs to lane 0 of warp s: it initialises the stage's barrier and issues every copy
    // into it, so the first copies leave before the block's first __syncthreads.
    const int pre = min(nstage, my_tiles);
    const bool issuer = (tid & 31) == 0 && (tid >> 5) < nstage;
    if (issuer) {
        const int s = tid >> 5;
        mbar_init(&bars[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (s < pre) issue_tile(s);
    }
    for (int it = 0; it < pre; ++it) fill_pos(it);

    // ---- this lane group's query ------------------------------------------------------------
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
    __syncthreads();

    bool timed_out = false;
    for (int it = 0; it < my_tiles; ++it) {
        const int st = it % nstage;
        const uint32_t parity = static_cast<uint32_t>(it / nstage) & 1u;
        // warp-uniform outcome, so the shuffles below always see whole warps
        if (__any_sync(0xffffffffu, !mbar_wait(&bars[st], parity))) { timed_out = true; break; }
        const unsigned char* sK = stage_mem + st * 2 * kTileBytes;
        const unsigned char* sV = sK + kTileBytes;
        const int* kp = kpos + st * TK;
        const int rows = tile_info(it).rows;
        for (int base = 0; base < rows; base += G * kUnroll) {  // same trip count for every group
            const int j0 = base + kg;
            float s[kUnroll];
            bool ok[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int jj = j0 + u * G;
                ok[u] = kp[jj] <= my_qpos;
                float kf[E];
                Vec16<T>::unpack(*reinterpret_cast<const uint4*>(sK + jj * ROWB + lig * 16), kf);
                float d = 0.f;
#pragma unroll
                for (int e = 0; e < E; ++e) d = fmaf(qf[e], kf[e], d);
                s[u] = d;
            }
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) {
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) s[u] += __shfl_xor_sync(0xffffffffu, s[u], o);
            }
            float m_new = m;
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                s[u] = ok[u] ? s[u] : kNeg;
                m_new = fmaxf(m_new, s[u]);
            }
            const float corr = exp2f(m - m_new);
            m = m_new;
            l *= corr;
#pragma unroll
            for (int e = 0; e < E; ++e) acc[e] *= corr;
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                if (ok[u]) {
                    const float p = exp2f(s[u] - m_new);
                    l += p;
                    float vf[E];
                    Vec16<T>::unpack(*reinterpret_cast<const uint4*>(sV + (j0 + u * G) * ROWB + lig * 16), vf);
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[e] = fmaf(p, vf[e], acc[e]);
                }
            }
        }
        if (it + nstage < my_tiles) {
            __syncthreads();  // every group is done with this stage
            if (issuer && (tid >> 5) == st) issue_tile(it + nstage);
            fill_pos(it + nstage);
            __syncthreads();
        }
    }
    if (timed_out) {
        // give the copies in flight one more bounded chance to land, flag the failure, leave
        for (int s = 0; s < nstage; ++s) (void)mbar_try_wait(&bars[s], 0);
        if (tid == 0) atomicExch(dev_status, DODO_DEV_WAIT_TIMEOUT);
        return;
    }

    // ---- merge the lane groups of each query ------------------------------------------------
#pragma unroll
    for (int e = 0; e < E; ++e) red[gid * (DH + 2) + lig * E + e] = acc[e];
    if (lig == 0) { red[gid * (DH + 2) + DH] = m; red[gid * (DH + 2) + DH + 1] = l; }
    __syncthreads();

    const int qrow0 = sq.q_row0 + q_first;
    for (int i = tid; i < QT * DH; i += kThreads) {
        const int q2 = i / DH, dim = i % DH;
        if (q2 >= nq) continue;
        float M = kNeg;
#pragma unroll
        for (int gg = 0; gg < G; ++gg) M = fmaxf(M, red[(q2 * G + gg) * (DH + 2) + DH]);
        float L = 0.f, o = 0.f;
#pragma unroll
        for (int gg = 0; gg < G; ++gg) {
            const float* rg = red + (q2 * G + gg) * (DH + 2);
            const float wgt = exp2f(rg[DH] - M);
            L = fmaf(rg[DH + 1], wgt, L);
            o = fmaf(rg[dim], wgt, o);
        }
        const size_t orow = static_cast<size_t>(qrow0 + q2) * H + h;
        if (nchunk == 1) {
            store_out(O + orow * DH + dim, L > 0.f ? o / L : 0.f);
            if (lse != nullptr && dim == 0)
                lse[orow] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
        } else {
            float* pr = partials + (static_cast<size_t>(sq.part0) +
                                    (static_cast<size_t>(q_first + q2) * H + h) * nchunk + chunk) * (DH + 2);
            pr[dim] = o;
            if (dim == 0) { pr[DH] = M; pr[DH + 1] = L; }
        }
    }
    if (nchunk == 1) return;

    // ---- last chunk to arrive merges the partials of its (query tile, head) ------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        int* tk = tickets + sq.tick0 + qtile * H + h;
        const int t = atomicAdd(tk, 1);
        s_flag = (t == nchunk - 1);
        if (s_flag) *tk = 0;
    }
    __syncthreads();
    if (!s_flag) return;
    __threadfence();
    for (int i = tid; i < QT * DH; i += kThreads) {
        const int q2 = i / DH, dim = i % DH;
        if (q2 >= nq) continue;
        const float* pr = partials + (static_cast<size_t>(sq.part0) +
                                      (static_cast<size_t>(q_first + q2) * H + h) * nchunk) * (DH + 2);
        float M = kNeg;
        for (int c = 0; c < nchunk; ++c) M = fmaxf(M, __ldcg(pr + c * (DH + 2) + DH));
        float L = 0.f, o = 0.f;
        for (int c = 0; c < nchunk; ++c) {
            const float* pc = pr + c * (DH + 2);
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

template <typename T, int DH, int QT>
int launch_t(dodo_ctx* ctx, int H, float sm_scale, const AttendPlan& plan, const AttendGroup& g,
             const void* Q, const AttendMaps& maps, const int32_t* cache_pos, void* O, float* lse,
             float* partials, int* tickets, int* dev_status, cudaStream_t st) {
    using C = Cfg<T, DH>;
    const int nstage = plan.stages;
    const size_t smem = 1024 + static_cast<size_t>(nstage) * 2 * kTileBytes +
                        static_cast<size_t>(nstage) * C::TK * sizeof(int) +
                        static_cast<size_t>(C::NG) * (DH + 2) * sizeof(float);
    auto kern = attend_kernel<T, DH, QT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "attend shared-memory attribute");
    const float scale_log2 = sm_scale * 1.4426950408889634f;
    kern<<<g.cta0[g.nseq], kThreads, smem, st>>>(static_cast<const T*>(Q), maps, g, cache_pos, H, scale_log2,
                                                 nstage, static_cast<T*>(O), lse, partials, tickets, dev_status);
    return dodo_check_cuda(ctx, cudaGetLastError(), "attend launch");
}

template <typename T, int DH>
int launch_qt(dodo_ctx* ctx, int H, float sm_scale, const AttendPlan& plan, const AttendGroup& g,
              const void* Q, const AttendMaps& maps, const int32_t* cache_pos, void* O, float* lse,
              float* partials, int* tickets, int* dev_status, cudaStream_t st) {
    constexpr int NG = Cfg<T, DH>::NG;
    switch (plan.qt) {
        case 1: return launch_t<T, DH, 1>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
        case 2: return launch_t<T, DH, 2>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
        case 4: return launch_t<T, DH, 4>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
        case 8:
            if constexpr (NG >= 8)
                return launch_t<T, DH, 8>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, dev_status, st);
        default: break;
    }
    return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "attend: query tile %d not built for this dtype/head size", plan.qt);
}

}  // namespace

int dodo_attend_tile_keys(int dtype, int dh) { return kTileBytes / (dh * static_cast<int>(dodo_elem_bytes(dtype))); }
int dodo_attend_box_rows() { return kBoxRows; }
int dodo_attend_max_qt(int dtype, int dh) {
    const int ng = kThreads / (dh * static_cast<int>(dodo_elem_bytes(dtype)) / 16);
    return ng >= 8 ? 8 : ng;
}

int dodo_launch_attend(dodo_ctx* ctx, int dtype, int H, int dh, float sm_scale, const AttendPlan& plan,
                       const AttendGroup& g, const void* Q, const AttendMaps& maps,
                       const int32_t* cache_pos, void* O, float* lse, float* partials, int* tickets,
                       int* dev_status, cudaStream_t st) {
    if (g.cta0[g.nseq] == 0) return DODO_OK;
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
