// Attention of query tokens over [nugget cache ; local tokens] (Eq. 4, Eq. 9, Eq. 13, Eq. 16):
// split-K flash-decode kernel, HBM-bound.
//
// One thread block serves (sequence, query tile of QT tokens, head, key chunk).  Keys stream straight
// from global memory into registers -- no shared-memory staging: lanes are bundled LPR =
// head_dim*elem/16 per key row, each lane owning one 16-byte piece of the row, so a bundle reads a
// head's K (or V) row as one coalesced segment.  The bundles of a block take interleaved keys; a
// bundle issues the K and V loads of U keys at once and always keeps the next batch in flight while
// it reduces the current one (2*U to 4*U 16-byte loads outstanding per lane, which is what keeps HBM
// busy with only a few hundred threads per SM); for each of the QT queries it forms
// the dot products (a few FMAs plus a log2(LPR)-step butterfly), masks by position and updates a
// private online-softmax state (running max, sum, fp32 accumulator).  At the end the bundles are
// merged in shared memory.  Without split the block normalises and writes O; with several chunks per
// (query tile, head) it writes an unnormalised partial and takes a ticket, and the block holding the
// last ticket merges the partials by log-sum-exp.  No block waits for another.
#include "dodo_internal.cuh"
#include <type_traits>

namespace {

constexpr int kThreads = 256;
constexpr int kGranule = 8;           // keys per bundle in one planning granule ("tile")
constexpr int kMaxCluster = 8;        // portable cluster size: most chunks that merge in shared memory
constexpr int kPrefetchKeys = 32;     // rows at the end of a block's key list requested into L2 ahead of the dependency wait
constexpr float kNeg = -1.0e30f;      // finite stand-in for -inf in running maxima

template <typename T, int DH>
struct Cfg {
    static constexpr int E = 16 / sizeof(T);          // elements per lane
    static constexpr int LPR = DH / E;                // lanes per key row
    static constexpr int NB = kThreads / LPR;         // bundles per block
    static constexpr int RED = DH + 2;                // floats per (bundle, query) in the merge buffer
};

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ void store_out(float* p, float v) { *p = v; }
__device__ __forceinline__ void store_out(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

template <typename T, int DH, int QT, int U, bool kClustered>
__global__ void __launch_bounds__(kThreads)
attend_kernel(const T* __restrict__ Q, const AttendMaps src, const __grid_constant__ AttendGroup g,
              const int32_t* __restrict__ cache_pos, int H, float scale_log2, T* __restrict__ O,
              float* __restrict__ lse, float* __restrict__ partials, int* __restrict__ tickets, int early_cache) {
    using C = Cfg<T, DH>;
    constexpr int E = C::E, LPR = C::LPR, NB = C::NB, RED = C::RED;
    constexpr int TK = NB * kGranule;  // keys per planning granule

    extern __shared__ __align__(16) float red[];  // [NB][QT][RED]
    __shared__ int s_flag;

    const int tid = threadIdx.x;
    const int bundle = tid / LPR, lig = tid % LPR;
    // Clustered split: the chunks of a (query tile, head) are the thread blocks of one cluster and merge in
    // the shared memory of the cluster's first block.  Every block reports here that it has started; the
    // matching wait stands before the first store into another block's shared memory.
    constexpr bool clustered = kClustered;   // (launched with the cluster size g.cluster as an attribute)
    if (clustered) asm volatile("barrier.cluster.arrive.relaxed;" ::: "memory");

    // ---- which (sequence, query tile, head, chunk) ------------------------------------------
    const int bid = static_cast<int>(blockIdx.x);
    int b;
    if (g.uniform_ctas > 0) {
        b = bid / g.uniform_ctas;
    } else {
        b = 0;  // independent compares: the parameter loads overlap instead of chaining
#pragma unroll 8
        for (int i = 1; i < DODO_GROUP; ++i) b += (i < g.nseq && g.cta0[i] <= bid) ? 1 : 0;
    }
    const AttendSeq sq = g.seq[b];
    int r0 = bid - g.cta0[b];
    const int nchunk = sq.nchunk;
    const int chunk = r0 % nchunk; r0 /= nchunk;
    const int h = r0 % H;
    const int qtile = r0 / H;
    const int q_first = qtile * QT;
    const int nq = min(QT, sq.tq - q_first);
    // local rows that at least one query of the tile can see
    const int l_vis = max(0, min(sq.l_len, sq.q_pos0 + q_first + nq - 1 - sq.l_pos0 + 1));
    // this chunk's slice of the key list [nuggets ; local], in granules of TK keys per segment
    const int nt_c = (sq.c_len + TK - 1) / TK;
    const int t_begin = chunk * sq.ctiles, t_end = t_begin + sq.ctiles;
    const int c_begin = min(sq.c_len, t_begin * TK), c_end = min(sq.c_len, t_end * TK);
    const int l_begin = min(l_vis, max(0, t_begin - nt_c) * TK), l_end = min(l_vis, max(0, t_end - nt_c) * TK);

    const size_t row_elems = static_cast<size_t>(H) * DH;
    const size_t col = static_cast<size_t>(h) * DH + lig * E;

    // The chunk's keys as one list: first its nuggets (position from cache_pos), then its local
    // tokens (consecutive positions).  Batches of NB*U keys are software-pipelined: the loads of the
    // next batch are in flight while the current one is being reduced.
    const int n_c = c_end - c_begin, n_tot = n_c + (l_end - l_begin);
    const int c_row = sq.c_row0 + c_begin, l_row = sq.l_row0 + l_begin, l_pos = sq.l_pos0 + l_begin;
    const T* const cK = static_cast<const T*>(src.cK);
    const T* const cV = static_cast<const T*>(src.cV);
    const T* const lK = static_cast<const T*>(src.lK);
    const T* const lV = static_cast<const T*>(src.lV);

    // A ragged end of at most one key per bundle does not get a round trip of its own at the end of the
    // pipeline: it travels in a register set of one key, requested together with the first two batches.
    constexpr int kBatch = NB * U;
    const int r_tail = n_tot % kBatch;
    const bool has_tail = r_tail > 0 && r_tail <= NB && n_tot > 2 * kBatch;
    const int n_main = has_tail ? n_tot - r_tail : n_tot;
    // A batch that lies wholly in the nugget cache or wholly in the local segment needs no per-key bounds or
    // segment tests: one row pointer per operand and a fixed stride between the bundle's keys.  Batches at a
    // boundary take the general path.  (All of this is uniform over the block.)
    const size_t stride = static_cast<size_t>(NB) * row_elems;
    auto load_batch = [&](int base, uint4* kv, uint4* vv, int* kp) {
        if (base + NB * U <= n_c || (base >= n_c && base + NB * U <= n_main)) {
            const bool cached = base < n_c;
            const int j0 = base + bundle;
            const int row0 = cached ? c_row + j0 : l_row + (j0 - n_c);
            const T* pk = (cached ? cK : lK) + static_cast<size_t>(row0) * row_elems + col;
            const T* pv = (cached ? cV : lV) + static_cast<size_t>(row0) * row_elems + col;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                kv[u] = ld_stream16(pk + u * stride);
                vv[u] = ld_stream16(pv + u * stride);
            }
            if (cached) {
#pragma unroll
                for (int u = 0; u < U; ++u) kp[u] = __ldg(cache_pos + row0 + u * NB);
            } else {
#pragma unroll
                for (int u = 0; u < U; ++u) kp[u] = l_pos + (j0 - n_c) + u * NB;
            }
            return;
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int j = base + u * NB + bundle;
            kp[u] = 0x7fffffff;
            kv[u] = make_uint4(0, 0, 0, 0);
            vv[u] = make_uint4(0, 0, 0, 0);
            if (j < n_main) {
                const bool cached = j < n_c;
                const int row = cached ? c_row + j : l_row + (j - n_c);
                const size_t off = static_cast<size_t>(row) * row_elems + col;
                kv[u] = ld_stream16((cached ? cK : lK) + off);
                vv[u] = ld_stream16((cached ? cV : lV) + off);
                kp[u] = cached ? __ldg(cache_pos + row) : l_pos + (j - n_c);
            }
        }
    };
    // Programmatic dependent launch: this grid may start while the kernel before it on the stream is still
    // finishing, and nothing that kernel wrote is guaranteed visible before griddepcontrol.wait returns.
    // early_cache says that nothing directly before this launch writes the nugget cache (the host knows: the
    // launch before was an attend, which never does); only then are the first two batches of cache rows
    // requested ahead of the wait, so that they stream in while the previous kernel drains.  Otherwise (the
    // launch follows a gather, or anything unknown) the same rows only get a hint to L2 there and are loaded
    // after the wait.  Queries, local tokens and every output are touched only after the wait, in plain
    // stream order; the successor is released after the wait, so it overlaps this kernel and nothing earlier.
    uint4 kA[U], vA[U], kB[U], vB[U], kT[1], vT[1];
    int pA[U], pB[U], pT[1];
    auto load_tail = [&]() {
        const int j = n_main + bundle;
        pT[0] = 0x7fffffff;
        kT[0] = make_uint4(0, 0, 0, 0);
        vT[0] = make_uint4(0, 0, 0, 0);
        if (has_tail && j < n_tot) {
            const bool cached = j < n_c;
            const int row = cached ? c_row + j : l_row + (j - n_c);
            const size_t off = static_cast<size_t>(row) * row_elems + col;
            kT[0] = ld_stream16((cached ? cK : lK) + off);
            vT[0] = ld_stream16((cached ? cV : lV) + off);
            pT[0] = cached ? __ldg(cache_pos + row) : l_pos + (j - n_c);
        }
    };
    // Hints to L2 for the K and V rows of keys [j0, j1) of this block's list.  Legal before the wait whoever
    // writes the lines: L2 is the point of coherence, so a later write by the predecessor lands in the same
    // lines, and a hint reads nothing into this SM.
    constexpr int kLinesPerRow = DH * static_cast<int>(sizeof(T)) / 128;
    auto hint_rows = [&](int j0, int j1) {
        const int nl = max(0, j1 - j0);
        constexpr int kPerKey = kLinesPerRow * 2;   // a key's lines: its K row's, then its V row's (divisions by constants)
        for (int i = tid; i < nl * kPerKey; i += kThreads) {
            const int j = j0 + i / kPerKey, which = (i % kPerKey) / kLinesPerRow, part = i % kLinesPerRow;
            const bool cached = j < n_c;
            const T* base = cached ? (which ? cV : cK) : (which ? lV : lK);
            const int row = cached ? c_row + j : l_row + (j - n_c);
            const char* line = reinterpret_cast<const char*>(base + static_cast<size_t>(row) * row_elems + static_cast<size_t>(h) * DH) + part * 128;
            asm volatile("prefetch.global.L2 [%0];" :: "l"(line));
        }
    };
    // Ahead of the wait: (1) the query rows; (2) the last kPrefetchKeys keys of this block's list -- the rows
    // its final batch will ask for, local tokens included -- so that the end of the block's chain hits L2
    // (more than that loses: the hints compete with the predecessor's own last loads); (3) when the first two
    // batches may not be loaded yet, their rows.
    if (tid < QT * kLinesPerRow && tid / kLinesPerRow < nq) {
        const size_t qrow = static_cast<size_t>(sq.q_row0 + q_first + tid / kLinesPerRow) * H + h;
        const char* line = reinterpret_cast<const char*>(Q + qrow * DH) + (tid % kLinesPerRow) * 128;
        asm volatile("prefetch.global.L2 [%0];" :: "l"(line));
    }
    hint_rows(max(n_tot - kPrefetchKeys, min(n_c, 2 * kBatch)), n_tot);
    if (!early_cache) hint_rows(0, min(n_c, 2 * kBatch));
    const bool earlyA = early_cache && n_c >= kBatch, earlyB = early_cache && n_c >= 2 * kBatch;   // batch lies wholly in the cache
    const bool earlyT = early_cache && n_c >= n_tot;
    if (earlyA) load_batch(0, kA, vA, pA);
    if (earlyB) load_batch(kBatch, kB, vB, pB);
    if (earlyT) load_tail();
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (!earlyA) load_batch(0, kA, vA, pA);
    if (!earlyB) load_batch(kBatch, kB, vB, pB);
    if (!earlyT) load_tail();
    if constexpr (!kClustered) {
        // The third and fourth batch are asked for now (hints to L2) rather than after the first batch has been
        // reduced, so that HBM has requests during the query load and the first reduction.  Not in the cluster
        // form: its launches are one wave of blocks in step, always streaming, and the hints only cost issue slots.
        hint_rows(2 * kBatch, min(n_tot - kPrefetchKeys, 4 * kBatch));
    }

    // ---- the queries, pre-scaled so that softmax runs in base 2 --------------------------------
    float qf[QT][E];
    int qpos[QT];
#pragma unroll
    for (int qi = 0; qi < QT; ++qi) {
        uint4 qv = make_uint4(0, 0, 0, 0);
        qpos[qi] = static_cast<int>(0x80000000);  // a dead slot sees nothing
        if (qi < nq) {
            const size_t qrow = static_cast<size_t>(sq.q_row0 + q_first + qi) * H + h;
            qv = *reinterpret_cast<const uint4*>(Q + qrow * DH + lig * E);
            qpos[qi] = sq.q_pos0 + q_first + qi;
        }
        Vec16<T>::unpack(qv, qf[qi]);
#pragma unroll
        for (int e = 0; e < E; ++e) qf[qi][e] *= scale_log2;
    }
    float m[QT], l[QT], acc[QT][E];
#pragma unroll
    for (int qi = 0; qi < QT; ++qi) {
        m[qi] = kNeg; l[qi] = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) acc[qi][e] = 0.f;
    }


    // Packed fp32 pairs (fma.rn.f32x2): element pairs (2i, 2i+1) of a 16-byte piece share one FMA.
    auto reduce_n = [&](auto count, const uint4* kv, const uint4* vv, const int* kp) {
        constexpr int N = decltype(count)::value;   // keys per bundle in this batch
#pragma unroll
        for (int qi = 0; qi < QT; ++qi) {
            float s[N];
            bool allvis = true;
#pragma unroll
            for (int u = 0; u < N; ++u) {
                float kf[E];
                Vec16<T>::unpack(kv[u], kf);
                float2 d2 = make_float2(0.f, 0.f);
#pragma unroll
                for (int e = 0; e < E; e += 2)
                    d2 = __ffma2_rn(make_float2(qf[qi][e], qf[qi][e + 1]), make_float2(kf[e], kf[e + 1]), d2);
                s[u] = d2.x + d2.y;
                allvis = allvis && kp[u] <= qpos[qi];
            }
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) {
#pragma unroll
                for (int u = 0; u < N; ++u) s[u] += __shfl_xor_sync(0xffffffffu, s[u], o);
            }
            // whole warp sees every key of the batch (the usual case in decode): no per-key selects
            const bool fast = __all_sync(0xffffffffu, allvis);
            float m_new = m[qi];
#pragma unroll
            for (int u = 0; u < N; ++u) {
                if (!fast) s[u] = kp[u] <= qpos[qi] ? s[u] : kNeg;
                m_new = fmaxf(m_new, s[u]);
            }
            const float corr = ex2_approx(m[qi] - m_new);
            m[qi] = m_new;
            l[qi] *= corr;
            const float2 c2 = make_float2(corr, corr);
#pragma unroll
            for (int e = 0; e < E; e += 2) {
                const float2 a2 = __fmul2_rn(make_float2(acc[qi][e], acc[qi][e + 1]), c2);
                acc[qi][e] = a2.x; acc[qi][e + 1] = a2.y;
            }
            if (fast) {
#pragma unroll
                for (int u = 0; u < N; ++u) {
                    const float p = ex2_approx(s[u] - m_new);
                    l[qi] += p;
                    float vf[E];
                    Vec16<T>::unpack(vv[u], vf);
                    const float2 p2 = make_float2(p, p);
#pragma unroll
                    for (int e = 0; e < E; e += 2) {
                        const float2 a2 = __ffma2_rn(p2, make_float2(vf[e], vf[e + 1]), make_float2(acc[qi][e], acc[qi][e + 1]));
                        acc[qi][e] = a2.x; acc[qi][e + 1] = a2.y;
                    }
                }
            } else {
#pragma unroll
                for (int u = 0; u < N; ++u) {
                    // a masked key contributes exactly nothing (its V row may hold anything)
                    const bool vis = kp[u] <= qpos[qi];
                    const float p = vis ? ex2_approx(s[u] - m_new) : 0.f;
                    l[qi] += p;
                    float vf[E];
                    Vec16<T>::unpack(vv[u], vf);
#pragma unroll
                    for (int e = 0; e < E; ++e) acc[qi][e] = vis ? fmaf(p, vf[e], acc[qi][e]) : acc[qi][e];
                }
            }
        }
    };
    auto reduce_batch = [&](const uint4* kv, const uint4* vv, const int* kp) {
        reduce_n(std::integral_constant<int, U>(), kv, vv, kp);
    };
    for (int base = 0; base < n_main; base += 2 * kBatch) {
        reduce_batch(kA, vA, pA);
        load_batch(base + 2 * kBatch, kA, vA, pA);
        if (base + kBatch < n_main) reduce_batch(kB, vB, pB);
        load_batch(base + 3 * kBatch, kB, vB, pB);
    }
    if (has_tail) reduce_n(std::integral_constant<int, 1>(), kT, vT, pT);

    // ---- merge the bundles of each query -------------------------------------------------------
#pragma unroll
    for (int qi = 0; qi < QT; ++qi) {
        float* rb = red + (bundle * QT + qi) * RED;
#pragma unroll
        for (int e = 0; e < E; ++e) rb[lig * E + e] = acc[qi][e];
        if (lig == 0) { rb[DH] = m[qi]; rb[DH + 1] = l[qi]; }
    }
    __syncthreads();

    // merge of up to eight partial results at a time, all of their loads in flight together (the merge is
    // the tail of a launch): part(c, i) = float i of chunk c's record [DH values, maximum, sum]
    auto merge_chunks = [&](auto part, int dim, float& M, float& L, float& o) {
        M = kNeg; L = 0.f; o = 0.f;
        for (int c0 = 0; c0 < nchunk; c0 += 8) {
            float mv[8], lv[8], ov[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const bool live = c0 + u < nchunk;
                mv[u] = live ? part(c0 + u, DH) : kNeg;
                lv[u] = live ? part(c0 + u, DH + 1) : 0.f;
                ov[u] = live ? part(c0 + u, dim) : 0.f;
            }
            float M_new = M;
#pragma unroll
            for (int u = 0; u < 8; ++u) M_new = fmaxf(M_new, mv[u]);
            const float corr = ex2_approx(M - M_new);
            M = M_new;
            L *= corr;
            o *= corr;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const float wgt = ex2_approx(mv[u] - M);
                L = fmaf(lv[u], wgt, L);
                o = fmaf(ov[u], wgt, o);
            }
        }
    };

    float* const xred = red + NB * QT * RED;   // [chunk][QT][RED], used in the cluster's first block only
    uint32_t xred0 = 0;                        // ... and its address there, in the cluster's window
    if (clustered) {
        asm volatile("barrier.cluster.wait;" ::: "memory");
        asm("mapa.shared::cluster.u32 %0, %1, %2;"
            : "=r"(xred0) : "r"(static_cast<uint32_t>(__cvta_generic_to_shared(xred))), "r"(0));
    }
    const int qrow0 = sq.q_row0 + q_first;
    for (int i = tid; i < QT * DH; i += kThreads) {
        const int q2 = i / DH, dim = i % DH;
        if (q2 >= nq) continue;
        float M = kNeg;
#pragma unroll
        for (int bb = 0; bb < NB; ++bb) M = fmaxf(M, red[(bb * QT + q2) * RED + DH]);
        float L = 0.f, o = 0.f;
#pragma unroll
        for (int bb = 0; bb < NB; ++bb) {
            const float* rg = red + (bb * QT + q2) * RED;
            const float wgt = ex2_approx(rg[DH] - M);   // (arguments <= 0; a bundle that saw nothing has l = 0 and o = 0)
            L = fmaf(rg[DH + 1], wgt, L);
            o = fmaf(rg[dim], wgt, o);
        }
        const size_t orow = static_cast<size_t>(qrow0 + q2) * H + h;
        if (nchunk == 1) {
            store_out(O + orow * DH + dim, L > 0.f ? o / L : 0.f);
            if (lse != nullptr && dim == 0)
                lse[orow] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
        } else if (clustered) {
            const uint32_t rec = xred0 + static_cast<uint32_t>(((chunk * QT + q2) * RED) * sizeof(float));
            asm volatile("st.shared::cluster.f32 [%0], %1;" :: "r"(rec + dim * 4u), "f"(o) : "memory");
            if (dim == 0) {
                asm volatile("st.shared::cluster.f32 [%0], %1;" :: "r"(rec + DH * 4u), "f"(M) : "memory");
                asm volatile("st.shared::cluster.f32 [%0], %1;" :: "r"(rec + (DH + 1) * 4u), "f"(L) : "memory");
            }
        } else {
            float* pr = partials + (static_cast<size_t>(sq.part0) +
                                    (static_cast<size_t>(q_first + q2) * H + h) * nchunk + chunk) * RED;
            pr[dim] = o;
            if (dim == 0) { pr[DH] = M; pr[DH + 1] = L; }
        }
    }
    if (nchunk == 1) return;

    auto write_out = [&](int q2, int dim, float M, float L, float o) {
        const size_t orow = static_cast<size_t>(qrow0 + q2) * H + h;
        store_out(O + orow * DH + dim, L > 0.f ? o / L : 0.f);
        if (lse != nullptr && dim == 0)
            lse[orow] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
    };
    if (clustered) {
        // the stores above are released by the arrival; the first block acquires them and merges.  A block
        // that has arrived may exit: the wait counts only blocks still running.
        asm volatile("barrier.cluster.arrive.release;" ::: "memory");
        if (chunk != 0) return;
        asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
        for (int i = tid; i < QT * DH; i += kThreads) {
            const int q2 = i / DH, dim = i % DH;
            if (q2 >= nq) continue;
            float M, L, o;
            merge_chunks([&](int c, int f) { return xred[(c * QT + q2) * RED + f]; }, dim, M, L, o);
            write_out(q2, dim, M, L, o);
        }
        return;
    }

    // ---- last chunk to arrive merges the partials of its (query tile, head) ------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        int* tk = tickets + sq.tick0 + qtile * H + h;
        const int t = atomicAdd(tk, 1);
        s_flag = (t == nchunk - 1);
        if (s_flag) *tk = 0;  // leave the counter clean for the next launch
    }
    __syncthreads();
    if (!s_flag) return;
    __threadfence();
    for (int i = tid; i < QT * DH; i += kThreads) {
        const int q2 = i / DH, dim = i % DH;
        if (q2 >= nq) continue;
        const float* pr = partials + (static_cast<size_t>(sq.part0) +
                                      (static_cast<size_t>(q_first + q2) * H + h) * nchunk) * RED;
        float M, L, o;
        merge_chunks([&](int c, int f) { return __ldcg(pr + c * RED + f); }, dim, M, L, o);
        write_out(q2, dim, M, L, o);
    }
}

template <typename T, int DH, int QT>
constexpr size_t attend_smem(bool clustered) {
    return static_cast<size_t>(Cfg<T, DH>::NB + (clustered ? kMaxCluster : 0)) * QT * Cfg<T, DH>::RED * sizeof(float);
}

// Clusters of 2..kMaxCluster blocks of this kernel that the device holds at once (occupancy calculator).
template <typename T, int DH, int QT, int U>
void cluster_cap_t(int* cap) {
    auto kern = attend_kernel<T, DH, QT, U, true>;
    const size_t smem = attend_smem<T, DH, QT>(true);
    cap[0] = cap[1] = 0;
    if (smem > 40 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) {
        (void)cudaGetLastError();
        for (int c = 2; c <= kMaxCluster; ++c) cap[c] = 0;
        return;
    }
    for (int c = 2; c <= kMaxCluster; ++c) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(c * 64));
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = static_cast<unsigned>(c);
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) { (void)cudaGetLastError(); n = 0; }
        cap[c] = n;
    }
}

template <typename T, int DH, int QT, int U, bool kClustered>
int launch_k(dodo_ctx* ctx, int H, float sm_scale, const AttendGroup& g, const void* Q, const AttendMaps& src,
             const int32_t* cache_pos, void* O, float* lse, float* partials, int* tickets, bool early, cudaStream_t st) {
    using C = Cfg<T, DH>;
    const size_t smem = attend_smem<T, DH, QT>(kClustered);
    auto kern = attend_kernel<T, DH, QT, U, kClustered>;
    if (smem > 40 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "attend shared-memory attribute");
    }
    const float scale_log2 = sm_scale * 1.4426950408889634f;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(g.cta0[g.nseq]));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (kClustered) {      // the grid is a whole number of clusters: every sequence owns (units x chunks) blocks
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = static_cast<unsigned>(g.cluster);
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
    }
    const cudaError_t le = cudaLaunchKernelEx(&cfg, kern, static_cast<const T*>(Q), src, g, cache_pos, H, scale_log2,
                                              static_cast<T*>(O), lse, partials, tickets, early ? 1 : 0);
    return dodo_check_cuda(ctx, le, "attend launch");
}

template <typename T, int DH, int QT, int U>
int launch_t(dodo_ctx* ctx, int H, float sm_scale, const AttendGroup& g, const void* Q, const AttendMaps& src,
             const int32_t* cache_pos, void* O, float* lse, float* partials, int* tickets, bool early, cudaStream_t st) {
    return g.cluster > 1 ? launch_k<T, DH, QT, U, true>(ctx, H, sm_scale, g, Q, src, cache_pos, O, lse, partials, tickets, early, st)
                         : launch_k<T, DH, QT, U, false>(ctx, H, sm_scale, g, Q, src, cache_pos, O, lse, partials, tickets, early, st);
}

template <typename T, int DH>
int launch_qt(dodo_ctx* ctx, int H, float sm_scale, const AttendPlan& plan, const AttendGroup& g,
              const void* Q, const AttendMaps& src, const int32_t* cache_pos, void* O, float* lse,
              float* partials, int* tickets, bool early, cudaStream_t st) {
    switch (plan.qt) {
        case 1: return launch_t<T, DH, 1, 4>(ctx, H, sm_scale, g, Q, src, cache_pos, O, lse, partials, tickets, early, st);
        case 2: return launch_t<T, DH, 2, 4>(ctx, H, sm_scale, g, Q, src, cache_pos, O, lse, partials, tickets, early, st);
        case 4: return launch_t<T, DH, 4, 4>(ctx, H, sm_scale, g, Q, src, cache_pos, O, lse, partials, tickets, early, st);
        default: break;
    }
    return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "attend: query tile %d is not built", plan.qt);
}

}  // namespace

int dodo_attend_tile_keys(int dtype, int dh) {
    const int lpr = dh * static_cast<int>(dodo_elem_bytes(dtype)) / 16;
    return (kThreads / lpr) * kGranule;
}
int dodo_attend_max_qt(int dtype, int dh) { (void)dtype; (void)dh; return 4; }
int dodo_attend_max_cluster() { return kMaxCluster; }

const int* dodo_attend_cluster_cap(dodo_ctx* ctx, int dtype, int dh, int qt) {
    const int qi = qt == 1 ? 0 : qt == 2 ? 1 : qt == 4 ? 2 : -1;
    const int ki = (dtype == DODO_BF16 ? 0 : dtype == DODO_F32 ? 2 : -1), di = dh == 128 ? 0 : dh == 64 ? 1 : -1;
    if (qi < 0 || ki < 0 || di < 0) return nullptr;
    const int slot = (ki + di) * 3 + qi;
    if (!ctx->cluster_cap_set[slot]) {
        int* cap = ctx->cluster_cap[slot];
        switch (slot) {
            case 0: cluster_cap_t<__nv_bfloat16, 128, 1, 4>(cap); break;
            case 1: cluster_cap_t<__nv_bfloat16, 128, 2, 4>(cap); break;
            case 2: cluster_cap_t<__nv_bfloat16, 128, 4, 4>(cap); break;
            case 3: cluster_cap_t<__nv_bfloat16, 64, 1, 4>(cap); break;
            case 4: cluster_cap_t<__nv_bfloat16, 64, 2, 4>(cap); break;
            case 5: cluster_cap_t<__nv_bfloat16, 64, 4, 4>(cap); break;
            case 6: cluster_cap_t<float, 128, 1, 4>(cap); break;
            case 7: cluster_cap_t<float, 128, 2, 4>(cap); break;
            case 8: cluster_cap_t<float, 128, 4, 4>(cap); break;
            case 9: cluster_cap_t<float, 64, 1, 4>(cap); break;
            case 10: cluster_cap_t<float, 64, 2, 4>(cap); break;
            default: cluster_cap_t<float, 64, 4, 4>(cap); break;
        }
        ctx->cluster_cap_set[slot] = true;
    }
    return ctx->cluster_cap[slot];
}

int dodo_launch_attend(dodo_ctx* ctx, int dtype, int H, int dh, float sm_scale, const AttendPlan& plan,
                       const AttendGroup& g, const void* Q, const AttendMaps& maps,
                       const int32_t* cache_pos, void* O, float* lse, float* partials, int* tickets,
                       bool early_cache, cudaStream_t st) {
    if (g.cta0[g.nseq] == 0) return DODO_OK;
    if (dtype == DODO_BF16 && dh == 128)
        return launch_qt<__nv_bfloat16, 128>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, early_cache, st);
    if (dtype == DODO_BF16 && dh == 64)
        return launch_qt<__nv_bfloat16, 64>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, early_cache, st);
    if (dtype == DODO_F32 && dh == 128)
        return launch_qt<float, 128>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, early_cache, st);
    if (dtype == DODO_F32 && dh == 64)
        return launch_qt<float, 64>(ctx, H, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, tickets, early_cache, st);
    return dodo_fail(ctx, DODO_ERR_UNSUPPORTED, "attend: dtype %d with head size %d", dtype, dh);
}
