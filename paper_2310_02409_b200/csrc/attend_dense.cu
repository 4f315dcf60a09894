// Attention of a block of query tokens over [nugget cache ; local tokens] (Eq. 13, Eq. 9) on the
// 5th-generation tensor cores: tcgen05.mma with TMEM accumulators, operands staged by TMA.
// bf16, head size 128.  This is the dense case, where many queries share every K/V tile and the
// work is a contraction (about Tq flop per K/V byte); single-token decode stays on the HBM-bound
// kernel in attend.cu.
//
// A unit of work is (sequence, block of 256 query tokens, head): two query tiles of 128 rows that walk
// the same key tiles of 128 keys, so that every K and V tile is brought into shared memory once for 256
// queries.  One thread block per SM takes one unit, or, in the balanced form of the kernel, an equal
// share of all key tiles whatever units they belong to (see DenseWork below).  Tensor memory holds the
// scores S_t of query tile t in columns [128 t, 128 t + 128) and its output O_t in [256 + 128 t, + 128).
// Four roles, each waiting only for what it consumes:
//   loader (one lane of warp 9)  plain per-block TMA tensor copies with the 128-byte swizzle: the two Q
//       tiles once per unit, K tiles and V tiles through two-stage rings, as far ahead as the rings allow.
//   issuer (one lane of warp 8)  per key tile j, in this order: O_0 += P_0(j-1) V(j-1), S_0 = Q_0 K(j)^T,
//       O_1 += P_1(j-1) V(j-1), S_1 = Q_1 K(j)^T.  The tensor pipe executes in issue order, so S_t(j) may
//       overwrite P_t(j-1), which lives in the first 64 columns of S_t, and while one tile's scores are in
//       the softmax the pipe works on the other tile.  S = Q K^T is 8 x tcgen05.mma M128 N128 K16 (both
//       operands K-major in shared memory), O += P V is 8 x M128 N128 K16 (A = P read from tensor memory,
//       B = V MN-major, i.e. V rows as stored).  tcgen05.commit -> mbarriers publish S_t, free P_t / O_t and
//       hand ring stages back to the loader.
//   softmax of tile t (warps 4t .. 4t+3, one thread per query row = TMEM lane)  two passes over its row of
//       S_t with tcgen05.ld, 32 columns at a time: the row maximum (position mask only on tiles that need
//       one: key visible iff key_pos <= q_pos; rows past a segment's end carry INT_MAX), then the weights
//       in the base-2 domain with the scale folded into the exponent's FMA, written as bf16 pairs over the
//       columns they came from (tcgen05.st), and the fp32 row sum of the unrounded weights.  O_t stays in
//       TMEM across key tiles; it is rescaled (tcgen05.ld / st) only when a row's maximum has grown by
//       more than 2^8 since the reference maximum was last moved.
// One round to bf16 at the end; optional log-sum-exp (from the unrounded weights).
// V rows past the end of a segment are zeroed in shared memory before use, so that whatever lies
// behind a sequence's region (another sequence, unused capacity) can never reach the product P V.
// Every wait is bounded; on time-out a status word is set and the block runs on to its end, where
// it always frees its TMEM columns.
#include "dodo_internal.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int DH = 128;               // head size
constexpr int BM = 128;               // query rows per tile = TMEM lanes
constexpr int QT = 2;                 // query tiles per unit
constexpr int BU = QT * BM;           // query rows per unit
constexpr int BN = 128;               // keys per tile
constexpr int kSoftmaxThreads = QT * BM;          // one thread per query row; warps 4t .. 4t+3 serve tile t
constexpr int kIssuerWarp = kSoftmaxThreads / 32;
constexpr int kLoaderWarp = kIssuerWarp + 1;
constexpr int kThreads = kSoftmaxThreads + 64;
constexpr int kHalfBytes = BM * 128;     // 64 columns of a 128-row bf16 tile, rows of 128 bytes (BM == BN)
constexpr int kTileBytes = 2 * kHalfBytes;
constexpr int kStages = 2;               // K ring and V ring: two tiles each
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kTmemO = QT * BN;     // first output column
constexpr float kNeg = -1.0e30f;
constexpr int kBalanceMinTiles = 24;     // balance by default only when a unit has about this many key tiles
constexpr float kRescaleStep = 8.f;      // move a row's reference maximum only past this many octaves

// shared-memory map (bytes from the 1024-aligned base)
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + QT * kTileBytes;
constexpr int kOffV = kOffK + kStages * kTileBytes;
constexpr int kSmemBytes = kOffV + kStages * kTileBytes;

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

struct TileSrc {
    bool cache;
    int row0;   // first global row of the tile
    int rows;   // rows of the tile that belong to the segment
    int pos0;   // position of the tile's first row (local tiles)
};

// A unit of work is (sequence, block of 256 queries, head); its key list is cut into tiles of BN keys.
struct Unit {
    int i, qb, h;    // sequence of the group, query block, head
    int nq0, nq1;    // live rows of the two query tiles (nq1 = 0: the block has one tile only)
    int nt_c;        // key tiles in the nugget cache
    int l_vis;       // local rows at least one query of the block can see
    int n;           // key tiles in all
    int n0;          // ... of which the first query tile needs the first n0 (its queries come earlier)
    int ne;          // slots the unit takes in the balanced order: max(1, n), or that of the sequence's
                     // last query block when the blocks of a head walk the keys in step (width > 1)
};
__device__ __forceinline__ void unit_shape(const AttendSeq& sq, Unit& u) {
    const int q_first = u.qb * BU, nq = min(BU, sq.tq - q_first);
    u.nq0 = min(BM, nq);
    u.nq1 = nq - u.nq0;
    u.l_vis = max(0, min(sq.l_len, sq.q_pos0 + q_first + nq - 1 - sq.l_pos0 + 1));
    const int l_vis0 = max(0, min(sq.l_len, sq.q_pos0 + q_first + u.nq0 - 1 - sq.l_pos0 + 1));
    u.nt_c = (sq.c_len + BN - 1) / BN;
    u.n = u.nt_c + (u.l_vis + BN - 1) / BN;
    u.n0 = u.nt_c + (l_vis0 + BN - 1) / BN;
    u.ne = max(1, u.n);
}
// width > 1: every sequence has `width` query blocks; the slot count is the last (longest) block's
__device__ __forceinline__ void unit_shape(const AttendSeq& sq, Unit& u, int width) {
    unit_shape(sq, u);
    if (width > 1) {
        Unit last = u;
        last.qb = width - 1;
        unit_shape(sq, last);
        u.ne = last.ne;
    }
}
__device__ __forceinline__ TileSrc tile_src(const AttendSeq& sq, const Unit& u, int t) {
    TileSrc s;
    if (t < u.nt_c) {
        s.cache = true; s.row0 = sq.c_row0 + t * BN; s.rows = min(BN, sq.c_len - t * BN); s.pos0 = 0;
    } else {
        const int tl = t - u.nt_c;
        s.cache = false; s.row0 = sq.l_row0 + tl * BN; s.rows = min(BN, u.l_vis - tl * BN); s.pos0 = sq.l_pos0 + tl * BN;
    }
    return s;
}
// The unit after u in the order (sequence, query block, head), heads fastest; with width > 1 the query
// block stays what it is and the order is (sequence, head).  False past the last one.
__device__ __forceinline__ bool next_unit(const AttendGroup& g, int H, int width, Unit& u) {
    if (++u.h < H) return true;
    u.h = 0;
    if (width == 1) {
        if (++u.qb * BU < g.seq[u.i].tq) { unit_shape(g.seq[u.i], u); return true; }
        u.qb = 0;
    }
    while (++u.i < g.nseq)
        if (g.seq[u.i].tq > 0) { unit_shape(g.seq[u.i], u, width); return true; }
    return false;
}

// Two ways to spread the units over thread blocks.  Plain: block c takes unit c whole.  Balanced: work
// is counted in slots, one per key tile and one for a unit without any visible key (so that somebody
// writes its zeros); the units are laid end to end and block c of G takes the slots
// [c T / G, (c+1) T / G), whatever units they fall in.  A unit cut by a block boundary is finished
// through unnormalised partial results in the workspace: every block that holds a piece writes it,
// takes a ticket on the unit, and the block that draws the last ticket merges by log-sum-exp.  Nobody
// waits for anybody.  Balanced pays when the units alone would leave SMs idle or unevenly loaded and
// the key lists are long enough to hide the partials.
// In step (width W > 1, every sequence has W query blocks): thread blocks come in groups of W, block c =
// group c / W, query block c % W; the groups share out the slots of the (sequence, head) pairs, counted by
// the longest query block, and the W blocks of a group pass the same key tiles at about the same time, so
// that a head's K/V is fetched from HBM once and found in L2 by the other W - 1.
struct DenseWork {
    int total_slots;         // T
    int width;               // W
    float* partials;         // [2 * gridDim.x] x QT x (DH x BM outputs, BM maxima, BM sums), balanced only
    int* tickets;            // one arrival counter per unit of the launch, zero between launches
};
constexpr int kPartFloats = BM * DH + 2 * BM;      // one query tile's piece
constexpr int kPieceFloats = QT * kPartFloats;     // a unit's piece

__device__ __forceinline__ int block_start(int T, int G, int c) { return static_cast<int>(static_cast<long long>(c) * T / G); }
__device__ __forceinline__ int block_of(int T, int G, int x) {   // the block whose range holds slot x
    return static_cast<int>(((static_cast<long long>(x) + 1) * G - 1) / T);
}

template <bool kBalanced>
__global__ void __launch_bounds__(kThreads, 1)
attend_dense_kernel(const __grid_constant__ DenseMaps maps, const __grid_constant__ AttendGroup g,
                    const int32_t* __restrict__ cache_pos, int H, float scale_log2,
                    __nv_bfloat16* __restrict__ O, float* __restrict__ lse, const DenseWork work,
                    int* __restrict__ dev_status) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    __shared__ __align__(8) uint64_t bar_q, bar_s[QT], bar_p[QT], bar_o[QT];
    __shared__ __align__(8) uint64_t bar_kfull[kStages], bar_vfull[kStages], bar_kfree[kStages], bar_vfree[kStages];
    __shared__ uint32_t tmem_slot;
    __shared__ int first_masked[2];
    __shared__ int s_start[4];      // balanced: the block's first unit and tile (i, qb, h, t)
    __shared__ int s_last;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int bid = static_cast<int>(blockIdx.x);
    const int W = kBalanced ? work.width : 1;
    const int G = static_cast<int>(gridDim.x) / W, grp = bid / W;   // balanced: groups of W blocks share a slot range
    const int T = work.total_slots;

    // ---- barriers, TMEM, where this block starts ---------------------------------------------------
    if (tid == 0) {
        first_masked[0] = first_masked[1] = 0x7fffffff;
        mbar_init(&bar_q, 1);
        for (int t = 0; t < QT; ++t) { mbar_init(&bar_s[t], 1); mbar_init(&bar_p[t], BM / 32); mbar_init(&bar_o[t], 1); }
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bar_kfull[s], 1); mbar_init(&bar_vfull[s], 1); mbar_init(&bar_kfree[s], 1); mbar_init(&bar_vfree[s], 1);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (kBalanced) {
            // walk the (sequence, query block) groups up to the one that holds this block's first slot
            Unit w;
            w.i = 0; w.qb = 0; w.h = 0;
            int t = 0, acc = 0;
            const int x0 = block_start(T, G, grp);
            bool found = false;
            for (int i = 0; i < g.nseq && !found; ++i) {
                for (int qb = (W > 1 ? bid % W : 0); qb * BU < g.seq[i].tq && !found; qb += (W > 1 ? W : 1)) {
                    w.i = i; w.qb = qb;
                    unit_shape(g.seq[i], w, W);
                    const int span = w.ne * H;
                    if (x0 < acc + span) {
                        w.h = (x0 - acc) / w.ne;
                        t = (x0 - acc) % w.ne;
                        found = true;
                    }
                    acc += span;
                }
            }
            s_start[0] = w.i; s_start[1] = w.qb; s_start[2] = w.h; s_start[3] = t;
        }
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    bool stuck = false;

    // Every role goes through the same list of segments = (unit, key tiles [t0, t1)); plain: one whole unit.
    Unit u;
    int t0 = 0, x = 0, left;
    if (kBalanced) {
        u.i = s_start[0]; u.qb = s_start[1]; u.h = s_start[2]; t0 = s_start[3];
        unit_shape(g.seq[u.i], u, W);
        x = block_start(T, G, grp);                  // slot at which the segment starts
        left = block_start(T, G, grp + 1) - x;       // slots still to do
    } else {
        int b;
        if (g.uniform_ctas > 0) {
            b = bid / g.uniform_ctas;
        } else {
            b = 0;
#pragma unroll 8
            for (int i = 1; i < DODO_GROUP; ++i) b += (i < g.nseq && g.cta0[i] <= bid) ? 1 : 0;
        }
        const int r0 = bid - g.cta0[b];
        u.i = b; u.h = r0 % H; u.qb = r0 / H;
        unit_shape(g.seq[b], u);
        left = u.ne;
    }
    // Counters that run on through the block's segments: m = key tiles (ring stages, the K/V barriers),
    // c = key tiles a query tile has been through (phases of bar_s / bar_p / bar_o), seg = segments with
    // key tiles (phase of the Q barrier).  Completion number n of a barrier is waited for with parity n & 1;
    // no waiter can be a whole phase behind: every producer of completion n + 1 needs, directly or through
    // the in-order tensor pipe, something its consumer does after it has seen completion n.
    int m = 0, seg = 0;

    if (warp == kLoaderWarp) {
        // ============================ loader: Q, K and V copies ===========================================
        if (tid == kLoaderWarp * 32) {
            bool more = left > 0;
            while (more) {
                const AttendSeq sq = g.seq[u.i];
                const int t1 = min(u.ne, t0 + left);
                const int nreal = max(0, min(t1, u.n) - t0);   // key tiles of the segment
                const int h = u.h;
                if (nreal > 0) {
                    // Q of a later segment: free once the last Q K^T before it has completed (its K stage was freed then)
                    if (seg > 0 && !mbar_wait(&bar_kfree[(m - 1) % kStages], static_cast<uint32_t>((m - 1) / kStages) & 1u)) stuck = true;
                    const int q_row = sq.q_row0 + u.qb * BU;
                    const int ntile = u.nq1 > 0 ? 2 : 1;
                    mbar_expect_tx(&bar_q, ntile * kTileBytes);
                    for (int t = 0; t < ntile; ++t) {
                        tma_load_2d(base + kOffQ + t * kTileBytes, &maps.Q, h * DH, q_row + t * BM, &bar_q);
                        tma_load_2d(base + kOffQ + t * kTileBytes + kHalfBytes, &maps.Q, h * DH + 64, q_row + t * BM, &bar_q);
                    }
                    for (int j = 0; j < nreal; ++j, ++m) {
                        const int st = m % kStages;
                        const uint32_t ph = static_cast<uint32_t>(m / kStages) & 1u;
                        const TileSrc ts = tile_src(sq, u, t0 + j);
                        const CUtensorMap* mk = ts.cache ? &maps.cK : &maps.lK;
                        const CUtensorMap* mv = ts.cache ? &maps.cV : &maps.lV;
                        if (m >= kStages && !mbar_wait(&bar_kfree[st], ph ^ 1u)) stuck = true;
                        const uint32_t dk = base + kOffK + st * kTileBytes;
                        mbar_expect_tx(&bar_kfull[st], kTileBytes);
                        tma_load_2d(dk, mk, h * DH, ts.row0, &bar_kfull[st]);
                        tma_load_2d(dk + kHalfBytes, mk, h * DH + 64, ts.row0, &bar_kfull[st]);
                        if (m >= kStages && !mbar_wait(&bar_vfree[st], ph ^ 1u)) stuck = true;
                        const uint32_t dv = base + kOffV + st * kTileBytes;
                        mbar_expect_tx(&bar_vfull[st], kTileBytes);
                        tma_load_2d(dv, mv, h * DH, ts.row0, &bar_vfull[st]);
                        tma_load_2d(dv + kHalfBytes, mv, h * DH + 64, ts.row0, &bar_vfull[st]);
                    }
                    ++seg;
                }
                left -= (t1 - t0);
                x += (t1 - t0);
                t0 = 0;
                more = kBalanced && left > 0 && next_unit(g, H, W, u);
            }
            if (stuck) atomicOr(dev_status, DODO_DEV_WAIT_TIMEOUT);
        }
    } else if (warp == kIssuerWarp) {
        // ============================ issuer: S_t = Q_t K^T, O_t += P_t V ==================================
        if (tid == kIssuerWarp * 32) {
            int c[QT] = {0, 0};
            const uint32_t idesc = idesc_bf16(BN, false), idesc_pv = idesc_bf16(DH, true);
            bool more = left > 0;
            while (more) {
                const int t1 = min(u.ne, t0 + left);
                const int nreal = max(0, min(t1, u.n) - t0);
                if (nreal > 0) {
                    if (!mbar_wait(&bar_q, static_cast<uint32_t>(seg) & 1u)) stuck = true;
                    // iteration j issues the P V of key tile j - 1 and the Q K^T of key tile j, query tile 0 first
                    for (int j = 0; j <= nreal; ++j) {
                        const int mp = m + j - 1, mc = m + j;               // ring positions of key tiles j - 1 and j
                        const bool a_prev[QT] = {j > 0 && t0 + j - 1 < u.n0, j > 0 && u.nq1 > 0};
                        const bool a_cur[QT] = {j < nreal && t0 + j < u.n0, j < nreal && u.nq1 > 0};
                        bool v_ready = false, k_ready = false;
#pragma unroll
                        for (int t = 0; t < QT; ++t) {
                            if (a_prev[t]) {
                                // P_t(j-1) is in tensor memory and O_t carries the right scale (and, at the start
                                // of a segment, the softmax threads have taken the previous unit's O_t out)
                                if (!mbar_wait(&bar_p[t], static_cast<uint32_t>(c[t]) & 1u)) stuck = true;
                                if (!v_ready && !mbar_wait(&bar_vfull[mp % kStages], static_cast<uint32_t>(mp / kStages) & 1u)) stuck = true;
                                v_ready = true;
                                tc_fence_after();
                                const uint64_t b0 = desc_mnmajor(base + kOffV + (mp % kStages) * kTileBytes, kHalfBytes);
#pragma unroll
                                for (int i = 0; i < BN / 16; ++i)   // 16 keys of P = 8 columns of bf16 pairs
                                    mma_bf16_ts(tmem + kTmemO + t * DH, tmem + t * BN + i * 8,
                                                b0 + static_cast<uint64_t>((i * 2048) >> 4), idesc_pv, j > 1 || i > 0);
                                mma_commit(&bar_o[t]);
                                ++c[t];
                            }
                            if (a_cur[t]) {
                                if (!k_ready && !mbar_wait(&bar_kfull[mc % kStages], static_cast<uint32_t>(mc / kStages) & 1u)) stuck = true;
                                k_ready = true;
                                tc_fence_after();
                                // descriptors differ only in their start-address field (units of 16 bytes)
                                const uint64_t a0 = desc_kmajor(base + kOffQ + t * kTileBytes);
                                const uint64_t b0 = desc_kmajor(base + kOffK + (mc % kStages) * kTileBytes);
#pragma unroll
                                for (int i = 0; i < DH / 16; ++i)
                                    mma_bf16(tmem + t * BN, a0 + static_cast<uint64_t>(((i / 4) * kHalfBytes + (i % 4) * 32) >> 4),
                                             b0 + static_cast<uint64_t>(((i / 4) * kHalfBytes + (i % 4) * 32) >> 4), idesc, i > 0);
                                mma_commit(&bar_s[t]);
                            }
                        }
                        // everything that reads V(j-1) / K(j) has been issued: the stages go back when it completes
                        if (j > 0) mma_commit(&bar_vfree[mp % kStages]);
                        if (j < nreal) mma_commit(&bar_kfree[mc % kStages]);
                    }
                    m += nreal;
                    ++seg;
                }
                left -= (t1 - t0);
                x += (t1 - t0);
                t0 = 0;
                more = kBalanced && left > 0 && next_unit(g, H, W, u);
            }
            if (stuck) atomicOr(dev_status, DODO_DEV_WAIT_TIMEOUT);
        }
    } else {
        // ===================================== softmax ===========================================
        // Thread = query row `row` of query tile t = its TMEM lane.  Warps 4t .. 4t+3 cover the 128 lanes.
        const int t = warp >> 2, row = tid & (BM - 1);
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;   // this warp's TMEM lanes
        const uint32_t tmem_s = tmem + t * BN + lane_sel, tmem_o = tmem + kTmemO + t * DH + lane_sel;
        const float2 c2 = make_float2(scale_log2, scale_log2);
        int c = 0;                      // key tiles this query tile has been through
        bool first_seg = true;

        bool more = left > 0;
        while (more) {
            const AttendSeq sq = g.seq[u.i];
            const int ne = u.ne;
            const int t1 = min(ne, t0 + left);
            const int nreal = max(0, min(t1, u.n) - t0);                              // key tiles of the segment
            const int n_mine = t == 0 ? u.n0 : (u.nq1 > 0 ? u.n : 0);                  // key tiles this query tile needs
            const int mine = max(0, min(t1, n_mine) - t0);                             // ... of the segment
            const int h = u.h, q_first = u.qb * BU + t * BM;
            const int nq = t == 0 ? u.nq0 : u.nq1;
            const bool row_live = row < nq;
            const int my_qpos = row_live ? sq.q_pos0 + q_first + row : static_cast<int>(0x80000000);
            const int min_qpos = sq.q_pos0 + q_first;
            float m_ref = kNeg, l = 0.f;   // l: sum of the unrounded weights of the row

            if (nreal > 0) {
                // First cache tile holding a key that some query of the block must not see (nuggets normally
                // all precede the block, so this is nt_c and no cache tile pays for the position test).
                {
                    const int block_qpos = sq.q_pos0 + u.qb * BU;
                    int bad = 0x7fffffff;
                    for (int i = tid; i < sq.c_len; i += kSoftmaxThreads)
                        if (__ldg(cache_pos + sq.c_row0 + i) > block_qpos) bad = min(bad, i / BN);
                    if (bad != 0x7fffffff) atomicMin(&first_masked[seg & 1], bad);
                    if (kBalanced && tid == 0) first_masked[(seg + 1) & 1] = 0x7fffffff;   // for the next segment; its users are past
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                }
                const int first_bad = first_masked[seg & 1];

                for (int j = 0; j < mine; ++j, ++c) {
                    const int tt = t0 + j, mm = m + j;
                    const int st = mm % kStages;
                    const TileSrc ts = tile_src(sq, u, tt);
                    const bool need_mask = ts.rows < BN || (ts.cache ? tt >= first_bad : ts.pos0 + ts.rows - 1 > min_qpos);

                    if (!mbar_wait(&bar_s[t], static_cast<uint32_t>(c) & 1u)) stuck = true;
                    tc_fence_after();
                    // ---- pass 1: the row maximum of the raw scores (masked entries are written back as such) ----
                    float tmax = kNeg;
#pragma unroll 1
                    for (int cc = 0; cc < BN / 32; ++cc) {
                        uint32_t sv[32];
                        tmem_ld32(tmem_s + cc * 32, sv);
                        if (need_mask) {
#pragma unroll
                            for (int e = 0; e < 32; ++e) {
                                const int col = cc * 32 + e;
                                int kp = 0x7fffffff;
                                if (col < ts.rows) kp = ts.cache ? __ldg(cache_pos + ts.row0 + col) : ts.pos0 + col;
                                if (kp > my_qpos) sv[e] = __float_as_uint(kNeg);
                            }
                            tmem_st32(tmem_s + cc * 32, sv);
                        }
                        float a = fmaxf(__uint_as_float(sv[0]), __uint_as_float(sv[1]));
#pragma unroll
                        for (int e = 2; e < 32; e += 2) a = max3(a, __uint_as_float(sv[e]), __uint_as_float(sv[e + 1]));
                        tmax = fmaxf(tmax, a);
                    }
                    tmax = tmax > 0.5f * kNeg ? tmax * scale_log2 : kNeg;   // base-2 domain; kNeg = nothing visible

                    // move the reference maximum only when it pays; rescale O_t in TMEM when any row of the warp
                    // moved.  P V of the key tile before is complete: S_t of this one was issued behind it.
                    const bool grow = tmax > m_ref + kRescaleStep;
                    const float m_new = grow ? tmax : m_ref;
                    if (j > 0 && __any_sync(0xffffffffu, grow)) {
                        if (!mbar_wait(&bar_o[t], static_cast<uint32_t>(c - 1) & 1u)) stuck = true;
                        tc_fence_after();
                        const float corr = ex2_approx(m_ref - m_new);   // 1 for rows that did not move
                        l *= corr;
#pragma unroll 1
                        for (int cc = 0; cc < DH / 32; ++cc) {
                            uint32_t ov[32];
                            tmem_ld32(tmem_o + cc * 32, ov);
#pragma unroll
                            for (int e = 0; e < 32; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * corr);
                            tmem_st32(tmem_o + cc * 32, ov);
                        }
                    }
                    m_ref = m_new;

                    // rows of V past the segment's end must not reach P V (both query tiles do this, each ahead
                    // of its own P V)
                    if (ts.rows < BN) {
                        if (!mbar_wait(&bar_vfull[st], static_cast<uint32_t>(mm / kStages) & 1u)) stuck = true;
                        unsigned char* v0 = base_ptr + kOffV + st * kTileBytes;
                        for (int i = row; i < (BN - ts.rows) * 16; i += BM) {   // 16 x 16 bytes per row
                            const int vrow = ts.rows + i / 16, piece = i % 16;
                            *reinterpret_cast<uint4*>(v0 + (piece / 8) * kHalfBytes + vrow * 128 + (piece % 8) * 16) = make_uint4(0, 0, 0, 0);
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // zeroed V rows -> tensor core
                    }

                    // ---- pass 2: P = 2^(scale s - m_ref) as bf16 pairs into tensor memory, the A operand of P V
                    // (chunk cc of 32 keys lands in columns [16 cc, 16 cc + 16), which held scores read by then).
                    // Masked entries hold kNeg and come out as exactly 0 (the clamp keeps that true while the
                    // row has seen no visible key).
                    const float nm = -fmaxf(m_ref, -1.0e20f);
                    const float2 nm2 = make_float2(nm, nm);
                    float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll 1
                    for (int cc = 0; cc < BN / 32; ++cc) {
                        uint32_t sv[32], packed[16];
                        tmem_ld32(tmem_s + cc * 32, sv);
#pragma unroll
                        for (int e = 0; e < 16; e += 2) {
                            const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(sv[2 * e]), __uint_as_float(sv[2 * e + 1])), c2, nm2);
                            const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(sv[2 * e + 2]), __uint_as_float(sv[2 * e + 3])), c2, nm2);
                            const float2 p0 = make_float2(ex2_approx(x0.x), ex2_approx(x0.y));
                            const float2 p1 = make_float2(ex2_approx(x1.x), ex2_approx(x1.y));
                            packed[e] = pack_bf16(p0.x, p0.y);
                            packed[e + 1] = pack_bf16(p1.x, p1.y);
                            acc0 = __fadd2_rn(acc0, p0);
                            acc1 = __fadd2_rn(acc1, p1);
                        }
                        tmem_st16(tmem_s + cc * 16, packed);
                    }
                    l += (acc0.x + acc0.y) + (acc1.x + acc1.y);
                    tc_fence_before();
                    __syncwarp();                      // one arrival per warp
                    if ((tid & 31) == 0) mbar_arrive(&bar_p[t]);
                }
                if (mine > 0) {
                    if (!mbar_wait(&bar_o[t], static_cast<uint32_t>(c - 1) & 1u)) stuck = true;
                    tc_fence_after();
                }
            }

            const size_t orow = static_cast<size_t>(sq.q_row0 + q_first + row) * H + h;
            const bool whole = !kBalanced || (t0 == 0 && t1 == ne);
            if (whole) {
                // ---- normalise, round once, store ----------------------------------------------------------------
                const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll 1
                for (int cc = 0; cc < DH / 32; ++cc) {
                    uint32_t ov[32];
                    if (mine > 0) {
                        tmem_ld32(tmem_o + cc * 32, ov);
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) ov[e] = 0u;
                    }
                    if (row_live) {
                        uint4* dst = reinterpret_cast<uint4*>(O + orow * DH + cc * 32);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            dst[q] = make_uint4(
                                pack_bf16(__uint_as_float(ov[8 * q]) * inv, __uint_as_float(ov[8 * q + 1]) * inv),
                                pack_bf16(__uint_as_float(ov[8 * q + 2]) * inv, __uint_as_float(ov[8 * q + 3]) * inv),
                                pack_bf16(__uint_as_float(ov[8 * q + 4]) * inv, __uint_as_float(ov[8 * q + 5]) * inv),
                                pack_bf16(__uint_as_float(ov[8 * q + 6]) * inv, __uint_as_float(ov[8 * q + 7]) * inv));
                        }
                    }
                }
                if (row_live && lse != nullptr)
                    lse[orow] = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
            } else {
                // ---- a cut unit: unnormalised partial to the workspace; the last block to arrive merges --------
                // Layout per query tile [feature][row]: a warp's lanes are consecutive rows, so they write and read
                // consecutive floats.
                const int xu = x - t0;                                        // the unit's first slot
                const int c_first = block_of(T, G, xu), c_last = block_of(T, G, xu + ne - 1);
                float* ps = work.partials + static_cast<size_t>(2 * bid + (first_seg ? 0 : 1)) * kPieceFloats + t * kPartFloats;
                if (nq > 0) {
#pragma unroll 1
                    for (int cc = 0; cc < DH / 32; ++cc) {
                        uint32_t ov[32];
                        if (mine > 0) {
                            tmem_ld32(tmem_o + cc * 32, ov);
                        } else {   // this query tile sees none of the segment's keys
#pragma unroll
                            for (int e = 0; e < 32; ++e) ov[e] = 0u;
                        }
                        float* dst = ps + (cc * 32) * BM + row;
#pragma unroll
                        for (int e = 0; e < 32; ++e) dst[e * BM] = __uint_as_float(ov[e]);
                    }
                    ps[BM * DH + row] = m_ref;
                    ps[BM * DH + BM + row] = l;
                }
                __threadfence();
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (tid == 0) {
                    int* tk = work.tickets + g.cta0[u.i] + u.qb * H + h;
                    const int arrived = atomicAdd(tk, 1);
                    s_last = arrived == c_last - c_first;
                    if (s_last) *tk = 0;   // leave the counter clean for the next launch
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (s_last && nq > 0) {
                    __threadfence();
                    // group cg's piece of this unit is its first segment if cg starts inside the unit, else its last
                    auto piece = [&](int cg) {
                        return work.partials + static_cast<size_t>(2 * (cg * W + bid % W) + (block_start(T, G, cg) >= xu ? 0 : 1)) * kPieceFloats +
                               t * kPartFloats;
                    };
                    float M = kNeg;
                    for (int cg = c_first; cg <= c_last; ++cg) M = fmaxf(M, __ldcg(piece(cg) + BM * DH + row));
                    float L = 0.f;
                    for (int cg = c_first; cg <= c_last; ++cg) {
                        const float* pc = piece(cg);
                        L = fmaf(__ldcg(pc + BM * DH + BM + row), ex2_approx(__ldcg(pc + BM * DH + row) - M), L);
                    }
                    const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll 1
                    for (int cc = 0; cc < DH / 32; ++cc) {
                        float o[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = 0.f;
                        for (int cg = c_first; cg <= c_last; ++cg) {
                            const float* pc = piece(cg);
                            const float w = ex2_approx(__ldcg(pc + BM * DH + row) - M);
                            const float* src = pc + (cc * 32) * BM + row;
#pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = fmaf(__ldcg(src + e * BM), w, o[e]);
                        }
                        if (row_live) {
                            uint4* dst = reinterpret_cast<uint4*>(O + orow * DH + cc * 32);
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                dst[q] = make_uint4(pack_bf16(o[8 * q] * inv, o[8 * q + 1] * inv), pack_bf16(o[8 * q + 2] * inv, o[8 * q + 3] * inv),
                                                    pack_bf16(o[8 * q + 4] * inv, o[8 * q + 5] * inv), pack_bf16(o[8 * q + 6] * inv, o[8 * q + 7] * inv));
                        }
                    }
                    if (row_live && lse != nullptr)
                        lse[orow] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");   // s_last is free again
            }
            if (nreal > 0) { m += nreal; ++seg; }
            first_seg = false;
            left -= (t1 - t0);
            x += (t1 - t0);
            t0 = 0;
            more = kBalanced && left > 0 && next_unit(g, H, W, u);
        }
        if (stuck) atomicOr(dev_status, DODO_DEV_WAIT_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

}  // namespace

int dodo_dense_tile_queries() { return BM; }
int dodo_dense_unit_queries() { return BU; }
int dodo_dense_tile_keys() { return BN; }
size_t dodo_dense_workspace_bytes(int num_sms) { return static_cast<size_t>(2) * num_sms * kPieceFloats * sizeof(float); }

int dodo_launch_attend_dense(dodo_ctx* ctx, int H, float sm_scale, const AttendGroup& g, const DenseMaps& maps,
                             const int32_t* cache_pos, void* O, float* lse, void* workspace, size_t workspace_bytes,
                             int* tickets, int* dev_status, cudaStream_t st) {
    const int units = g.cta0[g.nseq];
    if (units == 0) return DODO_OK;
    // slots of work: one per key tile of a unit, one for a unit without visible keys (same rules as the kernel);
    // `in step` counts every (sequence, head) once, by its last query block
    auto unit_tiles = [](const AttendSeq& sq, int qb) {
        const int q_first = qb * BU, nq = sq.tq - q_first < BU ? sq.tq - q_first : BU;
        int l_vis = sq.q_pos0 + q_first + nq - 1 - sq.l_pos0 + 1;
        l_vis = l_vis < sq.l_len ? l_vis : sq.l_len;
        l_vis = l_vis > 0 ? l_vis : 0;
        return (sq.c_len + BN - 1) / BN + (l_vis + BN - 1) / BN;
    };
    long long total = 0, total_step = 0;
    int width = 0;           // query blocks per sequence if all sequences agree, else -1
    for (int i = 0; i < g.nseq; ++i) {
        const AttendSeq& sq = g.seq[i];
        if (sq.tq <= 0) continue;
        const int qblocks = (sq.tq + BU - 1) / BU;
        width = width == 0 || width == qblocks ? qblocks : -1;
        for (int qb = 0; qb < qblocks; ++qb) {
            const int n = unit_tiles(sq, qb);
            total += static_cast<long long>(n > 0 ? n : 1) * H;
        }
        const int n_last = unit_tiles(sq, qblocks - 1);
        total_step += static_cast<long long>(n_last > 0 ? n_last : 1) * H;
    }
    // Balanced when asked for, or (by default) when the units would leave the resident blocks (one per SM)
    // unevenly loaded and the key lists are long enough for the partial results to disappear in them.
    const int resident = ctx->num_sms;
    const bool room = total < 0x7fffffff && total >= 2 && workspace != nullptr && dodo_aligned16(workspace) &&
                      workspace_bytes >= dodo_dense_workspace_bytes(ctx->num_sms) && units <= DODO_NUM_TICKETS;
    const bool uneven = units % resident != 0 && units < 4 * resident;   // the last wave is not full and weighs
    const bool pays = uneven && total / units >= kBalanceMinTiles;
    const bool balanced = room && ctx->dense_balance != 2 && (pays || ctx->dense_balance == 1 || ctx->dense_balance == 3);
    const bool in_step = balanced && ctx->dense_balance != 3 && width >= 2 && width <= resident;
    DenseWork work;
    work.width = in_step ? width : 1;
    work.total_slots = !balanced ? 0 : static_cast<int>(in_step ? total_step : total);
    work.partials = static_cast<float*>(workspace);
    work.tickets = tickets;
    int grid = units;
    if (balanced) {
        long long groups = resident / work.width;
        if (groups > work.total_slots) groups = work.total_slots;
        grid = static_cast<int>(groups) * work.width;
    }
    const size_t smem = static_cast<size_t>(kSmemBytes) + 1024;
    auto kern = balanced ? attend_dense_kernel<true> : attend_dense_kernel<false>;
    if (!ctx->dense_attr_set[balanced ? 1 : 0]) {
        const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "dense attend shared-memory attribute");
        ctx->dense_attr_set[balanced ? 1 : 0] = true;
    }
    kern<<<grid, kThreads, smem, st>>>(maps, g, cache_pos, H, sm_scale * 1.4426950408889634f,
                                                               static_cast<__nv_bfloat16*>(O), lse, work, dev_status);
    return dodo_check_cuda(ctx, cudaGetLastError(), "dense attend launch");
}
