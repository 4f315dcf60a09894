// Attention of long blocks of query tokens over [nugget cache ; local tokens] (Eq. 13, Eq. 9) on tcgen05:
// the form with TWO query tiles per thread block.  bf16, head size 128.
//
// A unit of work is (sequence, pair of 128-query tiles, head); one thread block per SM.  Every K/V tile of 128
// keys is brought into shared memory once and serves both query tiles, and the two tiles' pipelines run in
// anti-phase: while the softmax threads of one tile work on their scores, the tensor core runs the other
// tile's products.  Roles:
//   producer (one lane of warp 16)   TMA tensor copies with the 128-byte swizzle (no multicast): the 256 query
//       rows once per unit, K and V tiles of 128 keys through a two-stage ring each.
//   issuer x, x = 0, 1 (one lane of warps 17, 18)   for its query tile: S_x = Q_x K^T as 8 x tcgen05.mma M128 N128
//       K16 into 128 TMEM columns, and O_x += P_x V as 8 x tcgen05.mma M128 N128 K16 (A = P_x read from tensor
//       memory, B = V rows as stored) into 128 more; P_x V of tile m is followed at once by Q_x K^T of tile m+1,
//       which may overwrite S_x because the tensor core runs one thread's instructions in order.
//   softmax x (warps 8x .. 8x+7; two threads per query row, 64 score columns each)   two passes over its part
//       of S_x out of tensor memory: maximum (exchanged between the row's two threads through shared memory),
//       then base-2 exponentials written back as bf16 pairs over the first 32 of the thread's own 64 columns.
//       O_x is rescaled only when a row's maximum has grown by more than 2^8 (then, and only then, these
//       threads wait for a P V).  Position masks only on tiles that need them; V rows past a segment's end are
//       zeroed in shared memory before use.
// Plain form: block = unit.  Balanced form: blocks take equal shares of all key tiles (see DenseWork2), cut
// units meet through partial results in the workspace; with several pairs per sequence the blocks of a group
// walk the keys in step so that a head's K/V comes from HBM once.
// Every wait is bounded; on time-out a status word is set and the block runs on to its end, where it always
// frees its tensor memory.
#include "dodo_internal.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int DH = 128;
constexpr int BM = 128;                 // query rows per tile = TMEM lanes
constexpr int BP = 2 * BM;              // query rows per unit (a pair of tiles)
constexpr int BN = 128;                 // keys per tile
constexpr int kGroupThreads = 256;      // softmax threads per query tile: two per row
constexpr int kSoftmaxThreads = 2 * kGroupThreads;
constexpr int kThreads = kSoftmaxThreads + 96;   // + producer, issuer 0, issuer 1
constexpr int kQHalfBytes = BP * 128;   // 64 columns of the 256 query rows: [tile 0 rows][tile 1 rows]
constexpr int kQBytes = 2 * kQHalfBytes;
constexpr int kKVHalfBytes = BN * 128;  // 64 columns of a 128-key tile
constexpr int kKVBytes = 2 * kKVHalfBytes;
constexpr int kStages = 2;
constexpr uint32_t kTmemCols = 512;     // S_0 [0,128), S_1 [128,256), O_0 [256,384), O_1 [384,512)
constexpr float kNeg = -1.0e30f;
constexpr float kRescaleStep = 8.f;

constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + kQBytes;
constexpr int kOffV = kOffK + kStages * kKVBytes;
constexpr int kOffXch = kOffV + kStages * kKVBytes;   // float[2 groups][2][2][BM]
constexpr int kSmemBytes = kOffXch + 2 * 2 * 2 * BM * 4;

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
    int row0, rows, pos0;
};
struct Unit {
    int i, p, h;     // sequence of the group, pair of query tiles, head
    int nt_c;        // key tiles in the nugget cache
    int l_vis;       // local rows the pair's last query can see
    int n;           // key tiles in all
    int ne;          // slots in the balanced order (>= 1; the sequence's last pair's when pairs walk in step)
};
__device__ __forceinline__ void unit_shape(const AttendSeq& sq, Unit& u) {
    const int q_first = u.p * BP, nq = min(BP, sq.tq - q_first);
    u.l_vis = max(0, min(sq.l_len, sq.q_pos0 + q_first + nq - 1 - sq.l_pos0 + 1));
    u.nt_c = (sq.c_len + BN - 1) / BN;
    u.n = u.nt_c + (u.l_vis + BN - 1) / BN;
    u.ne = max(1, u.n);
}
__device__ __forceinline__ void unit_shape(const AttendSeq& sq, Unit& u, int width) {
    unit_shape(sq, u);
    if (width > 1) {
        Unit last = u;
        last.p = width - 1;
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
__device__ __forceinline__ bool next_unit(const AttendGroup& g, int H, int width, Unit& u) {
    if (++u.h < H) return true;
    u.h = 0;
    if (width == 1) {
        if (++u.p * BP < g.seq[u.i].tq) { unit_shape(g.seq[u.i], u); return true; }
        u.p = 0;
    }
    while (++u.i < g.nseq)
        if (g.seq[u.i].tq > 0) { unit_shape(g.seq[u.i], u, width); return true; }
    return false;
}

// As in the one-tile kernel: T slots (one per key tile, one for a unit without keys), block group c of G takes
// [c T / G, (c+1) T / G); width W > 1 = every sequence has W pairs and the W blocks of a group, one per pair,
// share a slot range counted by the last pair.  A cut unit leaves two partials (one per query tile) per piece.
struct DenseWork2 {
    int total_slots;
    int width;
    float* partials;     // [2 * gridDim.x][2 tiles] x (DH x BM outputs, BM maxima, BM sums)
    int* tickets;        // [units][2 tiles]
};
constexpr int kPartFloats = BM * DH + 2 * BM;

__device__ __forceinline__ int block_start(int T, int G, int c) { return static_cast<int>(static_cast<long long>(c) * T / G); }
__device__ __forceinline__ int block_of(int T, int G, int x) { return static_cast<int>(((static_cast<long long>(x) + 1) * G - 1) / T); }

struct Bars {
    uint64_t q, kfull[kStages], vfull[kStages], kempty[kStages], vempty[kStages];
    uint64_t sready[2], pready[2], odone[2];
};

template <bool kBalanced>
__global__ void __launch_bounds__(kThreads, 1)
attend_dense2_kernel(const __grid_constant__ DenseMaps maps, const __grid_constant__ AttendGroup g,
                     const int32_t* __restrict__ cache_pos, int H, float scale_log2,
                     __nv_bfloat16* __restrict__ O, float* __restrict__ lse, const DenseWork2 work,
                     int* __restrict__ dev_status) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    __shared__ __align__(8) Bars bars;
    __shared__ uint32_t tmem_slot;
    __shared__ int first_masked[2][2];   // [query tile][segment parity]
    __shared__ int s_start[4];
    __shared__ int s_last[2];

    const int tid = threadIdx.x, warp = tid >> 5;
    const int bid = static_cast<int>(blockIdx.x);
    const int W = kBalanced ? work.width : 1;
    const int G = static_cast<int>(gridDim.x) / W, grp = bid / W;
    const int T = work.total_slots;

    if (tid == 0) {
        first_masked[0][0] = first_masked[0][1] = first_masked[1][0] = first_masked[1][1] = 0x7fffffff;
        mbar_init(&bars.q, 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&bars.kfull[s], 1); mbar_init(&bars.vfull[s], 1);
            mbar_init(&bars.kempty[s], 2); mbar_init(&bars.vempty[s], 2);   // both issuers release a stage
        }
        for (int x = 0; x < 2; ++x) { mbar_init(&bars.sready[x], 1); mbar_init(&bars.pready[x], kGroupThreads); mbar_init(&bars.odone[x], 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (kBalanced) {
            Unit w;
            w.i = 0; w.p = 0; w.h = 0;
            int t = 0, acc = 0;
            const int x0 = block_start(T, G, grp);
            bool found = false;
            for (int i = 0; i < g.nseq && !found; ++i) {
                for (int p = (W > 1 ? bid % W : 0); p * BP < g.seq[i].tq && !found; p += (W > 1 ? W : 1)) {
                    w.i = i; w.p = p;
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
            s_start[0] = w.i; s_start[1] = w.p; s_start[2] = w.h; s_start[3] = t;
        }
    }
    if (warp == 16) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    bool stuck = false;

    // All roles go through the same list of segments = (unit, key tiles [t0, t1)); plain: one whole unit.
    Unit u;
    int t0 = 0, x = 0, left;
    if (kBalanced) {
        u.i = s_start[0]; u.p = s_start[1]; u.h = s_start[2]; t0 = s_start[3];
        unit_shape(g.seq[u.i], u, W);
        x = block_start(T, G, grp);
        left = block_start(T, G, grp + 1) - x;
    } else {
        int b = 0;
#pragma unroll 8
        for (int i = 1; i < DODO_GROUP; ++i) b += (i < g.nseq && g.cta0[i] <= bid) ? 1 : 0;
        const int r0 = bid - g.cta0[b];
        u.i = b; u.h = r0 % H; u.p = r0 / H;
        unit_shape(g.seq[b], u);
        left = u.ne;
    }
    int it = 0;        // key tiles this block has been through: tile m uses ring stage m % 2, phase (m / 2) & 1
                       // of the stage barriers and phase m & 1 of the per-tile barriers
    int seg = 0;       // segments with key tiles so far (phase of the Q barrier)

    if (warp == 16) {
        // ============================================ producer ============================================
        if (tid == kSoftmaxThreads) {
            bool more = left > 0;
            while (more) {
                const AttendSeq sq = g.seq[u.i];
                const int t1 = min(u.ne, t0 + left);
                const int nreal = max(0, min(t1, u.n) - t0);
                const int h = u.h;
                if (nreal > 0) {
                    // Q of the previous segment is free once both issuers' last Q K^T have completed: their commits
                    // released the K stage of that tile
                    if (kBalanced && it >= 1 && !mbar_wait(&bars.kempty[(it - 1) % kStages], static_cast<uint32_t>((it - 1) / kStages) & 1u)) stuck = true;
                    const int q_row = sq.q_row0 + u.p * BP;
                    mbar_expect_tx(&bars.q, kQBytes);
                    tma_load_2d(base + kOffQ, &maps.Q, h * DH, q_row, &bars.q);
                    tma_load_2d(base + kOffQ + kQHalfBytes, &maps.Q, h * DH + 64, q_row, &bars.q);
                    for (int j = 0; j < nreal; ++j) {
                        const int m = it + j, st = m % kStages;
                        const TileSrc ts = tile_src(sq, u, t0 + j);
                        if (m >= kStages && !mbar_wait(&bars.kempty[st], static_cast<uint32_t>(m / kStages - 1) & 1u)) stuck = true;
                        const uint32_t dk = base + kOffK + st * kKVBytes;
                        mbar_expect_tx(&bars.kfull[st], kKVBytes);
                        tma_load_2d(dk, ts.cache ? &maps.cK : &maps.lK, h * DH, ts.row0, &bars.kfull[st]);
                        tma_load_2d(dk + kKVHalfBytes, ts.cache ? &maps.cK : &maps.lK, h * DH + 64, ts.row0, &bars.kfull[st]);
                        if (m >= kStages && !mbar_wait(&bars.vempty[st], static_cast<uint32_t>(m / kStages - 1) & 1u)) stuck = true;
                        const uint32_t dv = base + kOffV + st * kKVBytes;
                        mbar_expect_tx(&bars.vfull[st], kKVBytes);
                        tma_load_2d(dv, ts.cache ? &maps.cV : &maps.lV, h * DH, ts.row0, &bars.vfull[st]);
                        tma_load_2d(dv + kKVHalfBytes, ts.cache ? &maps.cV : &maps.lV, h * DH + 64, ts.row0, &bars.vfull[st]);
                    }
                    it += nreal;
                    ++seg;
                }
                left -= (t1 - t0);
                t0 = 0;
                more = kBalanced && left > 0 && next_unit(g, H, W, u);
            }
            if (stuck) atomicExch(dev_status, DODO_DEV_WAIT_TIMEOUT);
        }
    } else if (warp == 17 || warp == 18) {
        // ============================================ issuer of query tile qx ============================
        const int qx = warp - 17;
        if ((tid & 31) == 0) {
            const uint32_t tmem_s = tmem + qx * BN, tmem_o = tmem + 2 * BN + qx * DH;
            const uint32_t idesc_qk = idesc_bf16(BN, false), idesc_pv = idesc_bf16(DH, true);
            bool more = left > 0;
            while (more) {
                const int t1 = min(u.ne, t0 + left);
                const int nreal = max(0, min(t1, u.n) - t0);
                if (nreal > 0) {
                    auto issue_qk = [&](int m) {
                        const int st = m % kStages;
                        if (!mbar_wait(&bars.kfull[st], static_cast<uint32_t>(m / kStages) & 1u)) stuck = true;
                        tc_fence_after();
                        const uint64_t a0 = desc_kmajor(base + kOffQ + qx * (kQHalfBytes / 2)), b0 = desc_kmajor(base + kOffK + st * kKVBytes);
#pragma unroll
                        for (int i = 0; i < DH / 16; ++i)
                            mma_bf16(tmem_s, a0 + static_cast<uint64_t>(((i / 4) * kQHalfBytes + (i % 4) * 32) >> 4),
                                     b0 + static_cast<uint64_t>(((i / 4) * kKVHalfBytes + (i % 4) * 32) >> 4), idesc_qk, i > 0);
                        mma_commit(&bars.sready[qx]);
                        mma_commit(&bars.kempty[st]);
                    };
                    if (!mbar_wait(&bars.q, static_cast<uint32_t>(seg) & 1u)) stuck = true;
                    issue_qk(it);
                    for (int j = 0; j < nreal; ++j) {
                        const int m = it + j, st = m % kStages;
                        // P_x(m) is in tensor memory and O_x carries the right scale (and, at the start of a segment,
                        // the softmax threads have taken the previous unit's O_x out)
                        if (!mbar_wait(&bars.pready[qx], static_cast<uint32_t>(m) & 1u)) stuck = true;
                        if (!mbar_wait(&bars.vfull[st], static_cast<uint32_t>(m / kStages) & 1u)) stuck = true;
                        tc_fence_after();
                        const uint64_t b0 = desc_mnmajor(base + kOffV + st * kKVBytes, kKVHalfBytes);
#pragma unroll
                        for (int i = 0; i < BN / 16; ++i)   // 16 keys of P = 8 columns of bf16 pairs; keys 64.. sit 64 columns on
                            mma_bf16_ts(tmem_o, tmem_s + (i / 4) * 64 + (i % 4) * 8, b0 + static_cast<uint64_t>((i * 2048) >> 4), idesc_pv,
                                        j > 0 || i > 0);
                        mma_commit(&bars.odone[qx]);
                        mma_commit(&bars.vempty[st]);
                        if (j + 1 < nreal) issue_qk(m + 1);   // overwrites S_x/P_x(m): same thread, after P V (m)
                    }
                    it += nreal;
                    ++seg;
                }
                left -= (t1 - t0);
                t0 = 0;
                more = kBalanced && left > 0 && next_unit(g, H, W, u);
            }
            if (stuck) atomicExch(dev_status, DODO_DEV_WAIT_TIMEOUT);
        }
    } else {
        // ============================================ softmax of query tile qx ===========================
        // Thread pair (row, half): row = TMEM lane, half 0 owns score columns [0,64) and output columns [0,64).
        const int qx = tid >> 8, gt = tid & 255;
        const int row = gt & (BM - 1), half = gt >> 7;
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tmem_s = tmem + qx * BN + lane_sel + half * 64, tmem_o = tmem + 2 * BN + qx * DH + lane_sel + half * 64;
        float* xch = reinterpret_cast<float*>(base_ptr + kOffXch) + qx * 4 * BM;   // [2][2][BM] of this group
        const float2 c2 = make_float2(scale_log2, scale_log2);
        const int pair_bar = 2 + qx * 4 + (warp & 3);   // the two warps that share these 32 rows
        const int group_bar = 10 + qx;                  // the 256 threads of this query tile
        bool first_seg = true;

        bool more = left > 0;
        while (more) {
            const AttendSeq sq = g.seq[u.i];
            const int ne = u.ne;
            const int t1 = min(ne, t0 + left);
            const int nreal = max(0, min(t1, u.n) - t0);
            const int h = u.h, q_first = u.p * BP + qx * BM;
            const int nq = max(0, min(BM, sq.tq - q_first));
            const bool row_live = row < nq;
            const int my_qpos = row_live ? sq.q_pos0 + q_first + row : static_cast<int>(0x80000000);
            const int min_qpos = sq.q_pos0 + q_first;
            float m_ref = kNeg, l = 0.f;

            if (nreal > 0) {
                {   // first cache tile holding a key that some query of this tile must not see
                    int bad = 0x7fffffff;
                    for (int i = gt; i < sq.c_len; i += kGroupThreads)
                        if (__ldg(cache_pos + sq.c_row0 + i) > min_qpos) bad = min(bad, i / BN);
                    if (bad != 0x7fffffff) atomicMin(&first_masked[qx][seg & 1], bad);
                    if (kBalanced && gt == 0) first_masked[qx][(seg + 1) & 1] = 0x7fffffff;
                    asm volatile("bar.sync %0, 256;" ::"r"(group_bar) : "memory");
                }
                const int first_bad = first_masked[qx][seg & 1];

                for (int j = 0; j < nreal; ++j) {
                    const int t = t0 + j, m = it + j;
                    const int st = m % kStages;
                    const TileSrc ts = tile_src(sq, u, t);
                    const bool need_mask = ts.rows < BN || (ts.cache ? t >= first_bad : ts.pos0 + ts.rows - 1 > min_qpos);

                    if (!mbar_wait(&bars.sready[qx], static_cast<uint32_t>(m) & 1u)) stuck = true;
                    tc_fence_after();
                    // ---- pass 1: the row maximum of this thread's 64 raw scores -----------------------------------
                    float tmax = kNeg;
#pragma unroll 1
                    for (int cc = 0; cc < 2; ++cc) {
                        uint32_t sv[32];
                        tmem_ld32(tmem_s + cc * 32, sv);
                        if (need_mask) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) {
                                const int col = half * 64 + cc * 32 + c;
                                int kp = 0x7fffffff;
                                if (col < ts.rows) kp = ts.cache ? __ldg(cache_pos + ts.row0 + col) : ts.pos0 + col;
                                if (kp > my_qpos) sv[c] = __float_as_uint(kNeg);
                            }
                        }
#pragma unroll
                        for (int c = 0; c < 32; c += 2) tmax = max3(tmax, __uint_as_float(sv[c]), __uint_as_float(sv[c + 1]));
                    }
                    tmax = tmax > 0.5f * kNeg ? tmax * scale_log2 : kNeg;
                    float* xm = xch + (m & 1) * 2 * BM;
                    xm[half * BM + row] = tmax;
                    asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
                    tmax = fmaxf(tmax, xm[(half ^ 1) * BM + row]);

                    const bool grow = tmax > m_ref + kRescaleStep;
                    const float m_new = grow ? tmax : m_ref;
                    if (j > 0 && __any_sync(0xffffffffu, grow)) {
                        if (!mbar_wait(&bars.odone[qx], static_cast<uint32_t>(m - 1) & 1u)) stuck = true;
                        tc_fence_after();
                        const float corr = ex2_approx(m_ref - m_new);
                        l *= corr;
#pragma unroll 1
                        for (int c = 0; c < 2; ++c) {
                            uint32_t ov[32];
                            tmem_ld32(tmem_o + c * 32, ov);
#pragma unroll
                            for (int e = 0; e < 32; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * corr);
                            tmem_st32(tmem_o + c * 32, ov);
                        }
                    }
                    m_ref = m_new;

                    if (ts.rows < BN) {   // rows of V past the segment's end must not reach P V (both groups write the zeros)
                        if (!mbar_wait(&bars.vfull[st], static_cast<uint32_t>(m / kStages) & 1u)) stuck = true;
                        unsigned char* v0 = base_ptr + kOffV + st * kKVBytes;
                        for (int i = gt; i < (BN - ts.rows) * 16; i += kGroupThreads) {
                            const int vrow = ts.rows + i / 16, piece = i % 16;
                            *reinterpret_cast<uint4*>(v0 + (piece / 8) * kKVHalfBytes + vrow * 128 + (piece % 8) * 16) = make_uint4(0, 0, 0, 0);
                        }
                    }

                    // ---- pass 2: P = 2^(scale s - m_ref) as bf16 pairs over the first 32 of this thread's columns ----
                    const float nm = -fmaxf(m_ref, -1.0e20f);
                    const float2 nm2 = make_float2(nm, nm);
                    float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll 1
                    for (int cc = 0; cc < 2; ++cc) {
                        uint32_t sv[32];
                        tmem_ld32(tmem_s + cc * 32, sv);
                        if (need_mask) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) {
                                const int col = half * 64 + cc * 32 + c;
                                int kp = 0x7fffffff;
                                if (col < ts.rows) kp = ts.cache ? __ldg(cache_pos + ts.row0 + col) : ts.pos0 + col;
                                if (kp > my_qpos) sv[c] = __float_as_uint(kNeg);
                            }
                        }
                        uint32_t packed[16];
#pragma unroll
                        for (int c = 0; c < 16; c += 2) {
                            const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(sv[2 * c]), __uint_as_float(sv[2 * c + 1])), c2, nm2);
                            const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(sv[2 * c + 2]), __uint_as_float(sv[2 * c + 3])), c2, nm2);
                            const float2 p0 = make_float2(ex2_approx(x0.x), ex2_approx(x0.y));
                            const float2 p1 = make_float2(ex2_approx(x1.x), ex2_approx(x1.y));
                            packed[c] = pack_bf16(p0.x, p0.y);
                            packed[c + 1] = pack_bf16(p1.x, p1.y);
                            acc0 = __fadd2_rn(acc0, p0);
                            acc1 = __fadd2_rn(acc1, p1);
                        }
                        // columns [16 cc, 16 cc + 16) of this thread's part: scores already read (cc = 0) or further on
                        tmem_st16(tmem_s + cc * 16, packed);
                    }
                    l += (acc0.x + acc0.y) + (acc1.x + acc1.y);
                    if (ts.rows < BN) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    tc_fence_before();
                    mbar_arrive(&bars.pready[qx]);
                }

                asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
                xch[half * BM + row] = l;
                asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
                l += xch[(half ^ 1) * BM + row];
                if (kBalanced) asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
                if (!mbar_wait(&bars.odone[qx], static_cast<uint32_t>(it + nreal - 1) & 1u)) stuck = true;
                tc_fence_after();
            }

            const size_t orow = static_cast<size_t>(sq.q_row0 + q_first + row) * H + h;
            const bool whole = !kBalanced || (t0 == 0 && t1 == ne);
            if (whole) {
                const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll 1
                for (int c = 0; c < 2; ++c) {
                    uint32_t ov[32];
                    if (nreal > 0) {
                        tmem_ld32(tmem_o + c * 32, ov);
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) ov[e] = 0u;
                    }
                    if (row_live) {
                        uint4* dst = reinterpret_cast<uint4*>(O + orow * DH + half * 64 + c * 32);
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
                if (row_live && half == 0 && lse != nullptr)
                    lse[orow] = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
            } else {
                // a cut unit: this tile's unnormalised partial to the workspace; the last piece to arrive merges
                const int xu = x - t0;
                const int c_first = block_of(T, G, xu), c_last = block_of(T, G, xu + ne - 1);
                float* ps = work.partials + (static_cast<size_t>(2 * bid + (first_seg ? 0 : 1)) * 2 + qx) * kPartFloats;
#pragma unroll 1
                for (int c = 0; c < 2; ++c) {
                    uint32_t ov[32];
                    if (nreal > 0) {
                        tmem_ld32(tmem_o + c * 32, ov);
                    } else {
#pragma unroll
                        for (int e = 0; e < 32; ++e) ov[e] = 0u;
                    }
                    float* dst = ps + (half * 64 + c * 32) * BM + row;
#pragma unroll
                    for (int e = 0; e < 32; ++e) dst[e * BM] = __uint_as_float(ov[e]);
                }
                if (half == 0) { ps[BM * DH + row] = m_ref; ps[BM * DH + BM + row] = l; }
                __threadfence();
                asm volatile("bar.sync %0, 256;" ::"r"(group_bar) : "memory");
                if (gt == 0) {
                    int* tk = work.tickets + (g.cta0[u.i] + u.p * H + h) * 2 + qx;
                    const int arrived = atomicAdd(tk, 1);
                    s_last[qx] = arrived == c_last - c_first;
                    if (s_last[qx]) *tk = 0;
                }
                asm volatile("bar.sync %0, 256;" ::"r"(group_bar) : "memory");
                if (s_last[qx]) {
                    __threadfence();
                    auto piece = [&](int c) -> const float* {
                        return work.partials + (static_cast<size_t>(2 * (c * W + bid % W) + (block_start(T, G, c) >= xu ? 0 : 1)) * 2 + qx) * kPartFloats;
                    };
                    float M = kNeg;
                    for (int c = c_first; c <= c_last; ++c) M = fmaxf(M, __ldcg(piece(c) + BM * DH + row));
                    float L = 0.f;
                    for (int c = c_first; c <= c_last; ++c) {
                        const float* pc = piece(c);
                        L = fmaf(__ldcg(pc + BM * DH + BM + row), ex2_approx(__ldcg(pc + BM * DH + row) - M), L);
                    }
                    const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll 1
                    for (int cc = 0; cc < 2; ++cc) {
                        float o[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = 0.f;
                        for (int c = c_first; c <= c_last; ++c) {
                            const float* pc = piece(c);
                            const float w = ex2_approx(__ldcg(pc + BM * DH + row) - M);
                            const float* src = pc + (half * 64 + cc * 32) * BM + row;
#pragma unroll
                            for (int e = 0; e < 32; ++e) o[e] = fmaf(__ldcg(src + e * BM), w, o[e]);
                        }
                        if (row_live) {
                            uint4* dst = reinterpret_cast<uint4*>(O + orow * DH + half * 64 + cc * 32);
#pragma unroll
                            for (int q = 0; q < 4; ++q)
                                dst[q] = make_uint4(pack_bf16(o[8 * q] * inv, o[8 * q + 1] * inv), pack_bf16(o[8 * q + 2] * inv, o[8 * q + 3] * inv),
                                                    pack_bf16(o[8 * q + 4] * inv, o[8 * q + 5] * inv), pack_bf16(o[8 * q + 6] * inv, o[8 * q + 7] * inv));
                        }
                    }
                    if (row_live && half == 0 && lse != nullptr)
                        lse[orow] = L > 0.f ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
                }
                asm volatile("bar.sync %0, 256;" ::"r"(group_bar) : "memory");
            }
            if (nreal > 0) { it += nreal; ++seg; }
            first_seg = false;
            left -= (t1 - t0);
            x += (t1 - t0);
            t0 = 0;
            more = kBalanced && left > 0 && next_unit(g, H, W, u);
        }
        if (stuck) atomicExch(dev_status, DODO_DEV_WAIT_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 16)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

}  // namespace

int dodo_dense2_pair_queries() { return BP; }
int dodo_dense2_tile_keys() { return BN; }

int dodo_launch_attend_dense2(dodo_ctx* ctx, int H, float sm_scale, const AttendGroup& g, const DenseMaps& maps,
                              const int32_t* cache_pos, void* O, float* lse, void* workspace, size_t workspace_bytes,
                              int* tickets, int* dev_status, cudaStream_t st) {
    const int units = g.cta0[g.nseq];   // planned with query tiles of BP rows
    if (units == 0) return DODO_OK;
    auto unit_tiles = [](const AttendSeq& sq, int p) {
        const int q_first = p * BP, nq = sq.tq - q_first < BP ? sq.tq - q_first : BP;
        int l_vis = sq.q_pos0 + q_first + nq - 1 - sq.l_pos0 + 1;
        l_vis = l_vis < sq.l_len ? l_vis : sq.l_len;
        l_vis = l_vis > 0 ? l_vis : 0;
        return (sq.c_len + BN - 1) / BN + (l_vis + BN - 1) / BN;
    };
    long long total = 0, total_step = 0;
    int width = 0;
    for (int i = 0; i < g.nseq; ++i) {
        const AttendSeq& sq = g.seq[i];
        if (sq.tq <= 0) continue;
        const int pairs = (sq.tq + BP - 1) / BP;
        width = width == 0 || width == pairs ? pairs : -1;
        for (int p = 0; p < pairs; ++p) {
            const int n = unit_tiles(sq, p);
            total += static_cast<long long>(n > 0 ? n : 1) * H;
        }
        const int n_last = unit_tiles(sq, pairs - 1);
        total_step += static_cast<long long>(n_last > 0 ? n_last : 1) * H;
    }
    const int resident = ctx->num_sms;   // one block per SM
    const bool room = total < 0x7fffffff && total >= 2 && workspace != nullptr && dodo_aligned16(workspace) &&
                      workspace_bytes >= dodo_dense_workspace_bytes(ctx->num_sms) && 2 * units <= DODO_NUM_TICKETS;
    const bool pays = units % resident != 0 && units < 4 * resident && total / units >= 24;
    const bool balanced = room && ctx->dense_balance != 2 && (pays || ctx->dense_balance == 1 || ctx->dense_balance == 3);
    const bool in_step = balanced && ctx->dense_balance != 3 && width >= 2 && width <= resident;
    DenseWork2 work;
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
    auto kern = balanced ? attend_dense2_kernel<true> : attend_dense2_kernel<false>;
    if (!ctx->dense2_attr_set[balanced ? 1 : 0]) {
        const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "dense attend (two query tiles) shared-memory attribute");
        ctx->dense2_attr_set[balanced ? 1 : 0] = true;
    }
    kern<<<grid, kThreads, smem, st>>>(maps, g, cache_pos, H, sm_scale * 1.4426950408889634f,
                                       static_cast<__nv_bfloat16*>(O), lse, work, dev_status);
    return dodo_check_cuda(ctx, cudaGetLastError(), "dense attend (two query tiles) launch");
}
