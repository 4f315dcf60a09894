// Attention of a block of query tokens over [nugget cache ; local tokens] (Eq. 13, Eq. 9) on the
// 5th-generation tensor cores: tcgen05.mma with TMEM accumulators, operands staged by TMA.
// bf16, head size 128.  This is the dense case, where many queries share every K/V tile and the
// work is a contraction (about Tq flop per K/V byte); single-token decode stays on the HBM-bound
// kernel in attend.cu.
//
// A unit of work is (sequence, tile of 128 query tokens, head).  A thread block takes one unit, or, in the
// balanced form of the kernel, an equal share of all key tiles whatever units they belong to (see
// DenseWork below).  Keys come in tiles of 64; tile m of a block uses S/P buffer m & 1 of tensor memory.
// Three roles, each waiting only for what it consumes:
//   issuer of Q K^T (one lane of warp 8)  plain per-block TMA tensor copies with the 128-byte swizzle bring the
//       Q tile once and K tiles through a two-stage ring; S = Q K^T as 8 x tcgen05.mma M128 N64 K16 (both
//       operands K-major in shared memory) into the tile's S buffer, as soon as K has landed and the buffer
//       is free, i.e. P V of the tile two before has completed: up to two tiles ahead of the softmax.
//   issuer of P V (one lane of warp 9)  V tiles through a two-stage ring; O += P V as 4 x tcgen05.mma M128
//       N128 K16 (A = P read from tensor memory, B = V MN-major, i.e. V rows as stored) into TMEM columns
//       [128,256) once the softmax threads have published P.
//   softmax (warps 0-7; two threads per query row = TMEM lane, each owning half of the score and output
//       columns)  reads its part of the row of S with tcgen05.ld, masks by position only on tiles that need
//       it (key visible iff key_pos <= q_pos; rows past a segment's end carry INT_MAX), keeps the running
//       max and sum in the base-2 domain and writes P as bf16 pairs over the first 32 columns of the S
//       buffer it came from.  O stays in TMEM across tiles; it is rescaled (tcgen05.ld / tcgen05.st) only
//       when a row's maximum has grown by more than 2^8 since the reference maximum was last moved, and
//       only then do these threads wait for a P V.
// Two blocks share an SM (96 KB of shared memory and 256 TMEM columns each) and fill each other's gaps.
// One round to bf16 at the end; optional log-sum-exp (from the unrounded weights).
// V rows past the end of a segment are zeroed in shared memory before use, so that whatever lies
// behind a sequence's region (another sequence, unused capacity) can never reach the product P V.
// Every wait is bounded; on time-out a status word is set and the block runs on to its end, where
// it always frees its TMEM columns.
//
// Gathered form (kGathered): there is no nugget cache.  The "cache" segment of a sequence is the list of its
// selected positions idx, and the K and V tiles of that segment are assembled in shared memory from the
// uncompressed K and V arrays by row-gather tensor copies (cp.async.bulk.tensor ... tile::gather4: four rows per
// instruction, named by four row coordinates, through a tensor map whose box is one row high), one selection
// serving the query block without a gather launch and without a cache written and read back (Sec. 2.1,
// Eq. 13).  The 32 gather copies of a 64-key tile are issued by the 32 lanes of the issuer's warp at once; the
// nuggets' positions for the mask are pos_base + idx.  Everything else is the same code.
#include "dodo_internal.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int DH = 128;               // head size
constexpr int BM = 128;               // query rows per block = TMEM lanes
constexpr int BN = 64;                // keys per tile (128 also works below: one block per SM then, measured slower)
constexpr int kSoftmaxThreads = 256;      // two threads per query row, each owning half of the columns
constexpr int kThreads = kSoftmaxThreads + 64;   // + the two issuer warps
constexpr int kQHalfBytes = 128 * 128;   // 64 columns of a 128-row bf16 tile, rows of 128 bytes
constexpr int kQBytes = 2 * kQHalfBytes;
constexpr int kKVHalfBytes = BN * 128;   // 64 columns of a 64-row tile
constexpr int kKVBytes = 2 * kKVHalfBytes;
constexpr int kStages = 2;              // 96 KB of shared memory per block: two blocks per SM
constexpr int kBlocksPerSM = BN == 64 ? 2 : 1;
constexpr uint32_t kTmemCols = BN == 64 ? 256 : 512;      // S of even / odd tiles: columns [0,64) / [64,128); P (bf16 pairs) of a tile takes over
                                         // the first 32 columns of its S once S is in registers; O: [128,256)
constexpr uint32_t kTmemO = 2 * BN;
constexpr float kNeg = -1.0e30f;
constexpr int kBalanceMinTiles = 48 * 64 / BN;      // balance by default only when a unit has about this many key tiles
constexpr float kRescaleStep = 8.f;      // move a row's reference maximum only past this many octaves

// shared-memory map (bytes from the 1024-aligned base)
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + kQBytes;
constexpr int kOffV = kOffK + kStages * kKVBytes;
constexpr int kOffXch = kOffV + kStages * kKVBytes;    // float[2][2][BM] row maxima / sums exchanged by a row's two threads
constexpr int kSmemBytes = kOffXch + 2 * 2 * BM * 4;

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

// A unit of work is (sequence, tile of 128 queries, head); its key list is cut into tiles of BN keys.
struct Unit {
    int i, qt, h;    // sequence of the group, query tile, head
    int nt_c;        // key tiles in the nugget cache
    int l_vis;       // local rows at least one query of the tile can see
    int n;           // key tiles in all
    int ne;          // slots the unit takes in the balanced order: max(1, n), or that of the sequence's
                     // last query tile when the query tiles of a head walk the keys in step (width > 1)
};
__device__ __forceinline__ void unit_shape(const AttendSeq& sq, Unit& u) {
    const int q_first = u.qt * BM, nq = min(BM, sq.tq - q_first);
    u.l_vis = max(0, min(sq.l_len, sq.q_pos0 + q_first + nq - 1 - sq.l_pos0 + 1));
    u.nt_c = (sq.c_len + BN - 1) / BN;
    u.n = u.nt_c + (u.l_vis + BN - 1) / BN;
    u.ne = max(1, u.n);
}
// width > 1: every sequence has `width` query tiles; the slot count is the last (longest) tile's
__device__ __forceinline__ void unit_shape(const AttendSeq& sq, Unit& u, int width) {
    unit_shape(sq, u);
    if (width > 1) {
        Unit last = u;
        last.qt = width - 1;
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
// The unit after u in the order (sequence, query tile, head), heads fastest; with width > 1 the query
// tile stays what it is and the order is (sequence, head).  False past the last one.
__device__ __forceinline__ bool next_unit(const AttendGroup& g, int H, int width, Unit& u) {
    if (++u.h < H) return true;
    u.h = 0;
    if (width == 1) {
        if (++u.qt * BM < g.seq[u.i].tq) { unit_shape(g.seq[u.i], u); return true; }
        u.qt = 0;
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
// In step (width W > 1, every sequence has W query tiles): blocks come in groups of W, block c = group c / W,
// query tile c % W; the groups share out the slots of the (sequence, head) pairs, counted by the longest
// query tile, and the W blocks of a group pass the same key tiles at about the same time, so that a
// head's K/V is fetched from HBM once and found in L2 by the other W - 1.
struct DenseWork {
    int total_slots;         // T
    int width;               // W
    float* partials;         // [2 * gridDim.x] x (DH x BM outputs, BM maxima, BM sums), balanced only
    int* tickets;            // one arrival counter per unit of the launch, zero between launches
};
constexpr int kPartFloats = BM * DH + 2 * BM;

__device__ __forceinline__ int block_start(int T, int G, int c) { return static_cast<int>(static_cast<long long>(c) * T / G); }
__device__ __forceinline__ int block_of(int T, int G, int x) {   // the block whose range holds slot x
    return static_cast<int>(((static_cast<long long>(x) + 1) * G - 1) / T);
}

__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* map, int x, int r0, int r1, int r2, int r3, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(smem_u32(bar))
        : "memory");
}

// Gathered form: the 32 lanes of a warp bring one 64-key tile (two halves of 64 columns) of the rows idx names:
// lane = (half, group of four keys).  Slots past the segment's end repeat its last row (they are masked, and
// their V rows zeroed, like every tile tail).  An index outside its sequence is clamped and reported.
__device__ __forceinline__ void gather_tile(uint32_t dst, const CUtensorMap* map, int col0, const int32_t* __restrict__ idx,
                                            int slot0, int rows, int src_row0, int src_n, uint64_t* bar, int* dev_status) {
    static_assert(BN == 64, "one gather copy per lane covers a 64-key tile");
    const int lane = threadIdx.x & 31, grp = lane & 15, half = lane >> 4;
    int r[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int j = min(4 * grp + e, rows - 1);
        int tok = __ldg(idx + slot0 + j);
        if (static_cast<unsigned>(tok) >= static_cast<unsigned>(src_n)) {
            atomicOr(dev_status, DODO_DEV_BAD_INDEX);
            tok = min(max(tok, 0), src_n - 1);
        }
        r[e] = src_row0 + tok;
    }
    tma_gather4(dst + half * kKVHalfBytes + grp * 512, map, col0 + half * 64, r[0], r[1], r[2], r[3], bar);
}

// cache_pos: positions of the cache rows; gathered form: the selected positions idx (sequence-local), and
// AttendSeq::c_row0 / c_len name a sequence's slots in it.
template <bool kBalanced, bool kGathered>
__global__ void __launch_bounds__(kThreads, kBlocksPerSM)
attend_dense_kernel(const __grid_constant__ DenseMaps maps, const __grid_constant__ AttendGroup g,
                    const int32_t* __restrict__ cache_pos, int H, float scale_log2,
                    __nv_bfloat16* __restrict__ O, float* __restrict__ lse, const DenseWork work,
                    int* __restrict__ dev_status, const __grid_constant__ DenseGather gs) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    __shared__ __align__(8) uint64_t bar_q, bar_s[2], bar_o[2], bar_pready[2], bar_kfull[kStages], bar_vfull[kStages];
    __shared__ uint32_t tmem_slot;
    __shared__ int first_masked[2];
    __shared__ int s_start[4];      // balanced: the block's first unit and tile (i, qt, h, t)
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
        for (int b = 0; b < 2; ++b) { mbar_init(&bar_s[b], 1); mbar_init(&bar_o[b], 1); mbar_init(&bar_pready[b], kSoftmaxThreads / 32); }
        for (int s = 0; s < kStages; ++s) { mbar_init(&bar_kfull[s], 1); mbar_init(&bar_vfull[s], 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (kBalanced) {
            // walk the (sequence, query tile) groups up to the one that holds this block's first slot
            Unit w;
            w.i = 0; w.qt = 0; w.h = 0;
            int t = 0, acc = 0;
            const int x0 = block_start(T, G, grp);
            bool found = false;
            for (int i = 0; i < g.nseq && !found; ++i) {
                for (int qt = (W > 1 ? bid % W : 0); qt * BM < g.seq[i].tq && !found; qt += (W > 1 ? W : 1)) {
                    w.i = i; w.qt = qt;
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
            s_start[0] = w.i; s_start[1] = w.qt; s_start[2] = w.h; s_start[3] = t;
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
    const uint32_t tmem_o = tmem + kTmemO;
    bool stuck = false;

    // Both roles go through the same list of segments = (unit, key tiles [t0, t1)); plain: one whole unit.
    Unit u;
    int t0 = 0, x = 0, left;
    if (kBalanced) {
        u.i = s_start[0]; u.qt = s_start[1]; u.h = s_start[2]; t0 = s_start[3];
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
        u.i = b; u.h = r0 % H; u.qt = r0 / H;
        unit_shape(g.seq[b], u);
        left = u.ne;
    }
    int it = 0;        // key tiles this block has been through (barrier phases and ring stages run on)
    int seg = 0;       // segments with key tiles so far (phase of the Q barrier)

    // Tile m of this block (m counts on through its segments) lives in S/P buffer m & 1 and in ring stage
    // m % kStages; the barriers of buffer b complete once per two tiles, so tile m waits for their phase m >> 1.
    // Nobody can be two phases ahead of a waiter: Q K^T of tile m+2 needs P V of tile m, which needs the softmax
    // of tile m, which needs Q K^T of tile m.
    if (warp == kSoftmaxThreads / 32) {
        // ============================ issuer of Q K^T: Q and K copies, S = Q K^T ============================
        const bool lead = (tid & 31) == 0;      // the issuing lane; gathered form: the other lanes help with the row copies
        if (kGathered || lead) {
            bool more = left > 0;
            while (more) {
                const AttendSeq sq = g.seq[u.i];
                const int ne = u.ne;
                const int t1 = min(ne, t0 + left);
                const int nreal = max(0, min(t1, u.n) - t0);   // this query tile's own key tiles in the segment
                const int h = u.h;
                if (nreal > 0) {
                    auto load_k = [&](int t, int m) {
                        const int st = m % kStages;
                        const TileSrc ts = tile_src(sq, u, t);
                        const CUtensorMap* mk = ts.cache ? &maps.cK : &maps.lK;
                        const uint32_t dk = base + kOffK + st * kKVBytes;
                        if (lead) mbar_expect_tx(&bar_kfull[st], kKVBytes);
                        if (kGathered && ts.cache) {
                            __syncwarp();      // the lead lane's waits for this stage are behind it
                            gather_tile(dk, mk, h * DH, cache_pos, ts.row0, ts.rows, gs.row0[u.i], gs.n[u.i], &bar_kfull[st], dev_status);
                        } else if (lead) {
                            tma_load_2d(dk, mk, h * DH, ts.row0, &bar_kfull[st]);
                            tma_load_2d(dk + kKVHalfBytes, mk, h * DH + 64, ts.row0, &bar_kfull[st]);
                        }
                    };
                    // a later segment: Q and the K stages are free once the last Q K^T before has completed
                    if (lead && kBalanced && it >= 1 && !mbar_wait(&bar_s[(it - 1) & 1], static_cast<uint32_t>((it - 1) >> 1) & 1u)) stuck = true;
                    const int q_row = sq.q_row0 + u.qt * BM;
                    if (lead) {
                        mbar_expect_tx(&bar_q, kQBytes);
                        tma_load_2d(base + kOffQ, &maps.Q, h * DH, q_row, &bar_q);
                        tma_load_2d(base + kOffQ + kQHalfBytes, &maps.Q, h * DH + 64, q_row, &bar_q);
                    }
                    for (int j = 0; j < min(kStages, nreal); ++j) load_k(t0 + j, it + j);
                    if (lead && !mbar_wait(&bar_q, static_cast<uint32_t>(seg) & 1u)) stuck = true;
                    for (int j = 0; j < nreal; ++j) {
                        const int m = it + j, b = m & 1, st = m % kStages;
                        // first of all the copy for the tile after this one: its K stage is the one of the tile
                        // before, free once that tile's Q K^T (issued an iteration ago) has completed
                        if (j >= 1 && j - 1 + kStages < nreal) {
                            if (lead && !mbar_wait(&bar_s[(m - 1) & 1], static_cast<uint32_t>((m - 1) >> 1) & 1u)) stuck = true;
                            load_k(t0 + j - 1 + kStages, m - 1 + kStages);
                        }
                        // the buffer is free once P V of the tile two before has consumed its P
                        if (lead && m >= 2 && !mbar_wait(&bar_o[b], static_cast<uint32_t>((m - 2) >> 1) & 1u)) stuck = true;
                        if (lead && !mbar_wait(&bar_kfull[st], static_cast<uint32_t>(m / kStages) & 1u)) stuck = true;
                        if (lead) {
                            tc_fence_after();
                            // descriptors differ only in their start-address field (units of 16 bytes)
                            const uint64_t a0 = desc_kmajor(base + kOffQ), b0 = desc_kmajor(base + kOffK + st * kKVBytes);
                            const uint32_t idesc = idesc_bf16(BN, false);
#pragma unroll
                            for (int i = 0; i < DH / 16; ++i)
                                mma_bf16(tmem + b * BN, a0 + static_cast<uint64_t>(((i / 4) * kQHalfBytes + (i % 4) * 32) >> 4),
                                         b0 + static_cast<uint64_t>(((i / 4) * kKVHalfBytes + (i % 4) * 32) >> 4), idesc, i > 0);
                            mma_commit(&bar_s[b]);
                        }
                    }
                    it += nreal;
                    ++seg;
                }
                left -= (t1 - t0);
                x += (t1 - t0);
                t0 = 0;
                more = kBalanced && left > 0 && next_unit(g, H, W, u);
            }
            if (stuck) atomicOr(dev_status, DODO_DEV_WAIT_TIMEOUT);
        }
    } else if (warp == kSoftmaxThreads / 32 + 1) {
        // ============================ issuer of P V: V copies, O += P V ==========================================
        const bool lead = (tid & 31) == 0;
        if (kGathered || lead) {
            bool more = left > 0;
            while (more) {
                const AttendSeq sq = g.seq[u.i];
                const int ne = u.ne;
                const int t1 = min(ne, t0 + left);
                const int nreal = max(0, min(t1, u.n) - t0);
                const int h = u.h;
                if (nreal > 0) {
                    auto load_v = [&](int t, int m) {
                        const int st = m % kStages;
                        const TileSrc ts = tile_src(sq, u, t);
                        const CUtensorMap* mv = ts.cache ? &maps.cV : &maps.lV;
                        const uint32_t dv = base + kOffV + st * kKVBytes;
                        if (lead) mbar_expect_tx(&bar_vfull[st], kKVBytes);
                        if (kGathered && ts.cache) {
                            __syncwarp();      // the lead lane's waits for this stage are behind it
                            gather_tile(dv, mv, h * DH, cache_pos, ts.row0, ts.rows, gs.row0[u.i], gs.n[u.i], &bar_vfull[st], dev_status);
                        } else if (lead) {
                            tma_load_2d(dv, mv, h * DH, ts.row0, &bar_vfull[st]);
                            tma_load_2d(dv + kKVHalfBytes, mv, h * DH + 64, ts.row0, &bar_vfull[st]);
                        }
                    };
                    // a later segment: the V stages are free once the last P V before has completed
                    if (lead && kBalanced && it >= 1 && !mbar_wait(&bar_o[(it - 1) & 1], static_cast<uint32_t>((it - 1) >> 1) & 1u)) stuck = true;
                    for (int j = 0; j < min(kStages, nreal); ++j) load_v(t0 + j, it + j);
                    for (int j = 0; j < nreal; ++j) {
                        const int m = it + j, b = m & 1, st = m % kStages;
                        // first the copy for the tile after this one: its V stage is the one of the tile before,
                        // free once that tile's P V has completed
                        if (j >= 1 && j - 1 + kStages < nreal) {
                            if (lead && !mbar_wait(&bar_o[(m - 1) & 1], static_cast<uint32_t>((m - 1) >> 1) & 1u)) stuck = true;
                            load_v(t0 + j - 1 + kStages, m - 1 + kStages);
                        }
                        // P(m) is in tensor memory and O carries the right scale (and, at the start of a segment,
                        // the softmax threads have taken the previous unit's O out)
                        if (lead && !mbar_wait(&bar_pready[b], static_cast<uint32_t>(m >> 1) & 1u)) stuck = true;
                        if (lead && !mbar_wait(&bar_vfull[st], static_cast<uint32_t>(m / kStages) & 1u)) stuck = true;
                        if (lead) {
                            tc_fence_after();
                            const uint64_t b0 = desc_mnmajor(base + kOffV + st * kKVBytes, kKVHalfBytes);
                            const uint32_t idesc = idesc_bf16(DH, true);
#pragma unroll
                            for (int i = 0; i < BN / 16; ++i)   // 16 keys of P = 8 columns of bf16 pairs
                                mma_bf16_ts(tmem_o, tmem + b * BN + i * 8, b0 + static_cast<uint64_t>((i * 2048) >> 4), idesc, j > 0 || i > 0);
                            mma_commit(&bar_o[b]);
                        }
                    }
                    it += nreal;
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
        // Thread pair (row, half): row = TMEM lane, half 0 owns score columns [0,32) and output
        // columns [0,64), half 1 the rest.  Warps w and w+4 cover the same 32 lanes.
        const int row = tid & (BM - 1), half = tid >> 7;
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;   // this warp's TMEM lanes
        float* xch = reinterpret_cast<float*>(base_ptr + kOffXch);                 // [2][2][BM]
        constexpr int HN = BN / 2;   // score columns per thread
        const float2 c2 = make_float2(scale_log2, scale_log2);
        const int pair_bar = 2 + (warp & 3);   // named barrier of the two warps that share these 32 rows
        bool first_seg = true;

        bool more = left > 0;
        while (more) {
            const AttendSeq sq = g.seq[u.i];
            const int ne = u.ne;
            const int t1 = min(ne, t0 + left);
            const int nreal = max(0, min(t1, u.n) - t0);   // this query tile's own key tiles in the segment
            const int h = u.h, q_first = u.qt * BM;
            const int nq = min(BM, sq.tq - q_first);
            const bool row_live = row < nq;
            const int my_qpos = row_live ? sq.q_pos0 + q_first + row : static_cast<int>(0x80000000);
            const int min_qpos = sq.q_pos0 + q_first;
            const int pos_add = kGathered ? gs.pos_base[u.i] : 0;     // gathered form: cache_pos holds sequence-local indices
            float m_ref = kNeg, l = 0.f;   // l: sum of the unrounded weights over this thread's columns

            if (nreal > 0) {
                // First cache tile holding a key that some query of this tile must not see (nuggets normally
                // all precede the block, so this is nt_c and no cache tile pays for the position test).
                {
                    int bad = 0x7fffffff;
                    for (int i = tid; i < sq.c_len; i += kSoftmaxThreads)
                        if (__ldg(cache_pos + sq.c_row0 + i) + pos_add > min_qpos) bad = min(bad, i / BN);
                    if (bad != 0x7fffffff) atomicMin(&first_masked[seg & 1], bad);
                    if (kBalanced && tid == 0) first_masked[(seg + 1) & 1] = 0x7fffffff;   // for the next segment; its users are past
                    asm volatile("bar.sync 1, 256;" ::: "memory");
                }
                const int first_bad = first_masked[seg & 1];

                for (int j = 0; j < nreal; ++j) {
                    const int t = t0 + j, m = it + j;
                    const int st = m % kStages;
                    const TileSrc ts = tile_src(sq, u, t);
                    // a position test only where some key of the tile may lie behind some query; a tile that is merely
                    // short masks its missing columns without looking anything up
                    const bool need_pos = ts.cache ? t >= first_bad : ts.pos0 + ts.rows - 1 > min_qpos;

                    const int sb = m & 1;                             // S/P buffer of this tile
                    const uint32_t tmem_sp = tmem + sb * BN + lane_sel;
                    if (!mbar_wait(&bar_s[sb], static_cast<uint32_t>(m >> 1) & 1u)) stuck = true;
                    tc_fence_after();
                    uint32_t sv[HN];   // raw scores q.k; the softmax scale enters in the exponent's FMA
#pragma unroll
                    for (int c = 0; c < HN / 32; ++c) tmem_ld32(tmem_sp + half * HN + c * 32, sv + c * 32);

                    if (need_pos) {
#pragma unroll
                        for (int c = 0; c < HN; ++c) {
                            const int col = half * HN + c;
                            int kp = 0x7fffffff;
                            if (col < ts.rows) kp = ts.cache ? __ldg(cache_pos + ts.row0 + col) + pos_add : ts.pos0 + col;
                            if (kp > my_qpos) sv[c] = __float_as_uint(kNeg);
                        }
                    } else if (ts.rows < BN) {
#pragma unroll
                        for (int c = 0; c < HN; ++c)
                            if (half * HN + c >= ts.rows || !row_live) sv[c] = __float_as_uint(kNeg);
                    }
                    float tmax = fmaxf(__uint_as_float(sv[0]), __uint_as_float(sv[1]));
#pragma unroll
                    for (int c = 2; c < HN; c += 2) tmax = max3(tmax, __uint_as_float(sv[c]), __uint_as_float(sv[c + 1]));
                    tmax = tmax > 0.5f * kNeg ? tmax * scale_log2 : kNeg;   // base-2 domain; kNeg = nothing visible
                    // the row's two threads agree on the tile maximum through shared memory
                    float* xm = xch + (m & 1) * 2 * BM;
                    xm[half * BM + row] = tmax;
                    asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
                    tmax = fmaxf(tmax, xm[(half ^ 1) * BM + row]);

                    // move the reference maximum only when it pays; rescale O in TMEM when any row of the warp moved,
                    // which needs P V of the tile before complete (at the start of a segment O holds nothing yet)
                    const bool grow = tmax > m_ref + kRescaleStep;
                    const float m_new = grow ? tmax : m_ref;
                    if (j > 0 && __any_sync(0xffffffffu, grow)) {
                        if (!mbar_wait(&bar_o[(m - 1) & 1], static_cast<uint32_t>((m - 1) >> 1) & 1u)) stuck = true;
                        tc_fence_after();
                        const float corr = ex2_approx(m_ref - m_new);   // 1 for rows that did not move
                        l *= corr;
#pragma unroll 1
                        for (int c = 0; c < DH / 64; ++c) {
                            uint32_t ov[32];
                            tmem_ld32(tmem_o + lane_sel + half * 64 + c * 32, ov);
#pragma unroll
                            for (int e = 0; e < 32; ++e) ov[e] = __float_as_uint(__uint_as_float(ov[e]) * corr);
                            tmem_st32(tmem_o + lane_sel + half * 64 + c * 32, ov);
                        }
                    }
                    m_ref = m_new;

                    // rows of V past the segment's end must not reach P V
                    if (ts.rows < BN) {
                        if (!mbar_wait(&bar_vfull[st], static_cast<uint32_t>(m / kStages) & 1u)) stuck = true;
                        unsigned char* v0 = base_ptr + kOffV + st * kKVBytes;
                        for (int i = tid; i < (BN - ts.rows) * 16; i += kSoftmaxThreads) {   // 16 x 16 bytes per row
                            const int vrow = ts.rows + i / 16, piece = i % 16;
                            *reinterpret_cast<uint4*>(v0 + (piece / 8) * kKVHalfBytes + vrow * 128 + (piece % 8) * 16) = make_uint4(0, 0, 0, 0);
                        }
                    }

                    // P = 2^(scale s - m_ref) as bf16 pairs into tensor memory, the A operand of P V (this
                    // thread: 32 keys = 16 columns of its lane).  Masked entries hold kNeg and come out as
                    // exactly 0 (the clamp keeps that true while the row has seen no visible key).
                    const float nm = -fmaxf(m_ref, -1.0e20f);
                    const float2 nm2 = make_float2(nm, nm);
                    float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
                    uint32_t packed[HN / 2];
#pragma unroll
                    for (int c = 0; c < HN / 2; c += 2) {
                        const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(sv[2 * c]), __uint_as_float(sv[2 * c + 1])), c2, nm2);
                        const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(sv[2 * c + 2]), __uint_as_float(sv[2 * c + 3])), c2, nm2);
                        const float2 p0 = make_float2(ex2_approx(x0.x), ex2_approx(x0.y));
                        const float2 p1 = make_float2(ex2_approx(x1.x), ex2_approx(x1.y));
                        packed[c] = pack_bf16(p0.x, p0.y);
                        packed[c + 1] = pack_bf16(p1.x, p1.y);
                        acc0 = __fadd2_rn(acc0, p0);
                        acc1 = __fadd2_rn(acc1, p1);
                    }
                    // (its columns are S columns of the row's first thread, which read them before the exchange above;
                    // the P of two tiles ago was consumed before this tile's Q K^T was even issued)
                    if constexpr (HN / 2 == 16) tmem_st16(tmem_sp + half * (HN / 2), packed);
                    else tmem_st32(tmem_sp + half * (HN / 2), packed);
                    l += (acc0.x + acc0.y) + (acc1.x + acc1.y);
                    if (ts.rows < BN) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // zeroed V rows -> tensor core
                    tc_fence_before();
                    __syncwarp();                      // one arrival per warp: 8 per tile on the barrier's word, not 256
                    if ((tid & 31) == 0) mbar_arrive(&bar_pready[sb]);
                }

                // ---- the row's two partial sums meet -----------------------------------------------------------
                asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");   // the last tile's exchange has been read
                xch[half * BM + row] = l;
                asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
                l += xch[(half ^ 1) * BM + row];
                if (kBalanced) asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");   // ... before the next segment writes there
                if (!mbar_wait(&bar_o[(it + nreal - 1) & 1], static_cast<uint32_t>((it + nreal - 1) >> 1) & 1u)) stuck = true;
                tc_fence_after();
            }

            const size_t orow = static_cast<size_t>(sq.q_row0 + q_first + row) * H + h;
            const bool whole = !kBalanced || (t0 == 0 && t1 == ne);
            if (whole) {
                // ---- normalise, round once, store ----------------------------------------------------------------
                const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll 1
                for (int c = 0; c < DH / 64; ++c) {
                    uint32_t ov[32];
                    if (nreal > 0) {
                        tmem_ld32(tmem_o + lane_sel + half * 64 + c * 32, ov);
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
                // ---- a cut unit: unnormalised partial to the workspace; the last block to arrive merges --------
                // Layout [feature][row]: a warp's lanes are consecutive rows, so they write and read consecutive floats.
                const int xu = x - t0;                                        // the unit's first slot
                const int c_first = block_of(T, G, xu), c_last = block_of(T, G, xu + ne - 1);
                float* ps = work.partials + static_cast<size_t>(2 * bid + (first_seg ? 0 : 1)) * kPartFloats;
#pragma unroll 1
                for (int c = 0; c < DH / 64; ++c) {
                    uint32_t ov[32];
                    if (nreal > 0) {
                        tmem_ld32(tmem_o + lane_sel + half * 64 + c * 32, ov);
                    } else {   // in step: this query tile sees none of the segment's keys
#pragma unroll
                        for (int e = 0; e < 32; ++e) ov[e] = 0u;
                    }
                    float* dst = ps + (half * 64 + c * 32) * BM + row;
#pragma unroll
                    for (int e = 0; e < 32; ++e) dst[e * BM] = __uint_as_float(ov[e]);
                }
                if (half == 0) { ps[BM * DH + row] = m_ref; ps[BM * DH + BM + row] = l; }
                __threadfence();
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (tid == 0) {
                    int* tk = work.tickets + g.cta0[u.i] + u.qt * H + h;
                    const int arrived = atomicAdd(tk, 1);
                    s_last = arrived == c_last - c_first;
                    if (s_last) *tk = 0;   // leave the counter clean for the next launch
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (s_last) {
                    __threadfence();
                    // group c's piece of this unit is its first segment if c starts inside the unit, else its last
                    float M = kNeg;
                    for (int c = c_first; c <= c_last; ++c) {
                        const float* pc = work.partials + static_cast<size_t>(2 * (c * W + bid % W) + (block_start(T, G, c) >= xu ? 0 : 1)) * kPartFloats;
                        M = fmaxf(M, __ldcg(pc + BM * DH + row));
                    }
                    float L = 0.f;
                    for (int c = c_first; c <= c_last; ++c) {
                        const float* pc = work.partials + static_cast<size_t>(2 * (c * W + bid % W) + (block_start(T, G, c) >= xu ? 0 : 1)) * kPartFloats;
                        L = fmaf(__ldcg(pc + BM * DH + BM + row), ex2_approx(__ldcg(pc + BM * DH + row) - M), L);
                    }
                    const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll 1
                    for (int cc = 0; cc < DH / 64; ++cc) {
                        float o[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) o[e] = 0.f;
                        for (int c = c_first; c <= c_last; ++c) {
                            const float* pc = work.partials + static_cast<size_t>(2 * (c * W + bid % W) + (block_start(T, G, c) >= xu ? 0 : 1)) * kPartFloats;
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
                asm volatile("bar.sync 1, 256;" ::: "memory");   // s_last is free again
            }
            if (nreal > 0) { it += nreal; ++seg; }
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
int dodo_dense_tile_keys() { return BN; }
size_t dodo_dense_workspace_bytes(int num_sms) { return static_cast<size_t>(2) * 2 * num_sms * kPartFloats * sizeof(float); }

int dodo_launch_attend_dense(dodo_ctx* ctx, int H, float sm_scale, const AttendGroup& g, const DenseMaps& maps,
                             const int32_t* cache_pos, void* O, float* lse, void* workspace, size_t workspace_bytes,
                             int* tickets, int* dev_status, const DenseGather* gather, cudaStream_t st) {
    const int units = g.cta0[g.nseq];
    if (units == 0) return DODO_OK;
    // slots of work: one per key tile of a unit, one for a unit without visible keys (same rules as the kernel);
    // `in step` counts every (sequence, head) once, by its last query tile
    auto unit_tiles = [](const AttendSeq& sq, int qt) {
        const int q_first = qt * BM, nq = sq.tq - q_first < BM ? sq.tq - q_first : BM;
        int l_vis = sq.q_pos0 + q_first + nq - 1 - sq.l_pos0 + 1;
        l_vis = l_vis < sq.l_len ? l_vis : sq.l_len;
        l_vis = l_vis > 0 ? l_vis : 0;
        return (sq.c_len + BN - 1) / BN + (l_vis + BN - 1) / BN;
    };
    long long total = 0, total_step = 0;
    int width = 0;           // query tiles per sequence if all sequences agree, else -1
    for (int i = 0; i < g.nseq; ++i) {
        const AttendSeq& sq = g.seq[i];
        if (sq.tq <= 0) continue;
        const int qtiles = (sq.tq + BM - 1) / BM;
        width = width == 0 || width == qtiles ? qtiles : -1;
        for (int qt = 0; qt < qtiles; ++qt) {
            const int n = unit_tiles(sq, qt);
            total += static_cast<long long>(n > 0 ? n : 1) * H;
        }
        const int n_last = unit_tiles(sq, qtiles - 1);
        total_step += static_cast<long long>(n_last > 0 ? n_last : 1) * H;
    }
    // Balanced when asked for, or (by default) when the units would leave the resident blocks (two per SM)
    // unevenly loaded and the key lists are long enough for the partial results to disappear in them.
    const int resident = kBlocksPerSM * ctx->num_sms;
    const bool room = total < 0x7fffffff && total >= 2 && workspace != nullptr && dodo_aligned16(workspace) &&
                      workspace_bytes >= dodo_dense_workspace_bytes(ctx->num_sms) && units <= DODO_NUM_TICKETS;
    const bool pays = units < resident && total / units >= kBalanceMinTiles;
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
    const bool gathered = gather != nullptr;
    auto kern = gathered ? (balanced ? attend_dense_kernel<true, true> : attend_dense_kernel<false, true>)
                         : (balanced ? attend_dense_kernel<true, false> : attend_dense_kernel<false, false>);
    const int slot = (gathered ? 2 : 0) + (balanced ? 1 : 0);
    if (!ctx->dense_attr_set[slot]) {
        const cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "dense attend shared-memory attribute");
        ctx->dense_attr_set[slot] = true;
    }
    DenseGather none;
    memset(&none, 0, sizeof none);
    kern<<<grid, kThreads, smem, st>>>(maps, g, cache_pos, H, sm_scale * 1.4426950408889634f,
                                       static_cast<__nv_bfloat16*>(O), lse, work, dev_status, gathered ? *gather : none);
    return dodo_check_cuda(ctx, cudaGetLastError(), "dense attend launch");
}
