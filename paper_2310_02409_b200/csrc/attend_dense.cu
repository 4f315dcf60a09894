// Attention of a block of query tokens over [nugget cache ; local tokens] (Eq. 13, Eq. 9) on the
// 5th-generation tensor cores: tcgen05.mma with TMEM accumulators, operands staged by TMA.
// bf16, head size 128.  This is the dense case, where many queries share every K/V tile and the
// work is a contraction (about Tq flop per K/V byte); single-token decode stays on the HBM-bound
// kernel in attend.cu.
//
// One thread block serves (sequence, tile of 128 query tokens, head) with two roles:
//   issuer (one lane of warp 8)  TMA tensor copies with the 128-byte swizzle (no multicast) bring the
//       Q tile once and K and V tiles of 64 keys through two two-stage rings (two blocks share an SM and
//       overlap each other's waits); it issues
//       S = Q K^T (8 x tcgen05.mma M128 N64 K16, both operands K-major in shared memory, into TMEM
//       columns [0,64)) and O += P V (4 x tcgen05.mma M128 N128 K16, A = P from TMEM columns [192,224),
//       B = V MN-major, i.e. V rows as stored, into TMEM columns [64,192)).  S of tile t+1 is issued as soon as the
//       softmax threads hold S of tile t in registers, so the tensor core works during the softmax.
//   softmax (warps 0-7; two threads per query row = TMEM lane, each owning half of the score and
//       output columns, so that two warps per scheduler hide each other's latencies)  reads its part
//       of the row of S with tcgen05.ld,
//       scales, masks by position only on tiles that need it (key visible iff key_pos <= q_pos; rows
//       past a segment's end carry INT_MAX), keeps the running max and sum in the base-2 domain and
//       writes P as bf16 pairs into tensor memory, from where P V reads its A operand.  O stays
//       in TMEM across tiles; it is rescaled (tcgen05.ld / tcgen05.st) only when a row's maximum
//       has grown by more than 2^8 since the reference maximum was last moved.
// One round to bf16 at the end; optional log-sum-exp (from the unrounded weights).
// V rows past the end of a segment are zeroed in shared memory before use, so that whatever lies
// behind a sequence's region (another sequence, unused capacity) can never reach the product P V.
// Every wait is bounded; on time-out a status word is set and the block runs on to its end, where
// it always frees its TMEM columns.
#include "dodo_internal.cuh"

namespace {

constexpr int DH = 128;               // head size
constexpr int BM = 128;               // query rows per block = TMEM lanes
constexpr int BN = 64;                // keys per tile
constexpr int kSoftmaxThreads = 256;      // two threads per query row, each owning half of the columns
constexpr int kThreads = kSoftmaxThreads + 32;
constexpr int kQHalfBytes = 128 * 128;   // 64 columns of a 128-row bf16 tile, rows of 128 bytes
constexpr int kQBytes = 2 * kQHalfBytes;
constexpr int kKVHalfBytes = BN * 128;   // 64 columns of a 64-row tile
constexpr int kKVBytes = 2 * kKVHalfBytes;
constexpr int kStages = 2;              // 96 KB of shared memory per block: two blocks per SM
constexpr uint32_t kTmemCols = 256;      // S: columns [0,64), O: [64,192), P (bf16 pairs): [192,224)
constexpr uint32_t kTmemP = 192;
constexpr int kWaitPolls = 1 << 22;
constexpr float kNeg = -1.0e30f;
constexpr float kRescaleStep = 8.f;      // move a row's reference maximum only past this many octaves

// shared-memory map (bytes from the 1024-aligned base)
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + kQBytes;
constexpr int kOffV = kOffK + kStages * kKVBytes;
constexpr int kOffXch = kOffV + kStages * kKVBytes;    // float[2][2][BM] row maxima / sums exchanged by a row's two threads
constexpr int kSmemBytes = kOffXch + 2 * 2 * BM * 4;

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
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (int i = 0; i < kWaitPolls; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

// Shared-memory matrix descriptors for tcgen05.mma, 128-byte swizzle, rows of 128 bytes, groups of
// eight rows 1024 bytes apart.  K-major: the contraction index runs along a row.  MN-major: the
// contraction index runs down the rows and `lbo_bytes` is the distance between 64-element column
// blocks.
__device__ __forceinline__ uint64_t desc_kmajor(uint32_t addr) {
    return static_cast<uint64_t>((addr & 0x3ffffu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ uint64_t desc_mnmajor(uint32_t addr, uint32_t lbo_bytes) {
    return static_cast<uint64_t>((addr & 0x3ffffu) >> 4) | (static_cast<uint64_t>(lbo_bytes >> 4) << 16) |
           (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, M = 128, N = n; B MN-major when asked.
__device__ __forceinline__ uint32_t idesc_bf16(uint32_t n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}
__device__ __forceinline__ void mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate ? 1u : 0u)
        : "memory");
}
// Same, with the A operand (bf16 pairs, K-major) read from tensor memory.
__device__ __forceinline__ void mma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, bool accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate ? 1u : 0u)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* v) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t* v) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
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
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
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

__global__ void __launch_bounds__(kThreads, 2)
attend_dense_kernel(const __grid_constant__ DenseMaps maps, const __grid_constant__ AttendGroup g,
                    const int32_t* __restrict__ cache_pos, int H, float scale_log2,
                    __nv_bfloat16* __restrict__ O, float* __restrict__ lse, int* __restrict__ dev_status) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* base_ptr = smem_raw + (base - smem_u32(smem_raw));
    __shared__ __align__(8) uint64_t bar_q, bar_s, bar_o, bar_sread, bar_pready, bar_kfull[kStages], bar_vfull[kStages];
    __shared__ uint32_t tmem_slot;
    __shared__ int first_masked;

    const int tid = threadIdx.x, warp = tid >> 5;

    // ---- which (sequence, query tile, head) ---------------------------------------------------
    const int bid = static_cast<int>(blockIdx.x);
    int b;
    if (g.uniform_ctas > 0) {
        b = bid / g.uniform_ctas;
    } else {
        b = 0;
#pragma unroll 8
        for (int i = 1; i < DODO_GROUP; ++i) b += (i < g.nseq && g.cta0[i] <= bid) ? 1 : 0;
    }
    const AttendSeq sq = g.seq[b];
    const int r0 = bid - g.cta0[b];
    const int h = r0 % H, qtile = r0 / H;
    const int q_first = qtile * BM;
    const int nq = min(BM, sq.tq - q_first);
    const int l_vis = max(0, min(sq.l_len, sq.q_pos0 + q_first + nq - 1 - sq.l_pos0 + 1));
    const int nt_c = (sq.c_len + BN - 1) / BN;
    const int ntiles = nt_c + (l_vis + BN - 1) / BN;
    auto tile_src = [&](int t) -> TileSrc {
        TileSrc s;
        if (t < nt_c) {
            s.cache = true; s.row0 = sq.c_row0 + t * BN; s.rows = min(BN, sq.c_len - t * BN); s.pos0 = 0;
        } else {
            const int tl = t - nt_c;
            s.cache = false; s.row0 = sq.l_row0 + tl * BN; s.rows = min(BN, l_vis - tl * BN); s.pos0 = sq.l_pos0 + tl * BN;
        }
        return s;
    };

    // ---- barriers, TMEM ------------------------------------------------------------------------
    if (tid == 0) {
        first_masked = nt_c;
        mbar_init(&bar_q, 1); mbar_init(&bar_s, 1); mbar_init(&bar_o, 1);
        mbar_init(&bar_sread, kSoftmaxThreads); mbar_init(&bar_pready, kSoftmaxThreads);
        for (int s = 0; s < kStages; ++s) { mbar_init(&bar_kfull[s], 1); mbar_init(&bar_vfull[s], 1); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
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
    const uint32_t tmem_s = tmem, tmem_o = tmem + BN;
    bool stuck = false;

    if (warp == kSoftmaxThreads / 32) {
        // ===================================== issuer ============================================
        if (tid == kSoftmaxThreads && ntiles > 0) {
            auto load_k = [&](int t) {
                const int st = t % kStages;
                const TileSrc ts = tile_src(t);
                const CUtensorMap* mk = ts.cache ? &maps.cK : &maps.lK;
                const uint32_t dk = base + kOffK + st * kKVBytes;
                mbar_expect_tx(&bar_kfull[st], kKVBytes);
                tma_load_2d(dk, mk, h * DH, ts.row0, &bar_kfull[st]);
                tma_load_2d(dk + kKVHalfBytes, mk, h * DH + 64, ts.row0, &bar_kfull[st]);
            };
            auto load_v = [&](int t) {
                const int st = t % kStages;
                const TileSrc ts = tile_src(t);
                const CUtensorMap* mv = ts.cache ? &maps.cV : &maps.lV;
                const uint32_t dv = base + kOffV + st * kKVBytes;
                mbar_expect_tx(&bar_vfull[st], kKVBytes);
                tma_load_2d(dv, mv, h * DH, ts.row0, &bar_vfull[st]);
                tma_load_2d(dv + kKVHalfBytes, mv, h * DH + 64, ts.row0, &bar_vfull[st]);
            };
            auto issue_qk = [&](int t) {
                const int st = t % kStages;
                if (!mbar_wait(&bar_kfull[st], static_cast<uint32_t>(t / kStages) & 1u)) stuck = true;
                tc_fence_after();
                // descriptors differ only in their start-address field (units of 16 bytes)
                const uint64_t a0 = desc_kmajor(base + kOffQ), b0 = desc_kmajor(base + kOffK + st * kKVBytes);
                const uint32_t idesc = idesc_bf16(BN, false);
#pragma unroll
                for (int i = 0; i < DH / 16; ++i)
                    mma_bf16(tmem_s, a0 + static_cast<uint64_t>(((i / 4) * kQHalfBytes + (i % 4) * 32) >> 4),
                             b0 + static_cast<uint64_t>(((i / 4) * kKVHalfBytes + (i % 4) * 32) >> 4), idesc, i > 0);
                mma_commit(&bar_s);
            };
            auto issue_pv = [&](int t) {
                const int st = t % kStages;
                if (!mbar_wait(&bar_vfull[st], static_cast<uint32_t>(t / kStages) & 1u)) stuck = true;
                tc_fence_after();
                const uint64_t b0 = desc_mnmajor(base + kOffV + st * kKVBytes, kKVHalfBytes);
                const uint32_t idesc = idesc_bf16(DH, true);
#pragma unroll
                for (int i = 0; i < BN / 16; ++i)   // 16 keys of P = 8 columns of bf16 pairs
                    mma_bf16_ts(tmem_o, tmem + kTmemP + i * 8, b0 + static_cast<uint64_t>((i * 2048) >> 4), idesc, t > 0 || i > 0);
                mma_commit(&bar_o);
            };

            mbar_expect_tx(&bar_q, kQBytes);
            tma_load_2d(base + kOffQ, &maps.Q, h * DH, sq.q_row0 + q_first, &bar_q);
            tma_load_2d(base + kOffQ + kQHalfBytes, &maps.Q, h * DH + 64, sq.q_row0 + q_first, &bar_q);
            for (int t = 0; t < min(kStages, ntiles); ++t) { load_k(t); load_v(t); }
            if (!mbar_wait(&bar_q, 0)) stuck = true;
            issue_qk(0);
            for (int t = 0; t < ntiles; ++t) {
                // S(t) is in the softmax threads' registers: S may be overwritten, K stage t is free
                if (!mbar_wait(&bar_sread, static_cast<uint32_t>(t) & 1u)) stuck = true;
                tc_fence_after();
                if (t + 1 < ntiles) issue_qk(t + 1);
                if (t + kStages < ntiles) load_k(t + kStages);
                // P(t) is in shared memory and O carries the right scale
                if (!mbar_wait(&bar_pready, static_cast<uint32_t>(t) & 1u)) stuck = true;
                // P V of tile t-1 has completed (the softmax threads waited for it before writing P(t));
                // checked here, before tile t is committed, so that the parity cannot be ambiguous
                if (t >= 1 && !mbar_wait(&bar_o, static_cast<uint32_t>(t - 1) & 1u)) stuck = true;
                tc_fence_after();
                issue_pv(t);
                if (t >= 1 && t - 1 + kStages < ntiles) load_v(t - 1 + kStages);   // that V stage is free
            }
            if (stuck) atomicExch(dev_status, DODO_DEV_WAIT_TIMEOUT);
        }
    } else {
        // ===================================== softmax ===========================================
        // Thread pair (row, half): row = TMEM lane, half 0 owns score columns [0,32) and output
        // columns [0,64), half 1 the rest.  Warps w and w+4 cover the same 32 lanes.
        const int row = tid & (BM - 1), half = tid >> 7;
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;   // this warp's TMEM lanes
        float* xch = reinterpret_cast<float*>(base_ptr + kOffXch);                 // [2][2][BM]
        const bool row_live = row < nq;
        const int my_qpos = row_live ? sq.q_pos0 + q_first + row : static_cast<int>(0x80000000);
        const int min_qpos = sq.q_pos0 + q_first;
        constexpr int HN = BN / 2;   // score columns per thread
        float m_ref = kNeg, l = 0.f;   // l: sum of the unrounded weights over this thread's columns

        // First cache tile holding a key that some query of this tile must not see (nuggets normally all
        // precede the block, so this is nt_c and no cache tile pays for the position test).
        {
            int bad = nt_c;
            for (int i = tid; i < sq.c_len; i += kSoftmaxThreads)
                if (__ldg(cache_pos + sq.c_row0 + i) > min_qpos) bad = min(bad, i / BN);
            if (bad < nt_c) atomicMin(&first_masked, bad);
            asm volatile("bar.sync 1, 256;" ::: "memory");
        }
        const int first_bad = first_masked;
        const float2 c2 = make_float2(scale_log2, scale_log2);
        const int pair_bar = 2 + (warp & 3);   // named barrier of the two warps that share these 32 rows

        for (int t = 0; t < ntiles; ++t) {
            const int st = t % kStages;
            const TileSrc ts = tile_src(t);
            const bool need_mask = ts.rows < BN || (ts.cache ? t >= first_bad : ts.pos0 + ts.rows - 1 > min_qpos);

            if (!mbar_wait(&bar_s, static_cast<uint32_t>(t) & 1u)) stuck = true;
            tc_fence_after();
            uint32_t sv[HN];   // raw scores q.k; the softmax scale enters in the exponent's FMA
            tmem_ld32(tmem_s + lane_sel + half * HN, sv);
            tc_fence_before();
            mbar_arrive(&bar_sread);

            if (need_mask) {
#pragma unroll
                for (int j = 0; j < HN; ++j) {
                    const int col = half * HN + j;
                    int kp = 0x7fffffff;
                    if (col < ts.rows) kp = ts.cache ? __ldg(cache_pos + ts.row0 + col) : ts.pos0 + col;
                    if (kp > my_qpos) sv[j] = __float_as_uint(kNeg);
                }
            }
            float tmax = fmaxf(__uint_as_float(sv[0]), __uint_as_float(sv[1]));
#pragma unroll
            for (int j = 2; j < HN; j += 2) tmax = max3(tmax, __uint_as_float(sv[j]), __uint_as_float(sv[j + 1]));
            tmax = tmax > 0.5f * kNeg ? tmax * scale_log2 : kNeg;   // base-2 domain; kNeg = nothing visible
            // the row's two threads agree on the tile maximum through shared memory
            float* xm = xch + (t & 1) * 2 * BM;
            xm[half * BM + row] = tmax;
            asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
            tmax = fmaxf(tmax, xm[(half ^ 1) * BM + row]);

            // everything of tile t-1 must have left P (and O must be complete) before we touch them
            if (t > 0) {
                if (!mbar_wait(&bar_o, static_cast<uint32_t>(t - 1) & 1u)) stuck = true;
                tc_fence_after();
            }
            // move the reference maximum only when it pays; rescale O in TMEM when any row of the warp moved
            const bool grow = tmax > m_ref + kRescaleStep;
            const float m_new = grow ? tmax : m_ref;
            if (t > 0 && __any_sync(0xffffffffu, grow)) {
                const float corr = ex2_approx(m_ref - m_new);   // 1 for rows that did not move
                l *= corr;
#pragma unroll 1
                for (int c = 0; c < DH / 64; ++c) {
                    uint32_t ov[32];
                    tmem_ld32(tmem_o + lane_sel + half * 64 + c * 32, ov);
#pragma unroll
                    for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * corr);
                    tmem_st32(tmem_o + lane_sel + half * 64 + c * 32, ov);
                }
            }
            m_ref = m_new;

            // rows of V past the segment's end must not reach P V
            if (ts.rows < BN) {
                if (!mbar_wait(&bar_vfull[st], static_cast<uint32_t>(t / kStages) & 1u)) stuck = true;
                unsigned char* v0 = base_ptr + kOffV + st * kKVBytes;
                for (int i = tid; i < (BN - ts.rows) * 16; i += kSoftmaxThreads) {   // 16 x 16 bytes per row
                    const int vrow = ts.rows + i / 16, piece = i % 16;
                    *reinterpret_cast<uint4*>(v0 + (piece / 8) * kKVHalfBytes + vrow * 128 + (piece % 8) * 16) = make_uint4(0, 0, 0, 0);
                }
            }

            // P = 2^(scale s - m_ref) as bf16 pairs into tensor memory, the A operand of P V (this thread:
            // 32 keys = 16 columns of its lane).  Masked entries hold kNeg and come out as exactly 0 (the
            // clamp keeps that true while the row has seen no visible key and m_ref is still kNeg).
            const float nm = -fmaxf(m_ref, -1.0e20f);
            const float2 nm2 = make_float2(nm, nm);
            float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
            uint32_t packed[HN / 2];
#pragma unroll
            for (int j = 0; j < HN / 2; j += 2) {
                const float2 x0 = __ffma2_rn(make_float2(__uint_as_float(sv[2 * j]), __uint_as_float(sv[2 * j + 1])), c2, nm2);
                const float2 x1 = __ffma2_rn(make_float2(__uint_as_float(sv[2 * j + 2]), __uint_as_float(sv[2 * j + 3])), c2, nm2);
                const float2 p0 = make_float2(ex2_approx(x0.x), ex2_approx(x0.y));
                const float2 p1 = make_float2(ex2_approx(x1.x), ex2_approx(x1.y));
                packed[j] = pack_bf16(p0.x, p0.y);
                packed[j + 1] = pack_bf16(p1.x, p1.y);
                acc0 = __fadd2_rn(acc0, p0);
                acc1 = __fadd2_rn(acc1, p1);
            }
            tmem_st16(tmem + kTmemP + lane_sel + half * (HN / 2), packed);
            l += (acc0.x + acc0.y) + (acc1.x + acc1.y);
            if (ts.rows < BN) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // zeroed V rows -> tensor core
            tc_fence_before();
            mbar_arrive(&bar_pready);
        }

        // ---- the row's two partial sums meet; normalise, round once, store ---------------------------
        asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");   // the last tile's exchange has been read
        xch[half * BM + row] = l;
        asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
        l += xch[(half ^ 1) * BM + row];
        if (ntiles > 0) {
            if (!mbar_wait(&bar_o, static_cast<uint32_t>(ntiles - 1) & 1u)) stuck = true;
            tc_fence_after();
        }
        const size_t orow = static_cast<size_t>(sq.q_row0 + q_first + row) * H + h;
        const float inv = l > 0.f ? 1.f / l : 0.f;
#pragma unroll 1
        for (int c = 0; c < DH / 64; ++c) {
            uint32_t ov[32];
            if (ntiles > 0) {
                tmem_ld32(tmem_o + lane_sel + half * 64 + c * 32, ov);
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) ov[j] = 0u;
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
        if (stuck) atomicExch(dev_status, DODO_DEV_WAIT_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

}  // namespace

int dodo_dense_tile_queries() { return BM; }
int dodo_dense_tile_keys() { return BN; }

int dodo_launch_attend_dense(dodo_ctx* ctx, int H, float sm_scale, const AttendGroup& g, const DenseMaps& maps,
                             const int32_t* cache_pos, void* O, float* lse, int* dev_status, cudaStream_t st) {
    if (g.cta0[g.nseq] == 0) return DODO_OK;
    const size_t smem = static_cast<size_t>(kSmemBytes) + 1024;
    cudaError_t e = cudaFuncSetAttribute(attend_dense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "dense attend shared-memory attribute");
    attend_dense_kernel<<<g.cta0[g.nseq], kThreads, smem, st>>>(maps, g, cache_pos, H, sm_scale * 1.4426950408889634f,
                                                                static_cast<__nv_bfloat16*>(O), lse, dev_status);
    return dodo_check_cuda(ctx, cudaGetLastError(), "dense attend launch");
}
