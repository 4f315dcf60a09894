// Two-layer Scorer (Eq. 6 with the feed-forward network of App. B.3): s_i = w2 . act(W1 x_i + b1) + b2 for every
// context token.  The first layer is a [tokens, d] x [d, dh] contraction (2 d dh flop per token against d e bytes:
// tensor-bound) and runs on tcgen05.mma with fp32 accumulators in tensor memory; bias, activation and the dot
// product with w2 happen in the epilogue straight out of tensor memory, so the hidden layer is never written.
//
// Work item = (block of 256 tokens, chunk of hidden units); a persistent thread block (one per SM) takes items
// round-robin.  Per item and per tile of 256 hidden units, K runs over d in steps of 64:
//   producer (one lane of warp 0)  plain per-block TMA tensor copies with the 128-byte swizzle: X rows 256 x 64 and
//       W1 rows 256 x 64 into a 3-stage ring (64 KB per stage);
//   issuer (one lane of warp 1)    per stage 4 K = 16 steps x 2 halves of the token block: tcgen05.mma M128 N256 K16,
//       both operands K-major in shared memory, accumulators = TMEM columns [0,256) and [256,512); a commit
//       frees the stage, the last one of a tile publishes the accumulators;
//   epilogue (warps 2-9, thread = token = TMEM lane of its half)  tcgen05.ld 32 columns at a time, + b1, activation,
//       times w2, summed into the token's partial score; then the accumulators are handed back.
// An item leaves one partial score per token in the workspace; a second, tiny kernel adds the chunks in a fixed
// order (+ b2), so scores are bit-reproducible from run to run, which the TopK that follows relies on.
// Every wait is bounded; on time-out a status word is set and the block runs on to its end and frees its TMEM.
#include "dodo_internal.cuh"
#include "select_block.cuh"
#include "sm100_ptx.cuh"

namespace {

using namespace sm100;

constexpr int BM = 256;                 // tokens per item: two accumulator halves of 128 TMEM lanes
constexpr int BN = 256;                 // hidden units per tile
constexpr int BK = 64;                  // features per stage: rows of 128 bytes
constexpr int kStages = 3;
constexpr int kABytes = BM * BK * 2;    // 32 KB
constexpr int kBBytes = BN * BK * 2;    // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kEpiThreads = 256;
constexpr int kThreads = 64 + kEpiThreads;
constexpr uint32_t kTmemCols = 512;
constexpr int kSmemBytes = kStages * kStageBytes;

struct MlpWork {
    int rows;          // tokens in all
    int row_blocks;    // ceil(rows / BM)
    int n_tiles;       // dh / BN
    int n_chunks;      // items per token block
    int k_steps;       // d / BK
};

__device__ __forceinline__ float activate(float v, int act) {
    if (act == DODO_ACT_RELU) return fmaxf(v, 0.f);
    if (act == DODO_ACT_GELU_TANH) return 0.5f * v * (1.f + tanhf(0.7978845608028654f * (v + 0.044715f * v * v * v)));
    return v;
}

__global__ void __launch_bounds__(kThreads, 1)
score_mlp_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w1,
                 const float* __restrict__ b1, const __nv_bfloat16* __restrict__ w2, int act, const MlpWork work,
                 float* __restrict__ partials, int* __restrict__ dev_status) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    __shared__ __align__(8) uint64_t bar_full[kStages], bar_empty[kStages], bar_acc_full, bar_acc_empty;
    __shared__ uint32_t tmem_slot;
    __shared__ float b1s[2][BN], w2s[2][BN];

    const int tid = threadIdx.x, warp = tid >> 5;
    const int items = work.row_blocks * work.n_chunks;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
        mbar_init(&bar_acc_full, 1);
        mbar_init(&bar_acc_empty, kEpiThreads);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_slot;
    bool stuck = false;

    if (warp == 0) {
        // ===================================== producer ==========================================
        if (tid == 0) {
            int cnt = 0;   // stages filled so far
            for (int item = blockIdx.x; item < items; item += gridDim.x) {
                const int rb = item / work.n_chunks, ch = item % work.n_chunks;
                const int nt0 = ch * work.n_tiles / work.n_chunks, nt1 = (ch + 1) * work.n_tiles / work.n_chunks;
                for (int nt = nt0; nt < nt1; ++nt) {
                    for (int ks = 0; ks < work.k_steps; ++ks, ++cnt) {
                        const int st = cnt % kStages;
                        // the stage is free once the MMAs of its previous use have completed
                        if (cnt >= kStages && !mbar_wait(&bar_empty[st], static_cast<uint32_t>(cnt / kStages - 1) & 1u)) stuck = true;
                        const uint32_t dst = base + st * kStageBytes;
                        mbar_expect_tx(&bar_full[st], kStageBytes);
                        tma_load_2d(dst, &map_x, ks * BK, rb * BM, &bar_full[st]);
                        tma_load_2d(dst + kABytes, &map_w1, ks * BK, nt * BN, &bar_full[st]);
                    }
                }
            }
            if (stuck) atomicOr(dev_status, DODO_DEV_WAIT_TIMEOUT);
        }
    } else if (warp == 1) {
        // ===================================== issuer ============================================
        if (tid == 32) {
            const uint32_t idesc = idesc_bf16(BN, false);
            int cnt = 0, tile = 0;   // stages consumed, accumulator tiles produced
            for (int item = blockIdx.x; item < items; item += gridDim.x) {
                const int ch = item % work.n_chunks;
                const int nt0 = ch * work.n_tiles / work.n_chunks, nt1 = (ch + 1) * work.n_tiles / work.n_chunks;
                for (int nt = nt0; nt < nt1; ++nt, ++tile) {
                    // the epilogue has taken the previous tile out of the accumulators
                    if (tile >= 1 && !mbar_wait(&bar_acc_empty, static_cast<uint32_t>(tile - 1) & 1u)) stuck = true;
                    tc_fence_after();
                    for (int ks = 0; ks < work.k_steps; ++ks, ++cnt) {
                        const int st = cnt % kStages;
                        if (!mbar_wait(&bar_full[st], static_cast<uint32_t>(cnt / kStages) & 1u)) stuck = true;
                        tc_fence_after();
                        const uint64_t a0 = desc_kmajor(base + st * kStageBytes), b0 = desc_kmajor(base + st * kStageBytes + kABytes);
#pragma unroll
                        for (int k16 = 0; k16 < BK / 16; ++k16) {
#pragma unroll
                            for (int half = 0; half < 2; ++half)
                                mma_bf16(tmem + half * BN, a0 + static_cast<uint64_t>((half * (kABytes / 2) + k16 * 32) >> 4),
                                         b0 + static_cast<uint64_t>((k16 * 32) >> 4), idesc, ks > 0 || k16 > 0);
                        }
                        mma_commit(&bar_empty[st]);
                    }
                    mma_commit(&bar_acc_full);
                }
            }
            if (stuck) atomicOr(dev_status, DODO_DEV_WAIT_TIMEOUT);
        }
    } else {
        // ===================================== epilogue ==========================================
        const int et = tid - 64;                                   // 0 .. 255
        const int half = et >> 7;                                  // accumulator half = tokens 128 half .. 128 half + 127
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;   // the TMEM lanes this warp may read
        const int row_in_block = half * 128 + (warp & 3) * 32 + (tid & 31);
        int tile = 0;
        for (int item = blockIdx.x; item < items; item += gridDim.x) {
            const int rb = item / work.n_chunks, ch = item % work.n_chunks;
            const int nt0 = ch * work.n_tiles / work.n_chunks, nt1 = (ch + 1) * work.n_tiles / work.n_chunks;
            float partial = 0.f;
            for (int nt = nt0; nt < nt1; ++nt, ++tile) {
                // this tile's biases and output weights, staged once for the 256 threads (two buffers: nobody is
                // two tiles behind, the barrier below sees to it)
                b1s[tile & 1][et] = __ldg(b1 + nt * BN + et);
                w2s[tile & 1][et] = __bfloat162float(w2[nt * BN + et]);
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (!mbar_wait(&bar_acc_full, static_cast<uint32_t>(tile) & 1u)) stuck = true;
                tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < BN / 32; ++c) {
                    uint32_t v[32];
                    tmem_ld32(tmem + lane_sel + half * BN + c * 32, v);
#pragma unroll
                    for (int e = 0; e < 32; ++e)
                        partial = fmaf(activate(__uint_as_float(v[e]) + b1s[tile & 1][c * 32 + e], act), w2s[tile & 1][c * 32 + e], partial);
                }
                tc_fence_before();
                mbar_arrive(&bar_acc_empty);
            }
            const int row = rb * BM + row_in_block;
            if (row < work.rows) partials[static_cast<size_t>(ch) * work.rows + row] = partial;
        }
        if (stuck) atomicOr(dev_status, DODO_DEV_WAIT_TIMEOUT);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

// scores[i] = b2 + the chunks' partial scores, added in chunk order
__global__ void score_mlp_reduce_kernel(const float* __restrict__ partials, int rows, int n_chunks, float b2,
                                        float* __restrict__ scores) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= rows) return;
    float s = 0.f;
    for (int c = 0; c < n_chunks; ++c) s += partials[static_cast<size_t>(c) * rows + i];
    scores[i] = s + b2;
}

// The same reduction fused with the per-sequence TopK (Eq. 14), as the linear Scorer has it: a block adds up the
// chunks of kReduceRows rows of one sequence, makes its scores visible and takes a ticket on the sequence; the
// block that draws the last ticket selects that sequence's nuggets out of L2.  No block waits for another.
constexpr int kReduceRows = 512;
constexpr int kReduceKeyCache = 4096;

__global__ void __launch_bounds__(kReduceRows)
score_mlp_reduce_select_kernel(const float* __restrict__ partials, int rows, int n_chunks, float b2, float* __restrict__ scores,
                               const __grid_constant__ ScoreSelectGroup g, uint32_t flags, int32_t* __restrict__ idx,
                               int* __restrict__ tickets) {
    __shared__ dodo_sel::SelectSmem sel;
    __shared__ uint32_t sel_keys[kReduceKeyCache];
    __shared__ int is_last;
    const int tid = threadIdx.x;
    int lo = 0, hi = g.nseq;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (g.blk0[mid] <= static_cast<int>(blockIdx.x)) lo = mid; else hi = mid;
    }
    const int b = lo, n = g.n[b];
    const int lrow = (static_cast<int>(blockIdx.x) - g.blk0[b]) * kReduceRows + tid;
    dodo_grid_dependency_sync();
    if (lrow < n) {
        const size_t i = static_cast<size_t>(g.row0[b]) + lrow;
        float s = 0.f;
        for (int c = 0; c < n_chunks; ++c) s += partials[static_cast<size_t>(c) * rows + i];
        scores[i] = s + b2;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const int nblk = g.blk0[b + 1] - g.blk0[b];
        const int t = atomicAdd(&tickets[b], 1);
        is_last = (t == nblk - 1);
        if (is_last) tickets[b] = 0;  // leave the counter clean for the next launch
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const int team = dodo_sel::select_team_threads(n, kReduceRows);
    if (tid >= team) return;
    dodo_sel::block_select(scores + g.row0[b], n, g.k[b], flags, idx + g.idx0[b], sel, sel_keys, kReduceKeyCache, team);
}

}  // namespace

int dodo_score_mlp_reduce_rows() { return kReduceRows; }
int dodo_score_mlp_fused_max_tokens() { return kReduceKeyCache; }

size_t dodo_score_mlp_partial_bytes(int rows, int dh) {
    return static_cast<size_t>(dh / BN > 0 ? dh / BN : 1) * static_cast<size_t>(rows > 0 ? rows : 0) * sizeof(float);
}
bool dodo_score_mlp_supported(int dtype, int d, int dh) { return dtype == DODO_BF16 && d > 0 && d % BK == 0 && dh > 0 && dh % BN == 0; }

// groups == NULL: plain reduction into scores.  Else the reduction of each launch group of sequences ends in that
// group's TopK (ngroups launches of the fused reduction).
int dodo_launch_score_mlp(dodo_ctx* ctx, const void* X, int rows, int d, const void* W1, const float* b1, const void* w2,
                          float b2, int dh, int act, float* scores, float* partials, const ScoreSelectGroup* groups, int ngroups,
                          uint32_t flags, int32_t* idx, cudaStream_t st) {
    if (rows == 0) return DODO_OK;
    CUtensorMap map_x, map_w1;
    int rc;
    if ((rc = dodo_encode_bf16_rows(ctx, &map_x, X, d, rows, BM)) != DODO_OK) return rc;
    if ((rc = dodo_encode_bf16_rows(ctx, &map_w1, W1, d, dh, BN)) != DODO_OK) return rc;
    MlpWork work;
    work.rows = rows;
    work.row_blocks = (rows + BM - 1) / BM;
    work.n_tiles = dh / BN;
    work.k_steps = d / BK;
    // enough items for every SM twice over where the hidden layer allows it
    int chunks = (2 * ctx->num_sms + work.row_blocks - 1) / work.row_blocks;
    work.n_chunks = chunks < 1 ? 1 : chunks > work.n_tiles ? work.n_tiles : chunks;
    const int items = work.row_blocks * work.n_chunks;
    const size_t smem = static_cast<size_t>(kSmemBytes) + 1024;
    if (!ctx->mlp_attr_set) {
        const cudaError_t e = cudaFuncSetAttribute(score_mlp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return dodo_check_cuda(ctx, e, "two-layer Scorer shared-memory attribute");
        ctx->mlp_attr_set = true;
    }
    score_mlp_kernel<<<items < ctx->num_sms ? items : ctx->num_sms, kThreads, smem, st>>>(
        map_x, map_w1, b1, static_cast<const __nv_bfloat16*>(w2), act, work, partials, ctx->dev_status);
    rc = dodo_check_cuda(ctx, cudaGetLastError(), "two-layer Scorer launch");
    if (rc != DODO_OK) return rc;
    if (groups == nullptr) {
        score_mlp_reduce_kernel<<<(rows + 255) / 256, 256, 0, st>>>(partials, rows, work.n_chunks, b2, scores);
        return dodo_check_cuda(ctx, cudaGetLastError(), "two-layer Scorer reduce launch");
    }
    for (int gi = 0; gi < ngroups; ++gi) {
        const ScoreSelectGroup& g = groups[gi];
        if (g.blk0[g.nseq] == 0) continue;
        rc = dodo_check_cuda(ctx, dodo_launch_dependent(score_mlp_reduce_select_kernel, dim3(static_cast<unsigned>(g.blk0[g.nseq])),
                                                        dim3(kReduceRows), 0, st, static_cast<const float*>(partials), rows, work.n_chunks,
                                                        b2, scores, g, flags, idx, ctx->tickets),
                             "two-layer Scorer reduce + select launch");
        if (rc != DODO_OK) return rc;
    }
    return DODO_OK;
}
