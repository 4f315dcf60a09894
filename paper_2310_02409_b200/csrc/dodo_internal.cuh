// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "dodo.h"

// Sequences per launch: per-sequence descriptors travel as kernel parameters (no staging copy);
// larger batches are cut into groups of this size.
#define DODO_GROUP 64

// Arrival counters owned by a context (ints).  Self-resetting: the block that takes the last
// ticket of a unit puts the counter back to zero.
#define DODO_NUM_TICKETS (64 * 1024)

struct dodo_ctx {
    int device;
    int num_sms;
    int max_smem_optin;
    int* tickets;               // device, DODO_NUM_TICKETS ints, zero between calls
    int* dev_status;            // device word: 0, or a DODO_DEV_* code left by a kernel
    int* top_hist;              // device, DODO_GROUP x 256 ints: counts of the scores' top key digits per sequence (fused score + select), zero between calls
    int* compress_state;        // device, DODO_FLAG_STRIDE * (1 + DODO_GROUP) ints: exit counter and per-sequence flags of dodo_compress, zero between calls
    int attend_target_ctas;     // split-K aims at about this many thread blocks per launch
    int dense_min_tq;           // query blocks at least this long go to the tensor-core kernel
    int dense_balance;          // 0 auto, 1 always, 2 never, 3 always but not in step: key tiles balanced over the resident blocks
    void* encode_tiled;         // cuTensorMapEncodeTiled, fetched through the runtime
    // recently encoded tensor maps (a map depends only on these host values, so reuse is exact)
    struct MapEntry { const void* base; int rows, width, box_rows; CUtensorMap map; } map_cache[16];
    int map_next;               // round-robin replacement
    bool dense_attr_set[4];     // shared-memory attribute of the four forms of the tensor-core kernel
    bool mlp_attr_set;          // ... and of the two-layer Scorer's kernel
    bool select_attr_set;       // ... and of the select / estimate kernels, with the keys they may cache
    int select_key_cap;
    int select_resident[9];     // resident clusters of the cluster select kernel by cluster size (0: not asked yet)
    int cluster_cap[12][9];     // per streaming attend kernel (dtype, dh, qt): resident clusters by cluster size
    bool cluster_cap_set[12];
    // True while nothing this context launched since its last attend has written a nugget cache: the next
    // streaming attend may then read cache rows ahead of its dependency wait (see dodo_attend in dodo.h).
    bool cache_clean;
    unsigned long long clean_capture_id;   // stream-capture sequence the flag was set in (0: none)
    char err[512];
};

int dodo_fail(dodo_ctx* ctx, int status, const char* fmt, ...);
int dodo_check_cuda(dodo_ctx* ctx, cudaError_t e, const char* what);

static inline size_t dodo_elem_bytes(int dtype) { return dtype == DODO_F32 ? 4u : 2u; }
static inline bool dodo_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---- score / select ---------------------------------------------------------------------------
struct ScoreSelectGroup {
    int nseq;
    int row0[DODO_GROUP];       // first packed row of the sequence
    int n[DODO_GROUP];          // tokens
    int k[DODO_GROUP];          // nuggets to keep
    int idx0[DODO_GROUP];       // first slot of the sequence in idx
    int blk0[DODO_GROUP + 1];   // prefix sum of score blocks per sequence
};

// mode 0: scores; 1: fused with the selection; 2: scores plus the counts of their top key digits in ctx->top_hist
// (row = the sequence's number in g), for a dodo_launch_select(..., counted = true) of the same g right behind it
int dodo_launch_score(dodo_ctx* ctx, const void* X, int dtype, int d, const void* w, float bias,
                      const ScoreSelectGroup& g, int mode, uint32_t flags, float* scores,
                      int32_t* idx, int* tickets, int* seq_flag, cudaStream_t st);
int dodo_launch_select(dodo_ctx* ctx, const float* scores, const ScoreSelectGroup& g, uint32_t flags,
                       int32_t* idx, bool counted, cudaStream_t st);
int dodo_score_rows_per_block();
int dodo_select_fused_max_tokens();   // longer sequences are selected by a launch of their own

// ---- two-layer Scorer --------------------------------------------------------------------------
size_t dodo_score_mlp_partial_bytes(int rows, int dh);
bool dodo_score_mlp_supported(int dtype, int d, int dh);
int dodo_launch_score_mlp(dodo_ctx* ctx, const void* X, int rows, int d, const void* W1, const float* b1, const void* w2,
                          float b2, int dh, int act, float* scores, float* partials, const ScoreSelectGroup* groups, int ngroups,
                          uint32_t flags, int32_t* idx, cudaStream_t st);
int dodo_score_mlp_reduce_rows();          // rows per block of the fused reduction (blk0 of its ScoreSelectGroup counts these)
int dodo_score_mlp_fused_max_tokens();     // longer sequences are selected by a launch of their own
// tensor map of a [rows, width] bf16 row-major array: box of 64 elements x box_rows rows, 128-byte swizzle (cached)
int dodo_encode_bf16_rows(dodo_ctx* ctx, CUtensorMap* map, const void* base, int width, int rows, int box_rows);

// ---- threshold selection ----------------------------------------------------------------------
struct ThresholdGroup {
    int nseq;
    int row0[DODO_GROUP];       // first packed score of the sequence
    int n[DODO_GROUP];          // tokens
    int out0[DODO_GROUP];       // count: slot in counts; select: first slot of the sequence in idx
    int cap[DODO_GROUP];        // select: slots the sequence owns
};
int dodo_launch_threshold(dodo_ctx* ctx, const float* scores, const ThresholdGroup& g, float lambda, bool select,
                          int32_t* out, cudaStream_t st);
int dodo_launch_estimate_threshold(dodo_ctx* ctx, const float* sample, int m, int k, float* lambda, cudaStream_t st);

// ---- gather -----------------------------------------------------------------------------------
struct GatherGroup {
    int nseq;
    int idx0[DODO_GROUP + 1];   // prefix of nuggets per sequence (slots in idx, absolute)
    int src_row0[DODO_GROUP];   // first packed K/V row of the sequence
    int n[DODO_GROUP];          // tokens of the sequence: an index outside [0, n) is reported, not followed
    int dst_row0[DODO_GROUP];   // first cache row to write (cache_off + cache_len)
    int pos_base[DODO_GROUP];
};

int dodo_launch_gather(dodo_ctx* ctx, const void* K, const void* V, size_t row_bytes,
                       const int32_t* idx, const GatherGroup& g, void* cacheK, void* cacheV,
                       int32_t* cache_pos, int* dev_status, cudaStream_t st);

// The gather of the compression step: launched behind a fused score + select launch that raises seq_flag[b *
// DODO_FLAG_STRIDE] once sequence b's indices are visible, it copies a sequence's rows as soon as that flag is up
// instead of waiting for the whole launch before it.  `state`: [0] blocks that have left, then the flags; the last
// block to leave puts all of it back to zero.
#define DODO_FLAG_STRIDE 32   // ints between two sequences' flags: one 128-byte line each
int dodo_launch_gather_flagged(dodo_ctx* ctx, const void* K, const void* V, size_t row_bytes, const int32_t* idx,
                               const GatherGroup& g, void* cacheK, void* cacheV, int32_t* cache_pos, int* state,
                               int* dev_status, cudaStream_t st);

// Layers of one multi-layer gather launch (kernel parameter: device pointers by value).
#define DODO_LAYER_GROUP 64
struct GatherLayers {
    int n;                      // layers in this launch
    int first;                  // non-zero: this launch also records the positions
    const unsigned char* K[DODO_LAYER_GROUP];
    const unsigned char* V[DODO_LAYER_GROUP];
    unsigned char* cacheK[DODO_LAYER_GROUP];
    unsigned char* cacheV[DODO_LAYER_GROUP];
};
int dodo_launch_gather_layers(dodo_ctx* ctx, const GatherLayers& lay, size_t row_bytes, const int32_t* idx,
                              const GatherGroup& g, int32_t* cache_pos, int* dev_status, cudaStream_t st);

// ---- mean pooling of even chunks (the comparison system of Sec. 5.1) ---------------------------------
struct PoolGroup {
    int nseq;
    int out0[DODO_GROUP + 1];   // prefix of pooled rows per sequence (within the launch group)
    int src_row0[DODO_GROUP];   // first packed K/V row of the sequence
    int n[DODO_GROUP];          // tokens
    int dst_row0[DODO_GROUP];   // first cache row to write (cache_off + cache_len)
    int pos_base[DODO_GROUP];
};
int dodo_launch_pool(dodo_ctx* ctx, const void* K, const void* V, int dtype, size_t row_bytes, int r, const PoolGroup& g,
                     void* cacheK, void* cacheV, int32_t* cache_pos, cudaStream_t st);

// ---- attend -----------------------------------------------------------------------------------
struct AttendSeq {
    int q_row0;     // first query row
    int tq;         // query tokens
    int q_pos0;
    int c_row0;     // first nugget-cache row
    int c_len;
    int l_row0;     // first local row
    int l_len;
    int l_pos0;
    int nchunk;     // key chunks per (query tile, head)
    int ctiles;     // key tiles per chunk
    int part0;      // first partial row in the workspace
    int tick0;      // first arrival counter
};

struct AttendGroup {
    int nseq;
    int uniform_ctas;               // > 0: every sequence owns this many thread blocks (no search)
    int cluster;                    // > 1: every sequence is cut into this many chunks and the chunks of a
                                    // (query tile, head) form one thread-block cluster (merge in shared memory)
    int cta0[DODO_GROUP + 1];       // prefix sum of thread blocks per sequence
    AttendSeq seq[DODO_GROUP];
};

struct AttendPlan {
    int qt;                     // queries per thread block (1, 2, 4; 128 on the tensor-core kernel)
    const int* cluster_cap;     // [chunks] -> clusters of that many blocks the device holds at once; NULL: never cluster
};

// Bits of the device status word
#define DODO_DEV_WAIT_TIMEOUT 1  // a bounded wait on a copy barrier ran out
#define DODO_DEV_BAD_INDEX 2     // a gather met an index outside its sequence and skipped that row

// Base addresses of the key/value sources of one attend call
struct AttendMaps {
    const void *cK, *cV, *lK, *lV;
};

// early_cache: the launch may read cache rows ahead of its dependency wait (nothing directly before it on the
// stream writes them); otherwise it only sends cache hints there and reads after the wait
int dodo_launch_attend(dodo_ctx* ctx, int dtype, int H, int dh, float sm_scale, const AttendPlan& plan,
                       const AttendGroup& g, const void* Q, const AttendMaps& maps,
                       const int32_t* cache_pos, void* O, float* lse, float* partials, int* tickets,
                       bool early_cache, cudaStream_t st);
// Host view of one dodo_attend call (the caller's tables, unchanged).
struct AttendShape {
    const int32_t *q_off, *q_pos0, *cache_off, *cache_len, *loc_off, *loc_len, *loc_pos0;
    int B, H, dh, dtype;
};
struct AttendTotals {
    int64_t units, work, target;   // (query tile, head) units; units x key tiles; block target
    bool split;
    int64_t part_rows, tick_rows;  // running totals over launch groups
};
void dodo_attend_plan_begin(const AttendShape& s, int target_ctas, AttendPlan& plan, AttendTotals& tot);
void dodo_attend_plan_group(const AttendShape& s, const AttendPlan& plan, AttendTotals& tot, int b0, int nb,
                            AttendGroup& g);
// ---- dense (tensor-core) attend ----------------------------------------------------------------
struct DenseMaps {
    CUtensorMap Q, cK, cV, lK, lV;   // boxes of 64 elements x 128 rows, 128-byte swizzle
};
int dodo_dense_tile_queries();
int dodo_dense_tile_keys();
// cache_box_rows: rows of the box of the cK / cV maps (the key tile; 1 for the gathered form's row copies)
int dodo_dense_encode_maps(dodo_ctx* ctx, const AttendShape& s, const void* Q, int q_rows, const void* cacheK,
                           const void* cacheV, int cache_rows, int cache_box_rows, const void* locK, const void* locV,
                           int loc_rows, DenseMaps& maps);
size_t dodo_dense_workspace_bytes(int num_sms);
// Gathered form of the tensor-core kernel: where the selected rows of each sequence of a launch group come from --
// first row of the sequence in the uncompressed K / V arrays, its token count, the position of its token 0.
struct DenseGather {
    int row0[DODO_GROUP];
    int n[DODO_GROUP];
    int pos_base[DODO_GROUP];
};
// gather == NULL: cache_pos are the positions of the cache rows and maps.cK / cV tile the cache.  Else: cache_pos
// is the index list, AttendSeq::c_row0 / c_len name each sequence's slots in it, and maps.cK / cV have boxes one
// row high over the uncompressed K / V.
int dodo_launch_attend_dense(dodo_ctx* ctx, int H, float sm_scale, const AttendGroup& g, const DenseMaps& maps,
                             const int32_t* cache_pos, void* O, float* lse, void* workspace, size_t workspace_bytes,
                             int* tickets, int* dev_status, const DenseGather* gather, cudaStream_t st);
int dodo_attend_tile_keys(int dtype, int dh);
int dodo_attend_max_qt(int dtype, int dh);
int dodo_attend_max_cluster();   // most chunks of one (query tile, head) that can merge inside a cluster
// Table for AttendPlan::cluster_cap of the kernel that serves (dtype, dh, qt), from the occupancy calculator
// (cached in the context); NULL if that kernel is not built.
const int* dodo_attend_cluster_cap(dodo_ctx* ctx, int dtype, int dh, int qt);

#ifdef __CUDACC__
// Programmatic dependent launch.  The library's streaming kernels are launched with programmatic stream
// serialization: their blocks may be scheduled while the kernel before them on the stream drains, which hides
// the launch latency of short dependent kernels.  Each of them calls dodo_grid_dependency_sync() before its
// first global-memory access (the wait returns once everything earlier on the stream has completed and its
// writes are visible) and releases its own successor right after, so that never more than one kernel runs ahead.
__device__ __forceinline__ void dodo_grid_dependency_sync() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
template <typename... KArgs, typename... Args>
cudaError_t dodo_launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_gpu(int* p, int v) {
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// 16 bytes of storage elements widened to fp32.
template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int kElems = 4;
    static __device__ __forceinline__ void unpack(const uint4& v, float* f) {
        f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int kElems = 8;
    static __device__ __forceinline__ void unpack(const uint4& v, float* f) {
        f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
        f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
        f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
        f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
    }
};

// Streaming 16-byte global load: read-only path, no L1 allocation.
__device__ __forceinline__ uint4 ld_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
#endif
