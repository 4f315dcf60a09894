// Host-side planning for the attend kernels: query-tile size, split-K chunking per sequence and launch
// groups, and the tensor maps of the tensor-core kernels.  No device work happens here.
#include <stdarg.h>

#include "dodo_internal.cuh"

namespace {

int seq_tiles(const AttendShape& s, int b, int TK) {
    return ((s.cache_len ? s.cache_len[b] : 0) + TK - 1) / TK + ((s.loc_len ? s.loc_len[b] : 0) + TK - 1) / TK;
}

}  // namespace

namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

// [rows, H*dh] bf16 tensor, box of 64 elements x box_rows rows, 128-byte swizzle
int encode_sw128(void* fn, CUtensorMap* map, const void* base, int width, int rows, int box_rows, char* err,
                 size_t err_len) {
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(width), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {dims[0] * 2};
    const cuuint32_t box[2] = {64, static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
        map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        if (err != nullptr && err_len > 0) snprintf(err, err_len, "cuTensorMapEncodeTiled failed with %d", static_cast<int>(r));
        return DODO_ERR_CUDA;
    }
    return DODO_OK;
}
}  // namespace

namespace {
// encode_sw128 through the context's small cache: serving loops pass the same buffers call after call
int cached_sw128(dodo_ctx* ctx, CUtensorMap* map, const void* base, int width, int rows, int box_rows, char* err,
                 size_t err_len) {
    const int n = static_cast<int>(sizeof ctx->map_cache / sizeof ctx->map_cache[0]);
    for (int i = 0; i < n; ++i) {
        const dodo_ctx::MapEntry& e = ctx->map_cache[i];
        if (e.base == base && e.rows == rows && e.width == width && e.box_rows == box_rows && base != nullptr) {
            *map = e.map;
            return DODO_OK;
        }
    }
    const int rc = encode_sw128(ctx->encode_tiled, map, base, width, rows, box_rows, err, err_len);
    if (rc != DODO_OK) return rc;
    dodo_ctx::MapEntry& e = ctx->map_cache[ctx->map_next];
    ctx->map_next = (ctx->map_next + 1) % n;
    e.base = base; e.rows = rows; e.width = width; e.box_rows = box_rows; e.map = *map;
    return DODO_OK;
}
}  // namespace

int dodo_encode_bf16_rows(dodo_ctx* ctx, CUtensorMap* map, const void* base, int width, int rows, int box_rows) {
    return cached_sw128(ctx, map, base, width, rows, box_rows, ctx->err, sizeof ctx->err);
}

int dodo_dense_encode_maps(dodo_ctx* ctx, const AttendShape& s, const void* Q, int q_rows, const void* cacheK,
                           const void* cacheV, int cache_rows, int cache_box_rows, const void* locK, const void* locV,
                           int loc_rows, DenseMaps& maps) {
    char* err = ctx->err;
    const size_t err_len = sizeof ctx->err;
    memset(&maps, 0, sizeof maps);
    int rc;
    if ((rc = cached_sw128(ctx, &maps.Q, Q, s.H * s.dh, q_rows, dodo_dense_tile_queries(), err, err_len)) != DODO_OK) return rc;
    if (cache_rows > 0) {
        if ((rc = cached_sw128(ctx, &maps.cK, cacheK, s.H * s.dh, cache_rows, cache_box_rows, err, err_len)) != DODO_OK) return rc;
        if ((rc = cached_sw128(ctx, &maps.cV, cacheV, s.H * s.dh, cache_rows, cache_box_rows, err, err_len)) != DODO_OK) return rc;
    }
    if (loc_rows > 0) {
        if ((rc = cached_sw128(ctx, &maps.lK, locK, s.H * s.dh, loc_rows, dodo_dense_tile_keys(), err, err_len)) != DODO_OK) return rc;
        if ((rc = cached_sw128(ctx, &maps.lV, locV, s.H * s.dh, loc_rows, dodo_dense_tile_keys(), err, err_len)) != DODO_OK) return rc;
    }
    return DODO_OK;
}

void dodo_attend_plan_begin(const AttendShape& s, int target_ctas, AttendPlan& plan, AttendTotals& tot) {
    const int TK = dodo_attend_tile_keys(s.dtype, s.dh);
    int max_tq = 0;
    for (int b = 0; b < s.B; ++b) {
        const int tq = s.q_off[b + 1] - s.q_off[b];
        max_tq = max_tq > tq ? max_tq : tq;
    }
    plan.qt = max_tq <= 1 ? 1 : max_tq <= 2 ? 2 : max_tq <= 4 ? 4 : 8;
    const int max_qt = dodo_attend_max_qt(s.dtype, s.dh);
    if (plan.qt > max_qt) plan.qt = max_qt;
    plan.cluster_cap = nullptr;
    tot.units = tot.work = tot.part_rows = tot.tick_rows = 0;
    for (int b = 0; b < s.B; ++b) {
        const int tq = s.q_off[b + 1] - s.q_off[b];
        if (tq == 0) continue;
        const int64_t qtiles = (tq + plan.qt - 1) / plan.qt;
        tot.units += qtiles * s.H;
        tot.work += qtiles * s.H * seq_tiles(s, b, TK);
    }
    tot.target = target_ctas;
    // split the keys only while there are too few (query tile, head) units to fill the device
    tot.split = tot.units < tot.target && tot.work > tot.units;
}

void dodo_attend_plan_group(const AttendShape& s, const AttendPlan& plan, AttendTotals& tot, int b0, int nb,
                            AttendGroup& g) {
    const int TK = dodo_attend_tile_keys(s.dtype, s.dh);
    g.nseq = nb;
    g.cta0[0] = 0;
    // first pass: the chunk count every sequence would take by itself
    int chunks[DODO_GROUP];
    int chunks_all = -1;   // that count if all sequences with queries share one, else 0
    int64_t units = 0;     // (query tile, head) units of the group
    for (int i = 0; i < nb; ++i) {
        const int b = b0 + i;
        const int tq = s.q_off[b + 1] - s.q_off[b];
        const int tiles = seq_tiles(s, b, TK);
        const int qtiles = (tq + plan.qt - 1) / plan.qt;
        int nchunk = 1;
        if (tot.split && tiles > 1) {
            // share of the target proportional to this sequence's work, rounded
            int64_t want = (static_cast<int64_t>(tiles) * tot.target + tot.work / 2) / tot.work;
            if (want < 1) want = 1;
            if (want > tiles) want = tiles;
            const int ct = static_cast<int>((tiles + want - 1) / want);
            nchunk = (tiles + ct - 1) / ct;
        }
        chunks[i] = nchunk;
        units += static_cast<int64_t>(qtiles) * s.H;
        if (qtiles > 0) chunks_all = (chunks_all < 0 || chunks_all == nchunk) ? nchunk : 0;
    }
    // Clusters: when every sequence takes the same number of chunks, the chunks of a unit can be the blocks of
    // one cluster and merge in shared memory instead of through the workspace.  Only while all clusters are
    // resident at once -- the shared-memory merge shortens the tail of a single wave, whereas with more
    // clusters than fit whole clusters queue where single blocks would backfill -- so the chunk count drops
    // to the largest cluster size that fits, if that keeps at least three quarters of the blocks.
    g.cluster = 0;
    if (plan.cluster_cap != nullptr && chunks_all >= 2) {
        int c = chunks_all < dodo_attend_max_cluster() ? chunks_all : dodo_attend_max_cluster();
        while (c >= 2 && units > plan.cluster_cap[c]) --c;
        if (c >= 2 && 4 * c >= 3 * chunks_all) g.cluster = c;
    }
    bool uniform = true;
    for (int i = 0; i < nb; ++i) {
        const int b = b0 + i;
        const int tq = s.q_off[b + 1] - s.q_off[b];
        const int cl = s.cache_len ? s.cache_len[b] : 0, ll = s.loc_len ? s.loc_len[b] : 0;
        const int tiles = seq_tiles(s, b, TK);
        const int qtiles = (tq + plan.qt - 1) / plan.qt;
        const int nchunk = g.cluster > 1 ? g.cluster : chunks[i];   // (a chunk past the last tile is empty)
        AttendSeq& q = g.seq[i];
        q.q_row0 = s.q_off[b];
        q.tq = tq;
        q.q_pos0 = s.q_pos0[b];
        q.c_row0 = s.cache_len ? s.cache_off[b] : 0;
        q.c_len = cl;
        q.l_row0 = ll > 0 ? s.loc_off[b] : 0;
        q.l_len = ll;
        q.l_pos0 = ll > 0 ? s.loc_pos0[b] : 0;
        q.nchunk = nchunk;
        q.ctiles = nchunk == 1 ? (tiles > 0 ? tiles : 1) : (tiles + nchunk - 1) / nchunk;
        q.part0 = static_cast<int>(tot.part_rows);
        q.tick0 = static_cast<int>(tot.tick_rows);
        if (nchunk > 1 && g.cluster == 0) {   // merged through the workspace: partial rows and a counter per unit
            tot.part_rows += static_cast<int64_t>(tq) * s.H * nchunk;
            tot.tick_rows += static_cast<int64_t>(qtiles) * s.H;
        }
        g.cta0[i + 1] = g.cta0[i] + qtiles * s.H * nchunk;
        if (g.cta0[i + 1] - g.cta0[i] != g.cta0[1]) uniform = false;
    }
    for (int i = nb; i < DODO_GROUP; ++i) g.cta0[i + 1] = g.cta0[nb];
    g.uniform_ctas = (uniform && nb > 0 && g.cta0[1] > 0) ? g.cta0[1] : 0;
}
