// Host-side planning for the attend kernel: query-tile size, split-K chunking per sequence, launch
// groups, and the TMA descriptors.  No device work happens here.
#include <stdarg.h>

#include "dodo_internal.cuh"

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

int encode_one(void* fn, CUtensorMap* map, const void* base, const AttendShape& s, int rows, int box_rows, char* err,
               size_t err_len) {
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(s.H) * static_cast<cuuint64_t>(s.dh),
                                static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {dims[0] * dodo_elem_bytes(s.dtype)};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(s.dh), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = reinterpret_cast<EncodeTiledFn>(fn)(
        map, s.dtype == DODO_BF16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
        const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        if (err != nullptr && err_len > 0) snprintf(err, err_len, "cuTensorMapEncodeTiled failed with %d", static_cast<int>(r));
        return DODO_ERR_CUDA;
    }
    return DODO_OK;
}

int seq_tiles(const AttendShape& s, int b, int TK) {
    return ((s.cache_len ? s.cache_len[b] : 0) + TK - 1) / TK + ((s.loc_len ? s.loc_len[b] : 0) + TK - 1) / TK;
}

}  // namespace

int dodo_attend_encode_maps(void* encode_fn, const AttendShape& s, const void* cacheK, const void* cacheV,
                            int cache_rows, const void* locK, const void* locV, int loc_rows, AttendMaps& maps,
                            char* err, size_t err_len) {
    memset(&maps, 0, sizeof maps);
    const int boxes[2] = {dodo_attend_tile_keys(s.dtype, s.dh), dodo_attend_box_rows()};
    int rc;
    for (int i = 0; i < 2; ++i) {
        if (cache_rows > 0) {
            if ((rc = encode_one(encode_fn, &maps.cK[i], cacheK, s, cache_rows, boxes[i], err, err_len)) != DODO_OK) return rc;
            if ((rc = encode_one(encode_fn, &maps.cV[i], cacheV, s, cache_rows, boxes[i], err, err_len)) != DODO_OK) return rc;
        }
        if (loc_rows > 0) {
            if ((rc = encode_one(encode_fn, &maps.lK[i], locK, s, loc_rows, boxes[i], err, err_len)) != DODO_OK) return rc;
            if ((rc = encode_one(encode_fn, &maps.lV[i], locV, s, loc_rows, boxes[i], err, err_len)) != DODO_OK) return rc;
        }
    }
    return DODO_OK;
}

void dodo_attend_plan_begin(const AttendShape& s, int stages, AttendPlan& plan, AttendTotals& tot) {
    int max_tq = 0;
    for (int b = 0; b < s.B; ++b) {
        const int tq = s.q_off[b + 1] - s.q_off[b];
        max_tq = max_tq > tq ? max_tq : tq;
    }
    plan.qt = max_tq <= 1 ? 1 : max_tq <= 2 ? 2 : max_tq <= 4 ? 4 : 8;
    const int max_qt = dodo_attend_max_qt(s.dtype, s.dh);
    if (plan.qt > max_qt) plan.qt = max_qt;
    plan.stages = stages;
    tot.max_units = 0;
    tot.max_blocks = 0;
}

// One launch group: the (unit, tile) list of its sequences is dealt in equal contiguous ranges to
// min(target_blocks, items) persistent blocks.
void dodo_attend_plan_group(const AttendShape& s, const AttendPlan& plan, int target_blocks, AttendTotals& tot,
                            int b0, int nb, AttendGroup& g) {
    const int TK = dodo_attend_tile_keys(s.dtype, s.dh);
    g.nseq = nb;
    g.tile0[0] = 0;
    int64_t units = 0;
    for (int i = 0; i < nb; ++i) {
        const int b = b0 + i;
        const int tq = s.q_off[b + 1] - s.q_off[b];
        const int cl = s.cache_len ? s.cache_len[b] : 0, ll = s.loc_len ? s.loc_len[b] : 0;
        const int qtiles = (tq + plan.qt - 1) / plan.qt;
        int tiles = seq_tiles(s, b, TK);
        if (tiles == 0) tiles = 1;  // a unit without keys still needs one (empty) item to write O = 0
        AttendSeq& q = g.seq[i];
        q.q_row0 = s.q_off[b];
        q.tq = tq;
        q.q_pos0 = s.q_pos0[b];
        q.c_row0 = s.cache_len ? s.cache_off[b] : 0;
        q.c_len = cl;
        q.l_row0 = ll > 0 ? s.loc_off[b] : 0;
        q.l_len = ll;
        q.l_pos0 = ll > 0 ? s.loc_pos0[b] : 0;
        q.tiles = tiles;
        q.units = qtiles * s.H;
        q.unit0 = static_cast<int>(units);
        q.pad = 0;
        units += q.units;
        g.tile0[i + 1] = g.tile0[i] + static_cast<long long>(q.units) * tiles;
    }
    for (int i = nb; i < DODO_GROUP; ++i) g.tile0[i + 1] = g.tile0[nb];
    const long long total = g.tile0[nb];
    g.nblocks = static_cast<int>(total < target_blocks ? total : target_blocks);
    if (units > tot.max_units) tot.max_units = units;
    if (g.nblocks > tot.max_blocks) tot.max_blocks = g.nblocks;
}
