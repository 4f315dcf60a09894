// dodo_attend_noalloc: the attention entry point for callers that must not allocate.
//
// dodo_attend needs two pieces of scratch in global memory: the split-K partial results (normally
// the caller's workspace) and the arrival counters (normally owned by a dodo_ctx, which
// dodo_create obtains with cudaMalloc).  Some users of this library cannot make either
// allocation: code running inside a serving engine whose memory pool has already claimed the
// whole device, plug-ins that are handed raw pointers and a stream but are forbidden to touch the
// allocator, and code on latency-critical paths where the implicit device synchronisation of
// cudaMalloc/cudaFree is not acceptable.  For them this file keeps the scratch in a fixed
// file-scope device array that is part of the loaded library image.
//
// Cost and limits: every GPU that loads the library holds kScratchBytes (4 MiB) until the process
// exits.  One call may cover at most DODO_GROUP (64) sequences, and its split-K plan must fit the
// array; otherwise the call is refused with DODO_ERR_CAPACITY before anything is launched.
//
// All calls share the one array, and it keeps whatever the previous call left there.  The
// counters, which must start at zero, are cleared on the caller's stream at the start of every
// call; the partial results are always written before they are read.  Two calls that overlap on the
// GPU (different streams, or different processes' threads on one device without ordering) race on
// the array and give wrong results: keep calls to this entry point ordered per device.
//
// There is no device status word here: the streaming attend kernel, the only one this entry point
// launches, has no bounded wait and follows no caller-supplied index, so it has nothing to report.
#include <stdarg.h>

#include <mutex>

#include "dodo_internal.cuh"

namespace {

constexpr size_t kScratchBytes = 4u << 20;          // the whole static scratch
constexpr size_t kCounterInts = 4096;               // arrival counters at the front ...
constexpr size_t kPartialOffset = kCounterInts * sizeof(int);  // ... then the partial results
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

struct DeviceSetup {
    bool ready;
    unsigned char* scratch;   // device address of g_noalloc_scratch on this device
    int num_sms;
};
DeviceSetup g_setup[kMaxDevices];
std::mutex g_setup_lock;      // host threads may make their first calls at the same time

int fail(char* err, size_t err_len, int status, const char* fmt, ...) {
    if (err != nullptr && err_len > 0) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(err, err_len, fmt, ap);
        va_end(ap);
    }
    return status;
}

// Once per device, with that device current: the name g_noalloc_scratch means nothing to a kernel
// when used from host code, so ask the runtime for the array's address on this device.
int setup_device(int device, DeviceSetup* out, char* err, size_t err_len) {
    std::lock_guard<std::mutex> hold(g_setup_lock);
    DeviceSetup& s = g_setup[device];
    if (s.ready) { *out = s; return DODO_OK; }
    void* ptr = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess || ptr == nullptr)
        return fail(err, err_len, DODO_ERR_CUDA, "cudaGetSymbolAddress(static scratch): %s", cudaGetErrorString(e));
    int major = 0, sms = 0;
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) return fail(err, err_len, DODO_ERR_CUDA, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
    if (major != 10) return fail(err, err_len, DODO_ERR_CUDA, "device %d is not sm_100", device);
    s.scratch = static_cast<unsigned char*>(ptr);
    s.num_sms = sms;
    s.ready = true;
    *out = s;
    return DODO_OK;
}

}  // namespace

extern "C" int dodo_attend_noalloc(const void* Q, const int32_t* q_off, const int32_t* q_pos0, int dtype, int H,
                                   int dh, float sm_scale, const void* cacheK, const void* cacheV,
                                   const int32_t* cache_pos, const int32_t* cache_off, const int32_t* cache_len,
                                   const void* locK, const void* locV, const int32_t* loc_off,
                                   const int32_t* loc_len, const int32_t* loc_pos0, int loc_rows, int B, void* O,
                                   float* lse, void* stream, char* err, size_t err_len) {
    if (err != nullptr && err_len > 0) err[0] = '\0';
    if (B < 0 || B > DODO_GROUP)
        return fail(err, err_len, B < 0 ? DODO_ERR_INVALID_ARG : DODO_ERR_CAPACITY,
                    "B = %d: this entry point takes 0..%d sequences per call", B, DODO_GROUP);
    if (dtype != DODO_F32 && dtype != DODO_BF16) return fail(err, err_len, DODO_ERR_UNSUPPORTED, "dtype %d", dtype);
    if (dh != 64 && dh != 128) return fail(err, err_len, DODO_ERR_UNSUPPORTED, "head size %d (supported: 64, 128)", dh);
    if (H <= 0) return fail(err, err_len, DODO_ERR_INVALID_ARG, "H = %d", H);
    if (q_off == nullptr || q_off[0] != 0) return fail(err, err_len, DODO_ERR_INVALID_ARG, "q_off must start at 0");
    for (int b = 0; b < B; ++b)
        if (q_off[b + 1] < q_off[b]) return fail(err, err_len, DODO_ERR_INVALID_ARG, "q_off must be non-decreasing");
    if (B > 0 && q_pos0 == nullptr) return fail(err, err_len, DODO_ERR_INVALID_ARG, "q_pos0 must not be NULL");
    if (q_off[B] == 0) return DODO_OK;
    if (Q == nullptr || O == nullptr || !dodo_aligned16(Q) || !dodo_aligned16(O))
        return fail(err, err_len, DODO_ERR_INVALID_ARG, "Q and O must be non-NULL and 16-byte aligned");
    bool any_cache = false, any_local = false;
    if (cache_len != nullptr) {
        if (cache_off == nullptr || cache_off[0] != 0) return fail(err, err_len, DODO_ERR_INVALID_ARG, "cache_off must start at 0");
        for (int b = 0; b < B; ++b) {
            if (cache_off[b + 1] < cache_off[b] || cache_len[b] < 0 || cache_len[b] > cache_off[b + 1] - cache_off[b])
                return fail(err, err_len, DODO_ERR_INVALID_ARG, "sequence %d: cache_len %d outside its region", b, cache_len[b]);
            any_cache = any_cache || cache_len[b] > 0;
        }
    }
    if (loc_len != nullptr) {
        for (int b = 0; b < B; ++b) {
            if (loc_len[b] < 0) return fail(err, err_len, DODO_ERR_INVALID_ARG, "sequence %d: negative loc_len", b);
            if (loc_len[b] > 0) {
                if (loc_off == nullptr || loc_pos0 == nullptr) return fail(err, err_len, DODO_ERR_INVALID_ARG, "loc_off and loc_pos0 must not be NULL");
                if (loc_off[b] < 0 || static_cast<int64_t>(loc_off[b]) + loc_len[b] > loc_rows)
                    return fail(err, err_len, DODO_ERR_INVALID_ARG, "sequence %d: local rows outside loc_rows = %d", b, loc_rows);
                any_local = true;
            }
        }
    }
    if (any_cache && (cacheK == nullptr || cacheV == nullptr || cache_pos == nullptr || !dodo_aligned16(cacheK) || !dodo_aligned16(cacheV)))
        return fail(err, err_len, DODO_ERR_INVALID_ARG, "cacheK, cacheV, cache_pos must be non-NULL, K/V 16-byte aligned");
    if (any_local && (locK == nullptr || locV == nullptr || !dodo_aligned16(locK) || !dodo_aligned16(locV)))
        return fail(err, err_len, DODO_ERR_INVALID_ARG, "locK and locV must be non-NULL and 16-byte aligned");

    // ---- per-device set-up (first call on a device; do it before any stream capture) -----------
    int device = -1;
    cudaError_t e = cudaGetDevice(&device);
    if (e != cudaSuccess || device < 0 || device >= kMaxDevices)
        return fail(err, err_len, DODO_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    DeviceSetup su;
    int rc = setup_device(device, &su, err, err_len);
    if (rc != DODO_OK) return rc;
    int* counters = reinterpret_cast<int*>(su.scratch);
    float* partials = reinterpret_cast<float*>(su.scratch + kPartialOffset);
    const size_t part_rows_cap = (kScratchBytes - kPartialOffset) / (static_cast<size_t>(dh + 2) * sizeof(float));

    // ---- plan: same rules as dodo_attend, with a split target sized for the fixed scratch --------
    AttendShape shp = {q_off, q_pos0, cache_off, cache_len, loc_off, loc_len, loc_pos0, B, H, dh, dtype};
    AttendPlan plan;
    AttendTotals tot;
    dodo_attend_plan_begin(shp, 2 * su.num_sms, plan, tot);
    AttendGroup g;
    dodo_attend_plan_group(shp, plan, tot, 0, B, g);
    if (static_cast<size_t>(tot.part_rows) > part_rows_cap || static_cast<size_t>(tot.tick_rows) > kCounterInts)
        return fail(err, err_len, DODO_ERR_CAPACITY,
                    "this call needs %lld partial rows and %lld counters; the static scratch holds %zu rows at head "
                    "size %d and %zu counters -- use dodo_attend with a workspace for larger batches",
                    static_cast<long long>(tot.part_rows), static_cast<long long>(tot.tick_rows), part_rows_cap, dh,
                    kCounterInts);
    const AttendMaps maps = {any_cache ? cacheK : nullptr, any_cache ? cacheV : nullptr,
                             any_local ? locK : nullptr, any_local ? locV : nullptr};

    // the counters must start at zero; the array still holds the last call's
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    e = cudaMemsetAsync(su.scratch, 0, kPartialOffset, st);
    if (e != cudaSuccess) return fail(err, err_len, DODO_ERR_CUDA, "cudaMemsetAsync(static scratch): %s", cudaGetErrorString(e));

    dodo_ctx msg;   // host-side only: collects the launcher's error text
    memset(&msg, 0, sizeof msg);
    // (no cache row is read ahead of the launch's dependency wait: this entry point cannot know what precedes it)
    rc = dodo_launch_attend(&msg, dtype, H, dh, sm_scale, plan, g, Q, maps, cache_pos, O, lse, partials, counters,
                            false, st);
    if (rc != DODO_OK) return fail(err, err_len, rc, "%s", msg.err);
    return DODO_OK;
}
