// extern "C" boundary of the MoSKA library: argument validation and launch sequencing only.
#include <cmath>
#include <cstring>
#include <mutex>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

namespace moska {

char* last_error_buffer()
{
    static thread_local char buf[512] = {0};
    return buf;
}

int fail(int status, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(last_error_buffer(), 512, fmt, ap);
    va_end(ap);
    return status;
}

int check_shape(const moska_shape* s, bool needs_k)
{
    if (s == nullptr) return fail(MOSKA_ERR_INVALID_ARG, "shape is NULL");
    if (s->B < 0 || s->Hq <= 0 || s->Hkv <= 0 || s->C <= 0 || s->L <= 0)
        return fail(MOSKA_ERR_INVALID_ARG, "B >= 0 and Hq, Hkv, C, L > 0 required");
    if (s->Hq % s->Hkv != 0)
        return fail(MOSKA_ERR_INVALID_ARG, "Hq = %d is not a multiple of Hkv = %d", s->Hq, s->Hkv);
    if (s->Hq / s->Hkv > 8)
        return fail(MOSKA_ERR_UNSUPPORTED, "G = Hq / Hkv = %d > 8", s->Hq / s->Hkv);
    if (s->D != 64 && s->D != 128)
        return fail(MOSKA_ERR_UNSUPPORTED, "D = %d, only 64 and 128 are built", s->D);
    if (s->L % 128 != 0) return fail(MOSKA_ERR_UNSUPPORTED, "L = %d is not a multiple of 128", s->L);
    if (needs_k && (s->k < 1 || s->k > s->C))
        return fail(MOSKA_ERR_INVALID_ARG, "k = %d outside [1, C = %d]", s->k, s->C);
    if (s->shared_slots < 1 || s->n_unique_splits < 1)
        return fail(MOSKA_ERR_INVALID_ARG, "shared_slots and n_unique_splits must be >= 1");
    if (s->q_len < 0 || (s->q_len > 1 && s->B % s->q_len != 0))
        return fail(MOSKA_ERR_INVALID_ARG, "q_len = %d must be >= 0 and divide B = %d", s->q_len, s->B);
    if ((long long)s->B * s->Hkv * (long long)(s->k > 0 ? s->k : 1) > 0x7fffffffLL ||
        (long long)s->Hkv * s->C >= 0x7fffffffLL)
        return fail(MOSKA_ERR_UNSUPPORTED, "index range exceeds int32");
    return MOSKA_OK;
}

int check_device()
{
    static thread_local int cached_dev = -1;
    static thread_local int cached_major = 0;
    int dev = 0;
    MOSKA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev != cached_dev) {
        MOSKA_CUDA_TRY(cudaDeviceGetAttribute(&cached_major, cudaDevAttrComputeCapabilityMajor, dev));
        cached_dev = dev;
    }
    if (cached_major != 10)
        return fail(MOSKA_ERR_UNSUPPORTED, "device %d is compute capability %d.x, sm_100 required",
                    dev, cached_major);
    return MOSKA_OK;
}

}  // namespace moska

using namespace moska;

struct moska_profiler {
    int max_steps = 0;
    int n_steps = 0;
    cudaEvent_t* ev = nullptr;  // [max_steps][MOSKA_N_STAGES][2]
    bool* used = nullptr;       // [max_steps][MOSKA_N_STAGES]
    unsigned mask = ~0u;        // stages that are recorded (bit = stage index)
};

namespace {
// Records the begin/end event of one stage of the step being recorded (no-op without profiler).
inline cudaError_t prof_mark(moska_profiler* p, int stage, int which, cudaStream_t st)
{
    if (p == nullptr || p->n_steps >= p->max_steps || !((p->mask >> stage) & 1u)) return cudaSuccess;
    const int i = p->n_steps * MOSKA_N_STAGES + stage;
    p->used[i] = true;
    return cudaEventRecord(p->ev[2 * i + which], st);
}
}  // namespace

// One NVTX range per entry point (visible in a timeline profiler; a no-op when no tool is attached).
struct ApiRange {
    explicit ApiRange(const char* name) { nvtxRangePushA(name); }
    ~ApiRange() { nvtxRangePop(); }
    ApiRange(const ApiRange&) = delete;
    ApiRange& operator=(const ApiRange&) = delete;
};
#define MOSKA_API_RANGE() ApiRange api_range__(__func__)

#define MOSKA_TRY(expr)              \
    do {                             \
        int st__ = (expr);           \
        if (st__ != MOSKA_OK) return st__; \
    } while (0)

#define REQUIRE_PTR(p, align)                                                                   \
    do {                                                                                        \
        if ((p) == nullptr) return fail(MOSKA_ERR_INVALID_ARG, "%s is NULL", #p);               \
        if (!aligned((p), (align)))                                                             \
            return fail(MOSKA_ERR_INVALID_ARG, "%s is not %d-byte aligned", #p, (int)(align));  \
    } while (0)

extern "C" {

int moska_version(void) { return 100; }

const char* moska_last_error(void) { return last_error_buffer(); }

int moska_partial_slots(const moska_shape* shape)
{
    MOSKA_TRY(check_shape(shape, false));
    return shape->shared_slots + shape->n_unique_splits;
}

size_t moska_workspace_bytes(const moska_shape* shape)
{
    if (check_shape(shape, true) != MOSKA_OK) return 0;
    return ws_layout(shape).total;
}

int moska_default_unique_splits(int32_t B, int32_t Hkv, int32_t max_len)
{
    // Enough CTAs to fill 148 SMs several times over, but at least 512 tokens per split so the
    // per-CTA prologue and combine stay small next to the streaming loop.
    if (B <= 0 || Hkv <= 0 || max_len <= 0) return 1;
    const long long want_ctas = 148LL * 12;
    long long n = (want_ctas + (long long)B * Hkv - 1) / ((long long)B * Hkv);
    const long long cap = (max_len + 511) / 512;
    if (n > cap) n = cap;
    if (n < 1) n = 1;
    if (n > 64) n = 64;
    return (int)n;
}

int moska_default_unique_splits_fp8(int32_t B, int32_t Hkv, int32_t max_len)
{
    // The FP8 kernel's CTAs stream half the bytes per token, three of them per SM.  Its time is
    // about  n len / S  +  n s ov / S  +  a len / s  (n = B Hkv CTAs per split, S = CTA slots, ov =
    // fixed cost of a CTA in tokens, a len / s = the tail while the last CTAs run alone), smallest
    // at s = sqrt(a len S / (n ov)); a = 0.7 and ov = 128 tokens fit the measured sweeps.
    if (B <= 0 || Hkv <= 0 || max_len <= 0) return 1;
    const double slots = 148.0 * 3.0, n = (double)B * Hkv;
    long long s = llround(sqrt(0.7 * max_len * slots / (n * 128.0)));
    const long long cap = (max_len + 511) / 512;
    if (s > cap) s = cap;
    if (s < 1) s = 1;
    if (s > 64) s = 64;
    return (int)s;
}

int moska_build_chunk_summaries(const uint16_t* k_shared, float* summaries,
                                const moska_shape* shape, moska_stream stream)
{
    MOSKA_API_RANGE();
    MOSKA_TRY(check_shape(shape, false));
    REQUIRE_PTR(k_shared, 16);
    REQUIRE_PTR(summaries, 16);
    MOSKA_TRY(check_device());
    return launch_summaries(k_shared, summaries, shape, (cudaStream_t)stream);
}

int moska_build_chunk_summaries_attn(const uint16_t* k_shared, float* summaries, float probe_scale,
                                     const moska_shape* shape, moska_stream stream)
{
    MOSKA_API_RANGE();
    MOSKA_TRY(check_shape(shape, false));
    REQUIRE_PTR(k_shared, 16);
    REQUIRE_PTR(summaries, 16);
    if (!(probe_scale >= 0.f) || !std::isfinite(probe_scale))
        return fail(MOSKA_ERR_INVALID_ARG, "probe_scale must be finite and >= 0");
    MOSKA_TRY(check_device());
    return launch_summaries_attn(k_shared, summaries, probe_scale, shape, (cudaStream_t)stream);
}

namespace {
// SMs the persistent tensor-core kernel gets when it runs beside unique attention: both kernels'
// work is estimated (tensor-core items from the shape, unique attention from the token hint at
// 7 TB/s) and the SMs are divided so that neither waits for the other.  Unique attention keeps
// most of the HBM bandwidth on about half of the SMs; if it is the longer job the tensor-core
// kernel hides entirely on the remaining ones.
// Share of the SMs left to unique attention in that case (measured on the largest workload: 45-55 %
// is a flat optimum, 65 % is 0.5 % slower, 85 % 8 % slower; the other workloads do not care).
#ifndef MOSKA_HBM_SM_PCT
#define MOSKA_HBM_SM_PCT 55
#endif
int tc_sm_share(const moska_shape* s, bool dense, double unique_ms)
{
    int dev = 0, n_sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess)
        cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev);
    const double a = shared_tc_cost_sm_ms(s, dense);  // SM * ms
    int x;
    if (s->unique_tokens <= 0) {
        x = dense ? (n_sms * 4) / 5 : (n_sms * 35) / 100;  // no hint: tensor-heavy / HBM-heavy guess
    } else {
        const double b = unique_ms;
        const int hbm_sms = (n_sms * MOSKA_HBM_SM_PCT) / 100;
        if (a <= b * (n_sms - hbm_sms)) x = n_sms - hbm_sms;
        else x = (int)(a * n_sms / (a + b * 0.4 * n_sms));
    }
    if (x < 16) x = 16;
    if (x > n_sms) x = n_sms;
    return x;
}

#ifndef MOSKA_BESIDE_MS
#define MOSKA_BESIDE_MS 0.8
#endif
// The event pair that orders the side stream of a two-stream step after / before the main
// stream.  Events belong to the device they were created on, so there is one pair per (host
// thread, device ordinal), created on first use with that device current and kept.
int fork_join_events(cudaEvent_t* fork, cudaEvent_t* join)
{
    constexpr int kMaxDevices = 64;
    static thread_local cudaEvent_t ev[kMaxDevices][2] = {};
    int dev = 0;
    MOSKA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices)
        return fail(MOSKA_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
    if (ev[dev][0] == nullptr) {
        MOSKA_CUDA_TRY(cudaEventCreateWithFlags(&ev[dev][0], cudaEventDisableTiming));
        MOSKA_CUDA_TRY(cudaEventCreateWithFlags(&ev[dev][1], cudaEventDisableTiming));
    }
    *fork = ev[dev][0];
    *join = ev[dev][1];
    return MOSKA_OK;
}

// Validation + launch of the router; mark_groups also runs the grouping's first pass in it.
int route_impl(const uint16_t* q, const float* summaries, int32_t* topk_idx, float* topk_score,
               const moska_shape* shape, void* ws, size_t ws_bytes, bool mark_groups,
               cudaStream_t stream)
{
    MOSKA_TRY(check_shape(shape, true));
    REQUIRE_PTR(q, 16);
    REQUIRE_PTR(summaries, 16);
    REQUIRE_PTR(topk_idx, 4);
    if ((shape->C > kRouteSmallC || mark_groups) &&
        (ws == nullptr || !aligned(ws, 256) || ws_bytes < ws_layout(shape).total))
        return fail(MOSKA_ERR_WORKSPACE, "workspace missing, misaligned or smaller than %zu bytes",
                    ws_layout(shape).total);
    MOSKA_TRY(check_device());
    return launch_route(q, summaries, topk_idx, topk_score, shape, ws, mark_groups, stream);
}

int group_impl(const int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
               const moska_shape* shape, void* ws, size_t ws_bytes, bool premarked,
               cudaStream_t stream)
{
    MOSKA_TRY(check_shape(shape, true));
    REQUIRE_PTR(topk_idx, 4);
    REQUIRE_PTR(seg_offsets, 4);
    REQUIRE_PTR(seg_entries, 4);
    if (ws == nullptr || !aligned(ws, 256) || ws_bytes < ws_layout(shape).total)
        return fail(MOSKA_ERR_WORKSPACE, "workspace missing, misaligned or smaller than %zu bytes",
                    ws_layout(shape).total);
    MOSKA_TRY(check_device());
    return launch_group(topk_idx, seg_offsets, seg_entries, shape, ws, premarked, stream);
}
}  // namespace

int moska_route(const uint16_t* q, const float* summaries, int32_t* topk_idx, float* topk_score,
                const moska_shape* shape, void* ws, size_t ws_bytes, moska_stream stream)
{
    MOSKA_API_RANGE();
    return route_impl(q, summaries, topk_idx, topk_score, shape, ws, ws_bytes, false,
                      (cudaStream_t)stream);
}

int moska_group_by_chunk(const int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                         const moska_shape* shape, void* ws, size_t ws_bytes, moska_stream stream)
{
    MOSKA_API_RANGE();
    return group_impl(topk_idx, seg_offsets, seg_entries, shape, ws, ws_bytes, false,
                      (cudaStream_t)stream);
}

int moska_group_by_chunk_noalloc(const int32_t* topk_idx, int32_t* seg_offsets,
                                 int32_t* seg_entries, const moska_shape* shape,
                                 moska_stream stream)
{
    MOSKA_API_RANGE();
    MOSKA_TRY(check_shape(shape, true));
    REQUIRE_PTR(topk_idx, 4);
    REQUIRE_PTR(seg_offsets, 4);
    REQUIRE_PTR(seg_entries, 4);
    return launch_group_noalloc(topk_idx, seg_offsets, seg_entries, shape, (cudaStream_t)stream);
}

int moska_debug_check_workspace(void* ws, size_t ws_bytes, const moska_shape* shape,
                                moska_stream stream)
{
    MOSKA_API_RANGE();
    MOSKA_TRY(check_shape(shape, true));
#ifdef MOSKA_DEBUG_GUARDS
    if (ws == nullptr || !aligned(ws, 256) || ws_bytes < ws_layout(shape).total)
        return fail(MOSKA_ERR_WORKSPACE, "workspace missing, misaligned or smaller than %zu bytes",
                    ws_layout(shape).total);
    MOSKA_TRY(check_device());
    return launch_ws_guards(ws, ws_layout(shape), true, (cudaStream_t)stream, ws_layout(shape).total);
#else
    (void)ws; (void)ws_bytes; (void)stream;
    return fail(MOSKA_ERR_UNSUPPORTED, "this build of the library has no workspace guard words "
                                       "(compile with -DMOSKA_DEBUG_GUARDS)");
#endif
}

int moska_shared_attn(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                      const int32_t* topk_idx, const int32_t* seg_offsets,
                      const int32_t* seg_entries, float* o_part, float* lse_part,
                      float softmax_scale, const moska_shape* shape, void* ws, size_t ws_bytes,
                      moska_stream stream)
{
    MOSKA_API_RANGE();
    const bool dense = (topk_idx == nullptr && seg_offsets == nullptr && seg_entries == nullptr);
    MOSKA_TRY(check_shape(shape, !dense));
    REQUIRE_PTR(q, 16);
    REQUIRE_PTR(k_shared, 128);
    REQUIRE_PTR(v_shared, 128);
    REQUIRE_PTR(o_part, 32);
    REQUIRE_PTR(lse_part, 4);
    if (!dense) {
        REQUIRE_PTR(topk_idx, 4);
        REQUIRE_PTR(seg_offsets, 4);
        REQUIRE_PTR(seg_entries, 4);
        if (shape->shared_slots != shape->k)
            return fail(MOSKA_ERR_INVALID_ARG, "routed mode needs shared_slots == k");
        if (ws == nullptr || !aligned(ws, 256) || ws_bytes < ws_layout(shape).total)
            return fail(MOSKA_ERR_WORKSPACE, "workspace missing, misaligned or smaller than %zu bytes",
                        ws_layout(shape).total);
    } else if (shape->shared_slots > shape->C) {
        return fail(MOSKA_ERR_INVALID_ARG, "dense mode needs shared_slots <= C");
    }
    MOSKA_TRY(check_device());
    cudaStream_t st = (cudaStream_t)stream;
    const bool tc = shared_tc_supported(shape);
    if (dense) {
        // enough rows to fill a good part of a 128-row tile: tensor cores; else 16-row tiles
        if (tc && (long long)shape->B * (shape->Hq / shape->Hkv) >= kDenseTcMinRows)
            return launch_shared_tc(q, k_shared, v_shared, nullptr, o_part, lse_part, softmax_scale,
                                    shape, ws, true, 0, st);
        return launch_shared_small(q, k_shared, v_shared, nullptr, o_part, lse_part, softmax_scale,
                                   shape, ws, true, false, st);
    }
    // routed: the grouping pass cut every segment into work items for the kernel that serves the shape
    if (tc)
        MOSKA_TRY(launch_shared_tc(q, k_shared, v_shared, seg_entries, o_part, lse_part, softmax_scale,
                                   shape, ws, false, 0, st));
    return launch_shared_small(q, k_shared, v_shared, seg_entries, o_part, lse_part, softmax_scale,
                               shape, ws, false, tc, st);
}

int moska_shared_attn_fp8(const uint16_t* q, const uint8_t* k8_shared, const uint8_t* v8_shared,
                          const float* k_scale, const float* v_scale, const int32_t* topk_idx,
                          const int32_t* seg_offsets, const int32_t* seg_entries, float* o_part,
                          float* lse_part, float softmax_scale, const moska_shape* shape, void* ws,
                          size_t ws_bytes, moska_stream stream)
{
    MOSKA_API_RANGE();
    MOSKA_TRY(check_shape(shape, true));
    if (!shared_tc_supported(shape))
        return fail(MOSKA_ERR_UNSUPPORTED, "the FP8 shared store is built for D = 128");
    REQUIRE_PTR(q, 16);
    REQUIRE_PTR(k8_shared, 128);
    REQUIRE_PTR(v8_shared, 128);
    REQUIRE_PTR(k_scale, 4);
    REQUIRE_PTR(v_scale, 4);
    REQUIRE_PTR(o_part, 32);
    REQUIRE_PTR(lse_part, 4);
    const bool dense = (topk_idx == nullptr && seg_offsets == nullptr && seg_entries == nullptr);
    if (!dense) {
        REQUIRE_PTR(topk_idx, 4);
        REQUIRE_PTR(seg_offsets, 4);
        REQUIRE_PTR(seg_entries, 4);
        if (shape->shared_slots != shape->k)
            return fail(MOSKA_ERR_INVALID_ARG, "routed mode needs shared_slots == k");
    } else if (shape->shared_slots > shape->C) {
        return fail(MOSKA_ERR_INVALID_ARG, "dense mode needs shared_slots <= C");
    }
    // (dense mode too: the workspace holds the f16 copy of the queries)
    if (ws == nullptr || !aligned(ws, 256) || ws_bytes < ws_layout(shape).total)
        return fail(MOSKA_ERR_WORKSPACE, "workspace missing, misaligned or smaller than %zu bytes",
                    ws_layout(shape).total);
    MOSKA_TRY(check_device());
    // dense mode: every item on the tensor-core kernel; routed mode: segments of more than 8 rows
    // there, the 8-row tiles streamed
    MOSKA_TRY(launch_shared_tc_fp8(q, k8_shared, v8_shared, k_scale, v_scale, dense ? nullptr : seg_entries,
                                   o_part, lse_part, softmax_scale, shape, ws, dense, 0, (cudaStream_t)stream));
    if (dense) return MOSKA_OK;
    return launch_shared_small_fp8(q, k8_shared, v8_shared, k_scale, v_scale, seg_entries, o_part,
                                   lse_part, softmax_scale, shape, ws, (cudaStream_t)stream);
}

int moska_device_status(int32_t* status_host)
{
    if (status_host == nullptr) return fail(MOSKA_ERR_INVALID_ARG, "status_host is NULL");
    int v = 0;
    MOSKA_TRY(read_status(&v));
    *status_host = v;
    return MOSKA_OK;
}

int moska_unique_attn(const uint16_t* q, const uint16_t* k_unique, const uint16_t* v_unique,
                      const int64_t* kv_start, const int32_t* kv_len, float* o_part,
                      float* lse_part, float softmax_scale, const moska_shape* shape,
                      moska_stream stream)
{
    MOSKA_API_RANGE();
    MOSKA_TRY(check_shape(shape, false));
    if (shape->q_len > 1 && (shape->D != 128 || shape->q_len * (shape->Hq / shape->Hkv) > 16))
        return fail(MOSKA_ERR_UNSUPPORTED,
                    "q_len = %d needs D = 128 and q_len * G <= 16; pass the tokens as batch rows "
                    "with q_len = 1 and aliased kv_start instead", shape->q_len);
    REQUIRE_PTR(q, 16);
    REQUIRE_PTR(k_unique, 16);
    REQUIRE_PTR(v_unique, 16);
    REQUIRE_PTR(kv_start, 8);
    REQUIRE_PTR(kv_len, 4);
    REQUIRE_PTR(o_part, 16);
    REQUIRE_PTR(lse_part, 4);
    MOSKA_TRY(check_device());
    return launch_unique(q, k_unique, v_unique, kv_start, kv_len, o_part, lse_part, softmax_scale,
                         shape, (cudaStream_t)stream);
}

int moska_unique_attn_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8,
                          const float* k_scale, const float* v_scale, const int64_t* kv_start,
                          const int32_t* kv_len, float* o_part, float* lse_part,
                          float softmax_scale, const moska_shape* shape, moska_stream stream)
{
    MOSKA_API_RANGE();
    MOSKA_TRY(check_shape(shape, false));
    if (shape->D != 128) return fail(MOSKA_ERR_UNSUPPORTED, "FP8 unique attention is built for D = 128");
    if (shape->q_len > 1 && shape->q_len * (shape->Hq / shape->Hkv) > 8)
        return fail(MOSKA_ERR_UNSUPPORTED,
                    "FP8 unique attention with q_len = %d needs q_len * G <= 8; pass the tokens as "
                    "batch rows with q_len = 1 and aliased kv_start instead", shape->q_len);
    REQUIRE_PTR(q, 16);
    REQUIRE_PTR(k8, 16);
    REQUIRE_PTR(v8, 16);
    REQUIRE_PTR(k_scale, 4);
    REQUIRE_PTR(v_scale, 4);
    REQUIRE_PTR(kv_start, 8);
    REQUIRE_PTR(kv_len, 4);
    REQUIRE_PTR(o_part, 16);
    REQUIRE_PTR(lse_part, 4);
    MOSKA_TRY(check_device());
    return launch_unique_fp8(q, k8, v8, k_scale, v_scale, kv_start, kv_len, o_part, lse_part,
                             softmax_scale, shape, (cudaStream_t)stream);
}

int moska_merge(const float* o_part, const float* lse_part, uint16_t* out, float* out_f32,
                float* lse_out, const moska_shape* shape, moska_stream stream)
{
    MOSKA_API_RANGE();
    MOSKA_TRY(check_shape(shape, false));
    REQUIRE_PTR(o_part, 16);
    REQUIRE_PTR(lse_part, 4);
    REQUIRE_PTR(out, 8);
    MOSKA_TRY(check_device());
    if (out_f32 != nullptr && !aligned(out_f32, 16))
        return fail(MOSKA_ERR_INVALID_ARG, "out_f32 is not 16-byte aligned");
    return launch_merge(o_part, lse_part, out, out_f32, lse_out, shape, (cudaStream_t)stream);
}

int moska_gemv_baseline(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                        const int32_t* topk_idx, float* o_part, float* lse_part,
                        float softmax_scale, const moska_shape* shape, moska_stream stream)
{
    MOSKA_API_RANGE();
    const bool dense = topk_idx == nullptr;
    MOSKA_TRY(check_shape(shape, !dense));
    REQUIRE_PTR(q, 16);
    REQUIRE_PTR(k_shared, 16);
    REQUIRE_PTR(v_shared, 16);
    REQUIRE_PTR(o_part, 16);
    REQUIRE_PTR(lse_part, 4);
    MOSKA_TRY(check_device());
    if (!dense && shape->shared_slots != shape->k)
        return fail(MOSKA_ERR_INVALID_ARG, "routed mode needs shared_slots == k");
    if (dense && shape->shared_slots > shape->C)
        return fail(MOSKA_ERR_INVALID_ARG, "dense mode needs shared_slots <= C");
    return launch_gemv_baseline(q, k_shared, v_shared, topk_idx, o_part, lse_part, softmax_scale,
                                shape, (cudaStream_t)stream);
}

namespace {
// The private KV store of a decode step: bf16 (k, v) or FP8 E4M3 codes with per-token scales.
struct UniqueKv {
    const uint16_t* k = nullptr;
    const uint16_t* v = nullptr;
    const uint8_t* k8 = nullptr;
    const uint8_t* v8 = nullptr;
    const float* k_scale = nullptr;
    const float* v_scale = nullptr;
    bool fp8 = false;
};

int unique_impl(const uint16_t* q, const UniqueKv& kv, const int64_t* kv_start, const int32_t* kv_len,
                float* o_part, float* lse_part, float softmax_scale, const moska_shape* shape,
                cudaStream_t st)
{
    if (kv.fp8)
        return moska_unique_attn_fp8(q, kv.k8, kv.v8, kv.k_scale, kv.v_scale, kv_start, kv_len, o_part,
                                     lse_part, softmax_scale, shape, st);
    return moska_unique_attn(q, kv.k, kv.v, kv_start, kv_len, o_part, lse_part, softmax_scale, shape,
                             st);
}

// The shared store in FP8 (codes + one scale per (KV head, chunk)), when the step uses one.
struct SharedF8 {
    const uint8_t* k8 = nullptr;
    const uint8_t* v8 = nullptr;
    const float* k_scale = nullptr;
    const float* v_scale = nullptr;
};

// moska_decode_step_host: results of at least this many bytes leave the device in pieces, each
// copied while the next one is merged
#ifndef MOSKA_HOST_PIECES
#define MOSKA_HOST_PIECES 4
#endif
#ifndef MOSKA_HOST_Q_DIRECT
#define MOSKA_HOST_Q_DIRECT 1
#endif
constexpr size_t kHostPiecesMinBytes = 4u << 20;
constexpr int kHostPieces = MOSKA_HOST_PIECES;

int decode_step_impl(const uint16_t* q, const float* summaries, const uint16_t* k_shared,
                     const uint16_t* v_shared, const SharedF8* f8, const UniqueKv& kv, const int64_t* kv_start,
                     const int32_t* kv_len, int32_t* topk_idx, int32_t* seg_offsets,
                     int32_t* seg_entries, float* o_part, float* lse_part, uint16_t* out,
                     float* lse_out, float softmax_scale, const moska_shape* shape, void* ws,
                     size_t ws_bytes, moska_stream stream, moska_stream side_stream,
                     moska_profiler* prof, uint16_t* out_host = nullptr,
                     const uint16_t* q_host = nullptr)
{
    const bool dense = summaries == nullptr;
    cudaStream_t st = (cudaStream_t)stream, side = (cudaStream_t)side_stream;
    // q_host (moska_decode_step_host): the queries still have to be copied into q.  With two
    // streams and a page-locked source the copy runs on the side stream in front of the router
    // while unique attention, first on `stream`, reads its query rows straight from host memory.
    const size_t q_bytes = sizeof(uint16_t) * (size_t)shape->B * shape->Hq * shape->D;
    const uint16_t* q_unique = q;
    bool copy_on_side = false;
    if (q_host != nullptr) {
#if MOSKA_HOST_Q_DIRECT
        cudaPointerAttributes attr{};
        if (side != nullptr && q_bytes >= kHostPiecesMinBytes &&
            cudaPointerGetAttributes(&attr, q_host) == cudaSuccess && attr.type == cudaMemoryTypeHost &&
            attr.devicePointer != nullptr) {
            q_unique = static_cast<const uint16_t*>(attr.devicePointer);
            copy_on_side = true;
        }
        (void)cudaGetLastError();
#endif
        if (!copy_on_side)
            MOSKA_CUDA_TRY(cudaMemcpyAsync(const_cast<uint16_t*>(q), q_host, q_bytes, cudaMemcpyHostToDevice, st));
    }
    // the tensor-core kernel over whichever shared store the step has
    auto shared_tc = [&](bool dense_mode, int max_ctas, cudaStream_t s_) {
        if (f8 != nullptr)
            return launch_shared_tc_fp8(q, f8->k8, f8->v8, f8->k_scale, f8->v_scale,
                                        dense_mode ? nullptr : seg_entries, o_part, lse_part, softmax_scale,
                                        shape, ws, dense_mode, max_ctas, s_);
        return launch_shared_tc(q, k_shared, v_shared, dense_mode ? nullptr : seg_entries, o_part, lse_part,
                                softmax_scale, shape, ws, dense_mode, max_ctas, s_);
    };
    if (side == nullptr) {
        // one stream: route, group, unique, shared, merge
        if (!dense) {
            MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_ROUTE, 0, st));
            // the router also sets the grouping's request bits while it writes its picks
            MOSKA_TRY(route_impl(q, summaries, topk_idx, nullptr, shape, ws, ws_bytes, true, st));
            MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_ROUTE, 1, st));
            MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_GROUP, 0, st));
            MOSKA_TRY(group_impl(topk_idx, seg_offsets, seg_entries, shape, ws, ws_bytes, true, st));
            MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_GROUP, 1, st));
        }
        MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_UNIQUE, 0, st));
        MOSKA_TRY(unique_impl(q, kv, kv_start, kv_len, o_part, lse_part, softmax_scale, shape, st));
        MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_UNIQUE, 1, st));
        MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_SHARED, 0, st));
        if (f8 != nullptr)
            MOSKA_TRY(moska_shared_attn_fp8(q, f8->k8, f8->v8, f8->k_scale, f8->v_scale,
                                            dense ? nullptr : topk_idx, dense ? nullptr : seg_offsets,
                                            dense ? nullptr : seg_entries, o_part, lse_part, softmax_scale,
                                            shape, ws, ws_bytes, st));
        else
            MOSKA_TRY(moska_shared_attn(q, k_shared, v_shared, dense ? nullptr : topk_idx,
                                        dense ? nullptr : seg_offsets, dense ? nullptr : seg_entries,
                                        o_part, lse_part, softmax_scale, shape, ws, ws_bytes, st));
        MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_SHARED, 1, st));
    } else {
        // Two streams.  Unique attention (HBM-bound, thousands of short-lived CTAs) is enqueued
        // first on `stream`; everything else follows on the higher-priority side stream and takes
        // SMs over as unique-attention CTAs retire: the short routing and grouping kernels, the
        // streaming shared-attention tiles, and the persistent tensor-core kernel, which gets
        // only a share of the SMs so that unique attention keeps the others and HBM stays busy
        // while the tensor pipe works -- the single-GPU form of the paper's split into Shared-KV
        // and Unique-KV nodes (Section III-C).
        cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
        MOSKA_TRY(fork_join_events(&ev_fork, &ev_join));
        MOSKA_TRY(check_shape(shape, !dense));
        if (f8 != nullptr) {
            if (!shared_tc_supported(shape))
                return fail(MOSKA_ERR_UNSUPPORTED, "the FP8 shared store is built for D = 128");
            REQUIRE_PTR(f8->k8, 128);
            REQUIRE_PTR(f8->v8, 128);
            REQUIRE_PTR(f8->k_scale, 4);
            REQUIRE_PTR(f8->v_scale, 4);
            // (dense mode too: the workspace holds the f16 copy of the queries)
            if (ws == nullptr || !aligned(ws, 256) || ws_bytes < ws_layout(shape).total)
                return fail(MOSKA_ERR_WORKSPACE, "workspace missing, misaligned or smaller than %zu bytes",
                            ws_layout(shape).total);
        } else {
            REQUIRE_PTR(k_shared, 128);
            REQUIRE_PTR(v_shared, 128);
        }
        REQUIRE_PTR(o_part, 32);
        REQUIRE_PTR(lse_part, 4);
        if (dense && shape->shared_slots > shape->C)
            return fail(MOSKA_ERR_INVALID_ARG, "dense mode needs shared_slots <= C");
        if (!dense && shape->shared_slots != shape->k)
            return fail(MOSKA_ERR_INVALID_ARG, "routed mode needs shared_slots == k");
        MOSKA_CUDA_TRY(cudaEventRecord(ev_fork, st));
        MOSKA_CUDA_TRY(cudaStreamWaitEvent(side, ev_fork, 0));
        if (copy_on_side)
            MOSKA_CUDA_TRY(cudaMemcpyAsync(const_cast<uint16_t*>(q), q_host, q_bytes, cudaMemcpyHostToDevice, side));
        MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_UNIQUE, 0, st));
        MOSKA_TRY(unique_impl(q_unique, kv, kv_start, kv_len, o_part, lse_part, softmax_scale, shape, st));
        MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_UNIQUE, 1, st));
        if (!dense) {
            MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_ROUTE, 0, side));
            MOSKA_TRY(route_impl(q, summaries, topk_idx, nullptr, shape, ws, ws_bytes, true, side));
            MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_ROUTE, 1, side));
            MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_GROUP, 0, side));
            MOSKA_TRY(group_impl(topk_idx, seg_offsets, seg_entries, shape, ws, ws_bytes, true, side));
            MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_GROUP, 1, side));
        }
        MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_SHARED, 0, side));
        // (with the FP8 store the tensor-core kernel takes dense batches of any size)
        const bool tc = shared_tc_supported(shape) &&
                        (!dense || f8 != nullptr ||
                         (long long)shape->B * (shape->Hq / shape->Hkv) >= kDenseTcMinRows);
        // Sharing the SMs pays when unique attention runs long enough for the tensor-core kernel
        // to start beside it (the routing chain in front of it takes a few hundred microseconds
        // under contention); for a short unique attention the tensor-core items run after it, on
        // all SMs.
        const double unique_ms = (double)shape->unique_tokens * shape->Hkv *
                                 (kv.fp8 ? 2.0 * shape->D + 8.0 : 4.0 * shape->D) / 7.0e9;
        const bool beside = tc && (dense || unique_ms >= MOSKA_BESIDE_MS);
        if (tc && beside) MOSKA_TRY(shared_tc(dense, tc_sm_share(shape, dense, unique_ms), side));
        // the streaming tiles (every tile of a shape the tensor-core kernel does not serve, else the
        // 8-row tiles of routed mode) always run beside unique attention
        if (f8 != nullptr) {
            if (!dense)
                MOSKA_TRY(launch_shared_small_fp8(q, f8->k8, f8->v8, f8->k_scale, f8->v_scale, seg_entries,
                                                  o_part, lse_part, softmax_scale, shape, ws, side));
        } else if (!tc || !dense)
            MOSKA_TRY(launch_shared_small(q, k_shared, v_shared, dense ? nullptr : seg_entries, o_part,
                                          lse_part, softmax_scale, shape, ws, dense, tc, side));
        if (beside || !tc) MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_SHARED, 1, side));
        MOSKA_CUDA_TRY(cudaEventRecord(ev_join, side));
        MOSKA_CUDA_TRY(cudaStreamWaitEvent(st, ev_join, 0));
        if (tc && !beside) {
            MOSKA_TRY(shared_tc(false, 0, st));
            MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_SHARED, 1, st));
        }
    }
    MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_MERGE, 0, st));
    const long long rows = (long long)shape->B * shape->Hq;
    const size_t out_bytes = sizeof(uint16_t) * (size_t)rows * shape->D;
    if (out_host != nullptr && side != nullptr && out_bytes >= kHostPiecesMinBytes) {
        // result wanted in host memory: merge the rows in pieces on `stream` and copy every piece
        // on the side stream (idle by now) while the next one is merged
        REQUIRE_PTR(o_part, 16);
        REQUIRE_PTR(lse_part, 4);
        REQUIRE_PTR(out, 8);
        cudaEvent_t ev_piece = nullptr, ev_done = nullptr;
        MOSKA_TRY(fork_join_events(&ev_piece, &ev_done));
        const long long per = ((rows + kHostPieces - 1) / kHostPieces + 7) / 8 * 8;
        for (long long r0 = 0; r0 < rows; r0 += per) {
            const long long n = rows - r0 < per ? rows - r0 : per;
            MOSKA_TRY(launch_merge_rows(o_part, lse_part, out, nullptr, lse_out, shape, r0, n, st));
            MOSKA_CUDA_TRY(cudaEventRecord(ev_piece, st));
            MOSKA_CUDA_TRY(cudaStreamWaitEvent(side, ev_piece, 0));
            MOSKA_CUDA_TRY(cudaMemcpyAsync(out_host + r0 * shape->D, out + r0 * shape->D,
                                           sizeof(uint16_t) * (size_t)n * shape->D,
                                           cudaMemcpyDeviceToHost, side));
        }
        MOSKA_CUDA_TRY(cudaEventRecord(ev_done, side));
        MOSKA_CUDA_TRY(cudaStreamWaitEvent(st, ev_done, 0));
    } else {
        MOSKA_TRY(moska_merge(o_part, lse_part, out, nullptr, lse_out, shape, st));
        if (out_host != nullptr)
            MOSKA_CUDA_TRY(cudaMemcpyAsync(out_host, out, out_bytes, cudaMemcpyDeviceToHost, st));
    }
    MOSKA_CUDA_TRY(prof_mark(prof, MOSKA_STAGE_MERGE, 1, st));
    if (prof != nullptr && prof->n_steps < prof->max_steps) ++prof->n_steps;
    return MOSKA_OK;
}
}  // namespace

int moska_decode_step(const uint16_t* q, const float* summaries, const uint16_t* k_shared,
                      const uint16_t* v_shared, const uint16_t* k_unique,
                      const uint16_t* v_unique, const int64_t* kv_start, const int32_t* kv_len,
                      int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                      float* o_part, float* lse_part, uint16_t* out, float* lse_out,
                      float softmax_scale, const moska_shape* shape, void* ws, size_t ws_bytes,
                      moska_stream stream, moska_stream side_stream, moska_profiler* prof)
{
    MOSKA_API_RANGE();
    UniqueKv kv;
    kv.k = k_unique;
    kv.v = v_unique;
    return decode_step_impl(q, summaries, k_shared, v_shared, nullptr, kv, kv_start, kv_len, topk_idx,
                            seg_offsets, seg_entries, o_part, lse_part, out, lse_out, softmax_scale,
                            shape, ws, ws_bytes, stream, side_stream, prof);
}

int moska_decode_step_fp8shared(const uint16_t* q, const float* summaries, const uint8_t* k8_shared,
                                const uint8_t* v8_shared, const float* k_scale_shared,
                                const float* v_scale_shared, const uint16_t* k_unique,
                                const uint16_t* v_unique, const int64_t* kv_start, const int32_t* kv_len,
                                int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                                float* o_part, float* lse_part, uint16_t* out, float* lse_out,
                                float softmax_scale, const moska_shape* shape, void* ws, size_t ws_bytes,
                                moska_stream stream, moska_stream side_stream, moska_profiler* prof)
{
    MOSKA_API_RANGE();
    UniqueKv kv;
    kv.k = k_unique;
    kv.v = v_unique;
    SharedF8 f8;
    f8.k8 = k8_shared;
    f8.v8 = v8_shared;
    f8.k_scale = k_scale_shared;
    f8.v_scale = v_scale_shared;
    return decode_step_impl(q, summaries, nullptr, nullptr, &f8, kv, kv_start, kv_len, topk_idx, seg_offsets,
                            seg_entries, o_part, lse_part, out, lse_out, softmax_scale, shape, ws, ws_bytes,
                            stream, side_stream, prof);
}

int moska_decode_step_fp8(const uint16_t* q, const float* summaries, const uint8_t* k8_shared,
                          const uint8_t* v8_shared, const float* k_scale_shared, const float* v_scale_shared,
                          const uint8_t* k8_unique, const uint8_t* v8_unique, const float* k_scale_unique,
                          const float* v_scale_unique, const int64_t* kv_start, const int32_t* kv_len,
                          int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries, float* o_part,
                          float* lse_part, uint16_t* out, float* lse_out, float softmax_scale,
                          const moska_shape* shape, void* ws, size_t ws_bytes, moska_stream stream,
                          moska_stream side_stream, moska_profiler* prof)
{
    MOSKA_API_RANGE();
    UniqueKv kv;
    kv.k8 = k8_unique;
    kv.v8 = v8_unique;
    kv.k_scale = k_scale_unique;
    kv.v_scale = v_scale_unique;
    kv.fp8 = true;
    SharedF8 f8;
    f8.k8 = k8_shared;
    f8.v8 = v8_shared;
    f8.k_scale = k_scale_shared;
    f8.v_scale = v_scale_shared;
    return decode_step_impl(q, summaries, nullptr, nullptr, &f8, kv, kv_start, kv_len, topk_idx, seg_offsets,
                            seg_entries, o_part, lse_part, out, lse_out, softmax_scale, shape, ws, ws_bytes,
                            stream, side_stream, prof);
}

int moska_decode_step_fp8kv(const uint16_t* q, const float* summaries, const uint16_t* k_shared,
                            const uint16_t* v_shared, const uint8_t* k8_unique,
                            const uint8_t* v8_unique, const float* k_scale, const float* v_scale,
                            const int64_t* kv_start, const int32_t* kv_len, int32_t* topk_idx,
                            int32_t* seg_offsets, int32_t* seg_entries, float* o_part,
                            float* lse_part, uint16_t* out, float* lse_out, float softmax_scale,
                            const moska_shape* shape, void* ws, size_t ws_bytes, moska_stream stream,
                            moska_stream side_stream, moska_profiler* prof)
{
    MOSKA_API_RANGE();
    UniqueKv kv;
    kv.k8 = k8_unique;
    kv.v8 = v8_unique;
    kv.k_scale = k_scale;
    kv.v_scale = v_scale;
    kv.fp8 = true;
    return decode_step_impl(q, summaries, k_shared, v_shared, nullptr, kv, kv_start, kv_len, topk_idx,
                            seg_offsets, seg_entries, o_part, lse_part, out, lse_out, softmax_scale,
                            shape, ws, ws_bytes, stream, side_stream, prof);
}

int moska_profiler_create(moska_profiler** out, int32_t max_steps)
{
    if (out == nullptr || max_steps < 1) return fail(MOSKA_ERR_INVALID_ARG, "profiler arguments");
    moska_profiler* p = new moska_profiler();
    p->max_steps = max_steps;
    const int n = max_steps * MOSKA_N_STAGES;
    p->ev = new cudaEvent_t[2 * n];
    p->used = new bool[n]();
    for (int i = 0; i < 2 * n; ++i) {
        cudaError_t e = cudaEventCreate(&p->ev[i]);
        if (e != cudaSuccess) {
            for (int j = 0; j < i; ++j) cudaEventDestroy(p->ev[j]);
            delete[] p->ev;
            delete[] p->used;
            delete p;
            return fail(MOSKA_ERR_CUDA, "cudaEventCreate failed: %s", cudaGetErrorString(e));
        }
    }
    *out = p;
    return MOSKA_OK;
}

void moska_profiler_destroy(moska_profiler* p)
{
    if (p == nullptr) return;
    for (int i = 0; i < 2 * p->max_steps * MOSKA_N_STAGES; ++i) cudaEventDestroy(p->ev[i]);
    delete[] p->ev;
    delete[] p->used;
    delete p;
}

int moska_profiler_select(moska_profiler* p, uint32_t stage_mask)
{
    if (p == nullptr) return fail(MOSKA_ERR_INVALID_ARG, "profiler is NULL");
    p->mask = stage_mask;
    return MOSKA_OK;
}

int moska_profiler_read(moska_profiler* p, float* stage_ms, int32_t* n_steps)
{
    if (p == nullptr || stage_ms == nullptr || n_steps == nullptr)
        return fail(MOSKA_ERR_INVALID_ARG, "profiler arguments");
    for (int s = 0; s < MOSKA_N_STAGES; ++s) stage_ms[s] = 0.f;
    for (int i = 0; i < p->n_steps * MOSKA_N_STAGES; ++i) {
        if (!p->used[i]) continue;
        MOSKA_CUDA_TRY(cudaEventSynchronize(p->ev[2 * i + 1]));
        float ms = 0.f;
        MOSKA_CUDA_TRY(cudaEventElapsedTime(&ms, p->ev[2 * i], p->ev[2 * i + 1]));
        stage_ms[i % MOSKA_N_STAGES] += ms;
        p->used[i] = false;
    }
    *n_steps = p->n_steps;
    p->n_steps = 0;
    return MOSKA_OK;
}

int moska_decode_step_host(const uint16_t* q_host, uint16_t* q_dev, const float* summaries,
                           const uint16_t* k_shared, const uint16_t* v_shared,
                           const uint16_t* k_unique, const uint16_t* v_unique,
                           const int64_t* kv_start, const int32_t* kv_len, int32_t* topk_idx,
                           int32_t* seg_offsets, int32_t* seg_entries, float* o_part,
                           float* lse_part, uint16_t* out_dev, uint16_t* out_host,
                           float softmax_scale, const moska_shape* shape, void* ws,
                           size_t ws_bytes, moska_stream stream, moska_stream side_stream,
                           moska_profiler* prof)
{
    MOSKA_API_RANGE();
    MOSKA_TRY(check_shape(shape, summaries != nullptr));
    if (q_host == nullptr || q_dev == nullptr || out_dev == nullptr || out_host == nullptr)
        return fail(MOSKA_ERR_INVALID_ARG, "q_host, q_dev, out_dev and out_host must not be NULL");
    if (!aligned(q_host, 16))
        return fail(MOSKA_ERR_INVALID_ARG, "q_host is not 16-byte aligned");
    cudaStream_t st = (cudaStream_t)stream;
    UniqueKv kv;
    kv.k = k_unique;
    kv.v = v_unique;
    MOSKA_TRY(decode_step_impl(q_dev, summaries, k_shared, v_shared, nullptr, kv, kv_start, kv_len,
                               topk_idx, seg_offsets, seg_entries, o_part, lse_part, out_dev, nullptr,
                               softmax_scale, shape, ws, ws_bytes, stream, side_stream, prof, out_host,
                               q_host));
    MOSKA_CUDA_TRY(cudaStreamSynchronize(st));
    return MOSKA_OK;
}

int moska_decode_step_fp8_host(const uint16_t* q_host, uint16_t* q_dev, const float* summaries,
                               const uint8_t* k8_shared, const uint8_t* v8_shared,
                               const float* k_scale_shared, const float* v_scale_shared,
                               const uint8_t* k8_unique, const uint8_t* v8_unique,
                               const float* k_scale_unique, const float* v_scale_unique,
                               const int64_t* kv_start, const int32_t* kv_len, int32_t* topk_idx,
                               int32_t* seg_offsets, int32_t* seg_entries, float* o_part, float* lse_part,
                               uint16_t* out_dev, uint16_t* out_host, float softmax_scale,
                               const moska_shape* shape, void* ws, size_t ws_bytes, moska_stream stream,
                               moska_stream side_stream, moska_profiler* prof)
{
    MOSKA_API_RANGE();
    MOSKA_TRY(check_shape(shape, true));
    if (q_host == nullptr || q_dev == nullptr || out_dev == nullptr || out_host == nullptr)
        return fail(MOSKA_ERR_INVALID_ARG, "q_host, q_dev, out_dev and out_host must not be NULL");
    if (!aligned(q_host, 16))
        return fail(MOSKA_ERR_INVALID_ARG, "q_host is not 16-byte aligned");
    UniqueKv kv;
    kv.k8 = k8_unique;
    kv.v8 = v8_unique;
    kv.k_scale = k_scale_unique;
    kv.v_scale = v_scale_unique;
    kv.fp8 = true;
    SharedF8 f8;
    f8.k8 = k8_shared;
    f8.v8 = v8_shared;
    f8.k_scale = k_scale_shared;
    f8.v_scale = v_scale_shared;
    MOSKA_TRY(decode_step_impl(q_dev, summaries, nullptr, nullptr, &f8, kv, kv_start, kv_len, topk_idx,
                               seg_offsets, seg_entries, o_part, lse_part, out_dev, nullptr, softmax_scale,
                               shape, ws, ws_bytes, stream, side_stream, prof, out_host, q_host));
    MOSKA_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return MOSKA_OK;
}

}  // extern "C"
