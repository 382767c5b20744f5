// Shared host/device helpers of the MoSKA CUDA library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdarg>
#include <cstdio>

#include "moska.h"

namespace moska {

// ---- error reporting -------------------------------------------------------------------------
char* last_error_buffer();  // thread-local, 512 bytes
int fail(int status, const char* fmt, ...);

#define MOSKA_CUDA_TRY(expr)                                                              \
    do {                                                                                  \
        cudaError_t err__ = (expr);                                                       \
        if (err__ != cudaSuccess)                                                         \
            return ::moska::fail(MOSKA_ERR_CUDA, "%s failed: %s", #expr,                  \
                                 cudaGetErrorString(err__));                              \
    } while (0)

#define MOSKA_LAUNCH_CHECK(name)                                                          \
    do {                                                                                  \
        cudaError_t err__ = cudaGetLastError();                                           \
        if (err__ != cudaSuccess)                                                         \
            return ::moska::fail(MOSKA_ERR_CUDA, "launch of %s failed: %s", name,         \
                                 cudaGetErrorString(err__));                              \
    } while (0)

#define MOSKA_TRY_STATUS(expr)                 \
    do {                                       \
        int st__ = (expr);                     \
        if (st__ != MOSKA_OK) return st__;     \
    } while (0)

// Validates the shape fields every entry point relies on; returns MOSKA_OK or a negative status.
int check_shape(const moska_shape* s, bool needs_k);
// MOSKA_OK if the current device is compute capability 10.x.
int check_device();

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// ---- workspace layout (route / group / shared attention) ---------------------------------------
// One work item of shared attention: `n_entries` consecutive entries of segment `key`,
// starting at seg_entries[entry_begin].
struct TileItem {
    int32_t key;          // h * C + c
    int32_t entry_begin;  // absolute index into seg_entries
    int32_t n_entries;    // requests in this tile (rows = n_entries * G)
    int32_t pad;
};

struct WsHeader {
    int32_t n_small_tiles;  // items in the second list: single-tile items (tensor-core shapes) or 16-row tiles
    int32_t n_big_tiles;    // items of two 128-row query tiles
    int32_t reserved;
    int32_t n_tiny_tiles;   // items in the 8-row tile list
    int32_t pad[60];
};
static_assert(sizeof(WsHeader) == 256, "header is one 256-byte block");

// A build with -DMOSKA_DEBUG_GUARDS leaves 256 guard bytes behind every region of the workspace,
// writes a pattern into them (and into the region's alignment padding) before the grouping passes
// and checks it after them; the work-list writes are also checked against the lists' capacity.
#ifdef MOSKA_DEBUG_GUARDS
constexpr size_t kGuardBytes = 256;
#else
constexpr size_t kGuardBytes = 0;
#endif
constexpr int kWsRegions = 7;  // bit sets, totals, three work lists, router scores, f16 queries

struct WsLayout {
    int32_t words;            // 32-bit words of one key's request bit set
    int32_t n_keys;           // Hkv * C
    int32_t small_entries;    // requests per small (16-row) tile
    int32_t tiny_entries;     // requests per 8-row tile
    int32_t big_entries;      // requests per big tile
    int32_t tc;               // 1: the tensor-core kernel serves this shape (two-tile + single-tile items)
    int64_t max_small, max_big;
    size_t off_hist, off_totals, off_small, off_big, off_tiny;
    size_t group_total;  // end of what the grouping passes and shared attention use
    size_t off_scores;   // router: fp32 scores [B * Hkv][C] (only when C > kRouteSmallC)
    size_t off_q16;      // FP8 shared store: the step's queries as f16 [B][Hq][D] (tensor-core shapes)
    size_t total;
    // debug build: guard words fill [guard_begin[r], guard_end[r]) behind region r's payload
    size_t guard_begin[kWsRegions], guard_end[kWsRegions];
};
WsLayout ws_layout(const moska_shape* s);
// Debug build (MOSKA_DEBUG_GUARDS): writes the guard words behind every workspace region
// (check = false) or compares them and raises MOSKA_ERR_CORRUPT in the device status word
// (check = true).  Other builds: does nothing.
// `ws_extent`: bytes of `ws` that exist (guard words beyond them are left alone).
int launch_ws_guards(void* ws, const WsLayout& lay, bool check, cudaStream_t st, size_t ws_extent);

constexpr int kRouteSmallC = 256;   // up to this many chunks the router keeps its scores in shared memory
constexpr int kSmallTileRows = 16;  // query rows of one small tile (two 8-row MMA column blocks)
constexpr int kBigTileRows = 128;   // query rows of one tensor-core (tcgen05) tile; a work item has one or two
constexpr int kDenseTcMinRows = 16; // dense mode: batches with fewer query rows per KV head take the streaming tiles

// ---- internal launchers (one per .cu file) -----------------------------------------------------
int launch_summaries(const uint16_t* k_shared, float* summaries, const moska_shape* s,
                     cudaStream_t st);
int launch_summaries_attn(const uint16_t* k_shared, float* summaries, float probe_scale,
                          const moska_shape* s, cudaStream_t st);
int launch_route(const uint16_t* q, const float* summaries, int32_t* topk_idx, float* topk_score,
                 const moska_shape* s, void* ws, bool mark_groups, cudaStream_t st);
int launch_group(const int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                 const moska_shape* s, void* ws, bool premarked, cudaStream_t st,
                 bool grouping_regions_only = false);
int launch_group_noalloc(const int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                         const moska_shape* s, cudaStream_t st);
int launch_shared_small(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                        const int32_t* seg_entries, float* o_part, float* lse_part, float scale,
                        const moska_shape* s, void* ws, bool dense, bool tiny_list_only, cudaStream_t st);
// Tensor-core (tcgen05) Shared KV Attention over the big-tile work list (routed) or over
// (KV head, run of chunks, 256 / G requests) items (dense).
bool shared_tc_supported(const moska_shape* s);
int launch_shared_tc(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                     const int32_t* seg_entries, float* o_part, float* lse_part, float scale,
                     const moska_shape* s, void* ws, bool dense, int max_ctas, cudaStream_t st);
// The same over a shared store of FP8 (E4M3) codes with one scale per (KV head, chunk); routed mode.
int launch_shared_tc_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8, const float* k_scale,
                         const float* v_scale, const int32_t* seg_entries, float* o_part, float* lse_part,
                         float scale, const moska_shape* s, void* ws, bool dense, int max_ctas, cudaStream_t st);
// Estimated SM-milliseconds of the tensor-core kernel for this shape (host, pure).
double shared_tc_cost_sm_ms(const moska_shape* s, bool dense);
// Device address (on the current device) of the library's sticky status word: kernels lower it
// with atomicMin to a negative moska_status when they detect a problem while running.
int status_word(int** out);
// Synchronises the device, returns the sticky status word and clears it.
int read_status(int* out);
int launch_unique(const uint16_t* q, const uint16_t* k_unique, const uint16_t* v_unique,
                  const int64_t* kv_start, const int32_t* kv_len, float* o_part, float* lse_part,
                  float scale, const moska_shape* s, cudaStream_t st);
// FP8 shared store: the grouping pass's 8-row tiles on the streaming block (routed mode)
int launch_shared_small_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8, const float* k_scale,
                            const float* v_scale, const int32_t* seg_entries, float* o_part,
                            float* lse_part, float scale, const moska_shape* s, void* ws, cudaStream_t st);
int launch_unique_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8, const float* k_scale,
                      const float* v_scale, const int64_t* kv_start, const int32_t* kv_len,
                      float* o_part, float* lse_part, float scale, const moska_shape* s,
                      cudaStream_t st);
int launch_gemv_baseline(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                         const int32_t* topk_idx, float* o_part, float* lse_part, float scale,
                         const moska_shape* s, cudaStream_t st);
int launch_merge(const float* o_part, const float* lse_part, uint16_t* out, float* out_f32,
                 float* lse_out, const moska_shape* s, cudaStream_t st);
int launch_merge_rows(const float* o_part, const float* lse_part, uint16_t* out, float* out_f32,
                      float* lse_out, const moska_shape* s, long long row0, long long rows,
                      cudaStream_t st);

}  // namespace moska
