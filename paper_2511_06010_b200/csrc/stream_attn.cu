// Kernels built on the streaming decode-attention block: Unique KV Attention, the unbatched
// per-request GEMV baseline over shared chunks, and Shared KV Attention for small query tiles.
#include <cstddef>
#include <type_traits>

#include "common.cuh"
#include "stream_attn.cuh"

namespace moska {
using namespace stream;

namespace {

template <int NT>
__device__ __forceinline__ void clear_rows(TileRows<NT>& rows)
{
    for (int i = threadIdx.x; i < NT * 8; i += kThreads) {
        rows.q[i] = nullptr;
        rows.o[i] = nullptr;
        rows.lse[i] = nullptr;
    }
}

// Token range of split `s` of a request with `len` unique tokens: equal parts rounded up to a
// whole number of CTA passes (kWarps * 16 tokens), so trailing splits of short requests are empty.
__device__ __forceinline__ void split_range(int len, int n_splits, int s, int& t0, int& t1)
{
    constexpr int kQuantum = kWarps * kTileTokens;
    int per = (len + n_splits - 1) / n_splits;
    per = (per + kQuantum - 1) / kQuantum * kQuantum;
    t0 = min(len, s * per);
    t1 = min(len, t0 + per);
}

// ---- Unique KV Attention (Section III-A): one CTA per (request, KV head, split) ----------------
template <int D>
__global__ void __launch_bounds__(kThreads, 3)
unique_attn_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_unique,
                   const uint16_t* __restrict__ v_unique, const int64_t* __restrict__ kv_start,
                   const int32_t* __restrict__ kv_len, float* __restrict__ o_part,
                   float* __restrict__ lse_part, float scale, int Hq, int Hkv, int n_splits,
                   int slot0, int n_slots)
{
    __shared__ TileRows<1> rows;
    __shared__ CombineSmem<D, 1> sm;
    const int G = Hq / Hkv;
    // KV heads of the same (request, split) sit in neighbouring CTAs: together they read whole
    // token rows of the [T][Hkv][D] store.
    const int h = blockIdx.x % Hkv;
    const int s = (blockIdx.x / Hkv) % n_splits;
    const int b = blockIdx.x / (Hkv * n_splits);
    clear_rows(rows);
    __syncthreads();
    if (threadIdx.x < G) {
        const int64_t r = (int64_t)b * Hq + h * G + threadIdx.x;
        rows.q[threadIdx.x] = q + r * D;
        rows.o[threadIdx.x] = o_part + (r * n_slots + slot0 + s) * D;
        rows.lse[threadIdx.x] = lse_part + r * n_slots + slot0 + s;
    }
    __syncthreads();
    int t0, t1;
    split_range(kv_len[b], n_splits, s, t0, t1);
    const int64_t stride = (int64_t)Hkv * D;
    const uint16_t* kb = k_unique + kv_start[b] * stride + (int64_t)h * D;
    const uint16_t* vb = v_unique + kv_start[b] * stride + (int64_t)h * D;
    attend_stream<D, 1>(rows, kb, vb, stride, t0, t1, scale, sm);
}

// ---- Unique KV Attention with K/V staged through shared memory (D = 128) -------------------------
__global__ void __launch_bounds__(kThreads, 2)
unique_staged_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_unique,
                     const uint16_t* __restrict__ v_unique, const int64_t* __restrict__ kv_start,
                     const int32_t* __restrict__ kv_len, float* __restrict__ o_part,
                     float* __restrict__ lse_part, float scale, int Hq, int Hkv, int n_splits,
                     int slot0, int n_slots)
{
    constexpr int D = 128;
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ TileRows<1> rows;
    const int G = Hq / Hkv;
    const int h = blockIdx.x % Hkv;
    const int s = (blockIdx.x / Hkv) % n_splits;
    const int b = blockIdx.x / (Hkv * n_splits);
    clear_rows(rows);
    __syncthreads();
    if (threadIdx.x < G) {
        const int64_t r = (int64_t)b * Hq + h * G + threadIdx.x;
        rows.q[threadIdx.x] = q + r * D;
        rows.o[threadIdx.x] = o_part + (r * n_slots + slot0 + s) * D;
        rows.lse[threadIdx.x] = lse_part + r * n_slots + slot0 + s;
    }
    __syncthreads();
    int t0, t1;
    split_range(kv_len[b], n_splits, s, t0, t1);
    const int64_t stride = (int64_t)Hkv * D;
    const uint16_t* kb = k_unique + kv_start[b] * stride + (int64_t)h * D;
    const uint16_t* vb = v_unique + kv_start[b] * stride + (int64_t)h * D;
    attend_stream_staged<1>(rows, kb, vb, stride, t0, t1, scale, ring);
}

// ---- Unique KV Attention for several query tokens per request (D = 128) -------------------------
// The q_len query tokens of request r are the batch rows r * q_len + i; token i sees the first
// kv_len[r] - (q_len - 1 - i) tokens of the request's context.  Their q_len * G query rows of one
// KV head share one pass over the request's K/V (one CTA per (request, KV head, split)).
template <int NT>
__global__ void __launch_bounds__(kThreads, 2)
unique_multi_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_unique,
                    const uint16_t* __restrict__ v_unique, const int64_t* __restrict__ kv_start,
                    const int32_t* __restrict__ kv_len, float* __restrict__ o_part,
                    float* __restrict__ lse_part, float scale, int Hq, int Hkv, int n_splits,
                    int slot0, int n_slots, int q_len)
{
    constexpr int D = 128;
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ TileRows<NT> rows;
    __shared__ int row_last[NT * 8];
    const int G = Hq / Hkv;
    const int h = blockIdx.x % Hkv;
    const int s = (blockIdx.x / Hkv) % n_splits;
    const int r = blockIdx.x / (Hkv * n_splits);
    const int len = kv_len[r];
    clear_rows(rows);
    if (threadIdx.x < NT * 8) row_last[threadIdx.x] = 0x7fffffff;
    __syncthreads();
    if (threadIdx.x < q_len * G) {
        const int i = threadIdx.x / G, g = threadIdx.x % G;
        const int64_t row = ((int64_t)r * q_len + i) * Hq + h * G + g;
        rows.q[threadIdx.x] = q + row * D;
        rows.o[threadIdx.x] = o_part + (row * n_slots + slot0 + s) * D;
        rows.lse[threadIdx.x] = lse_part + row * n_slots + slot0 + s;
        row_last[threadIdx.x] = len - 1 - (q_len - 1 - i);
    }
    __syncthreads();
    int t0, t1;
    split_range(len, n_splits, s, t0, t1);
    const int64_t stride = (int64_t)Hkv * D;
    const uint16_t* kb = k_unique + kv_start[r] * stride + (int64_t)h * D;
    const uint16_t* vb = v_unique + kv_start[r] * stride + (int64_t)h * D;
    attend_stream_staged<NT, true>(rows, kb, vb, stride, t0, t1, scale, ring, row_last);
}

// ---- per-request GEMV baseline over shared chunks: one CTA per (request, KV head, slot) ---------
template <int D>
__global__ void __launch_bounds__(kThreads, D == 128 ? 2 : 3)
gemv_baseline_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_shared,
                     const uint16_t* __restrict__ v_shared, const int32_t* __restrict__ topk_idx,
                     float* __restrict__ o_part, float* __restrict__ lse_part, float scale,
                     int Hq, int Hkv, int C, int L, int k, int shared_slots, int n_slots)
{
    // same streaming block as unique attention: staged through shared memory for D = 128
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ TileRows<1> rows;
    __shared__ typename std::conditional<D == 128, int, CombineSmem<D, 1>>::type sm;
    const int G = Hq / Hkv;
    const int j = blockIdx.x % shared_slots;
    const int h = (blockIdx.x / shared_slots) % Hkv;
    const int b = blockIdx.x / (shared_slots * Hkv);
    clear_rows(rows);
    __syncthreads();
    if (threadIdx.x < G) {
        const int64_t r = (int64_t)b * Hq + h * G + threadIdx.x;
        rows.q[threadIdx.x] = q + r * D;
        rows.o[threadIdx.x] = o_part + (r * n_slots + j) * D;
        rows.lse[threadIdx.x] = lse_part + r * n_slots + j;
    }
    __syncthreads();
    int64_t tok0;
    int n_tok;
    if (topk_idx != nullptr) {  // routed: slot j is chunk topk_idx[b][h][j]
        tok0 = ((int64_t)h * C + topk_idx[((int64_t)b * Hkv + h) * k + j]) * L;
        n_tok = L;
    } else {                    // dense: slot j is the j-th run of consecutive chunks
        const int run = (C + shared_slots - 1) / shared_slots;
        const int c0 = min(C, j * run), c1 = min(C, c0 + run);
        tok0 = ((int64_t)h * C + c0) * L;
        n_tok = (c1 - c0) * L;
    }
    if constexpr (D == 128)
        attend_stream_staged<1>(rows, k_shared + tok0 * D, v_shared + tok0 * D, D, 0, n_tok, scale, ring);
    else
        attend_stream<D, 1>(rows, k_shared + tok0 * D, v_shared + tok0 * D, D, 0, n_tok, scale, sm);
}

// ---- Shared KV Attention, small tiles (Section III-A) ------------------------------------------
// Routed mode: one CTA per work item = up to 16/G requests of one (KV head, chunk) segment; the
// chunk's K/V is streamed once for all of them.  Dense mode: one CTA per (KV head, run of chunks,
// group of 16/G requests).
template <int D, int NT>
__global__ void __launch_bounds__(kThreads, (NT == 1 && D != 128) ? 3 : 2)
shared_small_kernel(const uint16_t* __restrict__ q, const uint16_t* __restrict__ k_shared,
                    const uint16_t* __restrict__ v_shared, const int32_t* __restrict__ seg_entries,
                    const WsHeader* __restrict__ hdr, const TileItem* __restrict__ items,
                    float* __restrict__ o_part, float* __restrict__ lse_part, float scale, int B,
                    int Hq, int Hkv, int C, int L, int k, int shared_slots, int n_slots, int dense,
                    int n_tiles_offset)
{
    // D = 128: K/V staged through a shared-memory ring (the combine step reuses it); D = 64: the
    // register path with its own combine buffers
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ TileRows<NT> rows;
    __shared__ typename std::conditional<D == 128, int, CombineSmem<D, NT>>::type sm;
    const int G = Hq / Hkv;
    const int per_tile = NT * 8 / G;  // requests per tile
    // Routed mode: the CTAs walk the device-side tile list with the grid as their stride (the
    // host only knows an upper bound of its length).  Dense mode: one tile per CTA.
    // which header word counts this list: the 16-row (NT = 2) or the 8-row (NT = 1) tiles
    const int n_tiles = dense ? (int)gridDim.x : reinterpret_cast<const int32_t*>(hdr)[n_tiles_offset];
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        __syncthreads();  // the previous tile's row descriptors and combine buffers are done with
        clear_rows(rows);
        __syncthreads();
        int64_t tok0;
        int n_tok;
        if (!dense) {
            const TileItem it = items[tile];
            const int h = it.key / C;
            if (threadIdx.x < it.n_entries * G) {
                const int p = seg_entries[it.entry_begin + threadIdx.x / G];
                const int g = threadIdx.x % G;
                const int j = p % k, b = p / (k * Hkv);
                const int64_t r = (int64_t)b * Hq + h * G + g;
                rows.q[threadIdx.x] = q + r * D;
                rows.o[threadIdx.x] = o_part + (r * n_slots + j) * D;
                rows.lse[threadIdx.x] = lse_part + r * n_slots + j;
            }
            tok0 = (int64_t)it.key * L;
            n_tok = L;
        } else {
            const int b_tiles = (B + per_tile - 1) / per_tile;
            const int bt = tile % b_tiles;
            const int j = (tile / b_tiles) % shared_slots;
            const int h = tile / (b_tiles * shared_slots);
            const int b = bt * per_tile + threadIdx.x / G;
            if (threadIdx.x < per_tile * G && b < B) {
                const int64_t r = (int64_t)b * Hq + h * G + threadIdx.x % G;
                rows.q[threadIdx.x] = q + r * D;
                rows.o[threadIdx.x] = o_part + (r * n_slots + j) * D;
                rows.lse[threadIdx.x] = lse_part + r * n_slots + j;
            }
            const int run = (C + shared_slots - 1) / shared_slots;
            const int c0 = min(C, j * run), c1 = min(C, c0 + run);
            tok0 = ((int64_t)h * C + c0) * L;
            n_tok = (c1 - c0) * L;
        }
        __syncthreads();
        if constexpr (D == 128)
            attend_stream_staged<NT>(rows, k_shared + tok0 * D, v_shared + tok0 * D, D, 0, n_tok, scale, ring);
        else
            attend_stream<D, NT>(rows, k_shared + tok0 * D, v_shared + tok0 * D, D, 0, n_tok, scale, sm);
    }
}

}  // namespace

int launch_unique(const uint16_t* q, const uint16_t* k_unique, const uint16_t* v_unique,
                  const int64_t* kv_start, const int32_t* kv_len, float* o_part, float* lse_part,
                  float scale, const moska_shape* s, cudaStream_t st)
{
    const int n_slots = s->shared_slots + s->n_unique_splits;
    const long long grid = (long long)s->B * s->Hkv * s->n_unique_splits;
    if (grid == 0) return MOSKA_OK;
    if (grid > 0x7fffffffLL) return fail(MOSKA_ERR_UNSUPPORTED, "unique attention grid too large");
    if (s->q_len > 1) {
        // several query tokens per request: their rows share one pass over the request's K/V
        constexpr int kRing = kWarps * kStagedWarpBytes;
        const int rows = s->q_len * (s->Hq / s->Hkv);
        const unsigned grid_r = (unsigned)(grid / s->q_len);
        if (rows <= 8) {
            MOSKA_CUDA_TRY(cudaFuncSetAttribute(unique_multi_kernel<1>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, kRing));
            unique_multi_kernel<1><<<grid_r, kThreads, kRing, st>>>(
                q, k_unique, v_unique, kv_start, kv_len, o_part, lse_part, scale, s->Hq, s->Hkv,
                s->n_unique_splits, s->shared_slots, n_slots, s->q_len);
        } else {
            MOSKA_CUDA_TRY(cudaFuncSetAttribute(unique_multi_kernel<2>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, kRing));
            unique_multi_kernel<2><<<grid_r, kThreads, kRing, st>>>(
                q, k_unique, v_unique, kv_start, kv_len, o_part, lse_part, scale, s->Hq, s->Hkv,
                s->n_unique_splits, s->shared_slots, n_slots, s->q_len);
        }
        MOSKA_LAUNCH_CHECK("unique_multi_kernel");
        return MOSKA_OK;
    }
    if (s->D == 128) {
        constexpr int kRing = kWarps * kStagedWarpBytes;
        MOSKA_CUDA_TRY(cudaFuncSetAttribute(unique_staged_kernel,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, kRing));
        unique_staged_kernel<<<(unsigned)grid, kThreads, kRing, st>>>(
            q, k_unique, v_unique, kv_start, kv_len, o_part, lse_part, scale, s->Hq, s->Hkv,
            s->n_unique_splits, s->shared_slots, n_slots);
        MOSKA_LAUNCH_CHECK("unique_staged_kernel");
        return MOSKA_OK;
    }
    unique_attn_kernel<64><<<(unsigned)grid, kThreads, 0, st>>>(
        q, k_unique, v_unique, kv_start, kv_len, o_part, lse_part, scale, s->Hq, s->Hkv,
        s->n_unique_splits, s->shared_slots, n_slots);
    MOSKA_LAUNCH_CHECK("unique_attn_kernel");
    return MOSKA_OK;
}

int launch_gemv_baseline(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                         const int32_t* topk_idx, float* o_part, float* lse_part, float scale,
                         const moska_shape* s, cudaStream_t st)
{
    const int n_slots = s->shared_slots + s->n_unique_splits;
    const long long grid = (long long)s->B * s->Hkv * s->shared_slots;
    if (grid == 0) return MOSKA_OK;
    if (grid > 0x7fffffffLL) return fail(MOSKA_ERR_UNSUPPORTED, "baseline grid too large");
    if (s->D == 128) {
        constexpr int kRing = kWarps * kStagedWarpBytes;
        MOSKA_CUDA_TRY(cudaFuncSetAttribute(gemv_baseline_kernel<128>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, kRing));
        gemv_baseline_kernel<128><<<(unsigned)grid, kThreads, kRing, st>>>(
            q, k_shared, v_shared, topk_idx, o_part, lse_part, scale, s->Hq, s->Hkv, s->C, s->L,
            s->k, s->shared_slots, n_slots);
    } else
        gemv_baseline_kernel<64><<<(unsigned)grid, kThreads, 0, st>>>(
            q, k_shared, v_shared, topk_idx, o_part, lse_part, scale, s->Hq, s->Hkv, s->C, s->L,
            s->k, s->shared_slots, n_slots);
    MOSKA_LAUNCH_CHECK("gemv_baseline_kernel");
    return MOSKA_OK;
}

int launch_shared_small(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                        const int32_t* seg_entries, float* o_part, float* lse_part, float scale,
                        const moska_shape* s, void* ws, bool dense, bool tiny_list_only, cudaStream_t st)
{
    const int n_slots = s->shared_slots + s->n_unique_splits;
    const int G = s->Hq / s->Hkv;
    long long grid;
    const WsHeader* hdr = nullptr;
    const TileItem* items = nullptr;
    const TileItem* tiny_items = nullptr;
    if (dense) {
        const int per_tile = kSmallTileRows / G;
        grid = (long long)s->Hkv * s->shared_slots * ((s->B + per_tile - 1) / per_tile);
    } else {
        const WsLayout lay = ws_layout(s);
        // resident CTAs (2 per SM) a few times over; they stride through the device-side list
        int dev = 0, n_sms = 0;
        MOSKA_CUDA_TRY(cudaGetDevice(&dev));
        MOSKA_CUDA_TRY(cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev));
        grid = lay.max_small < 8LL * n_sms ? lay.max_small : 8LL * n_sms;
        hdr = reinterpret_cast<const WsHeader*>(ws);
        items = reinterpret_cast<const TileItem*>(static_cast<const char*>(ws) + lay.off_small);
        if (lay.tiny_entries > 0)
            tiny_items = reinterpret_cast<const TileItem*>(static_cast<const char*>(ws) + lay.off_tiny);
    }
    if (grid == 0) return MOSKA_OK;
    if (grid > 0x7fffffffLL) return fail(MOSKA_ERR_UNSUPPORTED, "shared attention grid too large");
    constexpr int kSmallWord = offsetof(WsHeader, n_small_tiles) / 4;
    constexpr int kTinyWord = offsetof(WsHeader, n_tiny_tiles) / 4;
    constexpr int kRing = kWarps * kStagedWarpBytes;
#define MOSKA_LAUNCH_SMALL(DD, NN, ITEMS, WORD)                                                        \
    do {                                                                                               \
        if (DD == 128)                                                                                 \
            MOSKA_CUDA_TRY(cudaFuncSetAttribute(shared_small_kernel<DD, NN>,                           \
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, kRing));  \
        shared_small_kernel<DD, NN><<<(unsigned)grid, kThreads, DD == 128 ? kRing : 0, st>>>(          \
            q, k_shared, v_shared, seg_entries, hdr, ITEMS, o_part, lse_part, scale, s->B, s->Hq,      \
            s->Hkv, s->C, s->L, s->k, s->shared_slots, n_slots, dense ? 1 : 0, WORD);                  \
    } while (0)
    if (!tiny_list_only) {  // (routed shapes of the tensor-core kernel: the second list is not ours)
        if (s->D == 128) {
            MOSKA_LAUNCH_SMALL(128, 2, items, kSmallWord);
        } else {
            MOSKA_LAUNCH_SMALL(64, 2, items, kSmallWord);
        }
    }
    if (!dense && tiny_items != nullptr) {
        MOSKA_LAUNCH_CHECK("shared_small_kernel");
        if (s->D == 128) {
            MOSKA_LAUNCH_SMALL(128, 1, tiny_items, kTinyWord);
        } else {
            MOSKA_LAUNCH_SMALL(64, 1, tiny_items, kTinyWord);
        }
    }
#undef MOSKA_LAUNCH_SMALL
    MOSKA_LAUNCH_CHECK("shared_small_kernel");
    return MOSKA_OK;
}

}  // namespace moska
