// Query aggregation by shared chunk (Section III-A): a deterministic, stable counting sort of the
// routed (request, KV head, slot) positions by key = h * C + chunk, entirely on the device, plus
// the tile work lists that shared attention walks.
//
// Determinism without ordered atomics: a request routes to k DIFFERENT chunks per KV head, so a
// segment (h, c) holds each request at most once and is fully described by a bit set over the
// requests.  Pass 1 sets bit b of row (h, c) for every routed pair (atomicOr: the result does
// not depend on the order; inside moska_decode_step the router does it while it writes its
// picks).  Pass 2 counts the bits per row and scans the counts into segment offsets and tile
// lists, pass 3 walks every row's bits in ascending request order and writes the positions,
// looking the slot j up in the request's (ascending) chunk list.
#include <mutex>

#include "common.cuh"

namespace moska {

WsLayout ws_layout(const moska_shape* s)
{
    WsLayout w{};
    const int G = s->Hq / s->Hkv;
    w.n_keys = s->Hkv * s->C;
    w.words = (s->B + 31) / 32 > 0 ? (s->B + 31) / 32 : 1;
    w.small_entries = kSmallTileRows / G;
    w.tiny_entries = 8 / G;  // requests whose rows fit one 8-row MMA column block (0: no such tiles)
    w.big_entries = 2 * (kBigTileRows / G);  // a tensor-core work item holds two 128-row tiles
    w.tc = shared_tc_supported(s) ? 1 : 0;
    const int64_t P = (int64_t)s->B * s->Hkv * s->k;
    const int64_t segs = P < w.n_keys ? P : w.n_keys;  // non-empty segments at most
    w.max_small = P / w.small_entries + segs;
    w.max_big = P / w.big_entries + segs;
    size_t off = sizeof(WsHeader);
    int r = 0;
    // a region of `bytes` at the next 256-byte boundary; returns its offset
    auto region = [&](size_t bytes) {
        const size_t begin = off;
        w.guard_begin[r] = begin + round_up(bytes, 4);
        off += round_up(bytes, 256) + kGuardBytes;
        w.guard_end[r] = off;
        ++r;
        return begin;
    };
    w.off_hist = region(sizeof(uint32_t) * (size_t)w.words * w.n_keys);
    w.off_totals = region(sizeof(int32_t) * (size_t)w.n_keys);
    w.off_small = region(sizeof(TileItem) * (size_t)w.max_small);
    w.off_big = region(sizeof(TileItem) * (size_t)w.max_big);
    w.off_tiny = region(sizeof(TileItem) * (size_t)segs);  // at most one 8-row tile per segment
    w.group_total = off;
    w.off_scores = off;
    if (s->C > kRouteSmallC) {
        region(sizeof(float) * (size_t)s->B * s->Hkv * s->C);
    } else {
        w.guard_begin[r] = w.guard_end[r] = off;
        ++r;
    }
    w.off_q16 = off;
    if (w.tc) {
        region(sizeof(uint16_t) * (size_t)s->B * s->Hq * s->D);
    } else {
        w.guard_begin[r] = w.guard_end[r] = off;
    }
    w.total = off;
    return w;
}

namespace {

#ifdef MOSKA_DEBUG_GUARDS
struct GuardRanges {
    size_t begin[kWsRegions], end[kWsRegions];
};

__device__ __forceinline__ uint32_t guard_word(size_t byte_offset)
{
    return 0xC0DEFACEu ^ static_cast<uint32_t>(byte_offset);
}

// One CTA per region: writes (check = 0) or compares (check = 1) the region's guard words.
__global__ void __launch_bounds__(256)
ws_guard_kernel(uint32_t* __restrict__ ws_words, GuardRanges g, int check, int* __restrict__ status)
{
    const int r = blockIdx.x;
    for (size_t o = g.begin[r] + 4 * (size_t)threadIdx.x; o < g.end[r]; o += 4 * (size_t)blockDim.x) {
        if (!check) ws_words[o >> 2] = guard_word(o);
        else if (ws_words[o >> 2] != guard_word(o)) atomicMin(status, (int)MOSKA_ERR_CORRUPT);
    }
}
#endif

// Pass 1: one thread per routed pair p = (b*Hkv + h)*k + j.  Also checks what the bit-set form
// relies on: every index inside [0, C) and every (b, h) list strictly ascending (hence distinct).
__global__ void __launch_bounds__(256)
group_mark_kernel(const int32_t* __restrict__ topk_idx, uint32_t* __restrict__ bitmap,
                  int* __restrict__ status, long long P, int Hkv, int C, int k, int words)
{
    const long long p = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= P) return;
    const int c = topk_idx[p];
    if (c < 0 || c >= C) {  // corrupt routing: record it, touch nothing
        atomicMin(status, (int)MOSKA_ERR_INVALID_ARG);
        return;
    }
    if (p % k != 0 && topk_idx[p - 1] >= c) atomicMin(status, (int)MOSKA_ERR_INVALID_ARG);
    const int h = (int)((p / k) % Hkv);
    const int b = (int)(p / ((long long)k * Hkv));
    atomicOr(&bitmap[((size_t)h * C + c) * words + (b >> 5)], 1u << (b & 31));
}

// Requests per key, for shapes whose bit sets are too wide to be counted inside the scan.
__global__ void __launch_bounds__(256)
group_count_kernel(const uint32_t* __restrict__ bitmap, int32_t* __restrict__ totals, int n_keys,
                   int words)
{
    const int key = blockIdx.x * blockDim.x + threadIdx.x;
    if (key >= n_keys) return;
    const uint32_t* row = bitmap + (size_t)key * words;
    int n = 0;
    for (int w = 0; w < words; ++w) n += __popc(row[w]);
    totals[key] = n;
}

// Exclusive scans over the keys, one CTA: entries -> seg_offsets; tiles -> work lists.
// Shapes the tensor-core kernel serves (tc): a segment's requests go, in order, to items of two
// 128-row query tiles (big_entries requests; a remainder of more than one tile's requests still
// forms one) and the rest, if any, to ONE item: a single-tile item in the second list, or, if it
// has at most tiny_entries requests (8 rows), an 8-row tile in the third (the streaming kernel:
// for one or two requests on a chunk nothing beats reading it straight through).  Other shapes:
// 16-row tiles in the second list and a last piece of at most tiny_entries requests in the third.
__global__ void __launch_bounds__(1024)
group_scan_kernel(const uint32_t* __restrict__ bitmap, int words, const int32_t* __restrict__ totals,
                  int32_t* __restrict__ seg_offsets,
                  WsHeader* __restrict__ hdr, TileItem* __restrict__ small_items,
                  TileItem* __restrict__ tiny_items, TileItem* __restrict__ big_items, int n_keys,
                  int small_entries, int tiny_entries, int big_entries, int tc, long long max_small,
                  long long max_big, long long max_tiny, int* __restrict__ status)
{
    __shared__ int4 warp_sum[32];
    __shared__ int4 carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    auto add = [](int4 a, int4 b) { return make_int4(a.x + b.x, a.y + b.y, a.z + b.z, a.w + b.w); };
    auto sub = [](int4 a, int4 b) { return make_int4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w); };
    auto shfl_up = [](int4 a, int off) {
        return make_int4(__shfl_up_sync(0xffffffffu, a.x, off), __shfl_up_sync(0xffffffffu, a.y, off),
                         __shfl_up_sync(0xffffffffu, a.z, off), __shfl_up_sync(0xffffffffu, a.w, off));
    };
    if (threadIdx.x == 0) carry = make_int4(0, 0, 0, 0);
    __syncthreads();
    for (int base = 0; base < n_keys; base += blockDim.x) {
        const int key = base + threadIdx.x;
        int n = 0;  // requests of this key: counted beforehand, or the population count of its bits
        if (key < n_keys) {
            if (totals != nullptr) n = totals[key];
            else
                for (int w = 0; w < words; ++w) n += __popc(bitmap[(size_t)key * words + w]);
        }
        int n_big = 0, n_small = 0, n_tiny = 0;
        int small_cap = small_entries;  // requests per item of the second list
        if (tc) {
            n_big = n / big_entries;
            const int rem = n - n_big * big_entries;
            small_cap = big_entries / 2;  // one 128-row query tile
            if (rem > small_cap) ++n_big;
            else if (rem > tiny_entries) n_small = 1;
            else if (rem > 0) n_tiny = 1;  // one 8-row column block: the streaming kernel's list
        } else {
            n_small = n / small_entries;
            const int last = n - n_small * small_entries;  // requests of the last, partial tile
            if (last > 0) {
                if (last <= tiny_entries) n_tiny = 1; else ++n_small;
            }
        }
        // x: entries, y: 16-row tiles, z: tensor-core items, w: 8-row tiles
        const int4 v = make_int4(n, n_small, n_big, n_tiny);
        int4 inc = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int4 t = shfl_up(inc, off);
            if (lane >= off) inc = add(inc, t);
        }
        if (lane == 31) warp_sum[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            const int4 w = warp_sum[lane];
            int4 winc = w;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int4 t = shfl_up(winc, off);
                if (lane >= off) winc = add(winc, t);
            }
            warp_sum[lane] = sub(winc, w);  // exclusive
        }
        __syncthreads();
        const int4 ex = add(add(carry, warp_sum[warp]), sub(inc, v));
        if (key < n_keys) {
            seg_offsets[key] = ex.x;
            int e = ex.x;
#ifdef MOSKA_DEBUG_GUARDS
            // the lists' capacities follow from the shape; a write beyond one is reported, not done
            if (ex.z + n_big > max_big || ex.y + n_small > max_small || ex.w + n_tiny > max_tiny) {
                atomicMin(status, (int)MOSKA_ERR_CORRUPT);
                n_big = n_small = n_tiny = 0;
            }
#endif
            for (int t = 0; t < n_big; ++t) {
                const int cnt = min(big_entries, ex.x + n - e);
                big_items[ex.z + t] = TileItem{key, e, cnt, 0};
                e += cnt;
            }
            for (int t = 0; t < n_small; ++t) {
                const int cnt = min(small_cap, ex.x + n - e);
                small_items[ex.y + t] = TileItem{key, e, cnt, 0};
                e += cnt;
            }
            if (n_tiny) tiny_items[ex.w] = TileItem{key, e, ex.x + n - e, 0};
        }
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1) carry = add(ex, v);
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        seg_offsets[n_keys] = carry.x;
        hdr->n_small_tiles = carry.y;
        hdr->n_big_tiles = carry.z;
        hdr->n_tiny_tiles = carry.w;
    }
}

// Pass 4: one warp per key walks the key's request bits in ascending order.
__global__ void __launch_bounds__(256)
group_emit_kernel(const int32_t* __restrict__ topk_idx, const uint32_t* __restrict__ bitmap,
                  const int32_t* __restrict__ seg_offsets, int32_t* __restrict__ seg_entries,
                  int* __restrict__ status, int n_keys, int Hkv, int C, int k, int words)
{
    const int key = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (key >= n_keys) return;
    const int begin = seg_offsets[key];
    if (seg_offsets[key + 1] == begin) return;
    const int h = key / C, c = key % C;
    const uint32_t* row = bitmap + (size_t)key * words;
    int rank0 = begin;
    for (int w0 = 0; w0 < words; w0 += 32) {
        const int w = w0 + lane;
        uint32_t bits = w < words ? row[w] : 0u;
        const int cnt = __popc(bits);
        int inc = cnt;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += t;
        }
        int rank = rank0 + inc - cnt;
        while (bits) {
            const int b = w * 32 + (__ffs(bits) - 1);
            bits &= bits - 1;
            // slot j of chunk c in the ascending list topk_idx[b][h][0..k)
            const int32_t* lst = topk_idx + ((size_t)b * Hkv + h) * k;
            int lo = 0, hi = k - 1;
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (lst[mid] < c) lo = mid + 1; else hi = mid;
            }
            if (lst[lo] != c) {
                // the list is not ascending (reported by the marking pass): find the slot by a
                // plain scan so that the entry written is a position that exists
                atomicMin(status, (int)MOSKA_ERR_INVALID_ARG);
                for (int j = 0; j < k; ++j)
                    if (lst[j] == c) {
                        lo = j;
                        break;
                    }
            }
            seg_entries[rank++] = (b * Hkv + h) * k + lo;
        }
        rank0 += __shfl_sync(0xffffffffu, inc, 31);
    }
}

}  // namespace

int launch_ws_guards(void* ws, const WsLayout& lay, bool check, cudaStream_t st, size_t ws_extent)
{
#ifdef MOSKA_DEBUG_GUARDS
    // only the regions that lie inside the buffer the caller really has: the built-in scratch of the
    // allocation-free grouping ends where the grouping's regions end
    GuardRanges g;
    for (int r = 0; r < kWsRegions; ++r) {
        const bool inside = lay.guard_end[r] <= ws_extent;
        g.begin[r] = inside ? lay.guard_begin[r] : 0;
        g.end[r] = inside ? lay.guard_end[r] : 0;
    }
    int* status = nullptr;
    MOSKA_TRY_STATUS(status_word(&status));
    ws_guard_kernel<<<kWsRegions, 256, 0, st>>>(static_cast<uint32_t*>(ws), g, check ? 1 : 0, status);
    MOSKA_LAUNCH_CHECK("ws_guard_kernel");
#else
    (void)ws; (void)lay; (void)check; (void)st; (void)ws_extent;
#endif
    return MOSKA_OK;
}

int launch_group(const int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                 const moska_shape* s, void* ws, bool premarked, cudaStream_t st, bool grouping_regions_only)
{
    const WsLayout lay = ws_layout(s);
    char* base = static_cast<char*>(ws);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(base);
    uint32_t* bitmap = reinterpret_cast<uint32_t*>(base + lay.off_hist);
    TileItem* small_items = reinterpret_cast<TileItem*>(base + lay.off_small);
    TileItem* big_items = reinterpret_cast<TileItem*>(base + lay.off_big);
    TileItem* tiny_items = reinterpret_cast<TileItem*>(base + lay.off_tiny);
    const long long P = (long long)s->B * s->Hkv * s->k;
    int* status = nullptr;
    MOSKA_TRY_STATUS(status_word(&status));
    // header and bit sets must start at zero; the router has done both passes already when the
    // two calls run back to back inside moska_decode_step
    if (!premarked) {
        MOSKA_CUDA_TRY(cudaMemsetAsync(base, 0, lay.off_totals, st));
        MOSKA_TRY_STATUS(launch_ws_guards(ws, lay, false, st, grouping_regions_only ? lay.group_total : lay.total));
    }
    if (!premarked && P > 0) {
        group_mark_kernel<<<(unsigned)((P + 255) / 256), 256, 0, st>>>(topk_idx, bitmap, status, P,
                                                                       s->Hkv, s->C, s->k, lay.words);
        MOSKA_LAUNCH_CHECK("group_mark_kernel");
    }
    int32_t* totals = nullptr;
    if (lay.words > 2) {  // wide bit sets: count them with a whole grid, not with the scan's one CTA
        totals = reinterpret_cast<int32_t*>(base + lay.off_totals);
        group_count_kernel<<<(lay.n_keys + 255) / 256, 256, 0, st>>>(bitmap, totals, lay.n_keys, lay.words);
        MOSKA_LAUNCH_CHECK("group_count_kernel");
    }
    group_scan_kernel<<<1, 1024, 0, st>>>(bitmap, lay.words, totals, seg_offsets, hdr, small_items, tiny_items, big_items,
                                          lay.n_keys, lay.small_entries, lay.tiny_entries,
                                          lay.big_entries, lay.tc, lay.max_small, lay.max_big,
                                          (long long)(P < lay.n_keys ? P : lay.n_keys), status);
    MOSKA_LAUNCH_CHECK("group_scan_kernel");
    group_emit_kernel<<<(lay.n_keys + 7) / 8, 256, 0, st>>>(topk_idx, bitmap, seg_offsets, seg_entries,
                                                            status, lay.n_keys, s->Hkv, s->C, s->k, lay.words);
    MOSKA_LAUNCH_CHECK("group_emit_kernel");
    return launch_ws_guards(ws, lay, true, st, grouping_regions_only ? lay.group_total : lay.total);
}

// ---- grouping without any caller- or library-side allocation -----------------------------------
// Scratch for moska_group_by_chunk_noalloc lives in the library image itself: every GPU that
// loads the library reserves these bytes until the process exits.
static __device__ __align__(256) unsigned char g_noalloc_scratch[MOSKA_NOALLOC_SCRATCH_BYTES];

int launch_group_noalloc(const int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                         const moska_shape* s, cudaStream_t st)
{
    const WsLayout lay = ws_layout(s);
    if (lay.group_total > (size_t)MOSKA_NOALLOC_SCRATCH_BYTES)
        return fail(MOSKA_ERR_WORKSPACE,
                    "shape needs %zu bytes of grouping scratch, the built-in buffer holds %zu "
                    "(use moska_group_by_chunk with a caller workspace)",
                    lay.group_total, (size_t)MOSKA_NOALLOC_SCRATCH_BYTES);
    MOSKA_TRY_STATUS(check_device());
    // `g_noalloc_scratch` names a host-side handle here, not a device address; the address on
    // the current device is looked up once per device and kept.
    constexpr int kMaxDevices = 64;
    static void* dev_ptr[kMaxDevices] = {nullptr};
    static std::mutex mtx;
    int dev = 0;
    MOSKA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices)
        return fail(MOSKA_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(mtx);
        if (dev_ptr[dev] == nullptr) {
            void* p = nullptr;
            const cudaError_t e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
            if (e != cudaSuccess || p == nullptr)
                return fail(MOSKA_ERR_CUDA, "cudaGetSymbolAddress(noalloc scratch) failed: %s",
                            cudaGetErrorString(e));
            dev_ptr[dev] = p;
        }
        scratch = dev_ptr[dev];
    }
    // launch_group clears the header and the bit sets itself, so the previous call's contents
    // never leak into this one.
    return launch_group(topk_idx, seg_offsets, seg_entries, s, scratch, false, st, true);
}

}  // namespace moska
