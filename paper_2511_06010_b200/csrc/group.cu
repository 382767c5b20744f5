// Query aggregation by shared chunk (Section III-A): a deterministic, stable counting sort of the
// routed (request, KV head, slot) positions by key = h * C + chunk, entirely on the device, plus
// the tile work lists that shared attention walks.
//
// Stability without ordered atomics: the requests are cut into `n_blocks` consecutive blocks.
// Pass 1 counts keys per block (atomic adds only accumulate counts, whose value does not depend
// on order).  Pass 2 turns the per-block counts of each key into per-block start ranks and the
// key totals.  Pass 3 scans the totals.  Pass 4 lets each block walk ITS requests in ascending
// order; within one request all keys are distinct (a request routes to k different chunks per
// head), so its threads bump different counters and no two writers race.
#include "common.cuh"

namespace moska {

WsLayout ws_layout(const moska_shape* s)
{
    WsLayout w{};
    const int G = s->Hq / s->Hkv;
    w.n_keys = s->Hkv * s->C;
    w.n_blocks = s->B < 64 ? (s->B > 0 ? s->B : 1) : 64;
    w.small_entries = kSmallTileRows / G;
    w.big_entries = kBigTileRows / G;
    w.big_min_entries = 0x7fffffff;  // no tensor-core tiles unless enabled below
    const int64_t P = (int64_t)s->B * s->Hkv * s->k;
    const int64_t segs = P < w.n_keys ? P : w.n_keys;  // non-empty segments at most
    w.max_small = P / w.small_entries + segs;
    w.max_big = P / w.big_entries + segs;
    size_t off = sizeof(WsHeader);
    w.off_hist = off;
    off += round_up(sizeof(int32_t) * (size_t)w.n_blocks * w.n_keys, 256);
    w.off_totals = off;
    off += round_up(sizeof(int32_t) * 3 * (size_t)w.n_keys, 256);
    w.off_small = off;
    off += round_up(sizeof(TileItem) * (size_t)w.max_small, 256);
    w.off_big = off;
    off += round_up(sizeof(TileItem) * (size_t)w.max_big, 256);
    w.total = off;
    return w;
}

namespace {

__device__ __forceinline__ void block_range(int B, int n_blocks, int blk, int& b0, int& b1)
{
    const int per = (B + n_blocks - 1) / n_blocks;
    b0 = min(B, blk * per);
    b1 = min(B, b0 + per);
}

__global__ void __launch_bounds__(256)
group_count_kernel(const int32_t* __restrict__ topk_idx, int32_t* __restrict__ hist,
                   WsHeader* __restrict__ hdr, int B, int Hkv, int C, int k, int n_keys)
{
    int b0, b1;
    block_range(B, gridDim.x, blockIdx.x, b0, b1);
    int32_t* my = hist + (size_t)blockIdx.x * n_keys;
    const int per_req = Hkv * k;
    for (int b = b0; b < b1; ++b)
        for (int i = threadIdx.x; i < per_req; i += blockDim.x) {
            const int c = topk_idx[(size_t)b * per_req + i];
            if (c < 0 || c >= C) {  // corrupt routing: record it, touch nothing
                atomicMin(&hdr->status, (int)MOSKA_ERR_INVALID_ARG);
                continue;
            }
            atomicAdd(&my[(i / k) * C + c], 1);
        }
}

// Per key: per-block counts -> per-block start ranks (in place), total count.
__global__ void __launch_bounds__(256)
group_colscan_kernel(int32_t* __restrict__ hist, int32_t* __restrict__ totals, int n_blocks,
                     int n_keys)
{
    const int key = blockIdx.x * blockDim.x + threadIdx.x;
    if (key >= n_keys) return;
    int run = 0;
    for (int blk = 0; blk < n_blocks; ++blk) {
        const int t = hist[(size_t)blk * n_keys + key];
        hist[(size_t)blk * n_keys + key] = run;
        run += t;
    }
    totals[key] = run;
}

// Exclusive scans over the keys, one CTA: entries -> seg_offsets; tiles -> work lists.
__global__ void __launch_bounds__(1024)
group_scan_kernel(const int32_t* __restrict__ totals, int32_t* __restrict__ seg_offsets,
                  WsHeader* __restrict__ hdr, TileItem* __restrict__ small_items,
                  TileItem* __restrict__ big_items, int n_keys, int small_entries,
                  int big_entries, int big_min_entries)
{
    __shared__ int3 warp_sum[32];
    __shared__ int3 carry;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry = make_int3(0, 0, 0);
    __syncthreads();
    for (int base = 0; base < n_keys; base += blockDim.x) {
        const int key = base + threadIdx.x;
        const int n = key < n_keys ? totals[key] : 0;
        // tensor-core tiles take whole multiples of big_entries, and a large enough remainder
        int n_big = n / big_entries;
        int rem = n - n_big * big_entries;
        if (rem >= big_min_entries) {
            ++n_big;
            rem = 0;
        }
        if (big_min_entries == 0x7fffffff) {
            n_big = 0;
            rem = n;
        }
        const int n_small = (rem + small_entries - 1) / small_entries;
        int3 v = make_int3(n, n_small, n_big);
        int3 inc = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int a = __shfl_up_sync(0xffffffffu, inc.x, off);
            const int b = __shfl_up_sync(0xffffffffu, inc.y, off);
            const int c = __shfl_up_sync(0xffffffffu, inc.z, off);
            if (lane >= off) {
                inc.x += a;
                inc.y += b;
                inc.z += c;
            }
        }
        if (lane == 31) warp_sum[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            int3 w = warp_sum[lane];
            int3 winc = w;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int a = __shfl_up_sync(0xffffffffu, winc.x, off);
                const int b = __shfl_up_sync(0xffffffffu, winc.y, off);
                const int c = __shfl_up_sync(0xffffffffu, winc.z, off);
                if (lane >= off) {
                    winc.x += a;
                    winc.y += b;
                    winc.z += c;
                }
            }
            warp_sum[lane] = make_int3(winc.x - w.x, winc.y - w.y, winc.z - w.z);  // exclusive
        }
        __syncthreads();
        const int3 wbase = warp_sum[warp];
        const int3 cr = carry;
        const int ex_n = cr.x + wbase.x + inc.x - v.x;
        const int ex_s = cr.y + wbase.y + inc.y - v.y;
        const int ex_b = cr.z + wbase.z + inc.z - v.z;
        if (key < n_keys) {
            seg_offsets[key] = ex_n;
            int e = ex_n;
            for (int t = 0; t < n_big; ++t) {
                const int cnt = min(big_entries, ex_n + n - e);
                big_items[ex_b + t] = TileItem{key, e, cnt, 0};
                e += cnt;
            }
            for (int t = 0; t < n_small; ++t) {
                const int cnt = min(small_entries, ex_n + n - e);
                small_items[ex_s + t] = TileItem{key, e, cnt, 0};
                e += cnt;
            }
        }
        __syncthreads();
        if (threadIdx.x == blockDim.x - 1)
            carry = make_int3(ex_n + v.x, ex_s + v.y, ex_b + v.z);
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        seg_offsets[n_keys] = carry.x;
        hdr->n_small_tiles = carry.y;
        hdr->n_big_tiles = carry.z;
    }
}

__global__ void __launch_bounds__(256)
group_scatter_kernel(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ seg_offsets,
                     int32_t* __restrict__ hist, int32_t* __restrict__ seg_entries, int B, int Hkv,
                     int C, int k, int n_keys)
{
    int b0, b1;
    block_range(B, gridDim.x, blockIdx.x, b0, b1);
    int32_t* my = hist + (size_t)blockIdx.x * n_keys;
    const int per_req = Hkv * k;
    for (int b = b0; b < b1; ++b) {
        for (int i = threadIdx.x; i < per_req; i += blockDim.x) {
            const int c = topk_idx[(size_t)b * per_req + i];
            if (c < 0 || c >= C) continue;
            const int key = (i / k) * C + c;
            const int rank = my[key];  // distinct keys within one request: no other writer now
            my[key] = rank + 1;
            seg_entries[seg_offsets[key] + rank] = b * per_req + i;
        }
        __syncthreads();  // the next request may hit the same keys
    }
}

}  // namespace

int launch_group(const int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                 const moska_shape* s, void* ws, cudaStream_t st)
{
    const WsLayout lay = ws_layout(s);
    char* base = static_cast<char*>(ws);
    WsHeader* hdr = reinterpret_cast<WsHeader*>(base);
    int32_t* hist = reinterpret_cast<int32_t*>(base + lay.off_hist);
    int32_t* totals = reinterpret_cast<int32_t*>(base + lay.off_totals);
    TileItem* small_items = reinterpret_cast<TileItem*>(base + lay.off_small);
    TileItem* big_items = reinterpret_cast<TileItem*>(base + lay.off_big);
    // header and histogram must start at zero
    MOSKA_CUDA_TRY(cudaMemsetAsync(base, 0, lay.off_totals, st));
    group_count_kernel<<<lay.n_blocks, 256, 0, st>>>(topk_idx, hist, hdr, s->B, s->Hkv, s->C, s->k,
                                                     lay.n_keys);
    MOSKA_LAUNCH_CHECK("group_count_kernel");
    group_colscan_kernel<<<(lay.n_keys + 255) / 256, 256, 0, st>>>(hist, totals, lay.n_blocks,
                                                                   lay.n_keys);
    MOSKA_LAUNCH_CHECK("group_colscan_kernel");
    group_scan_kernel<<<1, 1024, 0, st>>>(totals, seg_offsets, hdr, small_items, big_items,
                                          lay.n_keys, lay.small_entries, lay.big_entries,
                                          lay.big_min_entries);
    MOSKA_LAUNCH_CHECK("group_scan_kernel");
    group_scatter_kernel<<<lay.n_blocks, 256, 0, st>>>(topk_idx, seg_offsets, hist, seg_entries,
                                                       s->B, s->Hkv, s->C, s->k, lay.n_keys);
    MOSKA_LAUNCH_CHECK("group_scatter_kernel");
    return MOSKA_OK;
}

}  // namespace moska
