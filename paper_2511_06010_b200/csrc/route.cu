// Chunk router (Section III-B): inner product of the pooled query with every chunk summary,
// then an exact top-k with ties going to the lower chunk index.  One warp per (request, KV
// head); the warps of a CTA serve consecutive requests of the SAME KV head, so a tile of that
// head's summaries is staged in shared memory once and scored by all of them.
#include "common.cuh"

namespace moska {
namespace {

constexpr int kChunkTile = 32;  // summaries staged per pass: one chunk per lane

struct Best {
    float score;
    int idx;
};

// a is better than b: larger score, or equal score and lower index.
__device__ __forceinline__ bool better(float sa, int ia, float sb, int ib)
{
    return (sa > sb) || (sa == sb && ia < ib);
}

template <int D>
__global__ void __launch_bounds__(256)
route_kernel(const uint16_t* __restrict__ q, const float* __restrict__ summaries,
             int32_t* __restrict__ topk_idx, float* __restrict__ topk_score, int B, int Hq,
             int Hkv, int C, int k, uint32_t* __restrict__ mark, int mark_words)
{
    constexpr int PITCH = D + 4;  // floats; 16-byte aligned rows, conflict-free float4 reads
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int n_warps = blockDim.x >> 5;
    const int sel_words = (C + 31) / 32;
    float* tile = reinterpret_cast<float*>(smem_raw);                 // [kChunkTile][PITCH]
    float* qbar = tile + kChunkTile * PITCH;                          // [n_warps][D]
    float* score = qbar + n_warps * D;                                // [n_warps][C]
    uint32_t* taken = reinterpret_cast<uint32_t*>(score + (size_t)n_warps * C);  // [n_warps][sel_words]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int G = Hq / Hkv;
    const int h = blockIdx.x % Hkv;
    const int b = (blockIdx.x / Hkv) * n_warps + warp;
    const bool live = b < B;

    // pooled query: sum of the G query heads of the group, in fp32
    if (live) {
        for (int d = lane; d < D; d += 32) {
            float s = 0.f;
            for (int g = 0; g < G; ++g)
                s += __uint_as_float((uint32_t)q[((long long)b * Hq + h * G + g) * D + d] << 16);
            qbar[warp * D + d] = s;
        }
    }
    for (int i = lane; i < sel_words; i += 32) taken[warp * sel_words + i] = 0u;

    const float* sum_h = summaries + (long long)h * C * D;
    for (int c0 = 0; c0 < C; c0 += kChunkTile) {
        __syncthreads();  // previous tile fully consumed (and qbar visible on the first pass)
        const int n_c = min(kChunkTile, C - c0);
        for (int i = threadIdx.x; i < n_c * (D / 4); i += blockDim.x) {
            const int cc = i / (D / 4), d4 = i % (D / 4);
            const float4 v =
                __ldg(reinterpret_cast<const float4*>(sum_h + (long long)(c0 + cc) * D) + d4);
            *reinterpret_cast<float4*>(tile + cc * PITCH + d4 * 4) = v;
        }
        __syncthreads();
        if (live && lane < n_c) {
            const float4* row = reinterpret_cast<const float4*>(tile + lane * PITCH);
            const float4* qv = reinterpret_cast<const float4*>(qbar + warp * D);
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll 8
            for (int d4 = 0; d4 < D / 4; ++d4) {
                const float4 s = row[d4], x = qv[d4];
                a0 = fmaf(s.x, x.x, a0);
                a1 = fmaf(s.y, x.y, a1);
                a2 = fmaf(s.z, x.z, a2);
                a3 = fmaf(s.w, x.w, a3);
            }
            score[(size_t)warp * C + c0 + lane] = (a0 + a1) + (a2 + a3);
        }
    }
    __syncwarp();
    if (!live) return;

    // ---- exact top-k: k rounds of "best remaining chunk"; each lane caches the best of its own
    // candidates (chunks lane, lane+32, ...) and only the winning lane rescans.
    const float* sc = score + (size_t)warp * C;
    uint32_t* tk = taken + warp * sel_words;
    auto rescan = [&]() -> Best {
        Best bst{-INFINITY, 0x7fffffff};
        for (int c = lane; c < C; c += 32) {
            if (tk[c >> 5] & (1u << (c & 31))) continue;
            const float s = sc[c];
            if (bst.idx == 0x7fffffff || better(s, c, bst.score, bst.idx)) bst = Best{s, c};
        }
        return bst;
    };
    Best mine = rescan();
    for (int round = 0; round < k; ++round) {
        Best w = mine;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float os = __shfl_xor_sync(0xffffffffu, w.score, off);
            const int oi = __shfl_xor_sync(0xffffffffu, w.idx, off);
            const bool take = (w.idx == 0x7fffffff) ? (oi != 0x7fffffff)
                                                    : (oi != 0x7fffffff && better(os, oi, w.score, w.idx));
            if (take) w = Best{os, oi};
        }
        if (w.idx != 0x7fffffff && (w.idx & 31) == lane) {
            tk[w.idx >> 5] |= 1u << (w.idx & 31);
            mine = rescan();
        }
        __syncwarp();
    }

    // ---- emit the selected chunks in ascending index order
    const long long out_base = ((long long)b * Hkv + h) * k;
    int written = 0;
    for (int wd = 0; wd < sel_words; ++wd) {
        const uint32_t bits = tk[wd];
        if (bits & (1u << lane)) {
            const int pos = written + __popc(bits & ((1u << lane) - 1u));
            const int c = wd * 32 + lane;
            topk_idx[out_base + pos] = c;
            if (topk_score) topk_score[out_base + pos] = sc[c];
            // first pass of the grouping, done here when the caller runs both back to back
            if (mark) atomicOr(&mark[((size_t)h * C + c) * mark_words + (b >> 5)], 1u << (b & 31));
        }
        written += __popc(bits);
    }
}

// ---- Router for many chunks: a register-tiled fp32 product, then a selection pass ---------------
// The scores of a tile of requests against all chunk summaries of one KV head are a small GEMM
// [32 requests x D] . [D x C]:  one CTA keeps the 32 pooled queries in shared memory, streams the
// summaries in tiles of 64 chunks, and every thread accumulates a 4 x 4 block of scores in
// registers (each summary value is used for 32 requests, each query value for 64 chunks).  The
// scores go to a [B * Hkv][C] array in the workspace (it stays in L2); a second kernel selects the
// k best of every row, one warp per row.  Shared memory does not grow with C.
constexpr int kGemmRows = 32;      // requests per CTA
constexpr int kGemmChunks = 64;    // chunk summaries per tile
constexpr int kGemmThreads = 128;

template <int D>
__global__ void __launch_bounds__(kGemmThreads)
route_score_kernel(const uint16_t* __restrict__ q, const float* __restrict__ summaries,
                   float* __restrict__ scores, int B, int Hq, int Hkv, int C)
{
    constexpr int PITCH = D + 4;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* qs = reinterpret_cast<float*>(smem_raw);  // [32][PITCH] pooled queries
    float* ss = qs + kGemmRows * PITCH;              // [64][PITCH] summary tile

    const int tid = threadIdx.x;
    const int G = Hq / Hkv;
    const int h = blockIdx.y;
    const int b0 = blockIdx.x * kGemmRows;

    // pooled queries: sum of the G query heads of the group, in fp32 (rows past B are zero)
    for (int i = tid; i < kGemmRows * D; i += kGemmThreads) {
        const int r = i / D, d = i % D;
        float v = 0.f;
        if (b0 + r < B)
            for (int g = 0; g < G; ++g)
                v += __uint_as_float((uint32_t)q[((long long)(b0 + r) * Hq + h * G + g) * D + d] << 16);
        qs[r * PITCH + d] = v;
    }

    const int ty = tid >> 4, tx = tid & 15;  // rows 4 ty .. 4 ty + 3; chunks tx, tx + 16, tx + 32, tx + 48
    const float* sum_h = summaries + (long long)h * C * D;
    // blockIdx.z takes a contiguous share of the chunk tiles
    const int n_tiles = (C + kGemmChunks - 1) / kGemmChunks;
    const int per_z = (n_tiles + gridDim.z - 1) / gridDim.z;
    const int c_begin = blockIdx.z * per_z * kGemmChunks;
    const int c_end = min(C, c_begin + per_z * kGemmChunks);
    for (int c0 = c_begin; c0 < c_end; c0 += kGemmChunks) {
        const int n_c = min(kGemmChunks, C - c0);
        __syncthreads();  // previous tile's summaries are done with (and qs is visible)
        for (int i = tid; i < kGemmChunks * (D / 4); i += kGemmThreads) {
            const int cc = i / (D / 4), d4 = i % (D / 4);
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (cc < n_c) v = __ldg(reinterpret_cast<const float4*>(sum_h + (long long)(c0 + cc) * D) + d4);
            *reinterpret_cast<float4*>(ss + cc * PITCH + d4 * 4) = v;
        }
        __syncthreads();
        float acc[4][4];
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[r][i] = 0.f;
        const float* qrow = qs + (4 * ty) * PITCH;
#pragma unroll 2
        for (int d = 0; d < D; d += 4) {
            float4 a[4], sv[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) a[r] = *reinterpret_cast<const float4*>(qrow + r * PITCH + d);
#pragma unroll
            for (int i = 0; i < 4; ++i) sv[i] = *reinterpret_cast<const float4*>(ss + (tx + 16 * i) * PITCH + d);
            // every score sums its D products in ascending d, whichever thread computes it
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    acc[r][i] = fmaf(a[r].x, sv[i].x, acc[r][i]);
                    acc[r][i] = fmaf(a[r].y, sv[i].y, acc[r][i]);
                    acc[r][i] = fmaf(a[r].z, sv[i].z, acc[r][i]);
                    acc[r][i] = fmaf(a[r].w, sv[i].w, acc[r][i]);
                }
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int b = b0 + 4 * ty + r;
            if (b >= B) continue;
            float* out = scores + ((long long)b * Hkv + h) * C + c0;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (tx + 16 * i < n_c) out[tx + 16 * i] = acc[r][i];
        }
    }
}

// Exact top-k of every score row, one warp per (request, KV head), by radix selection: four passes
// over the row (8 bits each, most significant first) find the bit pattern T of the k-th largest
// score, a fifth pass in ascending chunk order emits every chunk with a larger score and, of those
// equal to T, the ones with the lowest indices -- the same set as k rounds of "best remaining
// chunk, ties to the lower index", already in ascending index order.  Every pass reads the row
// with coalesced, independent loads (it sits in L2).
__device__ __forceinline__ uint32_t sortable(float s)
{
    uint32_t u = __float_as_uint(s);
    if (u == 0x80000000u) u = 0u;  // -0 and +0 compare equal
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);  // ascending unsigned == ascending float
}

__global__ void __launch_bounds__(256)
route_select_kernel(const float* __restrict__ scores, int32_t* __restrict__ topk_idx,
                    float* __restrict__ topk_score, long long rows, int C, int k, int Hkv,
                    uint32_t* __restrict__ mark, int mark_words)
{
    __shared__ int hist[8][256];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + warp;
    if (row >= rows) return;
    const float* sc = scores + row * C;
    int* hw = hist[warp];
    uint32_t prefix = 0u, mask = 0u;  // bits of T fixed so far
    int need = k;                     // how many of the elements matching the prefix are wanted
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = lane; i < 256; i += 32) hw[i] = 0;
        __syncwarp();
        for (int c = lane; c < C; c += 32) {
            const uint32_t u = sortable(__ldg(sc + c));
            if ((u & mask) == prefix) atomicAdd(&hw[(u >> shift) & 255u], 1);
        }
        __syncwarp();
        // lane l owns bins 255 - 8 l ... 248 - 8 l (descending); find the bin where the count of
        // elements in higher bins first reaches `need`
        int cnt[8], mine = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            cnt[j] = hw[255 - 8 * lane - j];
            mine += cnt[j];
        }
        int above = mine;  // inclusive scan over lanes (lane 0 = highest bins)
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, above, off);
            if (lane >= off) above += t;
        }
        above -= mine;  // elements in bins above this lane's bins
        int sel_bin = -1, sel_above = 0;
        if (above < need && above + mine >= need) {
            int run = above;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (sel_bin < 0 && run + cnt[j] >= need) {
                    sel_bin = 255 - 8 * lane - j;
                    sel_above = run;
                }
                run += cnt[j];
            }
        }
        const unsigned who = __ballot_sync(0xffffffffu, sel_bin >= 0);
        const int src = __ffs(who) - 1;  // exactly one lane holds the crossing
        sel_bin = __shfl_sync(0xffffffffu, sel_bin, src);
        sel_above = __shfl_sync(0xffffffffu, sel_above, src);
        prefix |= static_cast<uint32_t>(sel_bin) << shift;
        mask |= 255u << shift;
        need -= sel_above;
        __syncwarp();
    }
    // prefix == T; `need` of the elements equal to T are taken, lowest indices first
    const long long out_base = row * k;
    int written = 0, ties_seen = 0;
    for (int c0 = 0; c0 < C; c0 += 32) {
        const int c = c0 + lane;
        const float s = c < C ? __ldg(sc + c) : 0.f;
        const uint32_t u = sortable(s);
        const bool gt = c < C && u > prefix, eq = c < C && u == prefix;
        const unsigned eq_bits = __ballot_sync(0xffffffffu, eq);
        const bool take = gt || (eq && ties_seen + __popc(eq_bits & ((1u << lane) - 1u)) < need);
        const unsigned take_bits = __ballot_sync(0xffffffffu, take);
        if (take) {
            const int pos = written + __popc(take_bits & ((1u << lane) - 1u));
            topk_idx[out_base + pos] = c;
            if (topk_score) topk_score[out_base + pos] = s;
            if (mark) {
                const int b = (int)(row / Hkv), h = (int)(row % Hkv);
                atomicOr(&mark[((size_t)h * C + c) * mark_words + (b >> 5)], 1u << (b & 31));
            }
        }
        written += __popc(take_bits);
        ties_seen += __popc(eq_bits);
    }
}

size_t route_smem_bytes(int D, int C, int n_warps)
{
    const size_t sel_words = (C + 31) / 32;
    return sizeof(float) * ((size_t)kChunkTile * (D + 4) + (size_t)n_warps * D + (size_t)n_warps * C) +
           sizeof(uint32_t) * n_warps * sel_words;
}

}  // namespace

int launch_route(const uint16_t* q, const float* summaries, int32_t* topk_idx, float* topk_score,
                 const moska_shape* s, void* ws, bool mark_groups, cudaStream_t st)
{
    // mark_groups: also do the first grouping pass (set bit b of row (h, chunk) for every routed
    // pair) into the workspace, which is cleared here; launch_group is then told to skip it
    uint32_t* mark = nullptr;
    int mark_words = 0;
    if (mark_groups) {
        const WsLayout lay = ws_layout(s);
        MOSKA_CUDA_TRY(cudaMemsetAsync(ws, 0, lay.off_totals, st));
        MOSKA_TRY_STATUS(launch_ws_guards(ws, lay, false, st, lay.total));
        mark = reinterpret_cast<uint32_t*>(static_cast<char*>(ws) + lay.off_hist);
        mark_words = lay.words;
    }
    if ((long long)s->B * s->Hkv == 0) return MOSKA_OK;
    // many chunks: tiled product into the workspace + selection; else one warp per request with
    // the scores in shared memory
    if (ws != nullptr && s->C > kRouteSmallC) {
        const WsLayout lay = ws_layout(s);
        float* scores = reinterpret_cast<float*>(static_cast<char*>(ws) + lay.off_scores);
        const size_t smem = sizeof(float) * (size_t)(kGemmRows + kGemmChunks) * (s->D + 4);
        // enough CTAs for about three per SM: split the chunk tiles over blockIdx.z
        const int row_tiles = (s->B + kGemmRows - 1) / kGemmRows;
        const int n_tiles = (s->C + kGemmChunks - 1) / kGemmChunks;
        int n_sms = 148, dev = 0;
        MOSKA_CUDA_TRY(cudaGetDevice(&dev));
        MOSKA_CUDA_TRY(cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev));
        int z = (3 * n_sms + row_tiles * s->Hkv - 1) / (row_tiles * s->Hkv);
        if (z > n_tiles) z = n_tiles;
        if (z < 1) z = 1;
        const dim3 grid((unsigned)row_tiles, (unsigned)s->Hkv, (unsigned)z);
        if (s->D == 128) {
            MOSKA_CUDA_TRY(cudaFuncSetAttribute(route_score_kernel<128>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            route_score_kernel<128><<<grid, kGemmThreads, smem, st>>>(q, summaries, scores, s->B, s->Hq,
                                                                     s->Hkv, s->C);
        } else {
            MOSKA_CUDA_TRY(cudaFuncSetAttribute(route_score_kernel<64>,
                                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            route_score_kernel<64><<<grid, kGemmThreads, smem, st>>>(q, summaries, scores, s->B, s->Hq,
                                                                    s->Hkv, s->C);
        }
        MOSKA_LAUNCH_CHECK("route_score_kernel");
        const long long rows = (long long)s->B * s->Hkv;
        route_select_kernel<<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(
            scores, topk_idx, topk_score, rows, s->C, s->k, s->Hkv, mark, mark_words);
        MOSKA_LAUNCH_CHECK("route_select_kernel");
        return MOSKA_OK;
    }
    int n_warps = 8;
    const size_t limit = 200 * 1024;
    while (n_warps > 1 && route_smem_bytes(s->D, s->C, n_warps) > limit) n_warps >>= 1;
    const size_t smem = route_smem_bytes(s->D, s->C, n_warps);
    if (smem > limit) return fail(MOSKA_ERR_UNSUPPORTED, "router: C = %d chunks exceed shared memory", s->C);
    const long long grid = (long long)s->Hkv * ((s->B + n_warps - 1) / n_warps);
    if (s->D == 128) {
        MOSKA_CUDA_TRY(cudaFuncSetAttribute(route_kernel<128>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        route_kernel<128><<<(unsigned)grid, n_warps * 32, smem, st>>>(
            q, summaries, topk_idx, topk_score, s->B, s->Hq, s->Hkv, s->C, s->k, mark, mark_words);
    } else {
        MOSKA_CUDA_TRY(cudaFuncSetAttribute(route_kernel<64>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        route_kernel<64><<<(unsigned)grid, n_warps * 32, smem, st>>>(
            q, summaries, topk_idx, topk_score, s->B, s->Hq, s->Hkv, s->C, s->k, mark, mark_words);
    }
    MOSKA_LAUNCH_CHECK("route_kernel");
    return MOSKA_OK;
}

}  // namespace moska
