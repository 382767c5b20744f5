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
             int Hkv, int C, int k)
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
        }
        written += __popc(bits);
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
                 const moska_shape* s, cudaStream_t st)
{
    if ((long long)s->B * s->Hkv == 0) return MOSKA_OK;
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
            q, summaries, topk_idx, topk_score, s->B, s->Hq, s->Hkv, s->C, s->k);
    } else {
        MOSKA_CUDA_TRY(cudaFuncSetAttribute(route_kernel<64>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
        route_kernel<64><<<(unsigned)grid, n_warps * 32, smem, st>>>(
            q, summaries, topk_idx, topk_score, s->B, s->Hq, s->Hkv, s->C, s->k);
    }
    MOSKA_LAUNCH_CHECK("route_kernel");
    return MOSKA_OK;
}

}  // namespace moska
