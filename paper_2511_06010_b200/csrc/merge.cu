// Log-sum-exp combination of the partial attention results of a row (shared slots + unique
// splits) and the chunk-summary precompute.  Both are plain streaming kernels.
#include <cuda_bf16.h>

#include "common.cuh"

namespace moska {
namespace {

// One warp per query row.  Lane i owns elements [4i, 4i+4) of the head dimension.
template <int D>
__global__ void __launch_bounds__(256)
merge_kernel(const float* __restrict__ o_part, const float* __restrict__ lse_part,
             uint16_t* __restrict__ out, float* __restrict__ out_f32, float* __restrict__ lse_out,
             long long rows, int n_slots)
{
    const int lane = threadIdx.x & 31;
    const long long r = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (r >= rows) return;
    const float* lse = lse_part + r * n_slots;
    float M = -INFINITY;
    for (int i = lane; i < n_slots; i += 32) M = fmaxf(M, lse[i]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));

    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float W = 0.f;
    const bool active = lane < D / 4;
    if (M != -INFINITY) {
        const float* o = o_part + r * n_slots * D + (active ? lane * 4 : 0);
        // Slots in groups of 32: lane i holds the weight of slot base + i; the partial rows are then
        // read four slots at a time with all four loads in flight (a slot of weight 0 is read but
        // not used: it holds no meaningful o).
        for (int base = 0; base < n_slots; base += 32) {
            const int mine = base + lane;
            const float w_mine = mine < n_slots ? __expf(lse[mine] - M) : 0.f;
            const int n = min(32, n_slots - base);
            for (int i0 = 0; i0 < n; i0 += 4) {
                float w[4];
                float4 v[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    w[j] = __shfl_sync(0xffffffffu, w_mine, (i0 + j) & 31);
                    const int slot = min(base + i0 + j, n_slots - 1);
                    v[j] = *reinterpret_cast<const float4*>(o + (long long)slot * D);
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    if (i0 + j >= n || w[j] == 0.f) continue;
                    W += w[j];
                    acc.x = fmaf(w[j], v[j].x, acc.x);
                    acc.y = fmaf(w[j], v[j].y, acc.y);
                    acc.z = fmaf(w[j], v[j].z, acc.z);
                    acc.w = fmaf(w[j], v[j].w, acc.w);
                }
            }
        }
        const float inv = 1.f / W;
        acc.x *= inv;
        acc.y *= inv;
        acc.z *= inv;
        acc.w *= inv;
    }
    if (active) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y);
        __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 packed;
        packed.x = *reinterpret_cast<uint32_t*>(&lo);
        packed.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(out + r * D + lane * 4) = packed;
        if (out_f32) *reinterpret_cast<float4*>(out_f32 + r * D + lane * 4) = acc;
    }
    if (lane == 0 && lse_out) lse_out[r] = (M == -INFINITY) ? -INFINITY : M + logf(W);
}

// One CTA per (KV head, chunk): fp32 column mean of the chunk's L keys.
template <int D>
__global__ void __launch_bounds__(256)
summaries_kernel(const uint16_t* __restrict__ k_shared, float* __restrict__ summaries, int L)
{
    constexpr int LANES = D / 8;          // threads covering one token row with 16-byte loads
    constexpr int GROUPS = 256 / LANES;   // token rows in flight per pass
    __shared__ float red[GROUPS][D];
    const int col = threadIdx.x % LANES, grp = threadIdx.x / LANES;
    const uint16_t* base = k_shared + (long long)blockIdx.x * L * D + col * 8;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int t = grp; t < L; t += GROUPS) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(base + (long long)t * D));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            acc[2 * i] += __uint_as_float(w[i] << 16);
            acc[2 * i + 1] += __uint_as_float(w[i] & 0xffff0000u);
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) red[grp][col * 8 + i] = acc[i];
    __syncthreads();
    if (threadIdx.x < D) {
        float s = 0.f;
        for (int gI = 0; gI < GROUPS; ++gI) s += red[gI][threadIdx.x];
        summaries[(long long)blockIdx.x * D + threadIdx.x] = s / (float)L;
    }
}

}  // namespace

int launch_merge(const float* o_part, const float* lse_part, uint16_t* out, float* out_f32,
                 float* lse_out, const moska_shape* s, cudaStream_t st)
{
    const long long rows = (long long)s->B * s->Hq;
    const int n_slots = s->shared_slots + s->n_unique_splits;
    if (rows == 0) return MOSKA_OK;
    const unsigned grid = (unsigned)((rows + 7) / 8);
    if (s->D == 128)
        merge_kernel<128><<<grid, 256, 0, st>>>(o_part, lse_part, out, out_f32, lse_out, rows, n_slots);
    else
        merge_kernel<64><<<grid, 256, 0, st>>>(o_part, lse_part, out, out_f32, lse_out, rows, n_slots);
    MOSKA_LAUNCH_CHECK("merge_kernel");
    return MOSKA_OK;
}

int launch_summaries(const uint16_t* k_shared, float* summaries, const moska_shape* s,
                     cudaStream_t st)
{
    const long long grid = (long long)s->Hkv * s->C;
    if (grid == 0) return MOSKA_OK;
    if (s->D == 128)
        summaries_kernel<128><<<(unsigned)grid, 256, 0, st>>>(k_shared, summaries, s->L);
    else
        summaries_kernel<64><<<(unsigned)grid, 256, 0, st>>>(k_shared, summaries, s->L);
    MOSKA_LAUNCH_CHECK("summaries_kernel");
    return MOSKA_OK;
}

}  // namespace moska
