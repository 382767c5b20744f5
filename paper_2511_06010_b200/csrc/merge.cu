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

// One CTA per (KV head, chunk): attention-pooled chunk embedding.  The chunk's mean key probes
// the chunk's own keys, w_t = softmax_t(scale * <mean, k_t>), embedding = sum_t w_t k_t; all in
// fp32, every sum in a fixed order.  The chunk (L * D * 2 bytes) is read three times, the second
// and third time from L2.  Dynamic shared memory: L floats (the scores).
template <int D>
__global__ void __launch_bounds__(256)
summaries_attn_kernel(const uint16_t* __restrict__ k_shared, float* __restrict__ summaries, int L,
                      float scale)
{
    constexpr int LANES = D / 8;          // threads covering one token row with 16-byte loads
    constexpr int GROUPS = 256 / LANES;   // token rows in flight per pass
    extern __shared__ float score[];      // [L]
    __shared__ float red[GROUPS][D];
    __shared__ float kbar[D];
    __shared__ float wred[8];
    __shared__ float stat[2];
    const int col = threadIdx.x % LANES, grp = threadIdx.x / LANES;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint16_t* base = k_shared + (long long)blockIdx.x * L * D + col * 8;
    auto load8 = [&](int t, float (&x)[8]) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(base + (long long)t * D));
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    };
    // column sums over the tokens, each thread its 8 columns of every GROUPS-th token, then over
    // the groups in ascending order
    auto reduce_columns = [&](const float (&acc)[8], float divide_by, float* dst) {
#pragma unroll
        for (int i = 0; i < 8; ++i) red[grp][col * 8 + i] = acc[i];
        __syncthreads();
        if (threadIdx.x < D) {
            float s = 0.f;
            for (int gI = 0; gI < GROUPS; ++gI) s += red[gI][threadIdx.x];
            dst[threadIdx.x] = s / divide_by;
        }
        __syncthreads();
    };
    // ---- pass 1: the mean key
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int t = grp; t < L; t += GROUPS) {
        float x[8];
        load8(t, x);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] += x[i];
    }
    reduce_columns(acc, (float)L, kbar);
    // ---- pass 2: scores, their maximum and the sum of the exponentials
    float kb[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) kb[i] = kbar[col * 8 + i];
    for (int t0 = 0; t0 < L; t0 += GROUPS) {  // every thread takes part in the shuffles
        const int t = t0 + grp;
        float d = 0.f;
        if (t < L) {
            float x[8];
            load8(t, x);
#pragma unroll
            for (int i = 0; i < 8; ++i) d = fmaf(kb[i], x[i], d);
        }
#pragma unroll
        for (int off = LANES / 2; off > 0; off >>= 1) d += __shfl_xor_sync(0xffffffffu, d, off);
        if (col == 0 && t < L) score[t] = scale * d;
    }
    __syncthreads();
    float m = -INFINITY;
    for (int t = threadIdx.x; t < L; t += 256) m = fmaxf(m, score[t]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
    if (lane == 0) wred[warp] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        float mm = wred[0];
        for (int w = 1; w < 8; ++w) mm = fmaxf(mm, wred[w]);
        stat[0] = mm;
    }
    __syncthreads();
    const float smax = stat[0];
    float z = 0.f;
    for (int t = threadIdx.x; t < L; t += 256) {
        const float e = expf(score[t] - smax);
        score[t] = e;  // the unnormalised weight
        z += e;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) z += __shfl_xor_sync(0xffffffffu, z, off);
    __syncthreads();  // every wred[] of the maximum has been read
    if (lane == 0) wred[warp] = z;
    __syncthreads();
    if (threadIdx.x == 0) {
        float zz = 0.f;
        for (int w = 0; w < 8; ++w) zz += wred[w];
        stat[1] = zz;
    }
    __syncthreads();
    // ---- pass 3: the weighted column sums
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;
    for (int t = grp; t < L; t += GROUPS) {
        float x[8];
        load8(t, x);
        const float w = score[t];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = fmaf(w, x[i], acc[i]);
    }
    reduce_columns(acc, stat[1], summaries + (long long)blockIdx.x * D);
}

}  // namespace

int launch_summaries_attn(const uint16_t* k_shared, float* summaries, float probe_scale,
                          const moska_shape* s, cudaStream_t st)
{
    const long long grid = (long long)s->Hkv * s->C;
    if (grid == 0) return MOSKA_OK;
    const size_t smem = sizeof(float) * (size_t)s->L;
    if (smem > 40 * 1024)
        return fail(MOSKA_ERR_UNSUPPORTED, "attention-pooled summaries are built for L <= 10240");
    if (s->D == 128)
        summaries_attn_kernel<128><<<(unsigned)grid, 256, smem, st>>>(k_shared, summaries, s->L, probe_scale);
    else
        summaries_attn_kernel<64><<<(unsigned)grid, 256, smem, st>>>(k_shared, summaries, s->L, probe_scale);
    MOSKA_LAUNCH_CHECK("summaries_attn_kernel");
    return MOSKA_OK;
}

int launch_merge_rows(const float* o_part, const float* lse_part, uint16_t* out, float* out_f32,
                      float* lse_out, const moska_shape* s, long long row0, long long rows,
                      cudaStream_t st)
{
    const int n_slots = s->shared_slots + s->n_unique_splits;
    if (rows <= 0) return MOSKA_OK;
    // rows [row0, row0 + rows) of every buffer
    o_part += row0 * n_slots * s->D;
    lse_part += row0 * n_slots;
    out += row0 * s->D;
    if (out_f32 != nullptr) out_f32 += row0 * s->D;
    if (lse_out != nullptr) lse_out += row0;
    const unsigned grid = (unsigned)((rows + 7) / 8);
    if (s->D == 128)
        merge_kernel<128><<<grid, 256, 0, st>>>(o_part, lse_part, out, out_f32, lse_out, rows, n_slots);
    else
        merge_kernel<64><<<grid, 256, 0, st>>>(o_part, lse_part, out, out_f32, lse_out, rows, n_slots);
    MOSKA_LAUNCH_CHECK("merge_kernel");
    return MOSKA_OK;
}

int launch_merge(const float* o_part, const float* lse_part, uint16_t* out, float* out_f32,
                 float* lse_out, const moska_shape* s, cudaStream_t st)
{
    return launch_merge_rows(o_part, lse_part, out, out_f32, lse_out, s, 0, (long long)s->B * s->Hq, st);
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
