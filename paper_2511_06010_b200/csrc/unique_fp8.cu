// Unique KV Attention over a private KV store kept in FP8 (E4M3) with one fp32 scale per (token,
// KV head): a CTA per (request, KV head, split) on the streaming block of f8_stream.cuh.
#include "common.cuh"
#include "f8_stream.cuh"

namespace moska {
namespace {
using namespace f8stream;

template <bool kMulti>  // several query tokens per request (q_len > 1)
__global__ void __launch_bounds__(kThreads, 3)
unique_fp8_kernel(const uint16_t* __restrict__ q, const uint8_t* __restrict__ k8,
                  const uint8_t* __restrict__ v8, const float* __restrict__ k_scale,
                  const float* __restrict__ v_scale, const int64_t* __restrict__ kv_start,
                  const int32_t* __restrict__ kv_len, float* __restrict__ o_part,
                  float* __restrict__ lse_part, float scale, int Hq, int Hkv, int n_splits,
                  int slot0, int n_slots, int q_len)
{
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ TileRows<1> rows;
    const int G = Hq / Hkv;
    const int h = blockIdx.x % Hkv;
    const int sp = (blockIdx.x / Hkv) % n_splits;
    const int b = blockIdx.x / (Hkv * n_splits);  // request
    // Query rows of this (request, KV head): row j = i * G + g' is head g' of query token i (one
    // token unless q_len > 1), a batch row of its own.
    if (!kMulti) q_len = 1;
    const int n_rows = q_len * G;
    if (threadIdx.x < 8) {
        const int j = threadIdx.x;
        const int64_t row = ((int64_t)b * q_len + j / G) * Hq + h * G + j % G;
        const bool live = j < n_rows;
        rows.q[j] = live ? q + row * kD8 : nullptr;
        rows.o[j] = live ? o_part + (row * n_slots + slot0 + sp) * kD8 : nullptr;
        rows.lse[j] = live ? lse_part + row * n_slots + slot0 + sp : nullptr;
    }
    __syncthreads();

    // token range of this split (same rule as the bf16 kernel: equal parts rounded up to 64)
    const int len = kv_len[b];
    int per = (len + n_splits - 1) / n_splits;
    per = (per + kWarps * kTileTokens - 1) / (kWarps * kTileTokens) * (kWarps * kTileTokens);
    const int t_begin = min(len, sp * per), t_end = min(len, t_begin + per);

    const int64_t row0 = kv_start[b] * Hkv + h;  // (token, head) row of the request's first token
    F8Source src;
    src.k_base = k8 + row0 * kD8;
    src.v_base = v8 + row0 * kD8;
    src.tok_stride = (int64_t)Hkv * kD8;
    src.ks_base = k_scale + row0;
    src.vs_base = v_scale + row0;
    src.scale_stride = Hkv;
    src.ksc = src.vsc = 1.f;
    f8_attend_stream<kMulti, true>(rows, src, t_begin, t_end, len, q_len, G, n_rows, scale, ring);
}

}  // namespace

int launch_unique_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8, const float* k_scale,
                      const float* v_scale, const int64_t* kv_start, const int32_t* kv_len,
                      float* o_part, float* lse_part, float scale, const moska_shape* s,
                      cudaStream_t st)
{
    const int n_slots = s->shared_slots + s->n_unique_splits;
    const int q_len = s->q_len > 1 ? s->q_len : 1;
    const long long grid = (long long)(s->B / q_len) * s->Hkv * s->n_unique_splits;
    if (grid == 0) return MOSKA_OK;
    if (grid > 0x7fffffffLL) return fail(MOSKA_ERR_UNSUPPORTED, "unique attention grid too large");
    if (q_len > 1) {
        MOSKA_CUDA_TRY(cudaFuncSetAttribute(unique_fp8_kernel<true>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, kF8RingBytes));
        unique_fp8_kernel<true><<<(unsigned)grid, kThreads, kF8RingBytes, st>>>(
            q, k8, v8, k_scale, v_scale, kv_start, kv_len, o_part, lse_part, scale, s->Hq, s->Hkv,
            s->n_unique_splits, s->shared_slots, n_slots, q_len);
    } else {
        MOSKA_CUDA_TRY(cudaFuncSetAttribute(unique_fp8_kernel<false>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, kF8RingBytes));
        unique_fp8_kernel<false><<<(unsigned)grid, kThreads, kF8RingBytes, st>>>(
            q, k8, v8, k_scale, v_scale, kv_start, kv_len, o_part, lse_part, scale, s->Hq, s->Hkv,
            s->n_unique_splits, s->shared_slots, n_slots, q_len);
    }
    MOSKA_LAUNCH_CHECK("unique_fp8_kernel");
    return MOSKA_OK;
}

}  // namespace moska
