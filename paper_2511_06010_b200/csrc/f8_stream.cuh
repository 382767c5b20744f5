// Streaming attention of up to 8 query rows over a token range kept in FP8 (E4M3), the block
// shared by Unique KV Attention over an FP8 private store (one scale per (token, KV head)) and by
// the 8-row tiles of Shared KV Attention over an FP8 shared store (one scale per chunk) -- the KV
// precision the paper's evaluation assumes (Section IV) on the memory-bound parts of the path
// (Section III-A), where it halves the bytes that bound the kernel.
//
// The CTA's warps take interleaved 16-token tiles, each warp copies whole token rows (128 bytes per
// 8 lanes, cp.async.cg) and, with per-token scales, the tile's 32 scales into its own
// shared-memory ring four tiles ahead, chunk j of token t stored at j ^ (t & 7).  The codes are
// widened to f16 in registers (cvt.f16x2.e4m3x2, exact) and fed to f16 warp MMAs with fp32
// accumulation:
//   S^T = (K8 Q^T) * k_scale[token]        scores, scaled per token row after the MMA
//   O^T += V8^T (P * v_scale[token])       the value scale folded into P, the row sum is not
// The head dimension is assigned to the fragment registers so that every 16-byte shared load of a
// quarter warp hits eight different chunk positions (K: lane c owns chunks 2c, 2c+1 of a row;
// V: lane group g owns chunk g, i.e. dimensions 16g .. 16g+15).
#pragma once
#include <cuda_fp16.h>

#include "stream_attn.cuh"

namespace moska {
namespace f8stream {
using namespace stream;

constexpr int kD8 = 128;                                  // head dimension (bytes per token row)
constexpr int kF8Depth = 4;                               // tiles in flight per warp
constexpr int kF8KvBytes = kTileTokens * kD8;             // K (or V) codes of one tile
constexpr int kF8TileBytes = 2 * kF8KvBytes + 128;        // K, V, 16 key scales, 16 value scales
constexpr int kF8WarpBytes = kF8Depth * kF8TileBytes;
constexpr int kF8RingBytes = kWarps * kF8WarpBytes;
static_assert(kF8RingBytes >= (int)sizeof(CombineSmem<kD8, 1>), "the combine step reuses the ring");

__device__ __forceinline__ void mma_f16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2,
                                              uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 "
        "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Two E4M3 codes (low byte -> low half) widened to two f16 values; exact.
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two_codes)
{
    uint32_t r;
    const unsigned short v = static_cast<unsigned short>(two_codes);
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(v));
    return r;
}

__device__ __forceinline__ uint32_t pack_f16(float lo, float hi)
{
    const __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

__device__ __forceinline__ void cp_async4(uint32_t smem_dst, const void* src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_dst), "l"(src) : "memory");
}

__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}

// Head dimension that lane group g holds as row g (half = 0) / row g + 8 (half = 1) of block mt.
__device__ __forceinline__ int v8_dim_of(int g, int mt, int half) { return 16 * g + 2 * mt + half; }

// Where the tokens of the range live and how they are scaled.
struct F8Source {
    const uint8_t* k_base;   // codes of the range's token 0 (this KV head)
    const uint8_t* v_base;
    int64_t tok_stride;      // bytes between consecutive tokens
    const float* ks_base;    // kTokenScales: scale of token 0; consecutive tokens scale_stride apart
    const float* vs_base;
    int64_t scale_stride;
    float ksc, vsc;          // !kTokenScales: one key and one value scale for the whole range
};

// Attention of the rows in `rows` (shared memory; q == nullptr marks a row that does not exist)
// over tokens [t_begin, t_end) of `src`; normalised partial output and log-sum-exp go to rows.o /
// rows.lse.  kMulti: the rows are q_len query tokens x G heads of one request, row j = i * G + g'
// sees the context up to q_len - 1 - i tokens before its end `len`.  `ring`: kF8RingBytes of
// dynamic shared memory, reused for the combination of the warps at the end.  Every thread of the
// CTA calls this after a __syncthreads() that follows the writes to `rows`.
template <bool kMulti, bool kTokenScales>
__device__ __forceinline__ void f8_attend_stream(const TileRows<1>& rows, const F8Source& src, int t_begin,
                                                 int t_end, int len, int q_len, int G, int n_rows,
                                                 float scale, unsigned char* ring)
{
    constexpr int D = kD8, MT = 8;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const float sl2 = scale * kLog2e;
    if (!kMulti) q_len = 1;

    // Q as the B operand in f16: step s = 4u + w covers dimensions 16 (2c + u) + 4 w .. + 3
    const uint16_t* qp = rows.q[g];
    const bool live = qp != nullptr;
    uint32_t qf[8][2];
#pragma unroll
    for (int s = 0; s < 8; ++s) {
        const int d0 = 16 * (2 * c + (s >> 2)) + 4 * (s & 3);
        float x[4] = {0.f, 0.f, 0.f, 0.f};
        if (live) {
            const uint2 raw = __ldg(reinterpret_cast<const uint2*>(qp + d0));
            x[0] = __uint_as_float(raw.x << 16);
            x[1] = __uint_as_float(raw.x & 0xffff0000u);
            x[2] = __uint_as_float(raw.y << 16);
            x[3] = __uint_as_float(raw.y & 0xffff0000u);
        }
        qf[s][0] = pack_f16(x[0], x[1]);
        qf[s][1] = pack_f16(x[2], x[3]);
    }

    float oacc[MT][4];
    float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) oacc[mt][0] = oacc[mt][1] = oacc[mt][2] = oacc[mt][3] = 0.f;

    const int n_tiles = (t_end - t_begin + kTileTokens - 1) / kTileTokens;
    const int last_tok = t_end - 1;
    // last visible token of the two query rows (columns 2c, 2c + 1) this lane holds scores of
    const int min_last = len - q_len;
    int lim0 = 0x7fffffff, lim1 = 0x7fffffff;
    if (2 * c < n_rows) lim0 = len - 1 - (q_len - 1 - (2 * c) / G);
    if (2 * c + 1 < n_rows) lim1 = len - 1 - (q_len - 1 - (2 * c + 1) / G);
    const int my_tiles = n_tiles > warp ? (n_tiles - warp + kWarps - 1) / kWarps : 0;
    const uint32_t ring_base = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) + warp * kF8WarpBytes;
    // 16-byte chunk `ch` (0..7) of token row t of the K (kv = 0) / V (kv = 1) tile in stage s
    auto slot = [&](int s, int kv, int t, int ch) {
        return ring_base + s * kF8TileBytes + kv * kF8KvBytes + t * 128 + ((ch ^ (t & 7)) << 4);
    };
    auto scale_slot = [&](int s, int kv, int t) {
        return ring_base + s * kF8TileBytes + 2 * kF8KvBytes + (kv * 16 + t) * 4;
    };
    auto issue = [&](int i) {
        const int s = i % kF8Depth;
        const int t0 = t_begin + (warp + i * kWarps) * kTileTokens;
        const int ch = lane & 7;
#pragma unroll
        for (int it = 0; it < 4; ++it) {  // 8 lanes per token row, four rows per instruction
            const int t = 4 * it + (lane >> 3);
            const int64_t off = (int64_t)min(t0 + t, last_tok) * src.tok_stride + 16 * ch;
            cp_async16(slot(s, 0, t, ch), src.k_base + off);
            cp_async16(slot(s, 1, t, ch), src.v_base + off);
        }
        if constexpr (kTokenScales) {
            const int t = lane & 15;
            const int64_t srow = (int64_t)min(t0 + t, last_tok) * src.scale_stride;
            cp_async4(scale_slot(s, lane >> 4, t), (lane < 16 ? src.ks_base : src.vs_base) + srow);
        }
    };
#pragma unroll
    for (int i = 0; i < kF8Depth; ++i) {
        if (i < my_tiles) issue(i);
        cp_async_commit();
    }

    for (int i = 0; i < my_tiles; ++i) {
        const int s = i % kF8Depth;
        const int t0 = t_begin + (warp + i * kWarps) * kTileTokens;
        cp_async_wait<kF8Depth - 1>();
        __syncwarp();
        // ---- S^T = K Q^T : K rows of tokens g and g + 8, chunks 2c and 2c + 1
        float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const uint4 ka = lds16(slot(s, 0, g, 2 * c + u));
            const uint4 kb = lds16(slot(s, 0, g + 8, 2 * c + u));
            const uint32_t wa[4] = {ka.x, ka.y, ka.z, ka.w}, wb[4] = {kb.x, kb.y, kb.z, kb.w};
#pragma unroll
            for (int w = 0; w < 4; ++w)
                mma_f16_16816(sc, e4m3x2_to_f16x2(wa[w]), e4m3x2_to_f16x2(wb[w]),
                              e4m3x2_to_f16x2(wa[w] >> 16), e4m3x2_to_f16x2(wb[w] >> 16),
                              qf[4 * u + w][0], qf[4 * u + w][1]);
        }
        float ksa = src.ksc, ksb = src.ksc, vsa = src.vsc, vsb = src.vsc;
        if constexpr (kTokenScales) {
            ksa = lds_f32(scale_slot(s, 0, g));
            ksb = lds_f32(scale_slot(s, 0, g + 8));
            vsa = lds_f32(scale_slot(s, 1, g));
            vsb = lds_f32(scale_slot(s, 1, g + 8));
        }
        sc[0] *= ksa;
        sc[1] *= ksa;
        sc[2] *= ksb;
        sc[3] *= ksb;
        const bool va = (t0 + g) <= last_tok, vb = (t0 + 8 + g) <= last_tok;
        if (!va) sc[0] = sc[1] = -INFINITY;
        if (!vb) sc[2] = sc[3] = -INFINITY;
        if (kMulti && t0 + kTileTokens - 1 > min_last) {  // the tile reaches past some row's context
            if (t0 + g > lim0) sc[0] = -INFINITY;
            if (t0 + g > lim1) sc[1] = -INFINITY;
            if (t0 + 8 + g > lim0) sc[2] = -INFINITY;
            if (t0 + 8 + g > lim1) sc[3] = -INFINITY;
        }
        float mx0 = fmaxf(sc[0], sc[2]), mx1 = fmaxf(sc[1], sc[3]);
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
            mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
        }
        const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);
        const bool grew = (mn0 > m_run[0]) | (mn1 > m_run[1]);
        float al0 = fast_exp2((m_run[0] - mn0) * sl2), al1 = fast_exp2((m_run[1] - mn1) * sl2);
        m_run[0] = mn0;
        m_run[1] = mn1;
        float ms0 = mn0 * sl2, ms1 = mn1 * sl2;
        // a row that has seen no token yet: keep its (empty) state free of inf - inf
        if (kMulti && mn0 == -INFINITY) { al0 = 1.f; ms0 = 0.f; }
        if (kMulti && mn1 == -INFINITY) { al1 = 1.f; ms1 = 0.f; }
        const float p0 = fast_exp2(fmaf(sc[0], sl2, -ms0)), p1 = fast_exp2(fmaf(sc[1], sl2, -ms1));
        const float p2 = fast_exp2(fmaf(sc[2], sl2, -ms0)), p3 = fast_exp2(fmaf(sc[3], sl2, -ms1));
        l_run[0] = fmaf(l_run[0], al0, p0 + p2);
        l_run[1] = fmaf(l_run[1], al1, p1 + p3);
        // P with the value scale of its token folded in, as the B operand of the second product
        const uint32_t pb0 = movmatrix_trans(pack_f16(p0 * vsa, p1 * vsa));
        const uint32_t pb1 = movmatrix_trans(pack_f16(p2 * vsb, p3 * vsb));
        if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                oacc[mt][0] *= al0;
                oacc[mt][1] *= al1;
                oacc[mt][2] *= al0;
                oacc[mt][3] *= al1;
            }
        }
        // ---- O^T += V^T P : chunk g of the V rows of tokens 2c, 2c+1, 2c+8, 2c+9
        const uint4 v0 = lds16(slot(s, 1, 2 * c, g)), v1 = lds16(slot(s, 1, 2 * c + 1, g));
        const uint4 v2 = lds16(slot(s, 1, 2 * c + 8, g)), v3 = lds16(slot(s, 1, 2 * c + 9, g));
        const uint32_t r0[4] = {v0.x, v0.y, v0.z, v0.w}, r1[4] = {v1.x, v1.y, v1.z, v1.w};
        const uint32_t r2[4] = {v2.x, v2.y, v2.z, v2.w}, r3[4] = {v3.x, v3.y, v3.z, v3.w};
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            // bytes 2mt, 2mt+1 of the chunk: [tok A dim 2mt, tok B dim 2mt, tok A dim 2mt+1, tok B dim 2mt+1]
            const uint32_t sel = (mt & 1) ? 0x7362u : 0x5140u;
            const uint32_t lo = __byte_perm(r0[mt >> 1], r1[mt >> 1], sel);
            const uint32_t hi = __byte_perm(r2[mt >> 1], r3[mt >> 1], sel);
            mma_f16_16816(oacc[mt], e4m3x2_to_f16x2(lo), e4m3x2_to_f16x2(lo >> 16), e4m3x2_to_f16x2(hi),
                          e4m3x2_to_f16x2(hi >> 16), pb0, pb1);
        }
        __syncwarp();
        if (i + kF8Depth < my_tiles) issue(i + kF8Depth);
        cp_async_commit();
    }
    cp_async_wait<0>();

    // ---- combine the warps through the (now idle) staging memory
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], off);
        l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], off);
    }
    __syncthreads();
    CombineSmem<D, 1>& sm = *reinterpret_cast<CombineSmem<D, 1>*>(ring);
    if (g == 0) {
        sm.m[warp][2 * c] = m_run[0];
        sm.m[warp][2 * c + 1] = m_run[1];
        sm.l[warp][2 * c] = l_run[0];
        sm.l[warp][2 * c + 1] = l_run[1];
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
        const int d0 = v8_dim_of(g, mt, 0), d1 = v8_dim_of(g, mt, 1);
        sm.o[warp][2 * c][d0] = oacc[mt][0];
        sm.o[warp][2 * c + 1][d0] = oacc[mt][1];
        sm.o[warp][2 * c][d1] = oacc[mt][2];
        sm.o[warp][2 * c + 1][d1] = oacc[mt][3];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 8 * D; i += kThreads) {
        const int r = i / D, d = i % D;
        if (rows.o[r] == nullptr) continue;
        float M = sm.m[0][r];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) M = fmaxf(M, sm.m[w][r]);
        float num = 0.f, den = 0.f;
        if (M != -INFINITY) {
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                const float a = fast_exp2((sm.m[w][r] - M) * sl2);
                num = fmaf(a, sm.o[w][r][d], num);
                den = fmaf(a, sm.l[w][r], den);
            }
        }
        rows.o[r][d] = den > 0.f ? num / den : 0.f;
        if (d == 0) *rows.lse[r] = den > 0.f ? M * scale + logf(den) : -INFINITY;
    }
}

}  // namespace f8stream
}  // namespace moska
