// Streaming decode attention of a few query rows over one K/V token stream.
//
// This is the memory-bound building block (Section III-A: attention over per-request KV is a
// GEMV-like pass limited by memory bandwidth).  Each K and V element is needed by all query rows
// of the tile (the G heads of a GQA group, or the rows of a few requests routed to the same
// chunk), so that reuse runs on warp-level tensor-core MMAs (mma.sync m16n8k16, bf16 -> fp32)
// and the kernel stays bound by HBM, not by FMA issue:
//
//   S^T[16 tokens x 8 rows]  = K_tile[16 x D]   * Q^T[D x 8]          (A = K, B = Q)
//   O^T[D x 8 rows]         += V_tile^T[D x 16] * P[16 tokens x 8]    (A = V^T, B = P)
//
// K and V go from global memory straight into MMA fragments with 16-byte loads: a contraction
// does not care in which order its index is visited, so the head dimension (for Q.K) and the
// output dimension (for P.V) are permuted such that every lane's fragment registers are
// contiguous bytes of a token row.  No shared memory and no barrier inside the token loop; the
// warps of a CTA take interleaved 16-token tiles and combine their running (max, sum, O) once
// at the end.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace moska {
namespace stream {

constexpr int kWarps = 4;             // warps per CTA
constexpr int kThreads = kWarps * 32;
constexpr int kTileTokens = 16;       // tokens per MMA step of one warp
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1,
                                               uint32_t a2, uint32_t a3, uint32_t b0,
                                               uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 "
        "{%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Transposes an 8x8 matrix of 16-bit values held one row-pair per lane (MMA fragment layout).
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x)
{
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

__device__ __forceinline__ uint4 ldg16(const uint16_t* p)
{
    return __ldg(reinterpret_cast<const uint4*>(p));
}

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// Query rows of one tile: NT column blocks of 8 rows.  Row i of the tile is `q_rows[i]` (a
// pointer to D bf16 values) or nullptr for padding; its result goes to slot pointers
// `o_rows[i]` (D floats) / `lse_rows[i]` (1 float).
template <int NT>
struct TileRows {
    const uint16_t* q[NT * 8];
    float* o[NT * 8];
    float* lse[NT * 8];
};

// Shared memory for the end-of-tile combination of the warps' partial results.
template <int D, int NT>
struct CombineSmem {
    float o[kWarps][NT * 8][D];
    float m[kWarps][NT * 8];
    float l[kWarps][NT * 8];
};

// Index of the head-dimension element that lane-group g holds as its e-th V element
// (e < D/8): 16-byte pieces of 8 elements, piece j of a row at element 64*j + 8*g.
__device__ __forceinline__ int v_dim_of(int g, int e) { return 64 * (e >> 3) + 8 * g + (e & 7); }

// Attention of the NT*8 rows in `rows` (shared-memory resident descriptor, filled by the
// caller, visible to all threads) over tokens [t_begin, t_end) of the stream
// k_base/v_base + token * tok_stride (elements).  All threads of the CTA must call this.
// Writes normalised o (fp32) and natural-log lse for every non-null row; a range without
// tokens gives lse = -inf, o = 0.
template <int D, int NT>
__device__ __forceinline__ void attend_stream(const TileRows<NT>& rows, const uint16_t* k_base,
                                              const uint16_t* v_base, int64_t tok_stride,
                                              int t_begin, int t_end, float scale,
                                              CombineSmem<D, NT>& sm)
{
    static_assert(D == 64 || D == 128, "head dimension");
    constexpr int KU = D / 32;   // 16-byte K loads per token row and lane
    constexpr int VL = D / 64;   // 16-byte V loads per token row and lane
    constexpr int MT = D / 16;   // 16-row blocks of O^T

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const float sl2 = scale * kLog2e;

    // Q as the B operand: row g of column block n, elements [32u + 8c, +8).
    uint4 qf[NT][KU];
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        const uint16_t* qp = rows.q[n * 8 + g];
#pragma unroll
        for (int u = 0; u < KU; ++u)
            qf[n][u] = qp ? ldg16(qp + 32 * u + 8 * c) : make_uint4(0, 0, 0, 0);
    }

    float oacc[NT][MT][4];
    float m_run[NT][2], l_run[NT][2];
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        m_run[n][0] = m_run[n][1] = -INFINITY;
        l_run[n][0] = l_run[n][1] = 0.f;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
            oacc[n][mt][0] = oacc[n][mt][1] = oacc[n][mt][2] = oacc[n][mt][3] = 0.f;
    }

    const int n_tok = t_end - t_begin;
    const int n_tiles = (n_tok + kTileTokens - 1) / kTileTokens;
    const int last_tok = t_end - 1;

    uint4 kA[KU], kB[KU];      // K rows of tokens g and g+8 of the tile
    uint4 vr[4][VL];           // V rows of tokens 2c, 2c+1, 2c+8, 2c+9 of the tile

    auto load_k = [&](int tile) {
        const int t0 = t_begin + tile * kTileTokens;
        const int ta = min(t0 + g, last_tok), tb = min(t0 + 8 + g, last_tok);
        const uint16_t* pa = k_base + (int64_t)ta * tok_stride + 8 * c;
        const uint16_t* pb = k_base + (int64_t)tb * tok_stride + 8 * c;
#pragma unroll
        for (int u = 0; u < KU; ++u) {
            kA[u] = ldg16(pa + 32 * u);
            kB[u] = ldg16(pb + 32 * u);
        }
    };
    auto load_v = [&](int tile) {
        const int t0 = t_begin + tile * kTileTokens;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int tt = min(t0 + 2 * c + (i & 1) + 8 * (i >> 1), last_tok);
            const uint16_t* p = v_base + (int64_t)tt * tok_stride + 8 * g;
#pragma unroll
            for (int j = 0; j < VL; ++j) vr[i][j] = ldg16(p + 64 * j);
        }
    };

    int tile = warp;
    if (tile < n_tiles) {
        load_k(tile);
        load_v(tile);
    }
    for (; tile < n_tiles; tile += kWarps) {
        const int t0 = t_begin + tile * kTileTokens;
        // ---- S^T = K Q^T
        float s[NT][4];
#pragma unroll
        for (int n = 0; n < NT; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
        for (int u = 0; u < KU; ++u) {
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                mma_bf16_16816(s[n], kA[u].x, kB[u].x, kA[u].y, kB[u].y, qf[n][u].x, qf[n][u].y);
                mma_bf16_16816(s[n], kA[u].z, kB[u].z, kA[u].w, kB[u].w, qf[n][u].z, qf[n][u].w);
            }
        }
        const int next = tile + kWarps;
        if (next < n_tiles) load_k(next);

        // ---- online softmax over the 16 tokens (rows of S^T) for query columns 2c, 2c+1
        const bool va = (t0 + g) <= last_tok, vb = (t0 + 8 + g) <= last_tok;
        uint32_t pb0[NT], pb1[NT];
        bool grew = false;
        float alpha[NT][2];
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            if (!va) s[n][0] = s[n][1] = -INFINITY;
            if (!vb) s[n][2] = s[n][3] = -INFINITY;
            float mx0 = fmaxf(s[n][0], s[n][2]), mx1 = fmaxf(s[n][1], s[n][3]);
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
            }
            const float mn0 = fmaxf(m_run[n][0], mx0), mn1 = fmaxf(m_run[n][1], mx1);
            grew |= (mn0 > m_run[n][0]) | (mn1 > m_run[n][1]);
            alpha[n][0] = fast_exp2((m_run[n][0] - mn0) * sl2);
            alpha[n][1] = fast_exp2((m_run[n][1] - mn1) * sl2);
            m_run[n][0] = mn0;
            m_run[n][1] = mn1;
            const float ms0 = mn0 * sl2, ms1 = mn1 * sl2;
            const float p0 = fast_exp2(fmaf(s[n][0], sl2, -ms0));
            const float p1 = fast_exp2(fmaf(s[n][1], sl2, -ms1));
            const float p2 = fast_exp2(fmaf(s[n][2], sl2, -ms0));
            const float p3 = fast_exp2(fmaf(s[n][3], sl2, -ms1));
            l_run[n][0] = fmaf(l_run[n][0], alpha[n][0], p0 + p2);
            l_run[n][1] = fmaf(l_run[n][1], alpha[n][1], p1 + p3);
            // P as the B operand of the second product: transpose [token][row] -> [row][token]
            pb0[n] = movmatrix_trans(pack_bf16(p0, p1));
            pb1[n] = movmatrix_trans(pack_bf16(p2, p3));
        }
        if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
            for (int n = 0; n < NT; ++n)
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    oacc[n][mt][0] *= alpha[n][0];
                    oacc[n][mt][1] *= alpha[n][1];
                    oacc[n][mt][2] *= alpha[n][0];
                    oacc[n][mt][3] *= alpha[n][1];
                }
        }

        // ---- O^T += V^T P : fragment rows g / g+8 of block mt are V elements mt / MT+mt
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            const int e0 = mt, e1 = MT + mt;
            const uint32_t sel0 = (e0 & 1) ? 0x7632u : 0x5410u;
            const uint32_t sel1 = (e1 & 1) ? 0x7632u : 0x5410u;
            auto word = [&](int i, int e) -> uint32_t {
                const uint4& r = vr[i][e >> 3];
                const int w = (e & 7) >> 1;
                return w == 0 ? r.x : (w == 1 ? r.y : (w == 2 ? r.z : r.w));
            };
            const uint32_t a0 = __byte_perm(word(0, e0), word(1, e0), sel0);
            const uint32_t a1 = __byte_perm(word(0, e1), word(1, e1), sel1);
            const uint32_t a2 = __byte_perm(word(2, e0), word(3, e0), sel0);
            const uint32_t a3 = __byte_perm(word(2, e1), word(3, e1), sel1);
#pragma unroll
            for (int n = 0; n < NT; ++n) mma_bf16_16816(oacc[n][mt], a0, a1, a2, a3, pb0[n], pb1[n]);
        }
        if (next < n_tiles) load_v(next);
    }

    // ---- combine the warps: per-lane sums of l over the 8 token lanes first
#pragma unroll
    for (int n = 0; n < NT; ++n) {
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            l_run[n][0] += __shfl_xor_sync(0xffffffffu, l_run[n][0], off);
            l_run[n][1] += __shfl_xor_sync(0xffffffffu, l_run[n][1], off);
        }
        if (g == 0) {
            sm.m[warp][n * 8 + 2 * c] = m_run[n][0];
            sm.m[warp][n * 8 + 2 * c + 1] = m_run[n][1];
            sm.l[warp][n * 8 + 2 * c] = l_run[n][0];
            sm.l[warp][n * 8 + 2 * c + 1] = l_run[n][1];
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            const int d0 = v_dim_of(g, mt), d1 = v_dim_of(g, MT + mt);
            sm.o[warp][n * 8 + 2 * c][d0] = oacc[n][mt][0];
            sm.o[warp][n * 8 + 2 * c + 1][d0] = oacc[n][mt][1];
            sm.o[warp][n * 8 + 2 * c][d1] = oacc[n][mt][2];
            sm.o[warp][n * 8 + 2 * c + 1][d1] = oacc[n][mt][3];
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < NT * 8 * D; i += kThreads) {
        const int r = i / D, d = i % D;
        float* orow = rows.o[r];
        if (orow == nullptr) continue;
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
        orow[d] = den > 0.f ? num / den : 0.f;
        if (d == 0) rows.lse[r][0] = den > 0.f ? M * scale + logf(den) : -INFINITY;
    }
}

// ---- the same block with K/V staged through shared memory ---------------------------------------
// attend_stream keeps the next tile's K/V in registers while it is in flight: the bytes a SM has
// in flight are bounded by its register file, and the 64-byte pieces of a K row that one load
// instruction fetches rely on L1 to be merged into whole lines.  Here a warp copies whole token
// rows (256 contiguous bytes per 16 lanes, cp.async.cg: L2 -> shared memory, no L1) into its own
// ring of tiles, kStagedDepth tiles ahead, and builds the MMA fragments from shared memory.
// The 16-byte chunks of token row t are stored at chunk ^ (t & 7), and the head dimension is
// assigned to the fragment registers such that every 16-byte shared load of a quarter warp hits
// eight different chunk positions (K: lane c owns chunks 2c, 2c+1 of each 128-byte half row;
// V: lane group g owns chunk g of each half row) -- no bank conflicts, no ldmatrix.
// Twice the bytes in flight per SM, fewer registers, and no dependence on the L1 / shared-memory
// carve-out: the kernel keeps its bandwidth when CTAs with large shared memory share the SM.
constexpr int kStagedDepth = 3;                                  // tiles in flight per warp
constexpr int kStagedTileBytes = 2 * kTileTokens * 256;          // K and V of one 16-token tile, D = 128
constexpr int kStagedWarpBytes = kStagedDepth * kStagedTileBytes;

__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ uint4 lds16(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "r"(addr));
    return v;
}

// D = 128, NT column blocks of 8 query rows, the kWarps warps of the CTA take interleaved tiles.
// `ring` is the CTA's staging memory (kWarps * kStagedWarpBytes bytes, 128-byte aligned); the
// final combination of the warps reuses it.  All threads of the CTA must call this.
// With kRowLast, row r only sees the tokens up to index row_last[r] of the stream (several query
// tokens of one request, each one token further into the same context); `row_last` is an array of
// NT * 8 ints visible to all threads.
template <int NT, bool kRowLast = false>
__device__ __forceinline__ void attend_stream_staged(const TileRows<NT>& rows, const uint16_t* k_base,
                                                     const uint16_t* v_base, int64_t tok_stride,
                                                     int t_begin, int t_end, float scale,
                                                     unsigned char* ring, const int* row_last = nullptr)
{
    constexpr int D = 128, KU = 4, VL = 2, MT = 8;
    static_assert(sizeof(CombineSmem<D, NT>) <= kWarps * kStagedWarpBytes, "the combine step reuses the ring");
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, c = lane & 3;
    const float sl2 = scale * kLog2e;
    // 16-byte chunk of a token row that lane c consumes as its u-th K piece
    auto k_chunk = [&](int u) { return 2 * c + (u & 1) + 8 * (u >> 1); };

    uint4 qf[NT][KU];  // Q as the B operand, in the same head-dimension order as the K pieces
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        const uint16_t* qp = rows.q[n * 8 + g];
#pragma unroll
        for (int u = 0; u < KU; ++u) qf[n][u] = qp ? ldg16(qp + 8 * k_chunk(u)) : make_uint4(0, 0, 0, 0);
    }
    float oacc[NT][MT][4];
    float m_run[NT][2], l_run[NT][2];
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        m_run[n][0] = m_run[n][1] = -INFINITY;
        l_run[n][0] = l_run[n][1] = 0.f;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) oacc[n][mt][0] = oacc[n][mt][1] = oacc[n][mt][2] = oacc[n][mt][3] = 0.f;
    }

    const int n_tok = t_end - t_begin;
    const int n_tiles = (n_tok + kTileTokens - 1) / kTileTokens;
    const int last_tok = t_end - 1;
    const int my_tiles = n_tiles > warp ? (n_tiles - warp + kWarps - 1) / kWarps : 0;
    // last visible token of the two query rows (columns 2c, 2c+1 of block n) this lane holds scores of
    int lim[NT][2];
    int min_last = last_tok;
    if constexpr (kRowLast) {
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            lim[n][0] = row_last[n * 8 + 2 * c];
            lim[n][1] = row_last[n * 8 + 2 * c + 1];
        }
        for (int r = 0; r < NT * 8; ++r) min_last = min(min_last, row_last[r]);
    }
    const uint32_t ring_base = static_cast<uint32_t>(__cvta_generic_to_shared(ring)) + warp * kStagedWarpBytes;
    // chunk `ch` of token row `t` (0..15) of the K (kv = 0) or V (kv = 1) tile in ring stage s
    auto slot = [&](int s, int kv, int t, int ch) {
        return ring_base + s * kStagedTileBytes + kv * (kTileTokens * 256) + t * 256 + ((ch ^ (t & 7)) << 4);
    };
    // cooperative copy of the i-th tile of this warp: 16 lanes per token row, two rows per instruction
    auto issue = [&](int i) {
        const int s = i % kStagedDepth;
        const int t0 = t_begin + (warp + i * kWarps) * kTileTokens;
        const int ch = lane & 15;
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int t = 2 * it + (lane >> 4);
            const int64_t off = (int64_t)min(t0 + t, last_tok) * tok_stride + 8 * ch;
            cp_async16(slot(s, 0, t, ch), k_base + off);
            cp_async16(slot(s, 1, t, ch), v_base + off);
        }
    };
#pragma unroll
    for (int i = 0; i < kStagedDepth; ++i) {
        if (i < my_tiles) issue(i);
        cp_async_commit();  // one group per ring stage, empty ones included
    }

    for (int i = 0; i < my_tiles; ++i) {
        const int s = i % kStagedDepth;
        const int t0 = t_begin + (warp + i * kWarps) * kTileTokens;
        cp_async_wait<kStagedDepth - 1>();  // this lane's copies of tile i have landed ...
        __syncwarp();                       // ... and so have the other lanes'
        uint4 kA[KU], kB[KU];               // K rows of tokens g and g+8
#pragma unroll
        for (int u = 0; u < KU; ++u) {
            kA[u] = lds16(slot(s, 0, g, k_chunk(u)));
            kB[u] = lds16(slot(s, 0, g + 8, k_chunk(u)));
        }
        float sc[NT][4];
#pragma unroll
        for (int n = 0; n < NT; ++n) sc[n][0] = sc[n][1] = sc[n][2] = sc[n][3] = 0.f;
#pragma unroll
        for (int u = 0; u < KU; ++u) {
#pragma unroll
            for (int n = 0; n < NT; ++n) {
                mma_bf16_16816(sc[n], kA[u].x, kB[u].x, kA[u].y, kB[u].y, qf[n][u].x, qf[n][u].y);
                mma_bf16_16816(sc[n], kA[u].z, kB[u].z, kA[u].w, kB[u].w, qf[n][u].z, qf[n][u].w);
            }
        }
        const bool va = (t0 + g) <= last_tok, vb = (t0 + 8 + g) <= last_tok;
        uint32_t pb0[NT], pb1[NT];
        bool grew = false;
        float alpha[NT][2];
#pragma unroll
        for (int n = 0; n < NT; ++n) {
            if (!va) sc[n][0] = sc[n][1] = -INFINITY;
            if (!vb) sc[n][2] = sc[n][3] = -INFINITY;
            if constexpr (kRowLast) {
                if (t0 + kTileTokens - 1 > min_last) {  // the tile reaches past some row's context
                    if (t0 + g > lim[n][0]) sc[n][0] = -INFINITY;
                    if (t0 + g > lim[n][1]) sc[n][1] = -INFINITY;
                    if (t0 + 8 + g > lim[n][0]) sc[n][2] = -INFINITY;
                    if (t0 + 8 + g > lim[n][1]) sc[n][3] = -INFINITY;
                }
            }
            float mx0 = fmaxf(sc[n][0], sc[n][2]), mx1 = fmaxf(sc[n][1], sc[n][3]);
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
            }
            const float mn0 = fmaxf(m_run[n][0], mx0), mn1 = fmaxf(m_run[n][1], mx1);
            grew |= (mn0 > m_run[n][0]) | (mn1 > m_run[n][1]);
            alpha[n][0] = fast_exp2((m_run[n][0] - mn0) * sl2);
            alpha[n][1] = fast_exp2((m_run[n][1] - mn1) * sl2);
            m_run[n][0] = mn0;
            m_run[n][1] = mn1;
            float ms0 = mn0 * sl2, ms1 = mn1 * sl2;
            if constexpr (kRowLast) {
                // a row that has seen no token yet: keep its (empty) state free of inf - inf
                if (mn0 == -INFINITY) { alpha[n][0] = 1.f; ms0 = 0.f; }
                if (mn1 == -INFINITY) { alpha[n][1] = 1.f; ms1 = 0.f; }
            }
            const float p0 = fast_exp2(fmaf(sc[n][0], sl2, -ms0)), p1 = fast_exp2(fmaf(sc[n][1], sl2, -ms1));
            const float p2 = fast_exp2(fmaf(sc[n][2], sl2, -ms0)), p3 = fast_exp2(fmaf(sc[n][3], sl2, -ms1));
            l_run[n][0] = fmaf(l_run[n][0], alpha[n][0], p0 + p2);
            l_run[n][1] = fmaf(l_run[n][1], alpha[n][1], p1 + p3);
            pb0[n] = movmatrix_trans(pack_bf16(p0, p1));
            pb1[n] = movmatrix_trans(pack_bf16(p2, p3));
        }
        if (__any_sync(0xffffffffu, grew)) {
#pragma unroll
            for (int n = 0; n < NT; ++n)
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    oacc[n][mt][0] *= alpha[n][0];
                    oacc[n][mt][1] *= alpha[n][1];
                    oacc[n][mt][2] *= alpha[n][0];
                    oacc[n][mt][3] *= alpha[n][1];
                }
        }
        uint4 vr[4][VL];  // V rows of tokens 2c, 2c+1, 2c+8, 2c+9: chunk g of each half row
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
            for (int j = 0; j < VL; ++j)
                vr[r][j] = lds16(slot(s, 1, 2 * c + (r & 1) + 8 * (r >> 1), g + 8 * j));
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            const int e0 = mt, e1 = MT + mt;
            const uint32_t sel0 = (e0 & 1) ? 0x7632u : 0x5410u;
            const uint32_t sel1 = (e1 & 1) ? 0x7632u : 0x5410u;
            auto word = [&](int r, int e) -> uint32_t {
                const uint4& x = vr[r][e >> 3];
                const int w = (e & 7) >> 1;
                return w == 0 ? x.x : (w == 1 ? x.y : (w == 2 ? x.z : x.w));
            };
            const uint32_t a0 = __byte_perm(word(0, e0), word(1, e0), sel0);
            const uint32_t a1 = __byte_perm(word(0, e1), word(1, e1), sel1);
            const uint32_t a2 = __byte_perm(word(2, e0), word(3, e0), sel0);
            const uint32_t a3 = __byte_perm(word(2, e1), word(3, e1), sel1);
#pragma unroll
            for (int n = 0; n < NT; ++n) mma_bf16_16816(oacc[n][mt], a0, a1, a2, a3, pb0[n], pb1[n]);
        }
        __syncwarp();  // every lane has read the stage into registers: refill it
        if (i + kStagedDepth < my_tiles) issue(i + kStagedDepth);
        cp_async_commit();
    }
    cp_async_wait<0>();

    // ---- combine the warps through the (now idle) staging memory
#pragma unroll
    for (int n = 0; n < NT; ++n)
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            l_run[n][0] += __shfl_xor_sync(0xffffffffu, l_run[n][0], off);
            l_run[n][1] += __shfl_xor_sync(0xffffffffu, l_run[n][1], off);
        }
    __syncthreads();  // every warp has left its ring
    CombineSmem<D, NT>& sm = *reinterpret_cast<CombineSmem<D, NT>*>(ring);
#pragma unroll
    for (int n = 0; n < NT; ++n) {
        if (g == 0) {
            sm.m[warp][n * 8 + 2 * c] = m_run[n][0];
            sm.m[warp][n * 8 + 2 * c + 1] = m_run[n][1];
            sm.l[warp][n * 8 + 2 * c] = l_run[n][0];
            sm.l[warp][n * 8 + 2 * c + 1] = l_run[n][1];
        }
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            const int d0 = v_dim_of(g, mt), d1 = v_dim_of(g, MT + mt);
            sm.o[warp][n * 8 + 2 * c][d0] = oacc[n][mt][0];
            sm.o[warp][n * 8 + 2 * c + 1][d0] = oacc[n][mt][1];
            sm.o[warp][n * 8 + 2 * c][d1] = oacc[n][mt][2];
            sm.o[warp][n * 8 + 2 * c + 1][d1] = oacc[n][mt][3];
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < NT * 8 * D; i += kThreads) {
        const int r = i / D, d = i % D;
        float* orow = rows.o[r];
        if (orow == nullptr) continue;
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
        orow[d] = den > 0.f ? num / den : 0.f;
        if (d == 0) rows.lse[r][0] = den > 0.f ? M * scale + logf(den) : -INFINITY;
    }
    __syncthreads();  // the ring may be refilled by a following call
}

}  // namespace stream
}  // namespace moska
