// Shared KV Attention on the 5th-generation tensor cores (Section III-A, Fig. 2a): the query rows
// of all requests routed to one shared chunk form the M dimension of one GEMM, so the chunk's K/V
// leaves HBM once however many requests attend to it.
//
// One CTA owns one work item: up to two tiles of 128 gathered query rows (the rows of 2 * 128 / G
// requests of one (KV head, chunk) segment, or of consecutive requests in dense mode) and a
// range of K/V tokens (one chunk, or a run of consecutive chunks in dense mode), walked in tiles
// of 128 tokens:
//
//   S_t = Q_t K_j^T          tcgen05.mma, A and B from shared memory, accumulator in TMEM
//   P_t = exp2(S_t - m_t)    one thread per query row: TMEM -> registers -> bf16 back into TMEM,
//                            over the columns of S_t
//   O_t += P_t V_j           tcgen05.mma, A = P_t from TMEM, B = V_j from shared memory (N-major)
//
// Warp roles: warps 0-3 / 4-7 are the softmax groups of query tile 0 / 1 (thread i owns row i =
// TMEM lane i), warp 8 streams K/V tiles with TMA into a ring of shared-memory slots, warp 9
// issues the MMAs.  The two query tiles alternate on the tensor pipe, so the softmax of one tile
// runs under the MMAs of the other; both tiles consume every K/V tile from the same shared-memory
// copy.  The running maximum is only raised when a row's maximum grew by more than 2^8 (the
// accumulator rescale is then done in TMEM by the row's owner), which is exact after the final
// division by the row sum.  TMEM: S_0, S_1, O_0, O_1 of 128 columns each = all 512 columns.
#include <cuda.h>
#include <cuda_bf16.h>

#include <mutex>

#include "common.cuh"
#include "sm100.cuh"

namespace moska {
namespace {
using namespace sm100;

constexpr int kD = 128;                        // head dimension this kernel is built for
constexpr int kKvTile = 128;                   // tokens per K/V tile
constexpr int kTileBytes = 128 * kD * 2;       // one Q, K or V tile in shared memory
constexpr int kHalfBytes = kTileBytes / 2;     // 64 head-dimension columns of a tile
constexpr int kStages = 4;                     // K/V ring slots
constexpr int kThreads = 320;                  // 8 softmax warps + TMA warp + MMA warp
constexpr int kLoadWarp = 8, kMmaWarp = 9;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;       // log2 units a row maximum may lag behind

struct __align__(1024) TcSmem {
    uint8_t q[2][kTileBytes];
    uint8_t kv[kStages][kTileBytes];
    uint64_t full[kStages], empty[kStages];
    uint64_t q_full[2], s_full[2], p_full[2], o_full[2];
    long long row_r[2 * kBigTileRows];  // global query row b * Hq + hq of each tile row, -1 = padding
    uint32_t tmem_base;
    int abort_flag;
};

struct TcParams {
    const uint16_t* q;
    const int32_t* seg_entries;
    const WsHeader* hdr;
    const TileItem* items;
    float* o_part;
    float* lse_part;
    int* status;
    float scale;
    int B, Hq, Hkv, C, L, k, shared_slots, n_slots, dense;
};

__device__ int g_tc_status = 0;  // sticky: first negative status raised by a tensor-core CTA

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void group_barrier(int id)
{
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(128) : "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
shared_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                 const TcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    TcSmem& sm = *reinterpret_cast<TcSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                            ~static_cast<uintptr_t>(1023));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = p.Hq / p.Hkv;
    const int per_tile = kBigTileRows / G;  // requests per query tile

    // ---- the work item of this CTA (uniform over the CTA) --------------------------------------
    int h, slot_dense = 0, entry_begin = 0, b0 = 0, n_e[2], n_kv_tiles;
    long long kv_row0;
    if (!p.dense) {
        if ((int)blockIdx.x >= p.hdr->n_big_tiles) return;
        const TileItem it = p.items[blockIdx.x];
        h = it.key / p.C;
        entry_begin = it.entry_begin;
        n_e[0] = min(it.n_entries, per_tile);
        n_e[1] = min(it.n_entries - n_e[0], per_tile);
        kv_row0 = (long long)it.key * p.L;
        n_kv_tiles = p.L / kKvTile;
    } else {
        const int b_tiles = (p.B + 2 * per_tile - 1) / (2 * per_tile);
        const int bt = blockIdx.x % b_tiles;
        slot_dense = (blockIdx.x / b_tiles) % p.shared_slots;
        h = blockIdx.x / (b_tiles * p.shared_slots);
        const int run = (p.C + p.shared_slots - 1) / p.shared_slots;
        const int c0 = min(p.C, slot_dense * run), c1 = min(p.C, c0 + run);
        b0 = bt * 2 * per_tile;
        n_e[0] = min(per_tile, p.B - b0);
        n_e[1] = max(0, min(per_tile, p.B - b0 - per_tile));
        kv_row0 = ((long long)h * p.C + c0) * p.L;
        n_kv_tiles = (c1 - c0) * (p.L / kKvTile);
    }
    const int nq = n_e[1] > 0 ? 2 : 1;

    // Row owned by a softmax thread: tile t, tile row i.
    const int t = warp >> 2;           // only meaningful for warps 0..7
    const int i = tid & 127;
    long long my_r = -1;
    int my_slot = 0;
    if (warp < 8 && i < n_e[t] * G) {
        const int e = i / G, g = i % G;
        int b;
        if (!p.dense) {
            const int pp = p.seg_entries[entry_begin + t * per_tile + e];
            my_slot = pp % p.k;
            b = pp / (p.k * p.Hkv);
        } else {
            my_slot = slot_dense;
            b = b0 + t * per_tile + e;
        }
        my_r = (long long)b * p.Hq + h * G + g;
    }
    if (n_kv_tiles == 0) {  // dense mode: a trailing slot without chunks
        if (my_r >= 0) {
            float4* o = reinterpret_cast<float4*>(p.o_part + (my_r * p.n_slots + my_slot) * kD);
            for (int d = 0; d < kD / 4; ++d) o[d] = make_float4(0.f, 0.f, 0.f, 0.f);
            p.lse_part[my_r * p.n_slots + my_slot] = -INFINITY;
        }
        return;
    }

    // ---- set-up: barriers, tensor memory --------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], 1);
        }
        for (int u = 0; u < 2; ++u) {
            mbar_init(&sm.q_full[u], 128);
            mbar_init(&sm.s_full[u], 1);
            mbar_init(&sm.p_full[u], 128);
            mbar_init(&sm.o_full[u], 1);
        }
        sm.abort_flag = 0;
        fence_mbar_init();
    }
    __syncwarp();
    if (warp == kLoadWarp) {
        tmem_alloc(&sm.tmem_base, 512);
        tmem_relinquish();
    }
    if (warp == kMmaWarp && lane == 0) {
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    volatile int* ab = &sm.abort_flag;

    if (warp < 8) {
        // =========================== softmax group of query tile t ==============================
        if (n_e[t] > 0) {
            sm.row_r[tid] = my_r;
            group_barrier(1 + t);
            // gather the tile's query rows into the 128-byte-swizzled K-major operand layout
            for (int idx = i; idx < kBigTileRows * 16; idx += 128) {
                const int row = idx >> 4, c = idx & 15;
                const long long rr = sm.row_r[t * kBigTileRows + row];
                uint4 val = make_uint4(0u, 0u, 0u, 0u);
                if (rr >= 0) val = __ldg(reinterpret_cast<const uint4*>(p.q + rr * kD + c * 8));
                uint8_t* dst = sm.q[t] + (c >> 3) * kHalfBytes + row * 128 + (((c & 7) ^ (row & 7)) << 4);
                *reinterpret_cast<uint4*>(dst) = val;
            }
            fence_proxy_async_smem();
            mbar_arrive(&sm.q_full[t]);

            const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
            const uint32_t t_s = tmem + lane_sel + t * 128;        // S_t, and P_t over its columns
            const uint32_t t_o = tmem + lane_sel + 256 + t * 128;  // O_t
            const float sl2 = p.scale * kLog2e;
            float m_ref = -INFINITY, l_sum = 0.f;
            bool alive = true;
            for (int j = 0; j < n_kv_tiles; ++j) {
                alive = __all_sync(0xffffffffu, mbar_wait(&sm.s_full[t], j & 1, ab));
                if (!alive) break;
                tc_fence_after_sync();
                // pass 1: row maximum of this tile's scores
                float mx = -INFINITY;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tmem_ld32(t_s + c * 32, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int x = 0; x < 32; ++x) mx = fmaxf(mx, __uint_as_float(r[x]));
                }
                if (j == 0) {
                    m_ref = mx;
                } else {
                    const bool need = (mx - m_ref) * sl2 > kRescaleThreshold;
                    if (__any_sync(0xffffffffu, need)) {
                        // every MMA issued before S_t(j), PV_t(j-1) included, has completed
                        const float alpha = need ? fast_exp2((m_ref - mx) * sl2) : 1.f;
                        if (need) m_ref = mx;
                        l_sum *= alpha;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t r[32];
                            tmem_ld32(t_o + c * 32, r);
                            tmem_ld_wait();
#pragma unroll
                            for (int x = 0; x < 32; ++x)
                                r[x] = __float_as_uint(__uint_as_float(r[x]) * alpha);
                            tmem_st32(t_o + c * 32, r);
                        }
                    }
                }
                // pass 2: P = exp2((S - m_ref) * scale * log2 e) as bf16 over the columns of S
                const float mb = m_ref * sl2;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tmem_ld32(t_s + c * 32, r);
                    tmem_ld_wait();
                    uint32_t pk[16];
#pragma unroll
                    for (int x = 0; x < 16; ++x) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(r[2 * x]), sl2, -mb));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(r[2 * x + 1]), sl2, -mb));
                        l_sum += p0 + p1;
                        __nv_bfloat162 b2 = __floats2bfloat162_rn(p0, p1);
                        pk[x] = *reinterpret_cast<uint32_t*>(&b2);
                    }
                    tmem_st16(t_s + c * 16, pk);
                }
                tmem_st_wait();
                tc_fence_before_sync();
                mbar_arrive(&sm.p_full[t]);
            }
            // epilogue: normalised partial output and log-sum-exp of the row
            if (alive) alive = __all_sync(0xffffffffu, mbar_wait(&sm.o_full[t], 0, ab));
            if (alive) {
                tc_fence_after_sync();
                const float inv = 1.f / l_sum;
                float4* o = my_r >= 0
                    ? reinterpret_cast<float4*>(p.o_part + (my_r * p.n_slots + my_slot) * kD)
                    : nullptr;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tmem_ld32(t_o + c * 32, r);
                    tmem_ld_wait();
                    if (o != nullptr) {
#pragma unroll
                        for (int x = 0; x < 8; ++x)
                            o[c * 8 + x] = make_float4(__uint_as_float(r[4 * x]) * inv,
                                                       __uint_as_float(r[4 * x + 1]) * inv,
                                                       __uint_as_float(r[4 * x + 2]) * inv,
                                                       __uint_as_float(r[4 * x + 3]) * inv);
                    }
                }
                if (my_r >= 0)
                    p.lse_part[my_r * p.n_slots + my_slot] = m_ref * p.scale + logf(l_sum);
            }
        }
    } else if (warp == kLoadWarp) {
        // =========================== TMA producer: K_0, V_0, K_1, V_1, ... =======================
        if (lane == 0) {
            const int n_loads = 2 * n_kv_tiles;
            int issued = 0;
            for (int ld = 0; ld < n_loads; ++ld) {
                const int s = ld % kStages;
                if (ld >= kStages && !mbar_wait(&sm.empty[s], ((ld / kStages) - 1) & 1, ab)) break;
                mbar_arrive_expect_tx(&sm.full[s], kTileBytes);
                const CUtensorMap* tm = (ld & 1) ? &tm_v : &tm_k;
                const int y = (int)(kv_row0 + (long long)(ld >> 1) * kKvTile);
                tma_load_2d(sm.kv[s], tm, 0, y, &sm.full[s]);
                tma_load_2d(sm.kv[s] + kHalfBytes, tm, 64, y, &sm.full[s]);
                issued = ld + 1;
            }
            if (*ab) {
                // giving up: let the copies still in flight land before the CTA leaves
                volatile int never = 0;
                for (int ld = max(0, issued - kStages); ld < issued; ++ld)
                    mbar_wait(&sm.full[ld % kStages], (ld / kStages) & 1, &never);
            }
        }
        __syncwarp();
    } else {
        // =========================== MMA issuer ===================================================
        if (lane == 0) {
            const uint32_t id_qk = idesc_bf16_f32(128, kKvTile, false);
            const uint32_t id_pv = idesc_bf16_f32(128, kD, true);
            const uint32_t q_addr[2] = {smem_u32(sm.q[0]), smem_u32(sm.q[1])};
            // S_t = Q_t K^T with K in ring slot s: 8 steps of 16 head-dimension columns
            auto issue_qk = [&](int tq, int s) {
                const uint32_t k_addr = smem_u32(sm.kv[s]);
#pragma unroll
                for (int ks = 0; ks < kD / 16; ++ks) {
                    const uint32_t off = (ks >> 2) * kHalfBytes + (ks & 3) * 32;
                    mma_ss(tmem + tq * 128, smem_desc_sw128(q_addr[tq] + off, 16, 1024),
                           smem_desc_sw128(k_addr + off, 16, 1024), id_qk, ks > 0);
                }
            };
            // O_t += P_t V with V in ring slot s: 8 steps of 16 tokens
            auto issue_pv = [&](int tq, int s, bool acc) {
                const uint32_t v_addr = smem_u32(sm.kv[s]);
#pragma unroll
                for (int ks = 0; ks < kKvTile / 16; ++ks)
                    mma_ts(tmem + 256 + tq * 128, tmem + tq * 128 + ks * 8,
                           smem_desc_sw128(v_addr + ks * 2048, kHalfBytes, 1024), id_pv,
                           acc || ks > 0);
            };
            bool ok = true;
            for (int tq = 0; tq < nq && ok; ++tq) ok = mbar_wait(&sm.q_full[tq], 0, ab);
            if (ok) ok = mbar_wait(&sm.full[0], 0, ab);  // K_0
            if (ok) {
                tc_fence_after_sync();
                for (int tq = 0; tq < nq; ++tq) {
                    issue_qk(tq, 0);
                    tc_commit(&sm.s_full[tq]);
                }
                tc_commit(&sm.empty[0]);
            }
            for (int j = 0; j < n_kv_tiles && ok; ++j) {
                const int ld_v = 2 * j + 1, ld_k = 2 * j + 2;
                const int s_v = ld_v % kStages, s_k = ld_k % kStages;
                ok = mbar_wait(&sm.full[s_v], (ld_v / kStages) & 1, ab);
                for (int tq = 0; tq < nq && ok; ++tq) {
                    ok = mbar_wait(&sm.p_full[tq], j & 1, ab);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_pv(tq, s_v, j > 0);
                    if (tq == nq - 1) tc_commit(&sm.empty[s_v]);
                    if (j + 1 < n_kv_tiles) {
                        if (tq == 0) {
                            ok = mbar_wait(&sm.full[s_k], (ld_k / kStages) & 1, ab);
                            if (!ok) break;
                            tc_fence_after_sync();
                        }
                        issue_qk(tq, s_k);
                        tc_commit(&sm.s_full[tq]);
                        if (tq == nq - 1) tc_commit(&sm.empty[s_k]);
                    } else {
                        tc_commit(&sm.o_full[tq]);
                    }
                }
            }
        }
        __syncwarp();
    }

    // ---- teardown -------------------------------------------------------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if (warp == kLoadWarp) tmem_dealloc(tmem, 512);
    if (tid == 0 && sm.abort_flag) atomicMin(p.status, (int)MOSKA_ERR_TIMEOUT);
}

// ---- host side ------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (no link against libcuda).
int encoder(EncodeTiledFn* out)
{
    static EncodeTiledFn fn = nullptr;
    static std::mutex mtx;
    std::lock_guard<std::mutex> lock(mtx);
    if (fn == nullptr) {
        void* sym = nullptr;
        cudaDriverEntryPointQueryResult res;
        MOSKA_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &res));
        if (sym == nullptr || res != cudaDriverEntryPointSuccess)
            return fail(MOSKA_ERR_CUDA, "the driver does not provide cuTensorMapEncodeTiled");
        fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    *out = fn;
    return MOSKA_OK;
}

// [rows][128] bf16 matrix, loaded in boxes of 128 rows x 64 columns with the 128-byte swizzle.
int make_kv_map(CUtensorMap* tm, const uint16_t* base, long long rows)
{
    EncodeTiledFn enc = nullptr;
    MOSKA_TRY_STATUS(encoder(&enc));
    const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kD * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kKvTile};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                           const_cast<uint16_t*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(MOSKA_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
    return MOSKA_OK;
}

}  // namespace

bool shared_tc_supported(const moska_shape* s) { return s->D == kD && s->L % kKvTile == 0; }

int launch_shared_tc(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                     const int32_t* seg_entries, float* o_part, float* lse_part, float scale,
                     const moska_shape* s, void* ws, bool dense, cudaStream_t st)
{
    const int G = s->Hq / s->Hkv;
    const int per_cta = 2 * (kBigTileRows / G);
    long long grid;
    TcParams p{};
    if (dense) {
        grid = (long long)s->Hkv * s->shared_slots * ((s->B + per_cta - 1) / per_cta);
    } else {
        const WsLayout lay = ws_layout(s);
        grid = lay.max_big;
        p.hdr = reinterpret_cast<const WsHeader*>(ws);
        p.items = reinterpret_cast<const TileItem*>(static_cast<const char*>(ws) + lay.off_big);
    }
    if (grid == 0) return MOSKA_OK;
    if (grid > 0x7fffffffLL) return fail(MOSKA_ERR_UNSUPPORTED, "shared attention grid too large");
    const long long kv_rows = (long long)s->Hkv * s->C * s->L;
    if (kv_rows > 0x7fffffffLL) return fail(MOSKA_ERR_UNSUPPORTED, "shared store exceeds 2^31 tokens");
    CUtensorMap tm_k, tm_v;
    MOSKA_TRY_STATUS(make_kv_map(&tm_k, k_shared, kv_rows));
    MOSKA_TRY_STATUS(make_kv_map(&tm_v, v_shared, kv_rows));
    int* status = nullptr;
    MOSKA_CUDA_TRY(cudaGetSymbolAddress(reinterpret_cast<void**>(&status), g_tc_status));
    p.q = q;
    p.seg_entries = seg_entries;
    p.o_part = o_part;
    p.lse_part = lse_part;
    p.status = status;
    p.scale = scale;
    p.B = s->B;
    p.Hq = s->Hq;
    p.Hkv = s->Hkv;
    p.C = s->C;
    p.L = s->L;
    p.k = s->k;
    p.shared_slots = s->shared_slots;
    p.n_slots = s->shared_slots + s->n_unique_splits;
    p.dense = dense ? 1 : 0;
    const int smem = (int)sizeof(TcSmem) + 1024;
    MOSKA_CUDA_TRY(cudaFuncSetAttribute(shared_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    shared_tc_kernel<<<(unsigned)grid, kThreads, smem, st>>>(tm_k, tm_v, p);
    MOSKA_LAUNCH_CHECK("shared_tc_kernel");
    return MOSKA_OK;
}

int read_tc_status(int* out)
{
    MOSKA_CUDA_TRY(cudaDeviceSynchronize());
    MOSKA_CUDA_TRY(cudaMemcpyFromSymbol(out, g_tc_status, sizeof(int)));
    const int zero = 0;
    MOSKA_CUDA_TRY(cudaMemcpyToSymbol(g_tc_status, &zero, sizeof(int)));
    return MOSKA_OK;
}

}  // namespace moska
