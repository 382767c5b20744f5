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
#include <cuda_fp16.h>

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
constexpr int kSubBytes = kTileBytes / 2;      // query sub-buffer for a tile of at most 64 rows
#ifndef MOSKA_TC_STAGES
#define MOSKA_TC_STAGES 4
#endif
constexpr int kStages = MOSKA_TC_STAGES;       // K/V ring slots (5 fill the 227 KB of an SM exactly)
// FP8 shared store: the tiles arrive as E4M3 codes (16 KB) in a ring of their own and are widened
// to f16 operand tiles by the two gather warps; fewer operand slots leave room for the codes.
constexpr int kCodeBytes = 128 * kD;           // one K or V tile of codes
#ifndef MOSKA_F8_CODE_STAGES
#define MOSKA_F8_CODE_STAGES 4
#define MOSKA_F8_OP_STAGES 3
#endif
constexpr int kCodeStages = MOSKA_F8_CODE_STAGES;
constexpr int kOpStagesF8 = MOSKA_F8_OP_STAGES;
constexpr int kThreads = 384;                  // 8 softmax warps, TMA warp, MMA warp, 2 gather warps
constexpr int kLoadWarp = 8, kMmaWarp = 9, kGatherWarp0 = 10;
// Per-thread register budgets after set-up.  The CTA is launched with kLaunchRegs per thread (the
// 64 K registers of an SM over 384 threads, rounded down to a multiple of 8); what the four other
// warps give back must cover what the eight softmax warps ask for, or their request never returns.
constexpr int kLaunchRegs = 168, kSoftmaxRegs = 208, kOtherRegs = 88;
static_assert(4 * (kLaunchRegs - kOtherRegs) >= 8 * (kSoftmaxRegs - kLaunchRegs),
              "setmaxnreg: the released registers do not cover the requested ones");
static_assert(kSoftmaxRegs % 8 == 0 && kOtherRegs % 8 == 0, "setmaxnreg takes multiples of 8");
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;
constexpr float kRescaleThreshold = 8.f;       // log2 units a row maximum may lag behind

// F: the shared store is FP8 (see above); otherwise bf16 tiles come straight from TMA.
template <bool F>
struct TcSmemT;

template <>
struct __align__(1024) TcSmemT<false> {
    static constexpr int kOp = kStages;  // operand (K/V) ring slots
    uint8_t q[2][kTileBytes];
    uint8_t kv[kStages][kTileBytes];
    uint64_t full[kStages], empty[kStages];
    uint64_t q_full[2][2], q_free[2][2];  // [slot][sub-buffer]; a full tile signals / frees [.][0] (both)
    uint64_t s_full[2], p_full[2], o_full[2];
    uint64_t x_full, x_free;      // split items: statistics of slot 1 published / O_1 read
    float stat_m[kBigTileRows];   // split items: running maximum and sum of slot 1's rows
    float stat_l[kBigTileRows];
    uint32_t tmem_base;
    int abort_flag;
};

template <>
struct __align__(1024) TcSmemT<true> {
    static constexpr int kOp = kOpStagesF8;
    uint8_t q[2][kTileBytes];
    uint8_t kv[kOpStagesF8][kTileBytes];     // f16 operand tiles written by the gather warps
    uint8_t codes[kCodeStages][kCodeBytes];  // E4M3 code tiles written by TMA
    uint64_t full[kOpStagesF8], empty[kOpStagesF8];
    uint64_t code_full[kCodeStages], code_empty[kCodeStages];
    uint64_t q_full[2][2], q_free[2][2];
    uint64_t s_full[2], p_full[2], o_full[2];
    uint64_t x_full, x_free;
    float stat_m[kBigTileRows];
    float stat_l[kBigTileRows];
    uint32_t tmem_base;
    int abort_flag;
};

static_assert(sizeof(TcSmemT<false>) + 1024 <= 232448 && sizeof(TcSmemT<true>) + 1024 <= 232448,
              "the CTA's shared memory exceeds the 227 KB an SM offers");

struct TcParams {
    const uint16_t* q;
    const int32_t* seg_entries;
    const WsHeader* hdr;
    const TileItem* items;    // items of two query tiles (more than 128 rows)
    const TileItem* singles;  // items of one query tile
    const float* k_scale;     // FP8 store: scale per (KV head, chunk) of the keys / values
    const float* v_scale;
    float* o_part;
    float* lse_part;
    int* status;
    float scale;
    int B, Hq, Hkv, C, L, k, shared_slots, n_slots, dense, n_items_dense;
};

__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
    return y;
}

// ---- packed fp32 arithmetic (two lanes per instruction) -------------------------------------------
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c)
{
    float2 d;
    asm("{\n"
        ".reg .b64 ra, rb, rc, rd;\n"
        "mov.b64 ra, {%2, %3};\n"
        "mov.b64 rb, {%4, %5};\n"
        "mov.b64 rc, {%6, %7};\n"
        "fma.rn.f32x2 rd, ra, rb, rc;\n"
        "mov.b64 {%0, %1}, rd;\n"
        "}\n"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}

__device__ __forceinline__ float2 fadd2(float2 a, float2 b)
{
    float2 d;
    asm("{\n"
        ".reg .b64 ra, rb, rd;\n"
        "mov.b64 ra, {%2, %3};\n"
        "mov.b64 rb, {%4, %5};\n"
        "add.rn.f32x2 rd, ra, rb;\n"
        "mov.b64 {%0, %1}, rd;\n"
        "}\n"
        : "=f"(d.x), "=f"(d.y)
        : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}

// One 32-byte store (sm_100): p must be 32-byte aligned.
__device__ __forceinline__ void st_global_v8(float* p, const float* v)
{
    asm volatile("st.global.v8.f32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "f"(v[0]),
                 "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
                 : "memory");
}

__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// One work unit of a CTA.  The CTA has two "slots" (t = 0, 1), each with its own S/P and O
// accumulator in TMEM, its own softmax warp group and its own query buffer.  Three forms:
//   two tiles  one item of more than 128 rows: its two query tiles run in the two slots over the
//              same K/V tiles (one shared-memory copy serves both);
//   pair       two different items of at most 128 rows each, one per slot, every slot over its own
//              item's K/V tiles (which alternate in the ring) -- nothing is shared and nothing is
//              merged, so one slot's epilogue and query gather run under the other slot's tiles;
//   split      a single item of at most 128 rows: both slots hold the same query tile, slot 0 takes
//              the even and slot 1 the odd K/V tiles, and the two partial softmax states are
//              combined at the end.
// In every form the tensor pipe has two independent dependency chains to alternate between.
enum : int { kTwoTiles = 0, kSplit = 1, kPair = 2 };

struct Unit {
    int mode;
    int n_kv;            // K/V tiles of 128 tokens of one item
    int h[2];            // KV head of the item whose rows sit in slot t
    int n_e[2];          // requests of that item's tile (split: slot 1 mirrors slot 0)
    int entry_begin[2];  // routed: first entry of the tile in seg_entries
    int b0[2];           // dense: first request of the tile
    int slot_dense;      // dense: partial slot (= run of chunks)
    int n_it[2];         // K/V tiles handled by slot 0 / 1
    long long kv_row0[2];  // first token row of the slot's K/V range in the [Hkv*C*L][D] store
    int key[2];            // h * C + chunk of the slot's item (dense: the run's first chunk): index of its scales
};

// Where the routed work lists end and how the single-tile items are scheduled on this grid: whole
// rounds of pairs (two items per CTA and round), and the remaining fewer than 2 * grid items one per
// unit in the split form, so that the last round still spreads over as many CTAs as it has items.
struct Schedule {
    int n_two, n_pairs, n_units;
};

__device__ __forceinline__ Schedule make_schedule(const TcParams& p)
{
    Schedule s;
    if (p.dense) {
        s.n_two = p.n_items_dense;
        s.n_pairs = 0;
        s.n_units = p.n_items_dense;
    } else {
        s.n_two = p.hdr->n_big_tiles;
        const int n1 = p.hdr->n_small_tiles;
        s.n_pairs = (n1 / (2 * (int)gridDim.x)) * (int)gridDim.x;
        s.n_units = s.n_two + s.n_pairs + (n1 - 2 * s.n_pairs);
    }
    return s;
}

// i-th single-tile item (the second work list)
__device__ __forceinline__ int4 single_item(const TcParams& p, int i)
{
    return __ldg(reinterpret_cast<const int4*>(p.singles + i));
}

__device__ __forceinline__ Unit decode_unit(const TcParams& p, const Schedule& sch, int unit, int G,
                                            int per_tile)
{
    Unit it;
    it.slot_dense = 0;
    it.key[0] = it.key[1] = 0;
    it.b0[0] = it.b0[1] = 0;
    if (!p.dense) {
        it.n_kv = p.L / kKvTile;
        if (unit < sch.n_two) {
            const int4 raw = __ldg(reinterpret_cast<const int4*>(p.items) + unit);  // TileItem
            it.mode = kTwoTiles;
            it.h[0] = it.h[1] = raw.x / p.C;
            it.entry_begin[0] = raw.y;
            it.entry_begin[1] = raw.y + per_tile;
            it.n_e[0] = min(raw.z, per_tile);
            it.n_e[1] = min(raw.z - it.n_e[0], per_tile);
            it.kv_row0[0] = it.kv_row0[1] = (long long)raw.x * p.L;
            it.key[0] = it.key[1] = raw.x;
        } else if (unit < sch.n_two + sch.n_pairs) {
            it.mode = kPair;
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int4 raw = single_item(p, 2 * (unit - sch.n_two) + t);
                it.h[t] = raw.x / p.C;
                it.entry_begin[t] = raw.y;
                it.n_e[t] = min(raw.z, per_tile);
                it.kv_row0[t] = (long long)raw.x * p.L;
                it.key[t] = raw.x;
            }
        } else {
            const int4 raw = single_item(p, 2 * sch.n_pairs + (unit - sch.n_two - sch.n_pairs));
            it.key[0] = it.key[1] = raw.x;
            it.mode = kSplit;
            it.h[0] = it.h[1] = raw.x / p.C;
            it.entry_begin[0] = it.entry_begin[1] = raw.y;
            it.n_e[0] = it.n_e[1] = min(raw.z, per_tile);
            it.kv_row0[0] = it.kv_row0[1] = (long long)raw.x * p.L;
        }
    } else {
        const int b_tiles = (p.B + 2 * per_tile - 1) / (2 * per_tile);
        const int bt = unit % b_tiles;
        it.slot_dense = (unit / b_tiles) % p.shared_slots;
        it.h[0] = it.h[1] = unit / (b_tiles * p.shared_slots);
        const int run = (p.C + p.shared_slots - 1) / p.shared_slots;
        const int c0 = min(p.C, it.slot_dense * run), c1 = min(p.C, c0 + run);
        it.b0[0] = bt * 2 * per_tile;
        it.b0[1] = it.b0[0] + per_tile;
        it.n_e[0] = min(per_tile, p.B - it.b0[0]);
        it.n_e[1] = max(0, min(per_tile, p.B - it.b0[1]));
        it.kv_row0[0] = it.kv_row0[1] = ((long long)it.h[0] * p.C + c0) * p.L;
        it.key[0] = it.key[1] = it.h[0] * p.C + c0;  // the run's first chunk (index of its scales)
        it.n_kv = (c1 - c0) * (p.L / kKvTile);
        it.entry_begin[0] = it.entry_begin[1] = 0;
        it.mode = kTwoTiles;
        if (it.n_e[1] == 0 && it.n_kv >= 2) {
            it.mode = kSplit;
            it.n_e[1] = it.n_e[0];
            it.b0[1] = it.b0[0];
        }
    }
    if (it.mode == kSplit && it.n_kv < 2) {  // a single K/V tile cannot be divided: slot 0 alone
        it.mode = kTwoTiles;
        it.n_e[1] = 0;
    }
    if (it.mode == kSplit) {
        it.n_it[0] = (it.n_kv + 1) >> 1;
        it.n_it[1] = it.n_kv >> 1;
    } else {
        it.n_it[0] = it.n_kv;
        it.n_it[1] = it.n_e[1] > 0 ? it.n_kv : 0;
    }
    return it;
}

// a[t] for t in {0, 1} without indexing the array at run time (keeps it in registers)
template <class T>
__device__ __forceinline__ T pick(const T (&a)[2], int t)
{
    return t ? a[1] : a[0];
}

// Query buffers.  Slot u owns 32 KB: one full tile (two 64-column halves of 128 rows, 16 KB apart),
// or two 16 KB sub-buffers for tiles of at most 64 rows (halves 8 KB apart).  The MMA always reads
// 128 rows; behind a short tile it reads whatever follows in shared memory (the other sub-buffer,
// the next slot's buffer, the start of the K/V ring) -- rows of the accumulator that no thread
// looks at.  Consecutive short tiles of a slot alternate between the two sub-buffers, so the next
// item's rows are gathered while the MMAs still read this item's.
struct QUse {
    bool present;  // the slot gathers a query tile of its own in this unit
    bool small;    // at most 64 rows: one sub-buffer
    int sub;       // sub-buffer (small), else 0
};

__device__ __forceinline__ QUse q_use(const Unit& it, int u, int G, uint32_t& n_small)
{
    QUse q;
    q.present = it.n_kv > 0 && it.n_e[u] > 0 && !(it.mode == kSplit && u == 1);
    q.small = it.n_e[u] * G <= 64;
    q.sub = 0;
    if (q.present && q.small) q.sub = (n_small++) & 1;
    return q;
}

// Roles of the third warp group (after it has given registers up): TMA producer, MMA issuer and
// the two query-gather warps.
// Two E4M3 codes (low byte -> low half) widened to two f16 values; exact.
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t two_codes)
{
    uint32_t r;
    const unsigned short v = static_cast<unsigned short>(two_codes);
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(r) : "h"(v));
    return r;
}

// Four E4M3 codes (one 32-bit word) widened to two f16 pairs: lo = codes 0, 1; hi = codes 2, 3.
__device__ __forceinline__ void e4m3x4_to_f16x4(uint32_t four_codes, uint32_t& lo, uint32_t& hi)
{
    asm("{\n"
        ".reg .b16 c01, c23;\n"
        "mov.b32 {c01, c23}, %2;\n"
        "cvt.rn.f16x2.e4m3x2 %0, c01;\n"
        "cvt.rn.f16x2.e4m3x2 %1, c23;\n"
        "}\n"
        : "=r"(lo), "=r"(hi)
        : "r"(four_codes));
}

template <bool F>
__device__ __forceinline__ void other_roles(TcSmemT<F>& sm, const CUtensorMap& tm_k, const CUtensorMap& tm_v,
                                         const CUtensorMap& tm_q, const TcParams& p, const Schedule& sch, int G,
                                         int per_tile, uint32_t tmem, int warp, int lane)
{
    constexpr int kOp = TcSmemT<F>::kOp;
    volatile int* ab = &sm.abort_flag;
    const int n_pos = p.B * p.Hkv * p.k;  // routed: valid entries of seg_entries are below this

    if (warp == kLoadWarp) {
        // =========================== TMA producer ================================================
        // two tiles: K_0 V_0 K_1 V_1 ... of the item; split: the same; pair: the two items' tiles
        // alternate, K_0 V_0 of slot 0's item, K_0 V_0 of slot 1's, K_1 V_1 of slot 0's, ...
        if (lane == 0) {
            uint32_t ld = 0;  // loads issued so far, over all units
            bool ok = true;
            for (int unit = blockIdx.x; unit < sch.n_units && ok; unit += gridDim.x) {
                const Unit it = decode_unit(p, sch, unit, G, per_tile);
                const int n_loads = (it.mode == kPair ? 4 : 2) * it.n_kv;
                for (int x = 0; x < n_loads; ++x, ++ld) {
                    const CUtensorMap* tm = (x & 1) ? &tm_v : &tm_k;
                    const int vt = x >> 1;  // tile in ring order
                    const int y = it.mode == kPair
                        ? (int)(it.kv_row0[vt & 1] + (long long)(vt >> 1) * kKvTile)
                        : (int)(it.kv_row0[0] + (long long)vt * kKvTile);
                    if constexpr (F) {
                        // one box of 128 code rows x 128 bytes into the code ring
                        const uint32_t s = ld % kCodeStages;
                        if (ld >= kCodeStages &&
                            !mbar_wait(&sm.code_empty[s], ((ld / kCodeStages) - 1) & 1, ab)) {
                            ok = false;
                            break;
                        }
                        mbar_arrive_expect_tx(&sm.code_full[s], kCodeBytes);
                        tma_load_2d(sm.codes[s], tm, 0, y, &sm.code_full[s]);
                    } else {
                        const uint32_t s = ld % kOp;
                        if (ld >= kOp && !mbar_wait(&sm.empty[s], ((ld / kOp) - 1) & 1, ab)) {
                            ok = false;
                            break;
                        }
                        mbar_arrive_expect_tx(&sm.full[s], kTileBytes);
                        tma_load_2d(sm.kv[s], tm, 0, y, &sm.full[s]);
                        tma_load_2d(sm.kv[s] + kHalfBytes, tm, 64, y, &sm.full[s]);
                    }
                }
            }
            if (*ab) {
                // giving up: let the copies still in flight land before the CTA leaves
                volatile int never = 0;
                if constexpr (F) {
                    for (uint32_t x = ld > kCodeStages ? ld - kCodeStages : 0; x < ld; ++x)
                        mbar_wait(&sm.code_full[x % kCodeStages], (x / kCodeStages) & 1, &never);
                } else {
                    for (uint32_t x = ld > kOp ? ld - kOp : 0; x < ld; ++x)
                        mbar_wait(&sm.full[x % kOp], (x / kOp) & 1, &never);
                }
            }
        }
        __syncwarp();
    } else if (warp >= kGatherWarp0) {
        // =========================== query gather of slot u ======================================
        // Brings the tile's query rows into the 128-byte-swizzled K-major operand layout as soon
        // as the MMAs have stopped reading the (sub-)buffer: TMA row gathers, four rows per copy
        // (lane l owns tile rows 4l .. 4l+3), so the copies do not queue behind the softmax
        // groups' result stores in the load/store pipe.  Rows past the item's last one hold
        // stale or repeated query rows; their results are never written.
        // FP8 store: the rows come from an f16 copy of the queries; once the unit's gather is on its
        // way the same warp, together with the other gather warp (64 token rows each), widens the
        // unit's code tiles into the operand ring.
        const int u = warp - kGatherWarp0;
        uint32_t n_small = 0;
        uint32_t arrivals[2] = {0, 0};  // uses of sub-buffer 0 / 1 so far (a full tile uses both)
        uint64_t* last_full = nullptr;  // barrier and phase of the last gather, for the abort path
        uint32_t last_phase = 0;
        uint32_t fills[2] = {0, 0};     // gathers signalled on q_full[u][0 / 1] so far
        uint32_t cv = 0;                // FP8 store: code tiles widened so far, over all units
        bool ok = true;
        // FP8 store: widens this warp's half (64 token rows) of every code tile of the unit.  In
        // step i the warp handles token rows R .. R+3, R = 64u + 4i, every lane 16 codes (dims
        // 16j .. 16j+15) of one row.  Both tiles carry the 128-byte swizzle (phase = row % 8, which
        // is one of two values per lane: even and odd steps).  A quarter warp (what one 16-byte
        // shared-memory access serves at a time) holds dims 0..63 of one row and dims 64..127 of
        // the next, so that its eight loads and its eight stores each fall on eight different
        // 16-byte bank groups.  The 16 values are pieces 2 (j % 4) and 2 (j % 4) + 1 of the row's
        // half j / 4 of the operand tile.
        uint32_t w_src[2], w_dst[2];
        {
            const int qw = lane >> 3, t = (lane >> 2) & 1, m = lane & 3;
            const int a0 = 2 * (qw >> 1) + t, j = 4 * (t ^ (qw & 1)) + m, r0 = u * 64 + a0;
#pragma unroll
            for (int ph = 0; ph < 2; ++ph) {
                const int a = a0 ^ (4 * ph);
                w_src[ph] = r0 * 128 + ((j ^ a) << 4);
                w_dst[ph] = (j >> 2) * kHalfBytes + r0 * 128 + (((2 * (j & 3)) ^ a) << 4);
            }
        }
        auto widen_unit = [&](const Unit& it) {
            if constexpr (F) {
                const int n_loads = (it.mode == kPair ? 4 : 2) * it.n_kv;
                for (int x = 0; x < n_loads && ok; ++x, ++cv) {
                    const uint32_t cs = cv % kCodeStages, os = cv % kOp;
                    bool w = mbar_wait(&sm.code_full[cs], (cv / kCodeStages) & 1, ab);
                    if (w && cv >= kOp) w = mbar_wait(&sm.empty[os], ((cv / kOp) - 1) & 1, ab);
                    ok = __all_sync(0xffffffffu, w);
                    if (!ok) break;
                    const uint8_t* src = sm.codes[cs];
                    uint8_t* dst = sm.kv[os];
                    // 16 steps of four token rows; every address is a per-lane base (one for each
                    // of the two swizzle phases a lane's rows alternate between) plus a constant
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int ph = i & 1;
                        const uint4 c = *reinterpret_cast<const uint4*>(src + w_src[ph] + i * 512);
                        uint4 lo, hi;
                        e4m3x4_to_f16x4(c.x, lo.x, lo.y);
                        e4m3x4_to_f16x4(c.y, lo.z, lo.w);
                        e4m3x4_to_f16x4(c.z, hi.x, hi.y);
                        e4m3x4_to_f16x4(c.w, hi.z, hi.w);
                        *reinterpret_cast<uint4*>(dst + w_dst[ph] + i * 512) = lo;
                        *reinterpret_cast<uint4*>(dst + (w_dst[ph] ^ 16) + i * 512) = hi;
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(&sm.full[os]);
                        mbar_arrive(&sm.code_empty[cs]);
                    }
                }
            }
        };
        for (int unit = blockIdx.x; unit < sch.n_units && ok; unit += gridDim.x) {
            const Unit it = decode_unit(p, sch, unit, G, per_tile);
            const QUse qu = q_use(it, u, G, n_small);
            if (!qu.present) {
                widen_unit(it);
                continue;
            }
            int rr[4];  // global query rows of tile rows 4 * lane .. 4 * lane + 3
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                const int i = 4 * lane + m;
                rr[m] = 0;
                if (i < it.n_e[u] * G) {
                    const int e = i / G, g = i % G;
                    int b;
                    if (!p.dense) {
                        const int pp = __ldg(p.seg_entries + it.entry_begin[u] + e);
                        b = (unsigned)pp < (unsigned)n_pos ? pp / (p.k * p.Hkv) : 0;
                    } else {
                        b = it.b0[u] + e;
                    }
                    rr[m] = b * p.Hq + it.h[u] * G + g;
                }
            }
            // the MMAs that read what is about to be overwritten must have completed
#pragma unroll
            for (int sb = 0; sb < 2; ++sb) {
                if (qu.small && sb != qu.sub) continue;
                if (arrivals[sb] > 0 && ok)
                    ok = __all_sync(0xffffffffu, mbar_wait(&sm.q_free[u][sb], (arrivals[sb] - 1) & 1, ab));
                ++arrivals[sb];
            }
            if (!ok) break;
            uint64_t* bar = &sm.q_full[u][qu.sub];
            last_full = bar;
            last_phase = fills[qu.sub]++ & 1;
            // only the groups of four rows that hold a query row are copied; the tile rows after
            // them keep whatever an earlier item left there
            const int n_groups = (it.n_e[u] * G + 3) >> 2;
            if (lane == 0) mbar_arrive_expect_tx(bar, n_groups * 2 * (4 * 128));
            __syncwarp();
            if (lane < n_groups) {
                uint8_t* dst = sm.q[u] + (qu.small ? qu.sub * kSubBytes : 0) + lane * (4 * 128);
                const int half = qu.small ? kSubBytes / 2 : kHalfBytes;
                tma_gather4_2d(dst, &tm_q, 0, rr[0], rr[1], rr[2], rr[3], bar);
                tma_gather4_2d(dst + half, &tm_q, 64, rr[0], rr[1], rr[2], rr[3], bar);
            }
            widen_unit(it);
        }
        if (*ab && last_full != nullptr) {
            // giving up: let the copies still in flight land before the CTA leaves
            volatile int never = 0;
            mbar_wait(last_full, last_phase, &never);
        }
    } else {
        // =========================== MMA issuer ===================================================
        if (lane == 0) {
            // bf16 operands, or (FP8 store) f16 operands: Q and P are then f16 as well
            const uint32_t id_qk = F ? idesc_f16_f32(128, kKvTile, false) : idesc_bf16_f32(128, kKvTile, false);
            const uint32_t id_pv = F ? idesc_f16_f32(128, kD, true) : idesc_bf16_f32(128, kD, true);
            // Operand descriptors differ only in their start-address field (low word, units of 16
            // bytes): build the constant parts once and add tile offsets per instruction, so that
            // issuing an MMA costs a handful of integer instructions.
            const uint64_t d_kmajor = smem_desc_sw128(0, 16, 1024);          // Q and K tiles
            const uint64_t d_nmajor = smem_desc_sw128(0, kHalfBytes, 1024);  // V tiles
            const uint32_t hi_k = static_cast<uint32_t>(d_kmajor >> 32);
            const uint32_t hi_n = static_cast<uint32_t>(d_nmajor >> 32);
            const uint32_t lo_q = static_cast<uint32_t>(d_kmajor) + (smem_u32(sm.q[0]) >> 4);
            const uint32_t lo_k = static_cast<uint32_t>(d_kmajor) + (smem_u32(sm.kv[0]) >> 4);
            const uint32_t lo_v = static_cast<uint32_t>(d_nmajor) + (smem_u32(sm.kv[0]) >> 4);
            auto desc = [](uint32_t hi, uint32_t lo) { return (static_cast<uint64_t>(hi) << 32) | lo; };
            // S_t = Q K^T, Q at descriptor address qa with its halves qh apart, K in ring slot s:
            // 8 steps of 16 head-dimension columns
            auto issue_qk = [&](int tq, uint32_t qa, uint32_t qh, uint32_t s) {
                const uint32_t b = lo_k + s * (kTileBytes >> 4);
#pragma unroll
                for (int ks = 0; ks < kD / 16; ++ks) {
                    const uint32_t sub = ((ks & 3) * 32) >> 4;
                    mma_ss(tmem + tq * 128, desc(hi_k, qa + (ks >> 2) * qh + sub),
                           desc(hi_k, b + (((ks >> 2) * kHalfBytes) >> 4) + sub), id_qk, ks > 0);
                }
            };
            // O_t += P_t V, V in ring slot s: 8 steps of 16 tokens
            auto issue_pv = [&](int tq, uint32_t s, bool acc) {
                const uint32_t b = lo_v + s * (kTileBytes >> 4);
#pragma unroll
                for (int ks = 0; ks < kKvTile / 16; ++ks)
                    mma_ts(tmem + 256 + tq * 128, tmem + tq * 128 + ks * 8,
                           desc(hi_n, b + ks * (2048 >> 4)), id_pv, acc || ks > 0);
            };
            uint32_t ld0 = 0;               // ring position of the unit's first load
            uint32_t pc[2] = {0, 0};
            uint32_t n_small[2] = {0, 0}, fills[2][2] = {{0, 0}, {0, 0}};
            int q_reads[2] = {0, 0};        // score MMAs of the unit that still have to read q[u]
            bool ok = true;
            for (int unit = blockIdx.x; unit < sch.n_units && ok; unit += gridDim.x) {
                const Unit it = decode_unit(p, sch, unit, G, per_tile);
                QUse qu[2];
                uint32_t qa[2], qh[2];
                for (int u = 0; u < 2; ++u) {
                    qu[u] = q_use(it, u, G, n_small[u]);
                    qa[u] = lo_q + ((u * kTileBytes + (qu[u].small ? qu[u].sub * kSubBytes : 0)) >> 4);
                    qh[u] = (qu[u].small ? kSubBytes / 2 : kHalfBytes) >> 4;
                }
                // ring position of the K tile of slot tq's x-th step (its V tile is the next one),
                // and whether that slot is the tile's last reader
                auto k_load = [&](int tq, int x) {
                    return ld0 + 2 * (it.mode == kTwoTiles ? x : 2 * x + tq);
                };
                auto last_reader = [&](int tq) {
                    return it.mode != kTwoTiles || it.n_it[1] == 0 || tq == 1;
                };
                auto wait_load = [&](uint32_t g) {
                    return mbar_wait(&sm.full[g % kOp], (g / kOp) & 1, ab);
                };
                auto issue_scores = [&](int tq, uint32_t s) {
                    const int u = it.mode == kSplit ? 0 : tq;
                    issue_qk(tq, qa[u], qh[u], s);
                    tc_commit(&sm.s_full[tq]);
                    if (--q_reads[u] == 0) {  // the gather warp may refill the (sub-)buffer
                        if (qu[u].small) {
                            tc_commit(&sm.q_free[u][qu[u].sub]);
                        } else {
                            tc_commit(&sm.q_free[u][0]);
                            tc_commit(&sm.q_free[u][1]);
                        }
                    }
                };
                q_reads[0] = it.mode == kSplit ? it.n_kv : it.n_it[0];
                q_reads[1] = it.mode == kSplit ? 0 : it.n_it[1];
                for (int u = 0; u < 2 && ok; ++u) {
                    if (!qu[u].present) continue;
                    uint64_t* bar;
                    bar = &sm.q_full[u][qu[u].sub];
                    ok = mbar_wait(bar, fills[u][qu[u].sub]++ & 1, ab);
                }
                // first scores of both slots
                for (int tq = 0; tq < 2 && ok; ++tq) {
                    if (it.n_it[tq] == 0) continue;
                    const uint32_t g = k_load(tq, 0);
                    ok = wait_load(g);
                    if (!ok) break;
                    tc_fence_after_sync();
                    issue_scores(tq, g % kOp);
                    if (last_reader(tq)) tc_commit(&sm.empty[g % kOp]);
                }
                for (int x = 0; x < it.n_it[0] && ok; ++x) {
                    for (int tq = 0; tq < 2 && ok; ++tq) {
                        if (x >= it.n_it[tq]) continue;
                        const uint32_t gv = k_load(tq, x) + 1;
                        ok = wait_load(gv) && mbar_wait(&sm.p_full[tq], pc[tq] & 1, ab);
                        if (!ok) break;
                        ++pc[tq];
                        tc_fence_after_sync();
                        issue_pv(tq, gv % kOp, x > 0);
                        if (last_reader(tq)) tc_commit(&sm.empty[gv % kOp]);
                        if (x + 1 < it.n_it[tq]) {
                            const uint32_t gk = k_load(tq, x + 1);
                            ok = wait_load(gk);
                            if (!ok) break;
                            tc_fence_after_sync();
                            issue_scores(tq, gk % kOp);
                            if (last_reader(tq)) tc_commit(&sm.empty[gk % kOp]);
                        } else {
                            tc_commit(&sm.o_full[tq]);
                        }
                    }
                }
                ld0 += (it.mode == kPair ? 4 : 2) * it.n_kv;
            }
        }
        __syncwarp();
    }
}

// FP8 shared store: the step's queries as f16 (the operand type of its MMAs), eight values per
// thread; round to nearest.
__global__ void __launch_bounds__(256)
q_to_f16_kernel(const uint4* __restrict__ q, uint4* __restrict__ q16, long long n_vec)
{
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_vec) return;
    uint4 v = q[i];
    auto cv = [](uint32_t w) {
        const __half2 h = __floats2half2_rn(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
        return *reinterpret_cast<const uint32_t*>(&h);
    };
    v.x = cv(v.x);
    v.y = cv(v.y);
    v.z = cv(v.z);
    v.w = cv(v.w);
    q16[i] = v;
}

template <bool F>
__global__ void __launch_bounds__(kThreads, 1)
shared_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                 const __grid_constant__ CUtensorMap tm_q, const TcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    TcSmemT<F>& sm = *reinterpret_cast<TcSmemT<F>*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                                    ~static_cast<uintptr_t>(1023));
    constexpr int kOp = TcSmemT<F>::kOp;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = p.Hq / p.Hkv;
    const int per_tile = kBigTileRows / G;  // requests per query tile
    const Schedule sch = make_schedule(p);
    if ((int)blockIdx.x >= sch.n_units) return;

    // ---- set-up: barriers, tensor memory --------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < kOp; ++s) {
            mbar_init(&sm.full[s], F ? 2 : 1);  // FP8 store: one arrival per widening warp
            mbar_init(&sm.empty[s], 1);
        }
        if constexpr (F) {
            for (int s = 0; s < kCodeStages; ++s) {
                mbar_init(&sm.code_full[s], 1);
                mbar_init(&sm.code_empty[s], 2);
            }
        }
        for (int u = 0; u < 2; ++u) {
            for (int sb = 0; sb < 2; ++sb) {
                mbar_init(&sm.q_full[u][sb], 1);
                mbar_init(&sm.q_free[u][sb], 1);
            }
            mbar_init(&sm.s_full[u], 1);
            mbar_init(&sm.p_full[u], 128);
            mbar_init(&sm.o_full[u], 1);
        }
        mbar_init(&sm.x_full, 128);
        mbar_init(&sm.x_free, 128);
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
        tma_prefetch_desc(&tm_q);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = sm.tmem_base;
    volatile int* ab = &sm.abort_flag;

    if (warp < 8) {
        // =========================== softmax group of slot t =====================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
        const int t = warp >> 2;
        const int i = tid & 127;  // tile row = TMEM lane
        const uint32_t lane_sel = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem + lane_sel + t * 128;        // S_t, and P_t over its columns
        const uint32_t t_o = tmem + lane_sel + 256 + t * 128;  // O_t
        const uint32_t t_o_other = tmem + lane_sel + 256 + (1 - t) * 128;
        const int n_pos = p.B * p.Hkv * p.k;
        uint32_t sc = 0, oc[2] = {0, 0}, xc = 0;  // barrier phases completed before this unit
        bool alive = true;
        for (int unit = blockIdx.x; unit < sch.n_units && alive; unit += gridDim.x) {
            const Unit it = decode_unit(p, sch, unit, G, per_tile);
            const int n_it = pick(it.n_it, t);
            const bool split = it.mode == kSplit;
            const uint32_t ph_o[2] = {oc[0] & 1u, oc[1] & 1u}, ph_x = xc & 1u;
            oc[0] += it.n_it[0] > 0;
            oc[1] += it.n_it[1] > 0;
            xc += split;
            // FP8 store: a chunk's key scale joins the softmax scale of its tiles; its value scale
            // joins the final normalisation (routed mode: one chunk per item) or, relative to the
            // scale of the run's first chunk, the P tile (dense mode: a run of chunks per item).
            // The running maximum is then kept in scaled log2 units, so that it carries across
            // chunks; with the bf16 store it stays in raw score units (`conv` converts).
            const int key0 = pick(it.key, t);
            const float v_ref = F ? __ldg(p.v_scale + key0) : 1.f;
            float ksc = F ? __ldg(p.k_scale + key0) : 1.f;
            float p_mul = 1.f;  // dense FP8: value scale of the tile's chunk / v_ref
            float sl2 = p.scale * kLog2e * ksc;
            const float conv = F ? 1.f : sl2;
            const int tiles_per_chunk = p.L / kKvTile;
            const int n_rows = pick(it.n_e, t) * G;
            // a warp none of whose rows exists skips the arithmetic (every row of the products
            // depends on its own query row only), but keeps every barrier in step
            const bool warp_live = (warp & 3) * 32 < n_rows;
            long long my_r = -1;
            int my_slot = 0;
            if (i < n_rows) {
                const int e = i / G, g = i % G;
                int b = -1;
                if (!p.dense) {
                    const int pp = __ldg(p.seg_entries + pick(it.entry_begin, t) + e);
                    if ((unsigned)pp < (unsigned)n_pos) {
                        my_slot = pp % p.k;
                        b = pp / (p.k * p.Hkv);
                    } else {
                        atomicMin(p.status, (int)MOSKA_ERR_INVALID_ARG);  // not a position of this batch
                    }
                } else {
                    my_slot = it.slot_dense;
                    b = pick(it.b0, t) + e;
                }
                if (b >= 0) my_r = (long long)b * p.Hq + pick(it.h, t) * G + g;
            }
            if (it.n_kv == 0) {  // dense mode: a trailing run without chunks
                if (my_r >= 0) {
                    float4* o = reinterpret_cast<float4*>(p.o_part + (my_r * p.n_slots + my_slot) * kD);
                    for (int d = 0; d < kD / 4; ++d) o[d] = make_float4(0.f, 0.f, 0.f, 0.f);
                    p.lse_part[my_r * p.n_slots + my_slot] = -INFINITY;
                }
                continue;
            }
            float m_ref = -INFINITY, l_sum = 0.f;
            for (int j = 0; j < n_it; ++j) {
                if constexpr (F) {
                    if (p.dense) {  // scales of the chunk this tile lies in (asked for before the wait)
                        const int tile = split ? 2 * j + t : j;
                        const int c = key0 + tile / tiles_per_chunk;
                        ksc = __ldg(p.k_scale + c);
                        p_mul = __ldg(p.v_scale + c) / v_ref;
                        sl2 = p.scale * kLog2e * ksc;
                    }
                }
                alive = __all_sync(0xffffffffu, mbar_wait(&sm.s_full[t], sc & 1, ab));
                if (!alive) break;
                ++sc;
                if (warp_live) {
                    tc_fence_after_sync();
                    // the row's 128 scores: four loads in flight, one wait
                    uint32_t r[4][32];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld32(t_s + c * 32, r[c]);
                    tmem_ld_wait();
                    // eight independent maximum chains of three-input maxima, then a tree
                    float mxs[8];
#pragma unroll
                    for (int x = 0; x < 8; ++x)
                        mxs[x] = fmaxf(__uint_as_float(r[0][2 * x]), __uint_as_float(r[0][2 * x + 1]));
#pragma unroll
                    for (int x = 8; x < 16; ++x)
                        mxs[x & 7] = fmax3(mxs[x & 7], __uint_as_float(r[0][2 * x]), __uint_as_float(r[0][2 * x + 1]));
#pragma unroll
                    for (int c = 1; c < 4; ++c)
#pragma unroll
                        for (int x = 0; x < 16; ++x)
                            mxs[x & 7] = fmax3(mxs[x & 7], __uint_as_float(r[c][2 * x]), __uint_as_float(r[c][2 * x + 1]));
                    float mx = fmaxf(fmaxf(fmaxf(mxs[0], mxs[1]), fmaxf(mxs[2], mxs[3])),
                                     fmaxf(fmaxf(mxs[4], mxs[5]), fmaxf(mxs[6], mxs[7])));
                    if constexpr (F) mx *= sl2;  // scaled log2 units
                    if (j == 0) {
                        m_ref = mx;
                    } else {
                        // rows that do not exist hold arbitrary bits: they never ask for a rescale
                        const bool need = i < n_rows && (mx - m_ref) * conv > kRescaleThreshold;
                        if (__any_sync(0xffffffffu, need)) {
                            // every MMA issued before S_t(j), PV_t(j-1) included, has completed
                            const float alpha = need ? fast_exp2((m_ref - mx) * conv) : 1.f;
                            if (need) m_ref = mx;
                            l_sum *= alpha;
#pragma unroll 1
                            for (int c = 0; c < 4; ++c) {
                                uint32_t o_acc[32];
                                tmem_ld32(t_o + c * 32, o_acc);
                                tmem_ld_wait();
#pragma unroll
                                for (int x = 0; x < 32; ++x)
                                    o_acc[x] = __float_as_uint(__uint_as_float(o_acc[x]) * alpha);
                                tmem_st32(t_o + c * 32, o_acc);
                            }
                        }
                    }
                    // P = exp2((S - m_ref) * scale * log2 e) as bf16, written over the columns of S
                    const float2 sl2_2 = make_float2(sl2, sl2);
                    const float2 nmb_2 = make_float2(-m_ref * conv, -m_ref * conv);
                    const float2 pmul_2 = make_float2(p_mul, p_mul);
                    float2 ls[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};  // partial row sums
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t pk[16];
#pragma unroll
                        for (int x = 0; x < 16; ++x) {
                            const float2 e = ffma2(make_float2(__uint_as_float(r[c][2 * x]),
                                                               __uint_as_float(r[c][2 * x + 1])),
                                                   sl2_2, nmb_2);
                            float2 pr;
                            pr.x = fast_exp2(e.x);
                            pr.y = fast_exp2(e.y);
                            ls[x & 1] = fadd2(ls[x & 1], pr);
                            if constexpr (F) {
                                const float2 ps = ffma2(pr, pmul_2, make_float2(0.f, 0.f));
                                const __half2 h2 = __floats2half2_rn(ps.x, ps.y);
                                pk[x] = *reinterpret_cast<const uint32_t*>(&h2);
                            } else {
                                const __nv_bfloat162 b2 = __floats2bfloat162_rn(pr.x, pr.y);
                                pk[x] = *reinterpret_cast<const uint32_t*>(&b2);
                            }
                        }
                        tmem_st16(t_s + c * 16, pk);
                    }
                    l_sum += (ls[0].x + ls[0].y) + (ls[1].x + ls[1].y);
                    tmem_st_wait();
                }
                tc_fence_before_sync();
                mbar_arrive(&sm.p_full[t]);
            }
            if (!alive) break;

            // ---- epilogue: normalised partial output and log-sum-exp of the row -----------------
            if (split && t == 1) {
                // publish this slot's statistics; slot 0's group combines and writes
                sm.stat_m[i] = m_ref;
                sm.stat_l[i] = l_sum;
                mbar_arrive(&sm.x_full);
                alive = __all_sync(0xffffffffu, mbar_wait(&sm.x_free, ph_x, ab));
                continue;
            }
            if (n_it == 0) continue;  // slot 1 of a unit with a single tile and a single K/V tile
            alive = __all_sync(0xffffffffu, mbar_wait(&sm.o_full[t], ph_o[t], ab));
            if (!alive) break;
            float a_mine = 1.f, a_other = 0.f, m_all = m_ref, den = l_sum;
            if (split) {
                alive = __all_sync(0xffffffffu, mbar_wait(&sm.o_full[1], ph_o[1], ab)) &&
                        __all_sync(0xffffffffu, mbar_wait(&sm.x_full, ph_x, ab));
                if (!alive) break;
                const float m1 = sm.stat_m[i], l1 = sm.stat_l[i];
                m_all = fmaxf(m_ref, m1);
                a_mine = fast_exp2((m_ref - m_all) * conv);
                a_other = fast_exp2((m1 - m_all) * conv);
                den = a_mine * l_sum + a_other * l1;
            }
            if (warp_live) {
                tc_fence_after_sync();
                const float inv = v_ref / den;
                a_mine *= inv;
                a_other *= inv;
                float4* o = my_r >= 0
                    ? reinterpret_cast<float4*>(p.o_part + (my_r * p.n_slots + my_slot) * kD)
                    : nullptr;
                // the whole accumulator row: four loads in flight, one wait (two rounds when a
                // second accumulator has to be folded in)
                uint32_t r[4][32];
#pragma unroll
                for (int c = 0; c < 4; ++c) tmem_ld32(t_o + c * 32, r[c]);
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int x = 0; x < 32; ++x) r[c][x] = __float_as_uint(__uint_as_float(r[c][x]) * a_mine);
                if (split) {
#pragma unroll
                    for (int hv = 0; hv < 2; ++hv) {
                        uint32_t r2[2][32];
                        tmem_ld32(t_o_other + hv * 64, r2[0]);
                        tmem_ld32(t_o_other + hv * 64 + 32, r2[1]);
                        tmem_ld_wait();
#pragma unroll
                        for (int c = 0; c < 2; ++c)
#pragma unroll
                            for (int x = 0; x < 32; ++x)
                                r[2 * hv + c][x] = __float_as_uint(
                                    fmaf(__uint_as_float(r2[c][x]), a_other, __uint_as_float(r[2 * hv + c][x])));
                    }
                }
                if (o != nullptr) {
                    // 32-byte stores: every instruction writes whole sectors of the row
#pragma unroll
                    for (int c = 0; c < 4; ++c)
#pragma unroll
                        for (int x = 0; x < 4; ++x)
                            st_global_v8(reinterpret_cast<float*>(o) + c * 32 + x * 8,
                                         reinterpret_cast<const float*>(&r[c][8 * x]));
                    p.lse_part[my_r * p.n_slots + my_slot] = (F ? m_all * kLn2 : m_all * p.scale) + logf(den);
                }
            }
            if (split) {
                tc_fence_before_sync();
                mbar_arrive(&sm.x_free);  // O_1 and the statistics may be overwritten
            }
        }
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
        other_roles<F>(sm, tm_k, tm_v, tm_q, p, sch, G, per_tile, tmem, warp, lane);
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

// The [rows][128] bf16 query matrix for row gathers: boxes of one row x 64 columns.
int make_q_map(CUtensorMap* tm, const uint16_t* base, long long rows)
{
    EncodeTiledFn enc = nullptr;
    MOSKA_TRY_STATUS(encoder(&enc));
    const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kD * 2};
    const cuuint32_t box[2] = {64, 1};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                           const_cast<uint16_t*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(MOSKA_ERR_CUDA, "cuTensorMapEncodeTiled failed for q (%d)", (int)r);
    return MOSKA_OK;
}

}  // namespace

bool shared_tc_supported(const moska_shape* s) { return s->D == kD && s->L % kKvTile == 0; }

namespace {

// [rows][128] matrix of E4M3 codes, loaded in boxes of 128 rows x 128 bytes with the 128-byte swizzle.
int make_code_map(CUtensorMap* tm, const uint8_t* base, long long rows)
{
    EncodeTiledFn enc = nullptr;
    MOSKA_TRY_STATUS(encoder(&enc));
    const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)kD};
    const cuuint32_t box[2] = {(cuuint32_t)kD, (cuuint32_t)kKvTile};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(base), dims, strides,
                           box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(MOSKA_ERR_CUDA, "cuTensorMapEncodeTiled failed for FP8 codes (%d)", (int)r);
    return MOSKA_OK;
}

// Common part of the two launchers.  k8 / v8 != nullptr selects the FP8 shared store.
int launch_tc(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared, const uint8_t* k8,
              const uint8_t* v8, const float* k_scale, const float* v_scale, const int32_t* seg_entries,
              float* o_part, float* lse_part, float scale, const moska_shape* s, void* ws, bool dense,
              int max_ctas, cudaStream_t st)
{
    const bool fp8 = k8 != nullptr;
    const int G = s->Hq / s->Hkv;
    const int per_cta = 2 * (kBigTileRows / G);
    long long grid;  // upper bound of the number of work items
    TcParams p{};
    if (dense) {
        grid = (long long)s->Hkv * s->shared_slots * ((s->B + per_cta - 1) / per_cta);
        p.n_items_dense = (int)grid;
    } else {
        const WsLayout lay = ws_layout(s);
        grid = lay.max_big + lay.max_small;
        p.hdr = reinterpret_cast<const WsHeader*>(ws);
        p.items = reinterpret_cast<const TileItem*>(static_cast<const char*>(ws) + lay.off_big);
        p.singles = reinterpret_cast<const TileItem*>(static_cast<const char*>(ws) + lay.off_small);
    }
    if (grid == 0) return MOSKA_OK;
    if (grid > 0x7fffffffLL) return fail(MOSKA_ERR_UNSUPPORTED, "shared attention grid too large");
    // persistent CTAs, one per SM, each walking the item list with the grid as its stride
    int dev = 0, n_sms = 0;
    MOSKA_CUDA_TRY(cudaGetDevice(&dev));
    MOSKA_CUDA_TRY(cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev));
    if (grid > n_sms) grid = n_sms;
    if (max_ctas > 0 && grid > max_ctas) grid = max_ctas;  // the caller keeps the other SMs for another kernel
    const long long kv_rows = (long long)s->Hkv * s->C * s->L;
    if (kv_rows > 0x7fffffffLL) return fail(MOSKA_ERR_UNSUPPORTED, "shared store exceeds 2^31 tokens");
    CUtensorMap tm_k, tm_v, tm_q;
    if (fp8) {
        MOSKA_TRY_STATUS(make_code_map(&tm_k, k8, kv_rows));
        MOSKA_TRY_STATUS(make_code_map(&tm_v, v8, kv_rows));
    } else {
        MOSKA_TRY_STATUS(make_kv_map(&tm_k, k_shared, kv_rows));
        MOSKA_TRY_STATUS(make_kv_map(&tm_v, v_shared, kv_rows));
    }
    const uint16_t* q_rows = q;
    if (fp8) {
        // the gathers read an f16 copy of the queries kept in the workspace
        const long long n_vec = (long long)s->B * s->Hq * kD / 8;
        uint16_t* q16 = reinterpret_cast<uint16_t*>(static_cast<char*>(ws) + ws_layout(s).off_q16);
        q_to_f16_kernel<<<(unsigned)((n_vec + 255) / 256), 256, 0, st>>>(
            reinterpret_cast<const uint4*>(q), reinterpret_cast<uint4*>(q16), n_vec);
        MOSKA_LAUNCH_CHECK("q_to_f16_kernel");
        q_rows = q16;
    }
    MOSKA_TRY_STATUS(make_q_map(&tm_q, q_rows, (long long)s->B * s->Hq));
    int* status = nullptr;
    MOSKA_TRY_STATUS(status_word(&status));
    p.q = q;
    p.seg_entries = seg_entries;
    p.k_scale = k_scale;
    p.v_scale = v_scale;
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
    if (fp8) {
        const int smem = (int)sizeof(TcSmemT<true>) + 1024;
        MOSKA_CUDA_TRY(cudaFuncSetAttribute(shared_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        shared_tc_kernel<true><<<(unsigned)grid, kThreads, smem, st>>>(tm_k, tm_v, tm_q, p);
    } else {
        const int smem = (int)sizeof(TcSmemT<false>) + 1024;
        MOSKA_CUDA_TRY(cudaFuncSetAttribute(shared_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
        shared_tc_kernel<false><<<(unsigned)grid, kThreads, smem, st>>>(tm_k, tm_v, tm_q, p);
    }
    MOSKA_LAUNCH_CHECK("shared_tc_kernel");
    return MOSKA_OK;
}

}  // namespace

int launch_shared_tc(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                     const int32_t* seg_entries, float* o_part, float* lse_part, float scale,
                     const moska_shape* s, void* ws, bool dense, int max_ctas, cudaStream_t st)
{
    return launch_tc(q, k_shared, v_shared, nullptr, nullptr, nullptr, nullptr, seg_entries, o_part, lse_part,
                     scale, s, ws, dense, max_ctas, st);
}

int launch_shared_tc_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8, const float* k_scale,
                         const float* v_scale, const int32_t* seg_entries, float* o_part, float* lse_part,
                         float scale, const moska_shape* s, void* ws, bool dense, int max_ctas,
                         cudaStream_t st)
{
    return launch_tc(q, nullptr, nullptr, k8, v8, k_scale, v_scale, seg_entries, o_part, lse_part, scale, s,
                     ws, dense, max_ctas, st);
}

// Measured on B200: an item costs about 6 us of fill, drain and epilogue plus 2.2 us per K/V
// tile with two query tiles (1.1 us with one, split between the two slots).
double shared_tc_cost_sm_ms(const moska_shape* s, bool dense)
{
    const int G = s->Hq / s->Hkv;
    const int per_cta = 2 * (kBigTileRows / G);
    double items, n_kv;
    bool two_tiles;
    if (dense) {
        items = (double)s->Hkv * s->shared_slots * ((s->B + per_cta - 1) / per_cta);
        n_kv = (double)((s->C + s->shared_slots - 1) / s->shared_slots) * (s->L / kKvTile);
        two_tiles = s->B * G > kBigTileRows;
    } else {
        const double P = (double)s->B * s->Hkv * s->k;
        const double segs = P < (double)s->Hkv * s->C ? P : (double)s->Hkv * s->C;
        items = 0.75 * (P / per_cta + segs);
        n_kv = s->L / kKvTile;
        two_tiles = P / segs > kBigTileRows / G;
    }
    return items * (6.0 + (two_tiles ? 2.2 : 1.1) * n_kv) * 1e-3;
}

}  // namespace moska
