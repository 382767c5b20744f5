// Shared KV Attention over an FP8 shared store, segments of at most 8 query rows (Section III-A
// with the KV precision of Section IV): one or two requests on a chunk are served best by reading
// the chunk's codes straight through, on the streaming block of f8_stream.cuh with the chunk's one
// key scale and one value scale.  The CTAs walk the grouping pass's list of 8-row tiles.
#include "common.cuh"
#include "f8_stream.cuh"

namespace moska {
namespace {
using namespace f8stream;

__global__ void __launch_bounds__(kThreads, 3)
shared_small_fp8_kernel(const uint16_t* __restrict__ q, const uint8_t* __restrict__ k8,
                        const uint8_t* __restrict__ v8, const float* __restrict__ k_scale,
                        const float* __restrict__ v_scale, const int32_t* __restrict__ seg_entries,
                        const WsHeader* __restrict__ hdr, const TileItem* __restrict__ items,
                        float* __restrict__ o_part, float* __restrict__ lse_part, int* __restrict__ status,
                        float scale, int B, int Hq, int Hkv, int C, int L, int k, int n_slots)
{
    extern __shared__ __align__(128) unsigned char ring[];
    __shared__ TileRows<1> rows;
    const int G = Hq / Hkv;
    const int n_pos = B * Hkv * k;  // valid entries of seg_entries are below this
    // the host only knows an upper bound of the list's length: the grid is the stride
    const int n_tiles = hdr->n_tiny_tiles;
    for (int tile = blockIdx.x; tile < n_tiles; tile += gridDim.x) {
        __syncthreads();  // the previous tile's row table and combine buffers are done with
        const TileItem it = items[tile];
        const int h = it.key / C;
        if (threadIdx.x < 8) {
            const int j = threadIdx.x;
            const uint16_t* qr = nullptr;
            float* orow = nullptr;
            float* lrow = nullptr;
            if (j < it.n_entries * G) {
                const int p = seg_entries[it.entry_begin + j / G];
                if ((unsigned)p < (unsigned)n_pos) {
                    const int slot = p % k, b = p / (k * Hkv);
                    const int64_t r = (int64_t)b * Hq + h * G + j % G;
                    qr = q + r * kD8;
                    orow = o_part + (r * n_slots + slot) * kD8;
                    lrow = lse_part + r * n_slots + slot;
                } else {
                    atomicMin(status, (int)MOSKA_ERR_INVALID_ARG);  // not a position of this batch
                }
            }
            rows.q[j] = qr;
            rows.o[j] = orow;
            rows.lse[j] = lrow;
        }
        __syncthreads();
        F8Source src;
        src.k_base = k8 + (int64_t)it.key * L * kD8;
        src.v_base = v8 + (int64_t)it.key * L * kD8;
        src.tok_stride = kD8;
        src.ks_base = src.vs_base = nullptr;
        src.scale_stride = 0;
        src.ksc = __ldg(k_scale + it.key);
        src.vsc = __ldg(v_scale + it.key);
        f8_attend_stream<false, false>(rows, src, 0, L, L, 1, G, it.n_entries * G, scale, ring);
    }
}

}  // namespace

int launch_shared_small_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8, const float* k_scale,
                            const float* v_scale, const int32_t* seg_entries, float* o_part,
                            float* lse_part, float scale, const moska_shape* s, void* ws, cudaStream_t st)
{
    const WsLayout lay = ws_layout(s);
    if (lay.tiny_entries == 0) return MOSKA_OK;  // G > 8: the grouping pass forms no 8-row tiles
    const long long P = (long long)s->B * s->Hkv * s->k;
    const long long segs = P < lay.n_keys ? P : lay.n_keys;  // the list's capacity
    int dev = 0, n_sms = 0;
    MOSKA_CUDA_TRY(cudaGetDevice(&dev));
    MOSKA_CUDA_TRY(cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev));
    // resident CTAs (3 per SM) a few times over; they stride through the device-side list
    const long long grid = segs < 12LL * n_sms ? segs : 12LL * n_sms;
    if (grid == 0) return MOSKA_OK;
    int* status = nullptr;
    MOSKA_TRY_STATUS(status_word(&status));
    const WsHeader* hdr = reinterpret_cast<const WsHeader*>(ws);
    const TileItem* items = reinterpret_cast<const TileItem*>(static_cast<const char*>(ws) + lay.off_tiny);
    MOSKA_CUDA_TRY(cudaFuncSetAttribute(shared_small_fp8_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        kF8RingBytes));
    shared_small_fp8_kernel<<<(unsigned)grid, kThreads, kF8RingBytes, st>>>(
        q, k8, v8, k_scale, v_scale, seg_entries, hdr, items, o_part, lse_part, status, scale, s->B, s->Hq,
        s->Hkv, s->C, s->L, s->k, s->shared_slots + s->n_unique_splits);
    MOSKA_LAUNCH_CHECK("shared_small_fp8_kernel");
    return MOSKA_OK;
}

}  // namespace moska
