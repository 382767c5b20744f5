/*
 * moska.h -- C ABI of the MoSKA decode-attention hot path for NVIDIA B200 (sm_100a).
 *
 * MoSKA (Mixture of Shared KV Attention) splits the KV context of a batch of decoding requests
 * into a large SHARED store, partitioned into chunks that many requests attend to, and a
 * per-request UNIQUE KV.  One decode step of one attention layer is
 *
 *   route  ->  group_by_chunk  ->  { shared_attn  ||  unique_attn }  ->  merge
 *
 * (Section III-A "Shared KV Attention", Section III-B "The MoSKA Architecture", Fig. 2.)
 *
 * Conventions that hold for every entry point
 * -------------------------------------------
 *  * All tensor arguments are DEVICE pointers owned by the caller, unless a parameter is
 *    documented as a host pointer.  The library never allocates, frees or keeps a pointer
 *    after the call returns.  Scratch memory comes from a caller-provided workspace.
 *  * Every call only enqueues work on `stream` and returns without synchronising, and nothing
 *    produced on the device is read back by the host.  The exceptions say so at their
 *    declaration: moska_device_status and the *_host forms of the step wait for the device.
 *  * bf16 tensors are passed as `const uint16_t*` (raw bfloat16 bit patterns).
 *  * Symbols: B requests, Hq query heads, Hkv KV heads, G = Hq / Hkv (1..8), D head dimension
 *    (64 or 128), C shared chunks of L tokens each, k chunks routed per (request, KV head).
 *    Query row r = b * Hq + hq; its KV head is h = hq / G.
 *  * Partial results: every query row owns `n_slots = shared_slots + n_unique_splits` slots.
 *        o_part   float [B][Hq][n_slots][D]   softmax-normalised partial output
 *        lse_part float [B][Hq][n_slots]      natural-log sum of exp(scale * q.k) over the
 *                                             tokens of that slot; -inf marks an empty slot
 *    Shared attention writes slots [0, shared_slots), unique attention writes slots
 *    [shared_slots, n_slots).  Both write EVERY slot of their range (empty ones as -inf, o = 0),
 *    so the caller never has to clear the buffers.
 *  * Return value: MOSKA_OK or a negative moska_status.  moska_last_error() gives a text for
 *    the last failure on the calling thread.  Invalid arguments are detected on the host
 *    before anything is launched.
 *  * What a kernel can only find out while it runs (routing indices that break the grouping's
 *    preconditions, an entry outside the batch, a bounded wait that ran out) goes to one sticky
 *    status word per device, read and cleared by moska_device_status().  A kernel that raises it
 *    never traps and never writes outside the caller's buffers; the results of that step are not
 *    valid.
 *  * Hidden state: none that outlives a call on the device side.  On the host side the library
 *    keeps, per device ordinal, the address of its status word (and of the built-in scratch of
 *    moska_group_by_chunk_noalloc), and per (host thread, device) the two CUDA events that order
 *    the side stream of a two-stream moska_decode_step; all are created on first use with that
 *    device current and are not valid across a cudaDeviceReset.
 */
#ifndef MOSKA_H_
#define MOSKA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum moska_status {
    MOSKA_OK              = 0,
    MOSKA_ERR_INVALID_ARG = -1, /* null pointer, k > C, Hq % Hkv != 0, misaligned pointer ...   */
    MOSKA_ERR_UNSUPPORTED = -2, /* D not in {64,128}, G > 8, L % 128 != 0, device is not sm_100 */
    MOSKA_ERR_WORKSPACE   = -3, /* workspace missing or smaller than moska_workspace_bytes()    */
    MOSKA_ERR_CUDA        = -4, /* a CUDA runtime call or kernel launch failed                  */
    MOSKA_ERR_TIMEOUT     = -5, /* device side: a bounded wait inside a kernel ran out          */
    MOSKA_ERR_CORRUPT     = -6  /* device side, debug build: workspace guard words overwritten  */
} moska_status;

/* Problem shape of one decode step of one layer. */
typedef struct moska_shape {
    int32_t B;               /* concurrent requests                                              */
    int32_t Hq;              /* query heads                                                      */
    int32_t Hkv;             /* KV heads, Hq % Hkv == 0, G = Hq / Hkv <= 8                       */
    int32_t D;               /* head dimension: 64 or 128                                        */
    int32_t C;               /* number of shared chunks                                          */
    int32_t L;               /* tokens per shared chunk, a multiple of 128                       */
    int32_t k;               /* chunks routed per (request, KV head), 1 <= k <= C                */
    int32_t shared_slots;    /* partial slots written by shared attention: k in routed mode;     */
                             /* in dense mode (no routing) the C chunks are cut into this many   */
                             /* runs of ceil(C / shared_slots) consecutive chunks                */
    int32_t n_unique_splits; /* partial slots written by unique attention (split-K), >= 1        */
    int64_t unique_tokens;   /* optional hint: the private tokens of all requests together, if   */
                             /* the host knows them, else 0.  Only moska_decode_step reads it,   */
                             /* to divide the SMs between shared and unique attention; results   */
                             /* never depend on it                                               */
    int32_t q_len;           /* query tokens per request (speculative decoding, chunked prefill;  */
                             /* Section II-A's multi-turn reuse): 0 or 1 = one.  With q_len > 1   */
                             /* the B batch rows are B / q_len requests, row b = r * q_len + i is */
                             /* token i of request r, kv_start / kv_len have B / q_len entries,   */
                             /* kv_len[r] counts the tokens the LAST query token sees and token i */
                             /* sees the first kv_len[r] - (q_len - 1 - i) of them.  Routing and  */
                             /* shared attention treat every row as a request of its own; unique  */
                             /* attention reads the request's K/V once for all its rows (needs    */
                             /* D = 128 and q_len * G <= 16; <= 8 with the FP8 store)             */
} moska_shape;

typedef void* moska_stream; /* a cudaStream_t */

/* Optional per-stage device timing of moska_decode_step (CUDA events recorded on the stream each
 * stage is launched on).  Stage order of the arrays below. */
enum { MOSKA_STAGE_ROUTE = 0, MOSKA_STAGE_GROUP, MOSKA_STAGE_SHARED, MOSKA_STAGE_UNIQUE,
       MOSKA_STAGE_MERGE, MOSKA_N_STAGES };
typedef struct moska_profiler moska_profiler;

/* Library version, major * 100 + minor. */
int moska_version(void);

/* Text of the last error raised on the calling thread ("" if none). Host pointer, never NULL. */
const char* moska_last_error(void);

/* Waits for the current device to finish, stores the sticky device-side status word in
 * *status_host (host pointer) and clears it.  0 means no kernel of the library raised anything.
 * MOSKA_ERR_TIMEOUT: a CTA of the tensor-core Shared KV Attention kernel gave up on one of its
 * bounded waits (TMA or MMA completion).  MOSKA_ERR_INVALID_ARG: a grouping call (either entry
 * point) met a chunk index outside [0, C) or a (request, KV head) list that is not strictly
 * ascending, or shared attention met an entry of seg_entries outside [0, B*Hkv*k).  In every
 * case the outputs of the steps since the last read are not valid.  MOSKA_ERR_CORRUPT (debug
 * build only): guard words of the workspace were overwritten or a work list would have overflowed.
 * The most negative code raised since the last read is the one reported. */
int moska_device_status(int32_t* status_host);

/* n_slots = shared_slots + n_unique_splits; negative status if the shape is invalid. Host only. */
int moska_partial_slots(const moska_shape* shape);

/* Bytes of workspace that moska_route / moska_group_by_chunk / moska_shared_attn[_fp8] need for
 * this shape (one workspace serves all of them; 256-byte aligned base required): the grouping's bit
 * sets and work lists, the router's scores beyond 256 chunks, and, for D = 128, room for an f16
 * copy of the queries (B*Hq*D*2 bytes, used by the FP8 shared store only).  Host only, pure.  */
size_t moska_workspace_bytes(const moska_shape* shape);

/* A reasonable n_unique_splits for a batch whose longest unique context has `max_len` tokens.
 * Host only, pure.                                                                              */
int moska_default_unique_splits(int32_t B, int32_t Hkv, int32_t max_len);

/* The same for a private store in FP8 (moska_unique_attn_fp8, moska_decode_step_fp8kv), whose
 * kernel has more and shorter-lived CTAs per SM.  Host only, pure.                             */
int moska_default_unique_splits_fp8(int32_t B, int32_t Hkv, int32_t max_len);

/*
 * Chunk embeddings used by the router (Section III-B: "precomputed chunk embeddings"; the
 * embedding of a chunk is the arithmetic mean of its L keys, per KV head).  Offline step.
 *   k_shared   bf16  [Hkv][C][L][D]   (16-byte aligned)
 *   summaries  float [Hkv][C][D]      out
 */
int moska_build_chunk_summaries(const uint16_t* k_shared, float* summaries,
                                const moska_shape* shape, moska_stream stream);

/*
 * A second training-free chunk embedding for the same `summaries` buffer (Section II-B and III-B
 * cite two lightweight routers: one pools a chunk's keys uniformly -- the mean above -- the other
 * weights a chunk's tokens by an attention pass inside the chunk).  Here the chunk's mean key
 * kbar probes the chunk's own keys:
 *     w_t = softmax_t(probe_scale * <kbar, k_t>),   summaries[h][c] = sum_t w_t k_t,
 * so tokens aligned with the chunk's centre count more and outliers less; probe_scale = 0 gives
 * the mean.  Everything downstream (moska_route and on) is unchanged.  Offline step; fp32.
 *   probe_scale  finite, >= 0 (1/sqrt(D) is the natural choice); L <= 10240
 */
int moska_build_chunk_summaries_attn(const uint16_t* k_shared, float* summaries, float probe_scale,
                                     const moska_shape* shape, moska_stream stream);

/*
 * Router (Section III-B): relevance of chunk c for (request b, KV head h) is the inner product
 * of the pooled query  qbar[b][h] = sum_{g<G} q[b][h*G+g]  with summaries[h][c]; the k chunks
 * with the largest score are selected, exact ties going to the lower chunk index.
 *   q           bf16  [B][Hq][D]
 *   summaries   float [Hkv][C][D]
 *   topk_idx    int32 [B][Hkv][k]   out, chunk indices in ASCENDING order
 *   topk_score  float [B][Hkv][k]   out, score of topk_idx[...] (same order); may be NULL
 * Up to 256 chunks one warp scores and selects for one (b, h) out of shared memory and `ws` may
 * be NULL; beyond that the scores are computed as a tiled fp32 product into `ws` (which must
 * then hold moska_workspace_bytes(); the grouping call may reuse the same workspace afterwards)
 * and selected by one warp per (b, h).
 */
int moska_route(const uint16_t* q, const float* summaries, int32_t* topk_idx, float* topk_score,
                const moska_shape* shape, void* ws, size_t ws_bytes, moska_stream stream);

/*
 * Query aggregation (Section III-A: the N concurrent queries that hit the same shared chunk are
 * gathered into one query matrix).  Let p = (b*Hkv + h)*k + j be the flat position of the j-th
 * routed chunk of (b, h) and key(p) = h*C + topk_idx[p].  This is a stable counting sort of the
 * positions by key:
 *   seg_offsets  int32 [Hkv*C + 1]  out, exclusive scan of the number of positions per key
 *   seg_entries  int32 [B*Hkv*k]    out, positions p, key-major, ascending p inside one key
 * The result is deterministic.  It also writes the tile work lists that moska_shared_attn
 * consumes into `ws` (give both calls the same, unmodified workspace).
 * Precondition (what moska_route produces): every list topk_idx[b][h][0..k) is STRICTLY ASCENDING,
 * hence without repeated chunks, and lies in [0, C).  The sort is done on one bit per (key,
 * request), which only describes such lists.  The marking pass checks it on the device: an index
 * outside [0, C) is skipped and a list out of order is flagged, both as MOSKA_ERR_INVALID_ARG in
 * the device status word (moska_device_status); seg_entries then still holds only positions that
 * exist, but a repeated or skipped chunk is missing from it, so the step's results are not valid.
 */
int moska_group_by_chunk(const int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                         const moska_shape* shape, void* ws, size_t ws_bytes, moska_stream stream);

/*
 * moska_group_by_chunk for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is a packaging variant of the call above.)
 *
 * Some hosts of this library may not call cudaMalloc at the point where they need the grouping:
 * a serving engine that gave all device memory to its own pool at start-up and has no bytes left
 * to carve a workspace from, or a latency-critical loop in which an allocation (which can
 * synchronise the whole device) is not acceptable.  For them the scratch of the grouping passes
 * lives in a fixed buffer of MOSKA_NOALLOC_SCRATCH_BYTES inside the library image; every GPU
 * that loads the library keeps that buffer until the process exits.  The call allocates and
 * frees nothing, neither directly nor through another library.
 *
 *   inputs / outputs      as moska_group_by_chunk (topk_idx in; seg_offsets, seg_entries out),
 *                         same precondition on topk_idx, same report through moska_device_status
 *   limit                 shapes whose grouping scratch (moska_workspace_bytes) exceeds the
 *                         buffer are rejected with MOSKA_ERR_WORKSPACE before anything runs
 *   first call            the first call on each device looks up the buffer's device address
 *                         (with that device current); make it before any stream capture
 *   shared state          all calls on a device use the same buffer and each call first clears
 *                         what it needs zeroed, so calls in stream order are independent; calls
 *                         that overlap on the GPU (different streams, no ordering) race
 *   work lists            the tile lists for moska_shared_attn stay inside the buffer and are not
 *                         exported; pair moska_shared_attn with moska_group_by_chunk instead
 */
#define MOSKA_NOALLOC_SCRATCH_BYTES (8u << 20)
int moska_group_by_chunk_noalloc(const int32_t* topk_idx, int32_t* seg_offsets,
                                 int32_t* seg_entries, const moska_shape* shape,
                                 moska_stream stream);

/*
 * Debug aid (no counterpart in the paper).  A library compiled with -DMOSKA_DEBUG_GUARDS
 * (`python -m paper_2511_06010_b200.build --debug` -> csrc/libmoska_debug.so) leaves 256 guard
 * bytes behind every region of the workspace (moska_workspace_bytes grows accordingly), fills them
 * and the regions' alignment padding with a pattern at the start of moska_route /
 * moska_group_by_chunk, compares them at the end of the grouping, and checks every work-list write
 * against the list's capacity.  This call compares the guard words once more, at any later point
 * (after shared attention, after the step): a mismatch raises MOSKA_ERR_CORRUPT in the device
 * status word (moska_device_status).  Nothing traps; a write beyond a list's capacity is skipped.
 *   ws, ws_bytes   the workspace the grouping call was given (device pointer, 256-byte aligned)
 * Returns MOSKA_ERR_UNSUPPORTED in a library built without the guard words (the regular build:
 * its workspace layout has no room for them and its kernels carry no checks).
 */
int moska_debug_check_workspace(void* ws, size_t ws_bytes, const moska_shape* shape,
                                moska_stream stream);

/*
 * Shared KV Attention (Section III-A, Fig. 2a): for every non-empty segment (h, c) the query rows
 * of all requests routed to chunk c form the rows of one Q matrix; S = scale * Q Kc^T, row-wise
 * softmax statistics and O = softmax(S) Vc are computed as one batched tensor-core product, so
 * the chunk's K/V tile leaves HBM once per step however many requests use it.
 * For entry p = (b*Hkv+h)*k + j and each g < G it writes slot j of row (b, h*G+g).
 *   q                      bf16 [B][Hq][D]
 *   k_shared, v_shared     bf16 [Hkv][C][L][D]   (128-byte aligned)
 *   topk_idx/seg_offsets/seg_entries   as produced by moska_route / moska_group_by_chunk,
 *       or all three NULL for DENSE mode: no routing, every row attends every chunk; run s of
 *       ceil(C/shared_slots) consecutive chunks goes to slot s (needs no prior grouping call).
 *   o_part, lse_part       see "Partial results" above; slots [0, shared_slots) are written
 *   softmax_scale          multiplies q.k before the softmax (usually 1/sqrt(D))
 */
int moska_shared_attn(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                      const int32_t* topk_idx, const int32_t* seg_offsets,
                      const int32_t* seg_entries, float* o_part, float* lse_part,
                      float softmax_scale, const moska_shape* shape, void* ws, size_t ws_bytes,
                      moska_stream stream);

/*
 * Shared KV Attention over a shared store kept in FP8 (E4M3), the KV precision the paper's
 * evaluation assumes (Section IV) applied to the batched product of Section III-A.  Token t of chunk
 * c of KV head h has key k_scale[h][c] * e4m3(k8[h][c][t][:]) and value v_scale[h][c] *
 * e4m3(v8[h][c][t][:]): ONE scale per (KV head, chunk) and tensor, so the key scale joins the softmax
 * scale and the value scale the final normalisation.  The code tiles arrive by TMA (half the bytes
 * of the bf16 store), are widened exactly to f16 in shared memory and multiplied on the tensor cores
 * with f16 Q and P and fp32 accumulation.  Routed or dense mode as for moska_shared_attn (in dense
 * mode a partial slot covers a run of chunks with different scales: the running maximum is kept in
 * scaled units and a chunk's value scale, relative to the run's first, joins its P tiles), D = 128.  Segments of at most 8 query rows are streamed by a
 * kernel of their own (codes widened in registers, f16 warp MMAs), as with the bf16 store.
 *   k8_shared, v8_shared  uint8 [Hkv][C][L][D]  OCP FP8 E4M3 codes (128-byte aligned)
 *   k_scale, v_scale      float [Hkv][C]        positive
 *   ws                    as for moska_shared_attn (the grouping's work lists); the call also keeps
 *                         an f16 copy of q in it, so it WRITES the workspace and needs it in dense
 *                         mode too
 * Chunk embeddings for the router are built from whichever copy of the keys the caller has in
 * bf16 (moska_build_chunk_summaries*); they are an offline step.
 */
int moska_shared_attn_fp8(const uint16_t* q, const uint8_t* k8_shared, const uint8_t* v8_shared,
                          const float* k_scale, const float* v_scale, const int32_t* topk_idx,
                          const int32_t* seg_offsets, const int32_t* seg_entries, float* o_part,
                          float* lse_part, float softmax_scale, const moska_shape* shape, void* ws,
                          size_t ws_bytes, moska_stream stream);

/*
 * Unique KV Attention (Section III-A: per-request attention over private KV, a memory-bound
 * GEMV-like pass).  Split-K over the request's tokens: each of the n_unique_splits slots holds
 * the partial result over a disjoint token range (which range is an implementation detail);
 * slots without tokens are written as lse = -inf, o = 0.
 *   k_unique, v_unique  bf16 [T_total][Hkv][D]  token-major ragged store (16-byte aligned)
 *   kv_start            int64 [B]  first token of request b in the store
 *   kv_len              int32 [B]  number of tokens of request b (0 allowed)
 */
int moska_unique_attn(const uint16_t* q, const uint16_t* k_unique, const uint16_t* v_unique,
                      const int64_t* kv_start, const int32_t* kv_len, float* o_part,
                      float* lse_part, float softmax_scale, const moska_shape* shape,
                      moska_stream stream);

/*
 * Unique KV Attention over a private KV store kept in FP8 (E4M3), the KV precision the paper's
 * evaluation assumes (Section IV) applied to the memory-bound per-request pass of Section III-A.
 * Token t of KV head h has key k_scale[t][h] * e4m3(k8[t][h][:]) and value v_scale[t][h] *
 * e4m3(v8[t][h][:]); everything else (split-K slots, empty requests, outputs) is as in
 * moska_unique_attn.  The codes are widened exactly to f16 and multiplied on tensor cores with
 * fp32 accumulation; P is rounded to f16.  D must be 128.
 *   k8, v8            uint8 [T_total][Hkv][D]   OCP FP8 E4M3 codes (16-byte aligned)
 *   k_scale, v_scale  float [T_total][Hkv]
 */
int moska_unique_attn_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8,
                          const float* k_scale, const float* v_scale, const int64_t* kv_start,
                          const int32_t* kv_len, float* o_part, float* lse_part,
                          float softmax_scale, const moska_shape* shape, moska_stream stream);

/*
 * Combination of the shared and unique partial results.  The paper leaves this step implicit;
 * the log-sum-exp merge is the only combination that equals softmax attention over the union of
 * the tokens (Section III-A/III-B).  Per row: M = max_i lse_i, w_i = exp(lse_i - M),
 * out = sum_i w_i o_i / sum_i w_i, lse = M + ln sum_i w_i.  Slots with lse = -inf contribute
 * nothing; if every slot is -inf then out = 0 and lse = -inf (never NaN).
 *   out      bf16  [B][Hq][D]        out
 *   out_f32  float [B][Hq][D]        out, unrounded copy; may be NULL
 *   lse_out  float [B][Hq]           out; may be NULL
 */
int moska_merge(const float* o_part, const float* lse_part, uint16_t* out, float* out_f32,
                float* lse_out, const moska_shape* shape, moska_stream stream);

/*
 * Measured comparison, not part of the method: the unbatched form that Shared KV Attention
 * replaces (Section I, Section III-A: one memory-bound GEMV pass per request over each routed
 * chunk).  Same results as moska_shared_attn, same slots; reads every routed chunk once per
 * (request, KV head) instead of once per step.  topk_idx == NULL selects dense mode.
 */
int moska_gemv_baseline(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                        const int32_t* topk_idx, float* o_part, float* lse_part,
                        float softmax_scale, const moska_shape* shape, moska_stream stream);

/* Creates a profiler able to hold `max_steps` recorded steps (host object owning CUDA events). */
int moska_profiler_create(moska_profiler** out, int32_t max_steps);
void moska_profiler_destroy(moska_profiler* prof);
/* Restricts recording to the stages whose bit (1 << MOSKA_STAGE_x) is set in stage_mask (all
 * stages by default).  Every recorded stage costs two event records per step on the stream it
 * runs on -- about 3 us per stage on a B200 -- so a caller timing whole steps records only the
 * stage it needs.  Stages that are not recorded read as 0. */
int moska_profiler_select(moska_profiler* prof, uint32_t stage_mask);
/* Waits for the recorded events, adds up the elapsed milliseconds per stage over the steps
 * recorded since the last read into stage_ms[MOSKA_N_STAGES] (host), stores their number in
 * *n_steps (host) and clears the profiler. */
int moska_profiler_read(moska_profiler* prof, float* stage_ms, int32_t* n_steps);

/*
 * One whole decode step on device buffers.  Without `side_stream` everything runs on `stream`
 * in the order route, group, unique, shared, merge.  With it, unique attention is enqueued first
 * on `stream`; route, group and shared attention follow on `side_stream` (both ordered after the
 * work already on `stream`), and the merge waits for both.  `side_stream` must have a HIGHER
 * priority than `stream`: its CTAs then take SMs over as unique-attention CTAs retire.  The
 * persistent tensor-core kernel of shared attention is given only a share of the SMs (derived
 * from the two kernels' estimated work, see shape->unique_tokens), so the HBM-bound unique
 * attention keeps running on the others: the two resource profiles overlap on one GPU.
 * Dense mode (no routing) when summaries == NULL.
 * Scratch buffers topk_idx [B*Hkv*k], seg_offsets [Hkv*C+1], seg_entries [B*Hkv*k], o_part,
 * lse_part and ws are caller-owned as in the individual calls.  `prof` may be NULL; otherwise
 * the step's stage boundaries are recorded into it (steps beyond its capacity are not recorded).
 */
int moska_decode_step(const uint16_t* q, const float* summaries, const uint16_t* k_shared,
                      const uint16_t* v_shared, const uint16_t* k_unique,
                      const uint16_t* v_unique, const int64_t* kv_start, const int32_t* kv_len,
                      int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                      float* o_part, float* lse_part, uint16_t* out, float* lse_out,
                      float softmax_scale, const moska_shape* shape, void* ws, size_t ws_bytes,
                      moska_stream stream, moska_stream side_stream, moska_profiler* prof);

/*
 * moska_decode_step with the private KV store in FP8 (E4M3 codes + per-(token, head) fp32 scales,
 * laid out as for moska_unique_attn_fp8); the shared store stays bf16.  Same schedule, buffers,
 * outputs and error behaviour; D must be 128.
 */
int moska_decode_step_fp8kv(const uint16_t* q, const float* summaries, const uint16_t* k_shared,
                            const uint16_t* v_shared, const uint8_t* k8_unique,
                            const uint8_t* v8_unique, const float* k_scale, const float* v_scale,
                            const int64_t* kv_start, const int32_t* kv_len, int32_t* topk_idx,
                            int32_t* seg_offsets, int32_t* seg_entries, float* o_part,
                            float* lse_part, uint16_t* out, float* lse_out, float softmax_scale,
                            const moska_shape* shape, void* ws, size_t ws_bytes, moska_stream stream,
                            moska_stream side_stream, moska_profiler* prof);

/*
 * moska_decode_step with the SHARED store in FP8 (laid out as for moska_shared_attn_fp8); the
 * private store stays bf16.  Same schedule, buffers, outputs and error behaviour (summaries NULL
 * selects dense mode); D = 128; the workspace is needed in dense mode too.
 */
int moska_decode_step_fp8shared(const uint16_t* q, const float* summaries, const uint8_t* k8_shared,
                                const uint8_t* v8_shared, const float* k_scale_shared,
                                const float* v_scale_shared, const uint16_t* k_unique,
                                const uint16_t* v_unique, const int64_t* kv_start, const int32_t* kv_len,
                                int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                                float* o_part, float* lse_part, uint16_t* out, float* lse_out,
                                float softmax_scale, const moska_shape* shape, void* ws, size_t ws_bytes,
                                moska_stream stream, moska_stream side_stream, moska_profiler* prof);

/*
 * moska_decode_step with BOTH stores in FP8, the KV precision of the paper's evaluation (Section
 * IV) on the whole path: the shared store as for moska_shared_attn_fp8 (one scale per (KV head,
 * chunk)), the private store as for moska_unique_attn_fp8 (one scale per (token, KV head)).  Same
 * schedule, buffers, outputs and error behaviour as moska_decode_step (summaries NULL selects dense
 * mode); D = 128; the workspace is needed in dense mode too.
 */
int moska_decode_step_fp8(const uint16_t* q, const float* summaries, const uint8_t* k8_shared,
                          const uint8_t* v8_shared, const float* k_scale_shared, const float* v_scale_shared,
                          const uint8_t* k8_unique, const uint8_t* v8_unique, const float* k_scale_unique,
                          const float* v_scale_unique, const int64_t* kv_start, const int32_t* kv_len,
                          int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries, float* o_part,
                          float* lse_part, uint16_t* out, float* lse_out, float softmax_scale,
                          const moska_shape* shape, void* ws, size_t ws_bytes, moska_stream stream,
                          moska_stream side_stream, moska_profiler* prof);

/*
 * moska_decode_step for a caller whose step inputs live in HOST memory: copies q_host (bf16
 * [B][Hq][D], ideally pinned) into q_dev, runs the step, copies `out` back into out_host (bf16
 * [B][Hq][D]) and waits for the stream.  The KV stores and all scratch stay on the device.
 * q_host must be 16-byte aligned.  With a side stream and buffers of 4 MiB or more the copies
 * leave the critical path: a PAGE-LOCKED q_host is copied on the side stream in front of the
 * router while unique attention reads its query rows straight from host memory, and the result
 * is merged in four row ranges, each copied to out_host on the side stream while the next one is
 * merged.  Pageable buffers and small ones take one copy before and one after the step.  Both
 * host buffers belong to the call until it returns.
 */
int moska_decode_step_host(const uint16_t* q_host, uint16_t* q_dev, const float* summaries,
                           const uint16_t* k_shared, const uint16_t* v_shared,
                           const uint16_t* k_unique, const uint16_t* v_unique,
                           const int64_t* kv_start, const int32_t* kv_len, int32_t* topk_idx,
                           int32_t* seg_offsets, int32_t* seg_entries, float* o_part,
                           float* lse_part, uint16_t* out_dev, uint16_t* out_host,
                           float softmax_scale, const moska_shape* shape, void* ws,
                           size_t ws_bytes, moska_stream stream, moska_stream side_stream,
                           moska_profiler* prof);

/*
 * moska_decode_step_fp8 (both stores in FP8, Section IV's precision) for a caller whose step inputs
 * live in HOST memory: q_host in, out_host out, the call returns when the result is there.  Copies,
 * their overlap with the step and the conditions on the host buffers are those of
 * moska_decode_step_host.
 */
int moska_decode_step_fp8_host(const uint16_t* q_host, uint16_t* q_dev, const float* summaries,
                               const uint8_t* k8_shared, const uint8_t* v8_shared,
                               const float* k_scale_shared, const float* v_scale_shared,
                               const uint8_t* k8_unique, const uint8_t* v8_unique,
                               const float* k_scale_unique, const float* v_scale_unique,
                               const int64_t* kv_start, const int32_t* kv_len, int32_t* topk_idx,
                               int32_t* seg_offsets, int32_t* seg_entries, float* o_part, float* lse_part,
                               uint16_t* out_dev, uint16_t* out_host, float softmax_scale,
                               const moska_shape* shape, void* ws, size_t ws_bytes, moska_stream stream,
                               moska_stream side_stream, moska_profiler* prof);

#ifdef __cplusplus
}
#endif
#endif /* MOSKA_H_ */
