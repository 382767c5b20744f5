/*
 * moska_oracle.c -- plain fp64 CPU statement of what the MoSKA decode-attention path computes.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call this file; it exists so that
 * the CUDA kernels can be compared with an independent, slow, obviously correct implementation.
 * It shares no code, header, table or helper with the CUDA library.
 *
 * Every function takes HOST pointers.  bf16 inputs arrive as raw bit patterns (uint16_t) and are
 * widened exactly to double; every sum, product, exp and log is done in double.  Loops follow
 * the definitions literally: no blocking, no fusion, no online softmax except where the staged
 * (per-chunk partial + merge) form is the thing being defined.  OpenMP only distributes
 * independent output rows over threads.
 *
 * What is pinned by independent checks (tests/test_oracle_pins.py): summaries, routing and its
 * tie-break, grouping, direct attention, the staged partials and the merge.  Routing QUALITY
 * (whether mean-key routing picks semantically right chunks) has no counterpart that can be run
 * without trained models: "parity unpinned" for that property only.
 *
 * Notation: B requests, Hq query heads, Hkv KV heads, G = Hq/Hkv, D head dim, C chunks of L
 * tokens, k routed chunks per (request, KV head).  Row r = b*Hq + hq, KV head h = hq / G.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* Exact widening of a bfloat16 bit pattern: bf16 is the upper half of an IEEE binary32. */
static double bf16_to_double(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Chunk embedding = arithmetic mean of the chunk's keys, per KV head (Section III-B,
 * "precomputed chunk embeddings"; mean-of-keys is the reading fixed by the workload definition).
 *   k_shared [Hkv][C][L][D] bf16 bits  ->  summaries [Hkv][C][D] double
 */
void oracle_chunk_summaries(const uint16_t* k_shared, double* summaries, int Hkv, int C, int L,
                            int D)
{
#pragma omp parallel for schedule(static)
    for (long hc = 0; hc < (long)Hkv * C; ++hc) {
        for (int d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int t = 0; t < L; ++t) acc += bf16_to_double(k_shared[(hc * L + t) * D + d]);
            summaries[hc * D + d] = acc / (double)L;
        }
    }
}

/*
 * Second training-free chunk embedding behind the same summaries buffer (Section II-B and III-B
 * cite two routers; the first pools a chunk's keys uniformly, which is the mean above; the
 * second weights a chunk's tokens by an attention pass inside the chunk).  The reading taken
 * here: the chunk's mean key kbar probes the chunk's own keys,
 *     w_t = softmax_t( scale * <kbar, k_t> ),   summary = sum_t w_t k_t,
 * i.e. one softmax-attention row with query kbar and the chunk's keys as both keys and values.
 * scale = 0 gives uniform weights, hence the mean.
 *   k_shared [Hkv][C][L][D] bf16 bits  ->  summaries [Hkv][C][D] double
 */
void oracle_chunk_summaries_attn(const uint16_t* k_shared, double* summaries, double scale,
                                 int Hkv, int C, int L, int D)
{
#pragma omp parallel for schedule(static)
    for (long hc = 0; hc < (long)Hkv * C; ++hc) {
        double* kbar = (double*)malloc(sizeof(double) * D);
        double* s = (double*)malloc(sizeof(double) * L);
        for (int d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int t = 0; t < L; ++t) acc += bf16_to_double(k_shared[(hc * L + t) * D + d]);
            kbar[d] = acc / (double)L;
        }
        double smax = -INFINITY;
        for (int t = 0; t < L; ++t) {
            double acc = 0.0;
            for (int d = 0; d < D; ++d) acc += kbar[d] * bf16_to_double(k_shared[(hc * L + t) * D + d]);
            s[t] = scale * acc;
            if (s[t] > smax) smax = s[t];
        }
        double den = 0.0;
        for (int t = 0; t < L; ++t) den += exp(s[t] - smax);
        for (int d = 0; d < D; ++d) {
            double acc = 0.0;
            for (int t = 0; t < L; ++t)
                acc += exp(s[t] - smax) * bf16_to_double(k_shared[(hc * L + t) * D + d]);
            summaries[hc * D + d] = acc / den;
        }
        free(kbar);
        free(s);
    }
}

/*
 * Router (Section III-B): score[b][h][c] = <sum_g q[b][h*G+g], summaries[h][c]>; the k chunks
 * of largest score are kept, exact ties going to the lower chunk index; the selected indices
 * are returned in ascending chunk order.  Selection is exhaustive: k passes, each taking the
 * best not-yet-taken chunk.
 *   scores_all (nullable) [B][Hkv][C] receives every score.
 *   topk_score (nullable) [B][Hkv][k] score of topk_idx, same order.
 */
void oracle_route(const uint16_t* q, const double* summaries, int32_t* topk_idx,
                  double* topk_score, double* scores_all, int B, int Hq, int Hkv, int D, int C,
                  int k)
{
    const int G = Hq / Hkv;
#pragma omp parallel for schedule(static)
    for (long bh = 0; bh < (long)B * Hkv; ++bh) {
        const int b = (int)(bh / Hkv), h = (int)(bh % Hkv);
        double* qbar = (double*)malloc(sizeof(double) * D);
        double* score = (double*)malloc(sizeof(double) * C);
        char* taken = (char*)calloc(C, 1);
        for (int d = 0; d < D; ++d) {
            double s = 0.0;
            for (int g = 0; g < G; ++g)
                s += bf16_to_double(q[((long)b * Hq + h * G + g) * D + d]);
            qbar[d] = s;
        }
        for (int c = 0; c < C; ++c) {
            double s = 0.0;
            for (int d = 0; d < D; ++d) s += qbar[d] * summaries[((long)h * C + c) * D + d];
            score[c] = s;
            if (scores_all) scores_all[bh * C + c] = s;
        }
        for (int j = 0; j < k; ++j) {
            int best = -1;
            for (int c = 0; c < C; ++c) {
                if (taken[c]) continue;
                if (best < 0 || score[c] > score[best]) best = c; /* strict >: lower index wins ties */
            }
            taken[best] = 1;
        }
        int j = 0;
        for (int c = 0; c < C; ++c) {
            if (!taken[c]) continue;
            topk_idx[bh * k + j] = c;
            if (topk_score) topk_score[bh * k + j] = score[c];
            ++j;
        }
        free(qbar);
        free(score);
        free(taken);
    }
}

/*
 * Query aggregation (Section III-A): positions p = (b*Hkv+h)*k + j listed per key = h*C +
 * topk_idx[p], keys ascending, p ascending inside a key.
 *   seg_offsets [Hkv*C + 1], seg_entries [B*Hkv*k]
 */
void oracle_group_by_chunk(const int32_t* topk_idx, int32_t* seg_offsets, int32_t* seg_entries,
                           int B, int Hkv, int C, int k)
{
    const long P = (long)B * Hkv * k;
    long n = 0;
    for (long key = 0; key < (long)Hkv * C; ++key) {
        seg_offsets[key] = (int32_t)n;
        for (long p = 0; p < P; ++p) {
            const int h = (int)((p / k) % Hkv);
            if ((long)h * C + topk_idx[p] == key) seg_entries[n++] = (int32_t)p;
        }
    }
    seg_offsets[(long)Hkv * C] = (int32_t)n;
}

/* Same result as oracle_group_by_chunk in O(P + Hkv*C) time, for the larger parity cases.
 * (Counting sort; pinned against the quadratic definition above and numpy's stable argsort.) */
void oracle_group_by_chunk_fast(const int32_t* topk_idx, int32_t* seg_offsets,
                                int32_t* seg_entries, int B, int Hkv, int C, int k)
{
    const long P = (long)B * Hkv * k, K = (long)Hkv * C;
    int32_t* fill = (int32_t*)calloc(K + 1, sizeof(int32_t));
    for (long p = 0; p < P; ++p) fill[(long)((p / k) % Hkv) * C + topk_idx[p] + 1]++;
    seg_offsets[0] = 0;
    for (long key = 0; key < K; ++key) seg_offsets[key + 1] = seg_offsets[key] + fill[key + 1];
    for (long key = 0; key < K; ++key) fill[key] = seg_offsets[key];
    for (long p = 0; p < P; ++p) {
        const long key = (long)((p / k) % Hkv) * C + topk_idx[p];
        seg_entries[fill[key]++] = (int32_t)p;
    }
    free(fill);
}

/*
 * Softmax attention of one query over an explicit list of n tokens (the plain definition):
 *   s_t = scale * <q, k_t>,  lse = ln sum_t exp(s_t),  out = sum_t exp(s_t - lse) v_t.
 * n == 0 gives lse = -inf and out = 0.  `kp[t]` / `vp[t]` point at the D bf16 values of token t.
 */
static void attend_tokens(const uint16_t* qrow, const uint16_t* const* kp,
                          const uint16_t* const* vp, long n, int D, double scale, double* out,
                          double* lse)
{
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    if (n == 0) {
        *lse = -INFINITY;
        return;
    }
    double* s = (double*)malloc(sizeof(double) * n);
    double m = -INFINITY;
    for (long t = 0; t < n; ++t) {
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += bf16_to_double(qrow[d]) * bf16_to_double(kp[t][d]);
        s[t] = scale * acc;
        if (s[t] > m) m = s[t];
    }
    double z = 0.0;
    for (long t = 0; t < n; ++t) z += exp(s[t] - m);
    *lse = m + log(z);
    for (long t = 0; t < n; ++t) {
        const double p = exp(s[t] - *lse);
        for (int d = 0; d < D; ++d) out[d] += p * bf16_to_double(vp[t][d]);
    }
    free(s);
}

/*
 * The definition of the whole step's result (Sections III-A and III-B): each query row attends,
 * with ONE softmax, to the concatenation of the tokens of its k routed shared chunks and of its
 * request's unique tokens.
 *   k_shared/v_shared [Hkv][C][L][D], k_unique/v_unique [T][Hkv][D], kv_start int64 [B],
 *   kv_len int32 [B], topk_idx [B][Hkv][k]  ->  out [B][Hq][D], lse [B][Hq]
 * use_shared / use_unique switch the two token sources on or off (both 1 for the full result).
 */
void oracle_attend_direct(const uint16_t* q, const uint16_t* k_shared, const uint16_t* v_shared,
                          const uint16_t* k_unique, const uint16_t* v_unique,
                          const int64_t* kv_start, const int32_t* kv_len,
                          const int32_t* topk_idx, double* out, double* lse, double scale, int B,
                          int Hq, int Hkv, int D, int C, int L, int k, int use_shared,
                          int use_unique)
{
    const int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (long r = 0; r < (long)B * Hq; ++r) {
        const int b = (int)(r / Hq), hq = (int)(r % Hq), h = hq / G;
        const long n_sh = use_shared ? (long)k * L : 0;
        const long n_un = use_unique ? (long)kv_len[b] : 0;
        const long n = n_sh + n_un;
        const uint16_t** kp = (const uint16_t**)malloc(sizeof(void*) * (n > 0 ? n : 1));
        const uint16_t** vp = (const uint16_t**)malloc(sizeof(void*) * (n > 0 ? n : 1));
        long i = 0;
        if (use_shared)
            for (int j = 0; j < k; ++j) {
                const long c = topk_idx[((long)b * Hkv + h) * k + j];
                for (int t = 0; t < L; ++t, ++i) {
                    kp[i] = k_shared + ((((long)h * C + c) * L + t) * D);
                    vp[i] = v_shared + ((((long)h * C + c) * L + t) * D);
                }
            }
        if (use_unique)
            for (long t = 0; t < n_un; ++t, ++i) {
                kp[i] = k_unique + (((long)kv_start[b] + t) * Hkv + h) * D;
                vp[i] = v_unique + (((long)kv_start[b] + t) * Hkv + h) * D;
            }
        attend_tokens(q + r * D, kp, vp, n, D, scale, out + r * D, lse + r);
        free(kp);
        free(vp);
    }
}

/*
 * Staged form, shared part: one partial per (row, routed chunk j) -- attention of the row over
 * the L tokens of chunk topk_idx[b][h][j] alone.
 *   ->  o_part [B][Hq][k][D], lse_part [B][Hq][k]
 */
void oracle_shared_partials(const uint16_t* q, const uint16_t* k_shared,
                            const uint16_t* v_shared, const int32_t* topk_idx, double* o_part,
                            double* lse_part, double scale, int B, int Hq, int Hkv, int D, int C,
                            int L, int k)
{
    const int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (long rj = 0; rj < (long)B * Hq * k; ++rj) {
        const long r = rj / k;
        const int j = (int)(rj % k);
        const int b = (int)(r / Hq), hq = (int)(r % Hq), h = hq / G;
        const long c = topk_idx[((long)b * Hkv + h) * k + j];
        const uint16_t** kp = (const uint16_t**)malloc(sizeof(void*) * L);
        const uint16_t** vp = (const uint16_t**)malloc(sizeof(void*) * L);
        for (int t = 0; t < L; ++t) {
            kp[t] = k_shared + ((((long)h * C + c) * L + t) * D);
            vp[t] = v_shared + ((((long)h * C + c) * L + t) * D);
        }
        attend_tokens(q + r * D, kp, vp, L, D, scale, o_part + rj * D, lse_part + rj);
        free(kp);
        free(vp);
    }
}

/*
 * Log-sum-exp combination of n_slots partial results per row (the step the paper leaves
 * implicit; it is the combination that equals one softmax over the union of the tokens):
 *   M = max_i lse_i, w_i = exp(lse_i - M), out = sum_i w_i o_i / sum_i w_i, lse = M + ln sum w_i.
 * All slots -inf  ->  out = 0, lse = -inf.
 *   o_part [rows][n_slots][D], lse_part [rows][n_slots]  ->  out [rows][D], lse [rows]
 */
void oracle_merge(const double* o_part, const double* lse_part, double* out, double* lse,
                  long rows, int n_slots, int D)
{
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r) {
        double M = -INFINITY;
        for (int i = 0; i < n_slots; ++i)
            if (lse_part[r * n_slots + i] > M) M = lse_part[r * n_slots + i];
        for (int d = 0; d < D; ++d) out[r * D + d] = 0.0;
        if (M == -INFINITY) {
            lse[r] = -INFINITY;
            continue;
        }
        double W = 0.0;
        for (int i = 0; i < n_slots; ++i) W += exp(lse_part[r * n_slots + i] - M);
        for (int i = 0; i < n_slots; ++i) {
            const double w = exp(lse_part[r * n_slots + i] - M) / W;
            if (w == 0.0) continue; /* an empty slot's o is unspecified beyond being finite */
            for (int d = 0; d < D; ++d) out[r * D + d] += w * o_part[(r * n_slots + i) * D + d];
        }
        lse[r] = M + log(W);
    }
}

/* ------------------------------------------------------------------------------------------------
 * FP8 (E4M3) private KV, the storage precision the paper's evaluation assumes (Section IV).
 *
 * Value of an OCP FP8 E4M3 code (1 sign bit, 4 exponent bits with bias 7, 3 mantissa bits; no
 * infinities; S.1111.111 is NaN; exponent field 0 holds the subnormals m/8 * 2^-6), written out
 * from the format's definition.
 */
double oracle_e4m3_value(uint8_t code)
{
    const int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m / 8.0, -6);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

/*
 * Unique KV Attention over an FP8 store (Section III-A with the KV precision of Section IV): token
 * t of KV head h has key  k_scale[t][h] * e4m3(k8[t][h][:])  and value  v_scale[t][h] *
 * e4m3(v8[t][h][:]); each query row attends with one softmax to its request's tokens.
 *   q bf16 [B][Hq][D]; k8, v8 uint8 [T][Hkv][D]; k_scale, v_scale float [T][Hkv];
 *   kv_start int64 [B], kv_len int32 [B]  ->  out [B][Hq][D], lse [B][Hq]
 */
void oracle_attend_unique_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8,
                              const float* k_scale, const float* v_scale, const int64_t* kv_start,
                              const int32_t* kv_len, double* out, double* lse, double scale, int B,
                              int Hq, int Hkv, int D)
{
    const int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (long r = 0; r < (long)B * Hq; ++r) {
        const int b = (int)(r / Hq), hq = (int)(r % Hq), h = hq / G;
        const long n = kv_len[b];
        double* o = out + r * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        if (n == 0) {
            lse[r] = -INFINITY;
            continue;
        }
        double* s = (double*)malloc(sizeof(double) * n);
        double m = -INFINITY;
        for (long t = 0; t < n; ++t) {
            const long row = ((long)kv_start[b] + t) * Hkv + h;
            double acc = 0.0;
            for (int d = 0; d < D; ++d)
                acc += bf16_to_double(q[r * D + d]) * ((double)k_scale[row] * oracle_e4m3_value(k8[row * D + d]));
            s[t] = scale * acc;
            if (s[t] > m) m = s[t];
        }
        double z = 0.0;
        for (long t = 0; t < n; ++t) z += exp(s[t] - m);
        lse[r] = m + log(z);
        for (long t = 0; t < n; ++t) {
            const long row = ((long)kv_start[b] + t) * Hkv + h;
            const double p = exp(s[t] - lse[r]);
            for (int d = 0; d < D; ++d)
                o[d] += p * ((double)v_scale[row] * oracle_e4m3_value(v8[row * D + d]));
        }
        free(s);
    }
}

/*
 * Shared KV Attention over an FP8 shared store (Section III-A with the KV precision of Section
 * IV).  Storage: E4M3 codes [Hkv][C][L][D] for keys and for values and ONE scale per (KV head,
 * chunk) for each, so token t of chunk c of head h has key  k_scale[h][c] * e4m3(k8[h][c][t][:])
 * and value  v_scale[h][c] * e4m3(v8[h][c][t][:]).  Staged form as oracle_shared_partials: one
 * partial per (row, routed chunk j), attention of the row over the L tokens of that chunk alone.
 *   ->  o_part [B][Hq][k][D], lse_part [B][Hq][k]
 */
void oracle_shared_partials_fp8(const uint16_t* q, const uint8_t* k8, const uint8_t* v8,
                                const float* k_scale, const float* v_scale,
                                const int32_t* topk_idx, double* o_part, double* lse_part,
                                double scale, int B, int Hq, int Hkv, int D, int C, int L, int k)
{
    const int G = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
    for (long rj = 0; rj < (long)B * Hq * k; ++rj) {
        const long r = rj / k;
        const int j = (int)(rj % k);
        const int b = (int)(r / Hq), hq = (int)(r % Hq), h = hq / G;
        const long hc = (long)h * C + topk_idx[((long)b * Hkv + h) * k + j];
        const double ksc = (double)k_scale[hc], vsc = (double)v_scale[hc];
        double* o = o_part + rj * D;
        double* s = (double*)malloc(sizeof(double) * L);
        double m = -INFINITY;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        for (int t = 0; t < L; ++t) {
            double acc = 0.0;
            for (int d = 0; d < D; ++d)
                acc += bf16_to_double(q[r * D + d]) * (ksc * oracle_e4m3_value(k8[(hc * L + t) * D + d]));
            s[t] = scale * acc;
            if (s[t] > m) m = s[t];
        }
        double z = 0.0;
        for (int t = 0; t < L; ++t) z += exp(s[t] - m);
        lse_part[rj] = m + log(z);
        for (int t = 0; t < L; ++t) {
            const double p = exp(s[t] - lse_part[rj]);
            for (int d = 0; d < D; ++d) o[d] += p * (vsc * oracle_e4m3_value(v8[(hc * L + t) * D + d]));
        }
        free(s);
    }
}
