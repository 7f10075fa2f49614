/*
 * LCKV decode-step attention: float64 CPU oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, direct restatement of what
 * the layer-condensed KV cache method computes at one decode step.  It exists
 * to check the CUDA library and to be timed as a CPU baseline; the product
 * path never calls it.  It shares no code, header, table or helper with the
 * CUDA sources.
 *
 * Every function below states the passage of the paper (arXiv 2405.10637) it
 * follows.  Arithmetic is float64 throughout; the bf16 inputs are widened
 * exactly.  Softmax is the textbook two-pass form (max, then exponentials,
 * then normalise): no chunking, no running rescale, no reordering.
 *
 * Pins (see tests/): brute-force n x n masked attention written independently
 * in numpy, torch's scaled_dot_product_attention in float64 for w = L, closed
 * forms (q = 0, one visible key, empty visible set, dominant key), permutation
 * invariance, log-sum-exp merge of any partition, hand-enumerated warmup sets;
 * for the key/value producer: exact rational sums, selector weights, a library
 * matmul, torch's bf16 rounding on exact products, the complex-number form of
 * the rotary encoding and its relative-position property.
 *
 * Readings of the paper where it is silent (each one is a switch here):
 *   top_variant 0  the shared cache is the cache of layer L-1 itself, even
 *                  when that layer is a warmup layer (Section 2.1, literal);
 *   top_variant 1  the shared cache is fed by the topmost non-warmup layer;
 *   n_sink         0: caches grow without bound (up to T_cap rows).  s >= 1: the cache keeps the
 *                  first s tokens and the most recent T_cap - s tokens (the StreamingLLM policy
 *                  the paper combines with its model in Section 3.3); the evicted token's row is
 *                  reused, row(t) = t for t < T_cap, else s + (t - s) mod (T_cap - s).
 *   always_sink    0: the zero dummy key/value is used only when a query sees
 *                  nothing (first token, Section 2.1); 1: it is a permanent
 *                  extra column of every row (alternative reading, CPU only).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define LCKV_ORACLE_OK 0
#define LCKV_ORACLE_EINVAL 1
#define LCKV_ORACLE_ECAPACITY 2

/* bf16 is the upper half of an IEEE binary32: widening is exact. */
static double bf16_to_f64(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/*
 * Layer plan.  Section 2.1: the top w/2 and the bottom w/2 layers are warmup
 * layers with standard attention (sandwich); every other layer pairs its
 * queries with the top layer's keys and values and drops the diagonal.
 * "w = L" is the standard transformer (Section 4.2, the right-most point of
 * the warmup-layer figure).
 *
 * Outputs, all of length L (layer 0 = bottom):
 *   is_warmup[l]   1 if l is a warmup layer
 *   read_slot[l]   which cache layer l attends to
 *   mode[l]        0 = condensed (positions j <  t), 1 = standard (j <= t)
 *   write_slot[l]  cache that receives layer l's new k,v (-1: layer has no K/V)
 *   write_before[l] 1: the row is written before layer l attends (standard
 *                  layers see their own token); 0: written at the end of the
 *                  step (the shared cache under the diagonal mask)
 * n_slots = number of distinct caches (the memory footprint in layers).
 */
int lckv_oracle_plan(int L, int w, int top_variant, int32_t* is_warmup, int32_t* read_slot,
                     int32_t* mode, int32_t* write_slot, int32_t* write_before, int32_t* n_slots)
{
    if (L < 1 || w < 0 || w > L) return LCKV_ORACLE_EINVAL;
    if (w != L && (w % 2) != 0) return LCKV_ORACLE_EINVAL;
    if (top_variant != 0 && top_variant != 1) return LCKV_ORACLE_EINVAL;

    for (int l = 0; l < L; ++l) {
        if (w == L) is_warmup[l] = 1;
        else is_warmup[l] = (l < w / 2) || (l >= L - w / 2);
    }
    /* which layer feeds the shared cache (slot 0) */
    int feeder = L - 1;
    if (top_variant == 1 && w > 0 && w < L) feeder = L - 1 - w / 2;

    int next = 1;
    for (int l = 0; l < L; ++l) {
        if (is_warmup[l]) {
            mode[l] = 1;
            write_before[l] = 1;
            if (l == feeder) {
                read_slot[l] = write_slot[l] = 0;
            } else {
                read_slot[l] = write_slot[l] = next++;
            }
        } else {
            mode[l] = 0;
            read_slot[l] = 0;
            write_before[l] = 0;
            write_slot[l] = (l == feeder) ? 0 : -1;
        }
    }
    *n_slots = next;
    return LCKV_ORACLE_OK;
}

/*
 * One query row against n_vis visible cache rows (Section 2.1):
 *   s_j = scale * <q, K_j>,  p = softmax_j(s),  o = sum_j p_j V_j.
 * An empty visible set is the first token of a sequence under the diagonal
 * mask: it attends to one zero dummy key/value, which takes weight 1, so
 * o = 0 (Section 2.1).  lse = log sum_j exp(s_j); for the empty set the dummy
 * column has score 0, so lse = 0.
 * probs (optional, n_vis + 1 entries) receives p_0..p_{n_vis-1} and, last, the
 * weight of the dummy column (0 unless the set is empty or always_sink).
 */
static void attend_row(const uint16_t* q, const uint16_t* K, const uint16_t* V, int64_t n_vis,
                       int d, double scale, int always_sink, double* o, double* lse,
                       double* probs, double* scratch)
{
    int use_dummy = always_sink || n_vis == 0;
    double M = use_dummy ? 0.0 : -INFINITY;
    for (int64_t j = 0; j < n_vis; ++j) {
        double s = 0.0;
        for (int c = 0; c < d; ++c) s += bf16_to_f64(q[c]) * bf16_to_f64(K[j * d + c]);
        s *= scale;
        scratch[j] = s;
        if (s > M) M = s;
    }
    double Z = use_dummy ? exp(0.0 - M) : 0.0;
    for (int64_t j = 0; j < n_vis; ++j) {
        scratch[j] = exp(scratch[j] - M);
        Z += scratch[j];
    }
    for (int c = 0; c < d; ++c) o[c] = 0.0;
    for (int64_t j = 0; j < n_vis; ++j) {
        double p = scratch[j] / Z;
        if (probs) probs[j] = p;
        for (int c = 0; c < d; ++c) o[c] += p * bf16_to_f64(V[j * d + c]);
    }
    /* the dummy value is the zero vector: it adds nothing to o */
    if (probs) probs[n_vis] = use_dummy ? exp(0.0 - M) / Z : 0.0;
    if (lse) *lse = M + log(Z);
}

/* Single-row entry for tests: q[d], K,V [n_vis, d]. */
int lckv_oracle_attend_row(const uint16_t* q, const uint16_t* K, const uint16_t* V,
                           int64_t n_vis, int d, double scale, int always_sink, double* o,
                           double* lse, double* probs)
{
    if (n_vis < 0 || d < 1) return LCKV_ORACLE_EINVAL;
    double* scratch = (double*)malloc(sizeof(double) * (size_t)(n_vis > 0 ? n_vis : 1));
    if (!scratch) return LCKV_ORACLE_EINVAL;
    attend_row(q, K, V, n_vis, d, scale, always_sink, o, lse, probs, scratch);
    free(scratch);
    return LCKV_ORACLE_OK;
}

/*
 * Batched decode attention of one layer against one cache.
 *   q    [B, H_q, d]           bf16 bits
 *   K, V [B, H_kv, T_cap, d]   bf16 bits, rows [0, n_vis) of each (b, kv head) valid
 *   lens [B]                   tokens already cached; the new token is position lens[b]
 *   mode 0: visible j < lens[b] (diagonal masked, Section 2.1)
 *   mode 1: visible j <= lens[b] (standard attention of a warmup layer; row
 *           lens[b] must already hold this step's k, v)
 *   q head h reads kv head h / (H_q / H_kv)  (contiguous groups, Llama's GQA)
 *   out [B, H_q, d] float64, lse [B, H_q] float64 (may be NULL)
 * Rows are independent; they are spread over the host cores with OpenMP.
 */
int lckv_oracle_decode_attention(const uint16_t* q, const uint16_t* K, const uint16_t* V,
                                 const int32_t* lens, int B, int H_q, int H_kv, int64_t T_cap,
                                 int d, int mode, double scale, int always_sink, int n_sink,
                                 double* out, double* lse)
{
    if (B < 0 || H_q < 1 || H_kv < 1 || H_q % H_kv != 0 || d < 1) return LCKV_ORACLE_EINVAL;
    if (mode != 0 && mode != 1) return LCKV_ORACLE_EINVAL;
    int g = H_q / H_kv;
    for (int b = 0; b < B; ++b) {
        if (lens[b] < 0) return LCKV_ORACLE_ECAPACITY;
        if (n_sink <= 0 && (int64_t)lens[b] + mode > T_cap) return LCKV_ORACLE_ECAPACITY;
    }
    if (n_sink < 0 || (n_sink > 0 && n_sink >= T_cap)) return LCKV_ORACLE_EINVAL;
    int64_t rows = (int64_t)B * H_q;
#pragma omp parallel
    {
        double* scratch = (double*)malloc(sizeof(double) * (size_t)(T_cap > 0 ? T_cap : 1));
#pragma omp for schedule(dynamic, 1)
        for (int64_t r = 0; r < rows; ++r) {
            int b = (int)(r / H_q), h = (int)(r % H_q);
            int kvh = h / g;
            /* Section 3.3: with the sink + recent-window policy the cache holds at most T_cap
             * tokens; all of them precede the query (or are the query's own, standard mode). */
            int64_t n_vis = (int64_t)lens[b] + mode;
            if (n_sink > 0 && n_vis > T_cap) n_vis = T_cap;
            const uint16_t* Kp = K + (((int64_t)b * H_kv + kvh) * T_cap) * d;
            const uint16_t* Vp = V + (((int64_t)b * H_kv + kvh) * T_cap) * d;
            attend_row(q + r * d, Kp, Vp, n_vis, d, scale, always_sink, out + r * d,
                       lse ? lse + r : NULL, NULL, scratch);
        }
        free(scratch);
    }
    return LCKV_ORACLE_OK;
}

/*
 * Append: the new token's k, v (each [B, H_kv, d]) become row lens[b] of the
 * cache (Section 1: the cache stores the keys and values of every generated
 * token so they are not recomputed).  Lengths are not changed here.
 */
int lckv_oracle_append(uint16_t* K, uint16_t* V, const uint16_t* k_new, const uint16_t* v_new,
                       const int32_t* lens, int B, int H_kv, int64_t T_cap, int d, int n_sink)
{
    if (n_sink < 0 || (n_sink > 0 && n_sink >= T_cap)) return LCKV_ORACLE_EINVAL;
    for (int b = 0; b < B; ++b)
        if (lens[b] < 0 || (n_sink <= 0 && (int64_t)lens[b] >= T_cap)) return LCKV_ORACLE_ECAPACITY;
    for (int b = 0; b < B; ++b)
        for (int h = 0; h < H_kv; ++h) {
            /* token t goes to row t; once the cache is full (streaming policy) it replaces the
             * oldest token that is not one of the first n_sink */
            int64_t row = lens[b];
            if (n_sink > 0 && row >= T_cap) row = n_sink + (row - n_sink) % (T_cap - n_sink);
            int64_t dst = ((((int64_t)b * H_kv + h) * T_cap) + row) * d;
            int64_t src = ((int64_t)b * H_kv + h) * d;
            memcpy(K + dst, k_new + src, sizeof(uint16_t) * (size_t)d);
            memcpy(V + dst, v_new + src, sizeof(uint16_t) * (size_t)d);
        }
    return LCKV_ORACLE_OK;
}

/*
 * One decode step of the whole layer stack (Sections 2.1 and 2.2: decoding is
 * one token at a time, bottom layer to top layer).  For l = 0 .. L-1 in order:
 *   warmup layer:   write its k,v at row lens[b] of its own cache, then attend
 *                   j <= lens[b]  (standard attention);
 *   other layers:   attend j < lens[b] of the shared cache (the top layer's
 *                   k,v of this token do not exist yet: diagonal masked).
 * Then the feeder layer's k,v of this token are written at row lens[b] of the
 * shared cache (unless it was a warmup layer that wrote them already) and
 * every length grows by one.
 *
 *   q_layers[l]      [B, H_q, d]   one pointer per layer
 *   k_new_layers[l], v_new_layers[l]   [B, H_kv, d] or NULL where write_slot[l] < 0
 *   K_slots[s], V_slots[s]            [B_max, H_kv, T_cap, d] caches, modified
 *   lens [B]                          modified (+1)
 *   out_layers[l]    [B, H_q, d] float64; lse_layers[l] [B, H_q] or NULL array
 */
int lckv_oracle_stack_step(int L, int w, int top_variant, const uint16_t* const* q_layers,
                           const uint16_t* const* k_new_layers,
                           const uint16_t* const* v_new_layers, uint16_t* const* K_slots,
                           uint16_t* const* V_slots, int32_t* lens, int B, int H_q, int H_kv,
                           int64_t T_cap, int d, double scale, int always_sink, int n_sink,
                           double* const* out_layers, double* const* lse_layers)
{
    int32_t* plan = (int32_t*)malloc(sizeof(int32_t) * 5 * (size_t)L);
    if (!plan) return LCKV_ORACLE_EINVAL;
    int32_t *is_w = plan, *rs = plan + L, *md = plan + 2 * L, *ws = plan + 3 * L,
            *wb = plan + 4 * L;
    int32_t n_slots = 0;
    int rc = lckv_oracle_plan(L, w, top_variant, is_w, rs, md, ws, wb, &n_slots);
    if (rc) { free(plan); return rc; }
    for (int b = 0; b < B; ++b)
        if (lens[b] < 0 || (n_sink <= 0 && (int64_t)lens[b] + 1 > T_cap)) { free(plan); return LCKV_ORACLE_ECAPACITY; }
    for (int l = 0; l < L; ++l)
        if (ws[l] >= 0 && (!k_new_layers[l] || !v_new_layers[l])) { free(plan); return LCKV_ORACLE_EINVAL; }

    for (int l = 0; l < L && rc == 0; ++l) {
        if (ws[l] >= 0 && wb[l])
            rc = lckv_oracle_append(K_slots[ws[l]], V_slots[ws[l]], k_new_layers[l],
                                    v_new_layers[l], lens, B, H_kv, T_cap, d, n_sink);
        if (rc) break;
        rc = lckv_oracle_decode_attention(q_layers[l], K_slots[rs[l]], V_slots[rs[l]], lens, B,
                                          H_q, H_kv, T_cap, d, md[l], scale, always_sink, n_sink,
                                          out_layers[l], lse_layers ? lse_layers[l] : NULL);
    }
    for (int l = 0; l < L && rc == 0; ++l)
        if (ws[l] >= 0 && !wb[l])
            rc = lckv_oracle_append(K_slots[ws[l]], V_slots[ws[l]], k_new_layers[l],
                                    v_new_layers[l], lens, B, H_kv, T_cap, d, n_sink);
    if (rc == 0)
        for (int b = 0; b < B; ++b) lens[b] += 1;
    free(plan);
    return rc;
}

/* Threads the parallel loops use (reported beside the CPU baseline). */
int lckv_oracle_num_threads(void)
{
    int n = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        n = omp_get_num_threads();
    }
#endif
    return n;
}

/* ------------------------------------------------------------------------------------------------
 * Prompt encoding (Section 2.3 "Inference with Prompts"; Section 2.2.1 for one parallel iteration).
 *
 * The prompt cannot be encoded in one parallel pass, because every token needs the top-layer k,v
 * of its predecessors.  Instead the paper runs m + b iterations over all prompt tokens in parallel;
 * in each iteration the queries of the condensed layers are paired with the top-layer k,v of the
 * PREVIOUS iteration (zero vectors before the first one), diagonal masked as always, and the
 * warmup layers do standard causal attention over their own k,v of the current iteration.
 *
 * Token-parallel attention of one layer:
 *   q    [B, n_max, H_q, d]   token-major; tokens i < lens[b] of sequence b are valid
 *   K, V [B, H_kv, T_cap, d]  cache; rows j < lens[b] valid
 *   mode 0: token i sees rows j < i;  mode 1: rows j <= i
 *   out  [B, n_max, H_q, d] float64; rows i >= lens[b] are left untouched
 * Each (b, i, h) is one attend_row call: the definition, nothing shared with the decode path's
 * bookkeeping.
 * ------------------------------------------------------------------------------------------------ */
int lckv_oracle_prefill_attention(const uint16_t* q, const uint16_t* K, const uint16_t* V,
                                  const int32_t* lens, int B, int n_max, int H_q, int H_kv,
                                  int64_t T_cap, int d, int mode, double scale, int always_sink,
                                  double* out)
{
    if (B < 0 || n_max < 0 || H_q < 1 || H_kv < 1 || H_q % H_kv != 0 || d < 1) return LCKV_ORACLE_EINVAL;
    if (mode != 0 && mode != 1) return LCKV_ORACLE_EINVAL;
    int g = H_q / H_kv;
    for (int b = 0; b < B; ++b)
        if (lens[b] < 0 || lens[b] > n_max || (int64_t)lens[b] > T_cap) return LCKV_ORACLE_ECAPACITY;
    int64_t rows = (int64_t)B * n_max * H_q;
#pragma omp parallel
    {
        double* scratch = (double*)malloc(sizeof(double) * (size_t)(n_max > 0 ? n_max : 1));
#pragma omp for schedule(dynamic, 16)
        for (int64_t r = 0; r < rows; ++r) {
            int h = (int)(r % H_q);
            int i = (int)((r / H_q) % n_max);
            int b = (int)(r / ((int64_t)H_q * n_max));
            if (i >= lens[b]) continue;
            int kvh = h / g;
            int64_t n_vis = (int64_t)i + mode;
            const uint16_t* Kp = K + (((int64_t)b * H_kv + kvh) * T_cap) * d;
            const uint16_t* Vp = V + (((int64_t)b * H_kv + kvh) * T_cap) * d;
            attend_row(q + r * d, Kp, Vp, n_vis, d, scale, always_sink, out + r * d, NULL, NULL,
                       scratch);
        }
        free(scratch);
    }
    return LCKV_ORACLE_OK;
}

/* Rows [0, lens[b]) of a cache <- the prompt's k, v ([B, n_max, H_kv, d], token-major). */
int lckv_oracle_prefill_write_kv(uint16_t* K, uint16_t* V, const uint16_t* k, const uint16_t* v,
                                 const int32_t* lens, int B, int n_max, int H_kv, int64_t T_cap,
                                 int d)
{
    for (int b = 0; b < B; ++b)
        if (lens[b] < 0 || lens[b] > n_max || (int64_t)lens[b] > T_cap) return LCKV_ORACLE_ECAPACITY;
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < lens[b]; ++i)
            for (int h = 0; h < H_kv; ++h) {
                int64_t dst = ((((int64_t)b * H_kv + h) * T_cap) + i) * d;
                int64_t src = (((int64_t)b * n_max + i) * H_kv + h) * d;
                memcpy(K + dst, k + src, sizeof(uint16_t) * (size_t)d);
                memcpy(V + dst, v + src, sizeof(uint16_t) * (size_t)d);
            }
    return LCKV_ORACLE_OK;
}

/*
 * One parallel iteration over the whole layer stack (Section 2.2.1 / 2.3), following the same
 * layer plan as a decode step: a warmup layer first stores its k,v of this iteration in its own
 * cache and then attends causally (j <= i); a condensed layer attends j < i over the shared
 * cache, which still holds the previous iteration's top-layer k,v; at the end of the iteration the
 * feeder layer's k,v of this iteration replace them.  Lengths do not change.
 */
int lckv_oracle_prefill_iteration(int L, int w, int top_variant, const uint16_t* const* q_layers,
                                  const uint16_t* const* k_layers, const uint16_t* const* v_layers,
                                  uint16_t* const* K_slots, uint16_t* const* V_slots,
                                  const int32_t* lens, int B, int n_max, int H_q, int H_kv,
                                  int64_t T_cap, int d, double scale, int always_sink,
                                  double* const* out_layers)
{
    int32_t* plan = (int32_t*)malloc(sizeof(int32_t) * 5 * (size_t)L);
    if (!plan) return LCKV_ORACLE_EINVAL;
    int32_t *is_w = plan, *rs = plan + L, *md = plan + 2 * L, *ws = plan + 3 * L, *wb = plan + 4 * L;
    int32_t n_slots = 0;
    int rc = lckv_oracle_plan(L, w, top_variant, is_w, rs, md, ws, wb, &n_slots);
    for (int l = 0; l < L && rc == 0; ++l)
        if (ws[l] >= 0 && (!k_layers[l] || !v_layers[l])) rc = LCKV_ORACLE_EINVAL;
    for (int l = 0; l < L && rc == 0; ++l) {
        if (ws[l] >= 0 && wb[l])
            rc = lckv_oracle_prefill_write_kv(K_slots[ws[l]], V_slots[ws[l]], k_layers[l],
                                              v_layers[l], lens, B, n_max, H_kv, T_cap, d);
        if (rc) break;
        rc = lckv_oracle_prefill_attention(q_layers[l], K_slots[rs[l]], V_slots[rs[l]], lens, B,
                                           n_max, H_q, H_kv, T_cap, d, md[l], scale, always_sink,
                                           out_layers[l]);
    }
    for (int l = 0; l < L && rc == 0; ++l)
        if (ws[l] >= 0 && !wb[l])
            rc = lckv_oracle_prefill_write_kv(K_slots[ws[l]], V_slots[ws[l]], k_layers[l],
                                              v_layers[l], lens, B, n_max, H_kv, T_cap, d);
    free(plan);
    return rc;
}

/* float64 -> bf16 bits, round to nearest, ties to even (the one rounding of a produced key or
 * value on its way into the bf16 cache).  The value is first rounded to binary32 by the C
 * conversion (itself to nearest even); double rounding cannot differ from direct rounding here
 * except on exact binary32 ties, which the callers' magnitudes make measure-zero events, and the
 * comparison that uses these bits allows one bf16 unit anyway. */
static uint16_t f64_to_bf16(double x)
{
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40u); /* NaN stays NaN */
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7fffu + lsb;
    return (uint16_t)(u >> 16);
}

/*
 * Keys and values of the new token (Section 2.1: W_K, W_V map a hidden representation to its key
 * and value; in the condensed model only the layers that own a cache still do this):
 *   k[b, f] = sum_c W_K[f, c] x[b, c],   v[b, f] = sum_c W_V[f, c] x[b, c],
 *   x [B, d_model], W [H_kv * d, d_model] (row f = output feature, as a linear layer stores it),
 *   feature f = kv head f / d, dimension f mod d.
 * Optional position encoding of the key (the paper's models are Llama models, whose keys are
 * rotated by their position before they are cached; the paper does not restate it, so it is a
 * switch: cos == NULL leaves k as projected).  Rotary embedding in the half-split pairing: with
 * p = lens[b] the token's position and i < d/2,
 *   k'[i]       = k[i] cos[p, i] - k[i + d/2] sin[p, i]
 *   k'[i + d/2] = k[i + d/2] cos[p, i] + k[i] sin[p, i].
 * cos, sin [n_pos, d/2] are inputs (float32 values, widened exactly).
 * Outputs: k_bits, v_bits [B, H_kv, d] bf16 (one rounding from float64); k_f64, v_f64 (optional)
 * the unrounded values.
 */
int lckv_oracle_project_kv(const uint16_t* x, const uint16_t* w_k, const uint16_t* w_v,
                           const float* cos_tab, const float* sin_tab, int n_pos,
                           const int32_t* lens, int B, int H_kv, int d, int d_model,
                           uint16_t* k_bits, uint16_t* v_bits, double* k_f64, double* v_f64)
{
    if (B < 1 || H_kv < 1 || d < 2 || (d & 1) || d_model < 1) return LCKV_ORACLE_EINVAL;
    if ((cos_tab == NULL) != (sin_tab == NULL)) return LCKV_ORACLE_EINVAL;
    const int half = d / 2;
    if (cos_tab)
        for (int b = 0; b < B; ++b)
            if (lens[b] < 0 || lens[b] >= n_pos) return LCKV_ORACLE_EINVAL;
    const int64_t F = (int64_t)H_kv * d;
    double* kp = (double*)malloc(sizeof(double) * (size_t)((int64_t)B * F));   /* projected keys */
    if (!kp) return LCKV_ORACLE_EINVAL;
#pragma omp parallel for schedule(static)
    for (int64_t bf = 0; bf < (int64_t)B * F; ++bf) {
        const int64_t b = bf / F, f = bf % F;
        double ks = 0.0, vs = 0.0;
        for (int c = 0; c < d_model; ++c) {
            const double xc = bf16_to_f64(x[b * d_model + c]);
            ks += bf16_to_f64(w_k[f * d_model + c]) * xc;
            vs += bf16_to_f64(w_v[f * d_model + c]) * xc;
        }
        kp[bf] = ks;
        if (v_f64) v_f64[bf] = vs;
        v_bits[bf] = f64_to_bf16(vs);
    }
    for (int64_t bh = 0; bh < (int64_t)B * H_kv; ++bh) {
        const int64_t b = bh / H_kv;
        const int64_t p = lens[b];
        double* kh = kp + bh * d;                      /* one head of one sequence */
        for (int i = 0; i < half && cos_tab; ++i) {
            const double cs = (double)cos_tab[p * half + i], sn = (double)sin_tab[p * half + i];
            const double lo = kh[i], hi = kh[i + half];
            kh[i] = lo * cs - hi * sn;
            kh[i + half] = hi * cs + lo * sn;
        }
        for (int i = 0; i < d; ++i) {
            if (k_f64) k_f64[bh * d + i] = kh[i];
            k_bits[bh * d + i] = f64_to_bf16(kh[i]);
        }
    }
    free(kp);
    return LCKV_ORACLE_OK;
}
