/*
 * PowerAttention CPU oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 statement of what the block-sparse attention path computes, written
 * from the paper's definitions.  Nothing in the product library links, imports or calls this
 * file; only tests, the smoke check and the benchmark's CPU-baseline leg do.
 *
 *   - Mask predicate: Algorithm 1 (Section 3.3).  The sink term is generalised from one block
 *     (kv_idx < B) to `sink_blocks` blocks (kv_idx < sink_blocks * B); the paper's setting is 1.
 *     The switch `use_power` turns the power-of-two term off, which gives the sliding-window
 *     baseline of Section 3.2 / Section 4.1 (local window plus sink blocks) from the same code.
 *   - Attention: Eq. (1) (Section 3.1), softmax normalised over the attended set A_i only.
 *     Full causal attention is the special case A_i = {j <= i} (Section 3.1).
 *   - Decode: the same row computation at the last cached position (Section 4.1: the same
 *     pattern is used in prefilling and decoding).
 *
 * There is no blocking, tiling or fusion here: each query row materialises its dense boolean
 * mask row from the token-level predicate and then evaluates Eq. (1) over the set bits with a
 * max-subtracted softmax.  Inputs are bfloat16 bit patterns widened exactly to fp64.
 *
 * Parity pins for every function in this file live in tests/test_oracle_*.py; none is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* bfloat16 is the upper half of an IEEE-754 binary32. */
static double bf16_to_double(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* True for 0, 1, 2, 4, 8, ...: at most one bit set. */
static int is_zero_or_power_of_two(int64_t d) { return (d & (d - 1)) == 0; }

/*
 * The mask of Algorithm 1 (Section 3.3) for one (query, key) token pair.  A key after the query
 * is never attended.  Otherwise let d >= 0 be the distance between the B-token blocks that hold
 * the two tokens; the key is attended when its block lies inside the local window (d < W), at a
 * power-of-two block distance (or in the query's own block, d = 0), or among the first
 * sink_blocks * B tokens of the sequence.
 */
int pa_oracle_mask(int64_t q_idx, int64_t kv_idx, int64_t B, int64_t W, int64_t sink_blocks,
                   int use_power)
{
    if (kv_idx > q_idx) return 0;
    const int64_t d = q_idx / B - kv_idx / B;
    if (d < W) return 1;
    if (use_power && is_zero_or_power_of_two(d)) return 1;
    return kv_idx < sink_blocks * B;
}

/* Dense mask row of query q over kv in [0, n_keys): row[kv] in {0,1}. */
void pa_oracle_mask_row(int64_t q_idx, int64_t n_keys, int64_t B, int64_t W, int64_t sink_blocks,
                        int use_power, uint8_t *row)
{
    for (int64_t kv = 0; kv < n_keys; ++kv)
        row[kv] = (uint8_t)pa_oracle_mask(q_idx, kv, B, W, sink_blocks, use_power);
}

/*
 * One row of Eq. (1): o = sum_{kv in A} softmax_A(scale * <q, k_kv>) v_kv and
 * lse = ln sum_{kv in A} exp(scale * <q, k_kv>).  k, v are rows of D bf16 values `kv_stride`
 * elements apart.  `scores` is scratch of n_keys doubles.  Returns the number of attended keys.
 */
static int64_t attend_row(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                          int64_t kv_stride, int64_t n_keys, int64_t D, double scale,
                          const uint8_t *mask_row, double *scores, double *o, double *lse)
{
    double m = -INFINITY;
    int64_t cnt = 0;
    for (int64_t kv = 0; kv < n_keys; ++kv) {
        if (!mask_row[kv]) continue;
        const uint16_t *kr = k + kv * kv_stride;
        double s = 0.0;
        for (int64_t d = 0; d < D; ++d) s += bf16_to_double(q[d]) * bf16_to_double(kr[d]);
        s *= scale;
        scores[kv] = s;
        if (s > m) m = s;
        ++cnt;
    }
    for (int64_t d = 0; d < D; ++d) o[d] = 0.0;
    if (cnt == 0) { /* cannot happen under a causal mask that keeps kv == q */
        *lse = -INFINITY;
        return 0;
    }
    double l = 0.0;
    for (int64_t kv = 0; kv < n_keys; ++kv) {
        if (!mask_row[kv]) continue;
        double p = exp(scores[kv] - m);
        l += p;
        const uint16_t *vr = v + kv * kv_stride;
        for (int64_t d = 0; d < D; ++d) o[d] += p * bf16_to_double(vr[d]);
    }
    for (int64_t d = 0; d < D; ++d) o[d] /= l;
    *lse = m + log(l);
    return cnt;
}

/*
 * Prefill rows.  Q [batch, N, Hq, D], K and V [batch, N, Hkv, D], contiguous bf16 bit patterns.
 * Query head h reads KV head floor(h / (Hq / Hkv)).  Only the query positions listed in
 * q_rows[n_rows] and the heads listed in heads[n_heads] are evaluated (pass all of them for
 * the whole problem).  dense_mask, if non-NULL, is an explicit [N, N] byte mask used instead
 * of the predicate (for masks that are not Algorithm 1, e.g. comparison patterns).
 * Outputs: O [batch, n_rows, n_heads, D] fp64, LSE [batch, n_heads, n_rows] fp64,
 * n_attended [n_rows] int64 (may be NULL).
 */
void pa_oracle_prefill(const uint16_t *Q, const uint16_t *K, const uint16_t *V, int64_t batch,
                       int64_t N, int64_t Hq, int64_t Hkv, int64_t D, double scale, int64_t B,
                       int64_t W, int64_t sink_blocks, int use_power, const uint8_t *dense_mask,
                       const int64_t *q_rows, int64_t n_rows, const int64_t *heads,
                       int64_t n_heads, double *O, double *LSE, int64_t *n_attended,
                       int n_threads)
{
    const int64_t G = Hq / Hkv;
    const int64_t total = batch * n_rows;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
#pragma omp parallel
    {
        uint8_t *row = (uint8_t *)malloc((size_t)N);
        double *scores = (double *)malloc((size_t)N * sizeof(double));
#pragma omp for schedule(dynamic, 1)
        for (int64_t t = 0; t < total; ++t) {
            const int64_t b = t / n_rows, ri = t % n_rows;
            const int64_t q = q_rows[ri];
            if (dense_mask)
                memcpy(row, dense_mask + q * N, (size_t)N);
            else
                pa_oracle_mask_row(q, N, B, W, sink_blocks, use_power, row);
            for (int64_t hi = 0; hi < n_heads; ++hi) {
                const int64_t h = heads[hi], hk = h / G;
                const uint16_t *qv = Q + ((b * N + q) * Hq + h) * D;
                const uint16_t *kb = K + (b * N * Hkv + hk) * D;
                const uint16_t *vb = V + (b * N * Hkv + hk) * D;
                double lse;
                int64_t cnt = attend_row(qv, kb, vb, Hkv * D, N, D, scale, row, scores,
                                         O + ((b * n_rows + ri) * n_heads + hi) * D, &lse);
                LSE[(b * n_heads + hi) * n_rows + ri] = lse;
                if (n_attended && b == 0 && hi == 0) n_attended[ri] = cnt;
            }
        }
        free(row);
        free(scores);
    }
}

/*
 * Decode.  q [batch, Hq, D]; caches [batch, max_len, Hkv, D]; lens[batch] counts the cached
 * keys INCLUDING the current token, so the query sits at position lens[b] - 1 and attends to
 * itself (causal is q_idx >= kv_idx).  The attended set is the mask row of that position.
 * Outputs: O [batch, Hq, D] fp64, LSE [batch, Hq] fp64, n_attended [batch] (may be NULL).
 */
void pa_oracle_decode(const uint16_t *q, const uint16_t *Kc, const uint16_t *Vc,
                      const int64_t *lens, int64_t batch, int64_t max_len, int64_t Hq,
                      int64_t Hkv, int64_t D, double scale, int64_t B, int64_t W,
                      int64_t sink_blocks, int use_power, double *O, double *LSE,
                      int64_t *n_attended, int n_threads)
{
    const int64_t G = Hq / Hkv;
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
#pragma omp parallel
    {
        uint8_t *row = (uint8_t *)malloc((size_t)max_len);
        double *scores = (double *)malloc((size_t)max_len * sizeof(double));
#pragma omp for schedule(dynamic, 1)
        for (int64_t t = 0; t < batch * Hq; ++t) {
            const int64_t b = t / Hq, h = t % Hq, hk = h / G;
            const int64_t L = lens[b];
            pa_oracle_mask_row(L - 1, L, B, W, sink_blocks, use_power, row);
            double lse;
            int64_t cnt = attend_row(q + (b * Hq + h) * D, Kc + (b * max_len * Hkv + hk) * D,
                                     Vc + (b * max_len * Hkv + hk) * D, Hkv * D, L, D, scale,
                                     row, scores, O + (b * Hq + h) * D, &lse);
            LSE[b * Hq + h] = lse;
            if (n_attended && h == 0) n_attended[b] = cnt;
        }
        free(row);
        free(scores);
    }
}

int pa_oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Backward of Eq. (1) (the paper trains with the mask, Section 4.1; it prints no gradient formulas,
 * these follow from differentiating Eq. (1)).  For one query row i with attended set A, weights
 * p_j = softmax_A(scale <q, k_j>) and output o = sum_j p_j v_j, and an upstream gradient g = dL/do:
 *     dL/dv_j  = p_j g
 *     dL/dp_j  = <g, v_j>
 *     dL/ds_j  = p_j (dL/dp_j - sum_k p_k dL/dp_k)          (softmax over A)
 *     dL/dq    = scale sum_j dL/ds_j k_j
 *     dL/dk_j  = scale dL/ds_j q
 * dK and dV sum over the query rows that attend to key j and over the query heads that share its
 * KV head.  Two plain passes, neither with any blocking: rows (dQ, and the per-row log-sum-exp and
 * sum_k p_k dL/dp_k), then keys (dK, dV), each re-evaluating the mask predicate pair by pair.
 * Q, dO [batch, N, Hq, D]; K, V [batch, N, Hkv, D] bf16 bit patterns; outputs fp64, same shapes.
 * k_rows (n_krows of them; NULL = every key) restricts the second pass to those key positions: the
 * other rows of dK and dV are left as they are.  The first pass always covers every query row, since
 * a key's gradient needs the log-sum-exp of every row that attends to it.
 */
void pa_oracle_backward(const uint16_t *Q, const uint16_t *K, const uint16_t *V, const uint16_t *dO,
                        int64_t batch, int64_t N, int64_t Hq, int64_t Hkv, int64_t D, double scale,
                        int64_t B, int64_t W, int64_t sink_blocks, int use_power,
                        const uint8_t *dense_mask, const int64_t *k_rows, int64_t n_krows, double *dQ,
                        double *dK, double *dV, int n_threads)
{
    const int64_t n_keys_out = k_rows ? n_krows : N;
    const int64_t G = Hq / Hkv;
    double *lse = (double *)malloc((size_t)(batch * Hq * N) * sizeof(double));
    double *dsum = (double *)malloc((size_t)(batch * Hq * N) * sizeof(double));
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
#pragma omp parallel
    {
        double *s = (double *)malloc((size_t)N * sizeof(double));
        double *dp = (double *)malloc((size_t)N * sizeof(double));
#pragma omp for schedule(dynamic, 4)
        for (int64_t t = 0; t < batch * Hq * N; ++t) {
            const int64_t b = t / (Hq * N), h = (t / N) % Hq, i = t % N, hk = h / G;
            const uint16_t *q = Q + ((b * N + i) * Hq + h) * D;
            const uint16_t *g = dO + ((b * N + i) * Hq + h) * D;
            double m = -INFINITY;
            for (int64_t j = 0; j < N; ++j) {
                const int on = dense_mask ? dense_mask[i * N + j] : pa_oracle_mask(i, j, B, W, sink_blocks, use_power);
                s[j] = -INFINITY;
                if (!on) continue;
                const uint16_t *k = K + ((b * N + j) * Hkv + hk) * D;
                const uint16_t *v = V + ((b * N + j) * Hkv + hk) * D;
                double acc = 0.0, gv = 0.0;
                for (int64_t d = 0; d < D; ++d) {
                    acc += bf16_to_double(q[d]) * bf16_to_double(k[d]);
                    gv += bf16_to_double(g[d]) * bf16_to_double(v[d]);
                }
                s[j] = acc * scale;
                dp[j] = gv;
                if (s[j] > m) m = s[j];
            }
            double l = 0.0, pd = 0.0;
            for (int64_t j = 0; j < N; ++j)
                if (s[j] != -INFINITY) l += exp(s[j] - m);
            double *dq = dQ + ((b * N + i) * Hq + h) * D;
            for (int64_t d = 0; d < D; ++d) dq[d] = 0.0;
            if (l == 0.0) { /* empty row: no gradient flows */
                lse[t] = INFINITY;
                dsum[t] = 0.0;
                continue;
            }
            for (int64_t j = 0; j < N; ++j)
                if (s[j] != -INFINITY) pd += exp(s[j] - m) / l * dp[j];
            for (int64_t j = 0; j < N; ++j) {
                if (s[j] == -INFINITY) continue;
                const double ds = exp(s[j] - m) / l * (dp[j] - pd);
                const uint16_t *k = K + ((b * N + j) * Hkv + hk) * D;
                for (int64_t d = 0; d < D; ++d) dq[d] += scale * ds * bf16_to_double(k[d]);
            }
            lse[t] = m + log(l);
            dsum[t] = pd;
        }
#pragma omp for schedule(dynamic, 4)
        for (int64_t t = 0; t < batch * Hkv * n_keys_out; ++t) {
            const int64_t b = t / (Hkv * n_keys_out), hk = (t / n_keys_out) % Hkv;
            const int64_t j = k_rows ? k_rows[t % n_keys_out] : t % n_keys_out;
            const uint16_t *k = K + ((b * N + j) * Hkv + hk) * D;
            const uint16_t *v = V + ((b * N + j) * Hkv + hk) * D;
            double *dk = dK + ((b * N + j) * Hkv + hk) * D;
            double *dv = dV + ((b * N + j) * Hkv + hk) * D;
            for (int64_t d = 0; d < D; ++d) dk[d] = dv[d] = 0.0;
            for (int64_t h = hk * G; h < (hk + 1) * G; ++h)
                for (int64_t i = 0; i < N; ++i) {
                    const int on = dense_mask ? dense_mask[i * N + j] : pa_oracle_mask(i, j, B, W, sink_blocks, use_power);
                    if (!on) continue;
                    const uint16_t *q = Q + ((b * N + i) * Hq + h) * D;
                    const uint16_t *g = dO + ((b * N + i) * Hq + h) * D;
                    double acc = 0.0, gv = 0.0;
                    for (int64_t d = 0; d < D; ++d) {
                        acc += bf16_to_double(q[d]) * bf16_to_double(k[d]);
                        gv += bf16_to_double(g[d]) * bf16_to_double(v[d]);
                    }
                    const double p = exp(acc * scale - lse[(b * Hq + h) * N + i]);
                    const double ds = p * (gv - dsum[(b * Hq + h) * N + i]);
                    for (int64_t d = 0; d < D; ++d) {
                        dv[d] += p * bf16_to_double(g[d]);
                        dk[d] += scale * ds * bf16_to_double(q[d]);
                    }
                }
        }
        free(s);
        free(dp);
    }
    free(lse);
    free(dsum);
}
