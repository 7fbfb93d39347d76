/*
 * CPU oracle for composed-cache query prefill (KV Packet serving path).
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64, written from the paper's definitions:
 * nothing here is tiled, fused, blocked or shared with the CUDA path.  Only tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it.
 *
 *   kvp_oracle_rope_rows       Eq. 1 (Section 2.1): k^{S+Delta} = R_{Theta,Delta} k^S, one
 *                              rotation by the integer offset Delta per 2-D pair.
 *   kvp_oracle_attention_rows  Section 3.2 step 4 / Fig. 2(d): each query token attends, with a
 *                              softmax, to every token of the concatenated packet caches and to
 *                              the query tokens up to and including itself.
 *
 * Every part is pinned by the CPU tests (brute-force dense-mask attention, RoPE identities,
 * closed forms, ordinary causal prefill, permutation invariance): no function is "parity unpinned".
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int kvp_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Eq. 1.  x, y: [n_rows][n_heads][d] (y may alias x).  Row r is rotated by delta[r] positions:
 * for pair index i in [0, d/2) with angle a = delta[r] * inv_freq[i] (fp64),
 *     (u, w) -> (u cos a - w sin a,  u sin a + w cos a).
 * pairing 0: the pair is (x[i], x[i + d/2]);  pairing 1: the pair is (x[2i], x[2i+1]).
 * V is never passed here: Eq. 1 rotates keys (and queries) only.
 */
void kvp_oracle_rope_rows(const double *x, double *y, long long n_rows, int n_heads, int d,
                          int pairing, const double *inv_freq, const long long *delta)
{
    const int half = d / 2;
#pragma omp parallel for schedule(static)
    for (long long r = 0; r < n_rows; ++r) {
        for (int h = 0; h < n_heads; ++h) {
            const double *xi = x + ((size_t)r * n_heads + h) * d;
            double *yo = y + ((size_t)r * n_heads + h) * d;
            for (int i = 0; i < half; ++i) {
                const double a = (double)delta[r] * inv_freq[i];
                const double c = cos(a), s = sin(a);
                const int ia = pairing ? 2 * i : i;
                const int ib = pairing ? 2 * i + 1 : i + half;
                const double u = xi[ia], w = xi[ib];
                yo[ia] = u * c - w * s;
                yo[ib] = u * s + w * c;
            }
        }
    }
}

/*
 * Attention of selected query rows over [prefix || causal query block].
 *
 *   K, V : [n_keys_total][n_kv_heads][d], n_keys_total = prefix_len + q_len.  Rows
 *          [0, prefix_len) are the composed (already re-based) packet caches, rows
 *          prefix_len + j are the query chunk's own keys/values.
 *   Q    : [q_len][n_q_heads][d]
 *   row r of the request is the pair (head rows_h[r], query token rows_i[r]).
 *
 * Query token i sees keys j in [0, prefix_len + i]  (prefix fully visible, query block
 * lower-triangular with the diagonal).  q head h reads kv head floor(h / (Hq/Hkv)).
 * Two-pass softmax:  s_j = scale <q, K_j>;  m = max_j s_j;  p_j = exp(s_j - m);
 *   out = sum_j p_j V_j / sum_j p_j;   lse = m + log sum_j p_j.
 * prob_sum[r] (optional) receives sum_j (p_j / sum p) as actually formed, for the rows-sum-to-1 pin.
 */
void kvp_oracle_attention_rows(const double *K, const double *V, const double *Q,
                               long long prefix_len, int q_len, int n_q_heads, int n_kv_heads, int d,
                               double scale, const int *rows_h, const int *rows_i, long long n_rows,
                               double *out, double *lse, double *prob_sum)
{
    const int group = n_q_heads / n_kv_heads;
    (void)q_len;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(prefix_len + q_len + 1));
#pragma omp for schedule(dynamic, 4)
        for (long long r = 0; r < n_rows; ++r) {
            const int h = rows_h[r], i = rows_i[r];
            const int hk = h / group;
            const long long n_vis = prefix_len + i + 1;
            const double *q = Q + ((size_t)i * n_q_heads + h) * d;
            double m = -INFINITY;
            for (long long j = 0; j < n_vis; ++j) {
                const double *k = K + ((size_t)j * n_kv_heads + hk) * d;
                double acc = 0.0;
                for (int c = 0; c < d; ++c) acc += q[c] * k[c];
                s[j] = acc * scale;
                if (s[j] > m) m = s[j];
            }
            double l = 0.0;
            for (long long j = 0; j < n_vis; ++j) {
                s[j] = exp(s[j] - m);
                l += s[j];
            }
            double *o = out + (size_t)r * d;
            for (int c = 0; c < d; ++c) o[c] = 0.0;
            double ps = 0.0;
            for (long long j = 0; j < n_vis; ++j) {
                const double p = s[j] / l;
                ps += p;
                const double *v = V + ((size_t)j * n_kv_heads + hk) * d;
                for (int c = 0; c < d; ++c) o[c] += p * v[c];
            }
            if (lse) lse[r] = m + log(l);
            if (prob_sum) prob_sum[r] = ps;
        }
        free(s);
    }
}
