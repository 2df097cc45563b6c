/*
 * LAGA per-rank hot path -- fp64 CPU ORACLE.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, obviously-correct statement of what one sequence-parallel rank computes
 * after the latent all-gather (paper Algorithm 1, steps 4 and 5) and of its backward (paper
 * Section 5.2).  It exists so that the tests, the smoke check and the benchmark's CPU-baseline leg
 * have something independent to compare the CUDA library with.  It shares no code, header, table or
 * helper with the CUDA path, and the product never calls it.
 *
 * Because LAGA reaches exactly the result of the explicit MLA form (Section 5.1, Propositions 1-2:
 * the same linear maps applied to the same tensor), the oracle is that explicit definition written
 * out, one softmax row at a time, in double precision on the caller's bf16 input bits:
 *
 *   step 4   KV[t, i*(d_n+d_v)+j] = sum_c c_kv[t,c] * W[c, i*(d_n+d_v)+j]
 *            K[t,i,0:d_n] = KV[t,i,0:d_n]      V[t,i,:] = KV[t,i,d_n:d_n+d_v]
 *   (2.1)    K[t,i,d_n:d_n+d_r] = k_pe[t,:]    (the rope key is shared by every head)
 *   step 5   x[t] = scale * <q[s,i,:], K[t,i,:]> for allowed t (t <= s when causal)
 *            m = max x, l = sum exp(x-m), LSE[s,i] = m + ln l, P[t] = exp(x[t]-LSE)
 *            O[s,i,:] = sum_t P[t] V[t,i,:]
 *   backward (chain rule through step 5 then step 4, Section 5.2)
 *            delta = <dO[s,i,:], O[s,i,:]>, dP[t] = <dO[s,i,:], V[t,i,:]>, dS[t] = P[t](dP[t]-delta)
 *            dQ[s,i,:] = scale * sum_t dS[t] K[t,i,:]
 *            dK[t,i,:] = scale * sum_s dS[s,t] q[s,i,:]     dV[t,i,:] = sum_s P[s,t] dO[s,i,:]
 *            dk_pe[t,:] = sum_i dK[t,i,d_n:]                (shared band: sum over the head shard)
 *            dKV[t, i*(d_n+d_v)+j] = dK[t,i,j] (j<d_n) | dV[t,i,j-d_n]
 *            dc_kv[t,c] = sum_n dKV[t,n] W[c,n]             dW[c,n] = sum_t c_kv[t,c] dKV[t,n]
 *
 * Readings where the paper is silent: the causal mask (t <= s), the softmax scale passed in by the
 * caller, the per-head interleaved column order of the W_kv_b shard, and natural-log LSE of the
 * scaled scores.  `kv_round_bf16` rounds K_nope and V to bf16 (round-to-nearest-even, straight from
 * fp64) after step 4: that is the explicit form as it runs in bf16, where per-head K/V are bf16
 * tensors.  The backward uses the oracle's own fp64 O.
 *
 * Pinned by tests that do not use this file's own arithmetic: brute-force S x S softmax, library
 * SDPA + autograd in fp64, finite differences, closed forms (q=0, S=1, row 0), the absorbed-form
 * identity, head-shard concatenation and trace identities.  No function here is "parity unpinned".
 *
 * All matrices are row-major, all pointers are host pointers, bf16 values are passed as uint16_t
 * bit patterns, every result is double.  Returns 0 on success, -1 on bad arguments, -2 on
 * allocation failure.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_bits_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* Round a double to the nearest bf16-representable value, ties to even, without going through
 * fp32 (which would round twice).  bf16 keeps 8 significant bits; its normal exponent range is
 * that of fp32, below which the spacing is fixed at 2^-133. */
double laga_oracle_round_bf16(double x) {
    if (x == 0.0 || isnan(x) || isinf(x)) return x;
    int e;
    (void)frexp(x, &e);            /* |x| = m * 2^e, m in [0.5, 1) */
    int ulp_exp = e - 8;           /* spacing of 8-significant-bit numbers around x */
    if (ulp_exp < -133) ulp_exp = -133;
    double scaled = ldexp(x, -ulp_exp);
    double r = nearbyint(scaled);  /* default rounding mode: to nearest, ties to even */
    double y = ldexp(r, ulp_exp);
    if (fabs(y) > 3.3895313892515355e38) y = copysign(INFINITY, x);
    return y;
}

int laga_oracle_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Algorithm 1 step 4 plus the key assembly of Section 2.1.
 * K: [h][S][d_n+d_r], V: [h][S][d_v] (head-major so one head's rows are contiguous). */
static void up_project(const uint16_t* c_kv, const uint16_t* k_pe, const uint16_t* w, int S, int h,
                       int d_c, int d_n, int d_r, int d_v, int kv_round_bf16, double* K, double* V) {
    const int d_qk = d_n + d_r, per_head = d_n + d_v, N = h * per_head;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < S; ++t) {
        for (int i = 0; i < h; ++i) {
            for (int j = 0; j < per_head; ++j) {
                double acc = 0.0;
                for (int c = 0; c < d_c; ++c)
                    acc += bf16_bits_to_f64(c_kv[(size_t)t * d_c + c]) *
                           bf16_bits_to_f64(w[(size_t)c * N + (size_t)i * per_head + j]);
                if (kv_round_bf16) acc = laga_oracle_round_bf16(acc);
                if (j < d_n) K[((size_t)i * S + t) * d_qk + j] = acc;
                else         V[((size_t)i * S + t) * d_v + (j - d_n)] = acc;
            }
            for (int r = 0; r < d_r; ++r)
                K[((size_t)i * S + t) * d_qk + d_n + r] = bf16_bits_to_f64(k_pe[(size_t)t * d_r + r]);
        }
    }
}

/* One softmax row of step 5: fills x[0..n_keys) with P, returns LSE.  n_keys = s+1 (causal) or S. */
static double softmax_row(const uint16_t* q_row, const double* K_head, int n_keys, int d_qk,
                          double scale, double* x) {
    double m = -INFINITY;
    for (int t = 0; t < n_keys; ++t) {
        double acc = 0.0;
        for (int d = 0; d < d_qk; ++d) acc += bf16_bits_to_f64(q_row[d]) * K_head[(size_t)t * d_qk + d];
        x[t] = scale * acc;
        if (x[t] > m) m = x[t];
    }
    double l = 0.0;
    for (int t = 0; t < n_keys; ++t) l += exp(x[t] - m);
    double lse = m + log(l);
    for (int t = 0; t < n_keys; ++t) x[t] = exp(x[t] - lse);
    return lse;
}

/* Forward for a chosen list of query rows (rows == NULL means all S rows, n_rows ignored).
 * out: [n_rows][h][d_v], lse: [n_rows][h].  k_nope_out [S][h][d_n] and v_out [S][h][d_v] are
 * optional (NULL to skip) copies of step 4's result. */
int laga_oracle_fwd_rows(const uint16_t* q, const uint16_t* c_kv, const uint16_t* k_pe,
                         const uint16_t* w_kv_b, int S, int h, int d_c, int d_nope, int d_rope,
                         int d_v, double softmax_scale, int causal, int kv_round_bf16,
                         const int* rows, int n_rows, double* out, double* lse, double* k_nope_out,
                         double* v_out) {
    if (!q || !c_kv || !k_pe || !w_kv_b || !out || !lse) return -1;
    if (S < 1 || h < 1 || d_c < 1 || d_nope < 1 || d_rope < 0 || d_v < 1) return -1;
    if (!rows) n_rows = S;
    const int d_qk = d_nope + d_rope;
    double* K = (double*)malloc(sizeof(double) * (size_t)h * S * d_qk);
    double* V = (double*)malloc(sizeof(double) * (size_t)h * S * d_v);
    if (!K || !V) { free(K); free(V); return -2; }
    up_project(c_kv, k_pe, w_kv_b, S, h, d_c, d_nope, d_rope, d_v, kv_round_bf16, K, V);
    if (k_nope_out)
        for (int t = 0; t < S; ++t) for (int i = 0; i < h; ++i) for (int j = 0; j < d_nope; ++j)
            k_nope_out[((size_t)t * h + i) * d_nope + j] = K[((size_t)i * S + t) * d_qk + j];
    if (v_out)
        for (int t = 0; t < S; ++t) for (int i = 0; i < h; ++i) for (int j = 0; j < d_v; ++j)
            v_out[((size_t)t * h + i) * d_v + j] = V[((size_t)i * S + t) * d_v + j];
    int fail = 0;
#pragma omp parallel
    {
        double* x = (double*)malloc(sizeof(double) * (size_t)S);
        if (!x) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for collapse(2) schedule(dynamic, 4)
            for (int r = 0; r < n_rows; ++r) {
                for (int i = 0; i < h; ++i) {
                    const int s = rows ? rows[r] : r;
                    const int n_keys = causal ? s + 1 : S;
                    const double* Kh = K + (size_t)i * S * d_qk;
                    const double* Vh = V + (size_t)i * S * d_v;
                    lse[(size_t)r * h + i] =
                        softmax_row(q + ((size_t)s * h + i) * d_qk, Kh, n_keys, d_qk, softmax_scale, x);
                    double* o = out + ((size_t)r * h + i) * d_v;
                    for (int j = 0; j < d_v; ++j) o[j] = 0.0;
                    for (int t = 0; t < n_keys; ++t)
                        for (int j = 0; j < d_v; ++j) o[j] += x[t] * Vh[(size_t)t * d_v + j];
                }
            }
        }
        free(x);
    }
    free(K); free(V);
    return fail ? -2 : 0;
}

/* Backward restricted to a list of query rows: dq [n_rows][h][d_n+d_r] (a row of dQ depends on that
 * query row only), plus the forward values out [n_rows][h][d_v] and lse [n_rows][h] it used. */
int laga_oracle_bwd_rows(const uint16_t* q, const uint16_t* c_kv, const uint16_t* k_pe,
                         const uint16_t* w_kv_b, const uint16_t* dout, int S, int h, int d_c, int d_nope,
                         int d_rope, int d_v, double softmax_scale, int causal, int kv_round_bf16,
                         const int* rows, int n_rows, double* dq, double* out, double* lse) {
    if (!q || !c_kv || !k_pe || !w_kv_b || !dout || !rows || !dq || !out || !lse) return -1;
    if (S < 1 || h < 1 || d_c < 1 || d_nope < 1 || d_rope < 0 || d_v < 1 || n_rows < 1) return -1;
    for (int r = 0; r < n_rows; ++r) if (rows[r] < 0 || rows[r] >= S) return -1;
    const int d_qk = d_nope + d_rope;
    double* K = (double*)malloc(sizeof(double) * (size_t)h * S * d_qk);
    double* V = (double*)malloc(sizeof(double) * (size_t)h * S * d_v);
    int fail = (!K || !V);
    if (fail) goto done;
    up_project(c_kv, k_pe, w_kv_b, S, h, d_c, d_nope, d_rope, d_v, kv_round_bf16, K, V);
#pragma omp parallel
    {
        double* x = (double*)malloc(sizeof(double) * (size_t)S);
        if (!x) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for collapse(2) schedule(dynamic, 1)
            for (int r = 0; r < n_rows; ++r) {
                for (int i = 0; i < h; ++i) {
                    const int s = rows[r];
                    const int n_allowed = causal ? s + 1 : S;
                    const double* Kh = K + (size_t)i * S * d_qk;
                    const double* Vh = V + (size_t)i * S * d_v;
                    const uint16_t* do_row = dout + ((size_t)s * h + i) * d_v;
                    double* o = out + ((size_t)r * h + i) * d_v;
                    double* dq_row = dq + ((size_t)r * h + i) * d_qk;
                    lse[(size_t)r * h + i] =
                        softmax_row(q + ((size_t)s * h + i) * d_qk, Kh, n_allowed, d_qk, softmax_scale, x);
                    for (int j = 0; j < d_v; ++j) o[j] = 0.0;
                    for (int t = 0; t < n_allowed; ++t)
                        for (int j = 0; j < d_v; ++j) o[j] += x[t] * Vh[(size_t)t * d_v + j];
                    double delta = 0.0;
                    for (int j = 0; j < d_v; ++j) delta += bf16_bits_to_f64(do_row[j]) * o[j];
                    for (int d = 0; d < d_qk; ++d) dq_row[d] = 0.0;
                    for (int t = 0; t < n_allowed; ++t) {
                        double dp = 0.0;
                        for (int j = 0; j < d_v; ++j) dp += bf16_bits_to_f64(do_row[j]) * Vh[(size_t)t * d_v + j];
                        double ds = x[t] * (dp - delta);
                        for (int d = 0; d < d_qk; ++d) dq_row[d] += softmax_scale * ds * Kh[(size_t)t * d_qk + d];
                    }
                }
            }
        }
        free(x);
    }
done:
    free(K); free(V);
    return fail ? -2 : 0;
}

/* Backward restricted to a list of key positions (for spot checks at sizes where the full backward
 * takes minutes).  For each listed key t it returns the same numbers the full backward would:
 * dk [n_keys][h][d_n+d_r], dv [n_keys][h][d_v], dk_pe [n_keys][d_r], dc_kv [n_keys][d_c].
 * Only the query rows that can attend to a listed key are visited (s >= min key when causal). */
int laga_oracle_bwd_keys(const uint16_t* q, const uint16_t* c_kv, const uint16_t* k_pe,
                         const uint16_t* w_kv_b, const uint16_t* dout, int S, int h, int d_c, int d_nope,
                         int d_rope, int d_v, double softmax_scale, int causal, int kv_round_bf16,
                         const int* keys, int n_keys, double* dk, double* dv, double* dk_pe,
                         double* dc_kv) {
    if (!q || !c_kv || !k_pe || !w_kv_b || !dout || !keys || !dk || !dv || !dk_pe || !dc_kv) return -1;
    if (S < 1 || h < 1 || d_c < 1 || d_nope < 1 || d_rope < 0 || d_v < 1 || n_keys < 1) return -1;
    const int d_qk = d_nope + d_rope, per_head = d_nope + d_v, N = h * per_head;
    int s_first = 0;
    if (causal) {
        s_first = keys[0];
        for (int k = 1; k < n_keys; ++k) if (keys[k] < s_first) s_first = keys[k];
    }
    for (int k = 0; k < n_keys; ++k) if (keys[k] < 0 || keys[k] >= S) return -1;
    double* K = (double*)malloc(sizeof(double) * (size_t)h * S * d_qk);
    double* V = (double*)malloc(sizeof(double) * (size_t)h * S * d_v);
    double* L = (double*)malloc(sizeof(double) * (size_t)h * S);
    double* D = (double*)malloc(sizeof(double) * (size_t)h * S);
    int fail = (!K || !V || !L || !D);
    if (fail) goto done;
    up_project(c_kv, k_pe, w_kv_b, S, h, d_c, d_nope, d_rope, d_v, kv_round_bf16, K, V);
#pragma omp parallel
    {
        double* x = (double*)malloc(sizeof(double) * (size_t)S);
        double* o = (double*)malloc(sizeof(double) * (size_t)d_v);
        if (!x || !o) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for collapse(2) schedule(dynamic, 4)
            for (int s = s_first; s < S; ++s) {
                for (int i = 0; i < h; ++i) {
                    const int n_allowed = causal ? s + 1 : S;
                    const double* Kh = K + (size_t)i * S * d_qk;
                    const double* Vh = V + (size_t)i * S * d_v;
                    const uint16_t* do_row = dout + ((size_t)s * h + i) * d_v;
                    L[(size_t)i * S + s] =
                        softmax_row(q + ((size_t)s * h + i) * d_qk, Kh, n_allowed, d_qk, softmax_scale, x);
                    for (int j = 0; j < d_v; ++j) o[j] = 0.0;
                    for (int t = 0; t < n_allowed; ++t)
                        for (int j = 0; j < d_v; ++j) o[j] += x[t] * Vh[(size_t)t * d_v + j];
                    double delta = 0.0;
                    for (int j = 0; j < d_v; ++j) delta += bf16_bits_to_f64(do_row[j]) * o[j];
                    D[(size_t)i * S + s] = delta;
                }
            }
        }
        free(x); free(o);
    }
    if (fail) goto done;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int k = 0; k < n_keys; ++k) {
        for (int i = 0; i < h; ++i) {
            const int t = keys[k];
            const double* Kh = K + (size_t)i * S * d_qk;
            const double* Vh = V + (size_t)i * S * d_v;
            double* dk_row = dk + ((size_t)k * h + i) * d_qk;
            double* dv_row = dv + ((size_t)k * h + i) * d_v;
            for (int d = 0; d < d_qk; ++d) dk_row[d] = 0.0;
            for (int j = 0; j < d_v; ++j) dv_row[j] = 0.0;
            for (int s = causal ? t : 0; s < S; ++s) {
                const uint16_t* q_row = q + ((size_t)s * h + i) * d_qk;
                const uint16_t* do_row = dout + ((size_t)s * h + i) * d_v;
                double acc = 0.0;
                for (int d = 0; d < d_qk; ++d) acc += bf16_bits_to_f64(q_row[d]) * Kh[(size_t)t * d_qk + d];
                double p = exp(softmax_scale * acc - L[(size_t)i * S + s]);
                double dp = 0.0;
                for (int j = 0; j < d_v; ++j) dp += bf16_bits_to_f64(do_row[j]) * Vh[(size_t)t * d_v + j];
                double ds = p * (dp - D[(size_t)i * S + s]);
                for (int d = 0; d < d_qk; ++d) dk_row[d] += softmax_scale * ds * bf16_bits_to_f64(q_row[d]);
                for (int j = 0; j < d_v; ++j) dv_row[j] += p * bf16_bits_to_f64(do_row[j]);
            }
        }
    }
    for (int k = 0; k < n_keys; ++k) {
        for (int r = 0; r < d_rope; ++r) {
            double acc = 0.0;
            for (int i = 0; i < h; ++i) acc += dk[((size_t)k * h + i) * d_qk + d_nope + r];
            dk_pe[(size_t)k * d_rope + r] = acc;
        }
        for (int c = 0; c < d_c; ++c) {
            double acc = 0.0;
            for (int i = 0; i < h; ++i)
                for (int j = 0; j < per_head; ++j) {
                    double g = (j < d_nope) ? dk[((size_t)k * h + i) * d_qk + j]
                                            : dv[((size_t)k * h + i) * d_v + (j - d_nope)];
                    acc += g * bf16_bits_to_f64(w_kv_b[(size_t)c * N + (size_t)i * per_head + j]);
                }
            dc_kv[(size_t)k * d_c + c] = acc;
        }
    }
done:
    free(K); free(V); free(L); free(D);
    return fail ? -2 : 0;
}

/* Backward.  Outputs: dq [S][h][d_n+d_r], dc_kv [S][d_c], dk_pe [S][d_r], dw [d_c][h*(d_n+d_v)].
 * Optional (NULL to skip): out [S][h][d_v], lse [S][h] (the forward it differentiates), and
 * dk_full [S][h][d_n+d_r], dv_full [S][h][d_v] (the per-head K/V gradients before they are
 * contracted back through W_kv_b). */
int laga_oracle_bwd(const uint16_t* q, const uint16_t* c_kv, const uint16_t* k_pe,
                    const uint16_t* w_kv_b, const uint16_t* dout, int S, int h, int d_c, int d_nope,
                    int d_rope, int d_v, double softmax_scale, int causal, int kv_round_bf16,
                    double* dq, double* dc_kv, double* dk_pe, double* dw, double* out, double* lse,
                    double* dk_full, double* dv_full) {
    if (!q || !c_kv || !k_pe || !w_kv_b || !dout || !dq || !dc_kv || !dk_pe || !dw) return -1;
    if (S < 1 || h < 1 || d_c < 1 || d_nope < 1 || d_rope < 0 || d_v < 1) return -1;
    const int d_qk = d_nope + d_rope, per_head = d_nope + d_v, N = h * per_head;
    double* K = (double*)malloc(sizeof(double) * (size_t)h * S * d_qk);
    double* V = (double*)malloc(sizeof(double) * (size_t)h * S * d_v);
    double* L = (double*)malloc(sizeof(double) * (size_t)h * S);     /* LSE   [h][S] */
    double* D = (double*)malloc(sizeof(double) * (size_t)h * S);     /* delta [h][S] */
    double* dK = (double*)calloc((size_t)h * S * d_qk, sizeof(double));
    double* dV = (double*)calloc((size_t)h * S * d_v, sizeof(double));
    int fail = (!K || !V || !L || !D || !dK || !dV);
    if (fail) goto done;
    up_project(c_kv, k_pe, w_kv_b, S, h, d_c, d_nope, d_rope, d_v, kv_round_bf16, K, V);

    /* Pass over query rows: forward row, delta, dS row, dQ. */
#pragma omp parallel
    {
        double* x = (double*)malloc(sizeof(double) * (size_t)S);
        double* o = (double*)malloc(sizeof(double) * (size_t)d_v);
        if (!x || !o) {
#pragma omp atomic write
            fail = 1;
        }
#pragma omp barrier
        if (!fail) {
#pragma omp for collapse(2) schedule(dynamic, 4)
            for (int s = 0; s < S; ++s) {
                for (int i = 0; i < h; ++i) {
                    const int n_keys = causal ? s + 1 : S;
                    const double* Kh = K + (size_t)i * S * d_qk;
                    const double* Vh = V + (size_t)i * S * d_v;
                    const uint16_t* q_row = q + ((size_t)s * h + i) * d_qk;
                    const uint16_t* do_row = dout + ((size_t)s * h + i) * d_v;
                    double row_lse = softmax_row(q_row, Kh, n_keys, d_qk, softmax_scale, x);
                    for (int j = 0; j < d_v; ++j) o[j] = 0.0;
                    for (int t = 0; t < n_keys; ++t)
                        for (int j = 0; j < d_v; ++j) o[j] += x[t] * Vh[(size_t)t * d_v + j];
                    double delta = 0.0;
                    for (int j = 0; j < d_v; ++j) delta += bf16_bits_to_f64(do_row[j]) * o[j];
                    L[(size_t)i * S + s] = row_lse;
                    D[(size_t)i * S + s] = delta;
                    if (out) for (int j = 0; j < d_v; ++j) out[((size_t)s * h + i) * d_v + j] = o[j];
                    if (lse) lse[(size_t)s * h + i] = row_lse;
                    double* dq_row = dq + ((size_t)s * h + i) * d_qk;
                    for (int d = 0; d < d_qk; ++d) dq_row[d] = 0.0;
                    for (int t = 0; t < n_keys; ++t) {
                        double dp = 0.0;
                        for (int j = 0; j < d_v; ++j)
                            dp += bf16_bits_to_f64(do_row[j]) * Vh[(size_t)t * d_v + j];
                        double ds = x[t] * (dp - delta);
                        for (int d = 0; d < d_qk; ++d)
                            dq_row[d] += softmax_scale * ds * Kh[(size_t)t * d_qk + d];
                    }
                }
            }
        }
        free(x); free(o);
    }
    if (fail) goto done;

    /* Pass over keys: dK[t], dV[t] as sums over the query rows that attend to t. */
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
    for (int t = 0; t < S; ++t) {
        for (int i = 0; i < h; ++i) {
            const double* Kh = K + (size_t)i * S * d_qk;
            const double* Vh = V + (size_t)i * S * d_v;
            double* dk_row = dK + ((size_t)i * S + t) * d_qk;
            double* dv_row = dV + ((size_t)i * S + t) * d_v;
            const int s_begin = causal ? t : 0;
            for (int s = s_begin; s < S; ++s) {
                const uint16_t* q_row = q + ((size_t)s * h + i) * d_qk;
                const uint16_t* do_row = dout + ((size_t)s * h + i) * d_v;
                double acc = 0.0;
                for (int d = 0; d < d_qk; ++d)
                    acc += bf16_bits_to_f64(q_row[d]) * Kh[(size_t)t * d_qk + d];
                double p = exp(softmax_scale * acc - L[(size_t)i * S + s]);
                double dp = 0.0;
                for (int j = 0; j < d_v; ++j)
                    dp += bf16_bits_to_f64(do_row[j]) * Vh[(size_t)t * d_v + j];
                double ds = p * (dp - D[(size_t)i * S + s]);
                for (int d = 0; d < d_qk; ++d)
                    dk_row[d] += softmax_scale * ds * bf16_bits_to_f64(q_row[d]);
                for (int j = 0; j < d_v; ++j) dv_row[j] += p * bf16_bits_to_f64(do_row[j]);
            }
        }
    }
    if (dk_full)
        for (int t = 0; t < S; ++t) for (int i = 0; i < h; ++i) for (int d = 0; d < d_qk; ++d)
            dk_full[((size_t)t * h + i) * d_qk + d] = dK[((size_t)i * S + t) * d_qk + d];
    if (dv_full)
        for (int t = 0; t < S; ++t) for (int i = 0; i < h; ++i) for (int j = 0; j < d_v; ++j)
            dv_full[((size_t)t * h + i) * d_v + j] = dV[((size_t)i * S + t) * d_v + j];

    /* Shared rope band: its gradient is the sum over this shard's heads (Section 5.3). */
#pragma omp parallel for schedule(static)
    for (int t = 0; t < S; ++t)
        for (int r = 0; r < d_rope; ++r) {
            double acc = 0.0;
            for (int i = 0; i < h; ++i) acc += dK[((size_t)i * S + t) * d_qk + d_nope + r];
            dk_pe[(size_t)t * d_rope + r] = acc;
        }

    /* Back through step 4: dKV = (dK_nope | dV) per head, then the two contractions with W and c_kv. */
#pragma omp parallel for schedule(static)
    for (int t = 0; t < S; ++t)
        for (int c = 0; c < d_c; ++c) {
            double acc = 0.0;
            for (int i = 0; i < h; ++i)
                for (int j = 0; j < per_head; ++j) {
                    double g = (j < d_nope) ? dK[((size_t)i * S + t) * d_qk + j]
                                            : dV[((size_t)i * S + t) * d_v + (j - d_nope)];
                    acc += g * bf16_bits_to_f64(w_kv_b[(size_t)c * N + (size_t)i * per_head + j]);
                }
            dc_kv[(size_t)t * d_c + c] = acc;
        }
#pragma omp parallel for collapse(2) schedule(static)
    for (int c = 0; c < d_c; ++c)
        for (int n = 0; n < N; ++n) {
            const int i = n / per_head, j = n % per_head;
            double acc = 0.0;
            for (int t = 0; t < S; ++t) {
                double g = (j < d_nope) ? dK[((size_t)i * S + t) * d_qk + j]
                                        : dV[((size_t)i * S + t) * d_v + (j - d_nope)];
                acc += bf16_bits_to_f64(c_kv[(size_t)t * d_c + c]) * g;
            }
            dw[(size_t)c * N + n] = acc;
        }
done:
    free(K); free(V); free(L); free(D); free(dK); free(dV);
    return fail ? -2 : 0;
}
