/*
 * CPU oracle for the SQuat KV-cache write path  --  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, single-threaded restatement of what the path computes, in fp64 (the
 * value quantizer is in IEEE binary32 because its result is compared bit for bit).
 * It shares no code with the CUDA library and is never called by it; only the tests,
 * the smoke check and the benchmark's CPU-baseline leg may use it.
 *
 * Each function follows one passage of the paper (SQuat, arXiv 2503.24358), in the
 * paper's order and notation, without blocking, fusion or reordering:
 *
 *   sqo_gram, sqo_jacobi_eig, sqo_query_subspace   Section 3.2, Algorithm 1 lines 5-6,
 *                                                  GQA rule of Appendix C
 *   sqo_update_matrices                            Prop. 1, Prop. 2, Lemma 3, Lemma 4,
 *                                                  Remark after Lemma 4, Alg. 1 lines 7-9
 *   sqo_quant_keys                                 Algorithm 1, function Quant; Eq. (3),
 *                                                  Eq. (update_block); Section 2 "Quantization"
 *   sqo_quant_values_f32 / _f64                    Section 2 "Quantization", Appendix C
 *                                                  (per-token value quantization)
 *   sqo_quant_keys_m16, sqo_quant_values_f32_m16,  the same with scale and zero-point stored in 16 bits
 *   sqo_half_round                                 (IEEE binary16, round to nearest even)
 *   sqo_dequant_keys / sqo_dequant_values          Section 2, deq(.)
 *   sqo_pack / sqo_unpack                          cache layout (the paper gives none; ours)
 *   sqo_kv_cache_bytes                             Appendix B, memory formula
 *   sqo_attention_decode                           Section 2 "(Masked) Attention mechanism": one decode step,
 *                                                  softmax(q K^T / sqrt(d)) V over the cached tokens (the
 *                                                  score vector w^deq of the proof of Theorem 1)
 *   sqo_rope_rows                                  Section 4, the variant that stores keys before the rotary
 *                                                  position embedding: the embedding a reader applies to
 *                                                  the dequantized rows (rotation of the channel pairs
 *                                                  (i, i + d/2) by pos * base^(-2i/d))
 *
 * Pins (tests, CPU only): the chain of Lemma 4 against direct inverses; B_t H_t against a
 * generic KKT solve of Eq. (2) and against the LDL^T factor of P_inv; lambda = 0 / r = 0
 * against ordinary round-to-nearest; the invariant delta^T P delta = e^T D^-1 e; idempotence;
 * chunking invariance; exhaustive search on tiny problems; the subspace against a library
 * SVD; the value path against a library float32 computation; the memory formula against
 * the worked example printed in Appendix B; the decode-step attention against a loop-by-loop
 * restatement, its closed forms (zero query = mean of the values, one dominant score) and the
 * bound of Theorem 1; the rotary embedding against explicit 2 x 2 rotation matrices, position 0,
 * norms, and the relative-position property of the scores.  The paper prints no input/output
 * pair for the quantizer itself.
 *
 * Readings of the paper where it is silent (same list as the design notes):
 *   - rounding is round-half-to-even;
 *   - a constant group (max = min) gets scale 0, all codes 0;
 *   - the grid of channel j is taken from the values AFTER the corrections of channels < j
 *     (Eq. (2) quantizes [k_{t-1}]_t; line order of Quant);
 *   - the value fed back is the one a reader of the cache reconstructs, i.e. computed from
 *     the stored float32 scale and zero-point;
 *   - scale and zero-point are stored as float32; in the 16-bit variant (the "KV size" columns of
 *     Tables 1-2 imply 16-bit metadata) they are stored as IEEE binary16: the float32 values rounded
 *     once more to nearest-even, and the rounding decision and the value fed back use the STORED
 *     values, so codes are clamped to [0, L] (a rounded zero-point can lie above the minimum);
 *   - channels are visited in natural order;
 *   - the rotary embedding (the paper only names it) pairs channel i with channel i + d/2 and
 *     uses the angles pos * base^(-2i/d), i < d/2: the convention of the Llama family the
 *     paper evaluates.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define SQO_OK 0
#define SQO_ERR_ARG 1
#define SQO_ERR_ALLOC 2
#define SQO_ERR_NUMERIC 3

/* ------------------------------------------------------------------------------------ */
/* Section 3.2 / Algorithm 1 line 5: Gram matrix M = Qc^T Qc of the stacked queries.      */
/* Qc is [N, d] row-major (all prompt tokens of all query heads that feed one KV head,    */
/* Appendix C "grouped-query attention").  M is [d, d].                                   */
int sqo_gram(const double *Qc, long N, int d, double *M)
{
    if (!Qc || !M || N < 0 || d <= 0) return SQO_ERR_ARG;
    for (int a = 0; a < d; ++a)
        for (int b = 0; b < d; ++b) M[a * d + b] = 0.0;
    for (long n = 0; n < N; ++n) {
        const double *q = Qc + n * d;
        for (int a = 0; a < d; ++a)
            for (int b = 0; b < d; ++b) M[a * d + b] += q[a] * q[b];
    }
    return SQO_OK;
}

/* Cyclic Jacobi eigen-decomposition of a symmetric matrix (textbook; Rutishauser's       */
/* rotation formulas).  On return mu[0] >= mu[1] >= ... and row i of V is the unit         */
/* eigenvector of mu[i].  A is destroyed.  Equal eigenvalues keep their original order.    */
int sqo_jacobi_eig(double *A, int d, double *mu, double *V)
{
    if (!A || !mu || !V || d <= 0) return SQO_ERR_ARG;
    /* E holds eigenvectors as columns while iterating */
    double *E = (double *)malloc(sizeof(double) * d * d);
    if (!E) return SQO_ERR_ALLOC;
    for (int i = 0; i < d; ++i)
        for (int j = 0; j < d; ++j) E[i * d + j] = (i == j) ? 1.0 : 0.0;
    double fro = 0.0;
    for (int i = 0; i < d * d; ++i) fro += A[i] * A[i];
    fro = sqrt(fro);
    for (int sweep = 0; sweep < 100; ++sweep) {
        double off = 0.0;
        for (int p = 0; p < d; ++p)
            for (int q = p + 1; q < d; ++q) off += 2.0 * A[p * d + q] * A[p * d + q];
        if (sqrt(off) <= 1e-15 * fro) break;
        for (int p = 0; p < d - 1; ++p) {
            for (int q = p + 1; q < d; ++q) {
                double apq = A[p * d + q];
                if (apq == 0.0) continue;
                double app = A[p * d + p], aqq = A[q * d + q];
                double theta = (aqq - app) / (2.0 * apq);
                double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
                double c = 1.0 / sqrt(t * t + 1.0), s = t * c;
                /* A <- J^T A J with J = [[c, s], [-s, c]] on the (p, q) plane */
                for (int k = 0; k < d; ++k) {
                    double akp = A[k * d + p], akq = A[k * d + q];
                    A[k * d + p] = c * akp - s * akq;
                    A[k * d + q] = s * akp + c * akq;
                }
                for (int k = 0; k < d; ++k) {
                    double apk = A[p * d + k], aqk = A[q * d + k];
                    A[p * d + k] = c * apk - s * aqk;
                    A[q * d + k] = s * apk + c * aqk;
                }
                for (int k = 0; k < d; ++k) {
                    double ekp = E[k * d + p], ekq = E[k * d + q];
                    E[k * d + p] = c * ekp - s * ekq;
                    E[k * d + q] = s * ekp + c * ekq;
                }
            }
        }
    }
    /* stable selection sort of the diagonal, descending */
    int *idx = (int *)malloc(sizeof(int) * d);
    if (!idx) { free(E); return SQO_ERR_ALLOC; }
    for (int i = 0; i < d; ++i) idx[i] = i;
    for (int i = 1; i < d; ++i) {               /* insertion sort: stable */
        int v = idx[i], j = i - 1;
        while (j >= 0 && A[idx[j] * d + idx[j]] < A[v * d + v]) { idx[j + 1] = idx[j]; --j; }
        idx[j + 1] = v;
    }
    for (int i = 0; i < d; ++i) {
        mu[i] = A[idx[i] * d + idx[i]];
        for (int k = 0; k < d; ++k) V[i * d + k] = E[k * d + idx[i]];
    }
    free(idx);
    free(E);
    return SQO_OK;
}

/* Algorithm 1 lines 5-6: Qhat = diag(Sigma[:r]) V[:r], with Sigma_i = sqrt(mu_i) the      */
/* singular values of Qc and V's rows its right singular vectors (= eigenvectors of the    */
/* Gram matrix).  Qhat is [r, d].  mu_out ([d]) and V_out ([d, d]) may be NULL.            */
int sqo_query_subspace(const double *Qc, long N, int d, int r, double *Qhat, double *mu_out, double *V_out)
{
    if (!Qc || r < 0 || r > d || d <= 0 || (r > 0 && !Qhat)) return SQO_ERR_ARG;
    double *M = (double *)malloc(sizeof(double) * d * d);
    double *mu = (double *)malloc(sizeof(double) * d);
    double *V = (double *)malloc(sizeof(double) * d * d);
    if (!M || !mu || !V) { free(M); free(mu); free(V); return SQO_ERR_ALLOC; }
    int rc = sqo_gram(Qc, N, d, M);
    if (rc == SQO_OK) rc = sqo_jacobi_eig(M, d, mu, V);
    if (rc == SQO_OK) {
        for (int i = 0; i < r; ++i) {
            double sigma = sqrt(mu[i] > 0.0 ? mu[i] : 0.0);
            for (int k = 0; k < d; ++k) Qhat[i * d + k] = sigma * V[i * d + k];
        }
        if (mu_out) memcpy(mu_out, mu, sizeof(double) * d);
        if (V_out) memcpy(V_out, V, sizeof(double) * d * d);
    }
    free(M); free(mu); free(V);
    return rc;
}

/* ------------------------------------------------------------------------------------ */
/* Inverse of a symmetric positive definite n x n matrix through its Cholesky factor.     */
static int spd_inverse(const double *S, int n, double *Sinv)
{
    double *L = (double *)calloc((size_t)n * n, sizeof(double));
    double *y = (double *)malloc(sizeof(double) * n);
    if (!L || !y) { free(L); free(y); return SQO_ERR_ALLOC; }
    for (int i = 0; i < n; ++i) {
        for (int j = 0; j <= i; ++j) {
            double s = S[i * n + j];
            for (int k = 0; k < j; ++k) s -= L[i * n + k] * L[j * n + k];
            if (i == j) {
                if (!(s > 0.0)) { free(L); free(y); return SQO_ERR_NUMERIC; }
                L[i * n + i] = sqrt(s);
            } else {
                L[i * n + j] = s / L[j * n + j];
            }
        }
    }
    for (int col = 0; col < n; ++col) {
        for (int i = 0; i < n; ++i) {              /* L y = e_col */
            double s = (i == col) ? 1.0 : 0.0;
            for (int k = 0; k < i; ++k) s -= L[i * n + k] * y[k];
            y[i] = s / L[i * n + i];
        }
        for (int i = n - 1; i >= 0; --i) {         /* L^T x = y */
            double s = y[i];
            for (int k = i + 1; k < n; ++k) s -= L[k * n + i] * Sinv[k * n + col];
            Sinv[i * n + col] = s / L[i * n + i];
        }
    }
    free(L); free(y);
    return SQO_OK;
}

/* Prop. 1 / Lemma 3 / Lemma 4 / Algorithm 1 lines 7-9.
 *
 *   P      = I + lambda Qhat^T Qhat             (= A_T^{-1}, Remark after Lemma 4)
 *   P_inv  = P^{-1}
 *   A_t^{-1} for t = T-1 .. 1 by Lemma 4:  A_t^{-1} = M - N^T O^{-1} N  where
 *            A_{t+1}^{-1} = [[M, N^T], [N, O]],  M is tg x tg, O is g x g
 *   U_t    = B_t H_t  (Lemma 3):  B_t = bottom-left (d - tg) x tg block of P_inv,
 *            H_t = last g columns of A_t^{-1}.
 *
 * The update matrices are returned assembled in one d x d matrix W (row-major):
 *   W[tg + i][(t-1)g + c] = U_t[i][c],  zero elsewhere,
 * so that Eq. (update_block) reads  k[j'] += sum_c d_c W[j'][(t-1)g + c]  for j' >= tg.
 *
 * Optional outputs (NULL to skip): P, P_inv (d x d each); Ainv_chain, the matrices
 * A_1^{-1}, ..., A_T^{-1} stored one after another (A_t^{-1} is tg x tg, row-major).
 */
int sqo_update_matrices(const double *Qhat, int r, int d, double lambda, int g,
                        double *W, double *P_out, double *Pinv_out, double *Ainv_chain)
{
    if (!W || d <= 0 || g <= 0 || d % g != 0 || r < 0 || r > d || !(lambda >= 0.0) || (r > 0 && !Qhat))
        return SQO_ERR_ARG;
    const int T = d / g;
    double *P = (double *)malloc(sizeof(double) * d * d);
    double *Pinv = (double *)malloc(sizeof(double) * d * d);
    double *Acur = (double *)malloc(sizeof(double) * d * d);   /* A_{t+1}^{-1}, (t+1)g square */
    double *Anew = (double *)malloc(sizeof(double) * d * d);
    double *Oinv = (double *)malloc(sizeof(double) * g * g);
    double *Obuf = (double *)malloc(sizeof(double) * g * g);
    double *OiN = (double *)malloc(sizeof(double) * g * d);
    int rc = SQO_OK;
    if (!P || !Pinv || !Acur || !Anew || !Oinv || !Obuf || !OiN) { rc = SQO_ERR_ALLOC; goto done; }

    for (int a = 0; a < d; ++a)
        for (int b = 0; b < d; ++b) {
            double s = (a == b) ? 1.0 : 0.0;
            for (int i = 0; i < r; ++i) s += lambda * Qhat[i * d + a] * Qhat[i * d + b];
            P[a * d + b] = s;
        }
    rc = spd_inverse(P, d, Pinv);
    if (rc != SQO_OK) goto done;
    if (P_out) memcpy(P_out, P, sizeof(double) * d * d);
    if (Pinv_out) memcpy(Pinv_out, Pinv, sizeof(double) * d * d);
    memset(W, 0, sizeof(double) * d * d);

    /* offsets of A_t^{-1} inside Ainv_chain */
    size_t *off = (size_t *)malloc(sizeof(size_t) * (T + 2));
    if (!off) { rc = SQO_ERR_ALLOC; goto done; }
    off[1] = 0;
    for (int t = 1; t <= T; ++t) off[t + 1] = off[t] + (size_t)(t * g) * (t * g);

    /* A_T^{-1} = P */
    int n = d;                                   /* current size (t+1) g */
    memcpy(Acur, P, sizeof(double) * d * d);
    if (Ainv_chain) memcpy(Ainv_chain + off[T], Acur, sizeof(double) * d * d);

    for (int t = T - 1; t >= 1; --t) {
        const int m = t * g;                     /* size of A_t^{-1} */
        /* O = bottom-right g x g block of A_{t+1}^{-1} */
        for (int a = 0; a < g; ++a)
            for (int b = 0; b < g; ++b) Obuf[a * g + b] = Acur[(m + a) * n + (m + b)];
        rc = spd_inverse(Obuf, g, Oinv);
        if (rc != SQO_OK) { free(off); goto done; }
        /* OiN = O^{-1} N,  N = rows m.., columns 0..m-1  (g x m) */
        for (int a = 0; a < g; ++a)
            for (int c = 0; c < m; ++c) {
                double s = 0.0;
                for (int b = 0; b < g; ++b) s += Oinv[a * g + b] * Acur[(m + b) * n + c];
                OiN[a * m + c] = s;
            }
        /* A_t^{-1} = M - N^T (O^{-1} N) */
        for (int a = 0; a < m; ++a)
            for (int c = 0; c < m; ++c) {
                double s = Acur[a * n + c];
                for (int b = 0; b < g; ++b) s -= Acur[(m + b) * n + a] * OiN[b * m + c];
                Anew[a * m + c] = s;
            }
        memcpy(Acur, Anew, sizeof(double) * m * m);
        n = m;
        if (Ainv_chain) memcpy(Ainv_chain + off[t], Acur, sizeof(double) * m * m);

        /* U_t = B_t H_t :  B_t = P_inv[m:, :m],  H_t = A_t^{-1}[:, m-g:m] */
        for (int i = 0; i < d - m; ++i)
            for (int c = 0; c < g; ++c) {
                double s = 0.0;
                for (int k = 0; k < m; ++k) s += Pinv[(m + i) * d + k] * Acur[k * m + (m - g + c)];
                W[(m + i) * d + (m - g + c)] = s;
            }
    }
    free(off);
done:
    free(P); free(Pinv); free(Acur); free(Anew); free(Oinv); free(Obuf); free(OiN);
    return rc;
}

/* ------------------------------------------------------------------------------------ */
/* Round a float32 to the nearest IEEE binary16 value (ties to even; subnormals kept; beyond
 * the largest finite binary16 value plus half a step: infinity), returned as a float32.
 * Written out on the bits: the exponent decides the spacing q of binary16 numbers around x
 * (2^(e-10) for normal results, 2^-24 below 2^-14), and x / q is rounded to an integer. */
float sqo_half_round(float x)
{
    if (x != x || x == INFINITY || x == -INFINITY || x == 0.0f) return x;
    const double ax = fabs((double)x);
    int e;
    (void)frexp(ax, &e);                      /* ax = f * 2^e, 0.5 <= f < 1  ->  2^(e-1) <= ax < 2^e */
    int qexp = (e - 1) - 10;                  /* spacing 2^qexp of binary16 numbers in [2^(e-1), 2^e) */
    if (qexp < -24) qexp = -24;               /* subnormal range: fixed spacing 2^-24 */
    const double q = ldexp(1.0, qexp);
    double r = nearbyint(ax / q) * q;         /* exact: ax / q is a double with few bits, round half to even */
    if (r >= 65520.0) r = INFINITY;           /* 65504 + half a step of 32 rounds up to 2^16: overflow */
    return (float)(x < 0.0f ? -r : r);
}

/* ------------------------------------------------------------------------------------ */
/* Algorithm 1, function Quant, applied to n/G consecutive groups of G tokens.
 *
 * K      [n, d] keys of one (batch, head), row = token; n % G == 0.
 * W      [d, d] assembled update matrix from sqo_update_matrices (NULL = no update).
 * codes  [n, d] one code per byte (not packed).
 * scale, zero  [n/G, d] float32: Delta and zero-point m of (group, channel)  (Section 2).
 * Khat   [n, d] the dequantized keys the cache reader reconstructs (may be NULL).
 * tval   [n, d] (x - zero)/scale before rounding, for tie diagnosis (may be NULL).
 * force  [n, d] int16: >= 0 forces that code instead of the rounded one (may be NULL);
 *        used to replay a run after a legitimate rounding tie was resolved the other way.
 *
 * For channel j = 0 .. d-1: the grid (m, Delta) is taken over the G tokens of the group on
 * the CURRENT (corrected) values; every token's element is rounded to the grid; the error
 * e = deq(qtz(x)) - x of each token is pushed onto its later channels, x[j'] += e W[j'][j]
 * (Eq. (3) for g = 1; Eq. (update_block) for g > 1, where W is zero inside a block so the
 * g channels of a block are quantized before any of them is corrected by the others).
 */
/* The general form.  meta16 != 0: scale and zero-point are stored as binary16 (sqo_half_round of the
 * float32 values); raw_scale / raw_zero [n/G, d] (may be NULL) receive the float32 values before that
 * rounding, for tie diagnosis; force_scale / force_zero [n/G, d] (may be NULL; NaN = not forced) replace
 * the stored values of single (group, channel) pairs, to replay a run after a legitimate tie of the
 * 16-bit rounding was resolved the other way. */
int sqo_quant_keys_m16(const double *K, long n, int d, int G, int bits, const double *W,
                       uint8_t *codes, float *scale, float *zero, double *Khat, double *tval,
                       const int16_t *force, int meta16, float *raw_scale, float *raw_zero,
                       const float *force_scale, const float *force_zero);

int sqo_quant_keys(const double *K, long n, int d, int G, int bits, const double *W,
                   uint8_t *codes, float *scale, float *zero, double *Khat, double *tval,
                   const int16_t *force)
{
    return sqo_quant_keys_m16(K, n, d, G, bits, W, codes, scale, zero, Khat, tval, force, 0, NULL, NULL, NULL, NULL);
}

int sqo_quant_keys_m16(const double *K, long n, int d, int G, int bits, const double *W,
                       uint8_t *codes, float *scale, float *zero, double *Khat, double *tval,
                       const int16_t *force, int meta16, float *raw_scale, float *raw_zero,
                       const float *force_scale, const float *force_zero)
{
    if (!K || !codes || !scale || !zero || n < 0 || d <= 0 || G <= 0 || n % G != 0 || bits < 1 || bits > 8)
        return SQO_ERR_ARG;
    const double L = (double)((1 << bits) - 1);
    double *X = (double *)malloc(sizeof(double) * (size_t)G * d);
    double *e = (double *)malloc(sizeof(double) * G);
    if (!X || !e) { free(X); free(e); return SQO_ERR_ALLOC; }
    for (long grp = 0; grp < n / G; ++grp) {
        const long t0 = grp * G;
        memcpy(X, K + t0 * d, sizeof(double) * (size_t)G * d);
        for (int j = 0; j < d; ++j) {
            double m = X[j], Mx = X[j];
            for (int i = 1; i < G; ++i) {
                double x = X[(size_t)i * d + j];
                if (x < m) m = x;
                if (x > Mx) Mx = x;
            }
            float zf = (float)m;                             /* stored zero-point */
            float sf = (float)((Mx - m) / L);                /* stored scale Delta */
            if (raw_zero) raw_zero[grp * d + j] = zf;
            if (raw_scale) raw_scale[grp * d + j] = sf;
            if (meta16) {
                zf = sqo_half_round(zf);
                sf = sqo_half_round(sf);
            }
            if (force_zero && force_zero[grp * d + j] == force_zero[grp * d + j]) zf = force_zero[grp * d + j];
            if (force_scale && force_scale[grp * d + j] == force_scale[grp * d + j]) sf = force_scale[grp * d + j];
            zero[grp * d + j] = zf;
            scale[grp * d + j] = sf;
            for (int i = 0; i < G; ++i) {
                const double x = X[(size_t)i * d + j];
                double c = 0.0, t = 0.0;
                if (sf > 0.0f) {
                    t = (x - (double)zf) / (double)sf;
                    c = nearbyint(t);                        /* round half to even */
                    if (c < 0.0) c = 0.0;
                    if (c > L) c = L;
                }
                if (force && force[(t0 + i) * d + j] >= 0) c = (double)force[(t0 + i) * d + j];
                const double xhat = (double)zf + (double)sf * c;      /* deq(qtz(x)) */
                codes[(t0 + i) * d + j] = (uint8_t)c;
                if (Khat) Khat[(t0 + i) * d + j] = xhat;
                if (tval) tval[(t0 + i) * d + j] = t;
                e[i] = xhat - x;
            }
            if (W) {
                for (int jp = j + 1; jp < d; ++jp) {
                    const double w = W[(size_t)jp * d + j];
                    if (w == 0.0) continue;
                    for (int i = 0; i < G; ++i) X[(size_t)i * d + jp] += e[i] * w;
                }
            }
        }
    }
    free(X); free(e);
    return SQO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* Per-token value quantization (Section 2 "Quantization" applied per token, Appendix C):
 * each token's d channels are split into d/G groups of G consecutive channels.
 * V [n, d]; codes [n, d] (one per byte); scale, zero [n, d/G].
 *
 * _f32: every operation is an IEEE binary32 operation in this order
 *         Delta = (M - m) / L ;  t = (x - m) / Delta ;  c = clamp(rint(t), 0, L)
 *       (compile without contraction or fast-math), so a float32 GPU kernel issuing the
 *       same operations produces identical bits.
 * _f64: the same in double, scale/zero rounded to float32 for storage and the rounding
 *       decision taken against the stored values, as for keys.
 */
int sqo_quant_values_f32(const float *V, long n, int d, int G, int bits,
                         uint8_t *codes, float *scale, float *zero)
{
    if (!V || !codes || !scale || !zero || n < 0 || d <= 0 || G <= 0 || d % G != 0 || bits < 1 || bits > 8)
        return SQO_ERR_ARG;
    const float L = (float)((1 << bits) - 1);
    const int ng = d / G;
    for (long i = 0; i < n; ++i)
        for (int q = 0; q < ng; ++q) {
            const float *x = V + i * d + q * G;
            float m = x[0], Mx = x[0];
            for (int c = 1; c < G; ++c) {
                if (x[c] < m) m = x[c];
                if (x[c] > Mx) Mx = x[c];
            }
            volatile float rng = Mx - m;
            volatile float delta = rng / L;
            scale[i * ng + q] = delta;
            zero[i * ng + q] = m;
            for (int c = 0; c < G; ++c) {
                float code = 0.0f;
                if (delta > 0.0f) {
                    volatile float num = x[c] - m;
                    volatile float t = num / delta;
                    code = nearbyintf(t);
                    if (code < 0.0f) code = 0.0f;
                    if (code > L) code = L;
                }
                codes[i * d + q * G + c] = (uint8_t)code;
            }
        }
    return SQO_OK;
}

/* The binary32 sequence with 16-bit metadata: Delta = half(Delta32), z = half(m), t = (x - z) / Delta,
 * c = clamp(rint(t), 0, L), every operation an IEEE binary32 operation on the rounded metadata. */
int sqo_quant_values_f32_m16(const float *V, long n, int d, int G, int bits,
                             uint8_t *codes, float *scale, float *zero)
{
    if (!V || !codes || !scale || !zero || n < 0 || d <= 0 || G <= 0 || d % G != 0 || bits < 1 || bits > 8)
        return SQO_ERR_ARG;
    const float L = (float)((1 << bits) - 1);
    const int ng = d / G;
    for (long i = 0; i < n; ++i)
        for (int q = 0; q < ng; ++q) {
            const float *x = V + i * d + q * G;
            float m = x[0], Mx = x[0];
            for (int c = 1; c < G; ++c) {
                if (x[c] < m) m = x[c];
                if (x[c] > Mx) Mx = x[c];
            }
            volatile float rng = Mx - m;
            volatile float delta32 = rng / L;
            const float delta = sqo_half_round(delta32);
            const float z = sqo_half_round(m);
            scale[i * ng + q] = delta;
            zero[i * ng + q] = z;
            for (int c = 0; c < G; ++c) {
                float code = 0.0f;
                if (delta > 0.0f && delta < INFINITY) {
                    volatile float num = x[c] - z;
                    volatile float t = num / delta;
                    code = nearbyintf(t);
                    if (code < 0.0f) code = 0.0f;
                    if (code > L) code = L;
                }
                codes[i * d + q * G + c] = (uint8_t)code;
            }
        }
    return SQO_OK;
}

int sqo_quant_values_f64(const double *V, long n, int d, int G, int bits,
                         uint8_t *codes, float *scale, float *zero)
{
    if (!V || !codes || !scale || !zero || n < 0 || d <= 0 || G <= 0 || d % G != 0 || bits < 1 || bits > 8)
        return SQO_ERR_ARG;
    const double L = (double)((1 << bits) - 1);
    const int ng = d / G;
    for (long i = 0; i < n; ++i)
        for (int q = 0; q < ng; ++q) {
            const double *x = V + i * d + q * G;
            double m = x[0], Mx = x[0];
            for (int c = 1; c < G; ++c) {
                if (x[c] < m) m = x[c];
                if (x[c] > Mx) Mx = x[c];
            }
            const float zf = (float)m, sf = (float)((Mx - m) / L);
            scale[i * ng + q] = sf;
            zero[i * ng + q] = zf;
            for (int c = 0; c < G; ++c) {
                double code = 0.0;
                if (sf > 0.0f) {
                    code = nearbyint((x[c] - (double)zf) / (double)sf);
                    if (code < 0.0) code = 0.0;
                    if (code > L) code = L;
                }
                codes[i * d + q * G + c] = (uint8_t)code;
            }
        }
    return SQO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* deq(c) = c * Delta + m  (Section 2).  Keys: scale/zero indexed [token / G][channel].   */
int sqo_dequant_keys(const uint8_t *codes, const float *scale, const float *zero,
                     long n, int d, int G, double *out)
{
    if (!codes || !scale || !zero || !out || n < 0 || d <= 0 || G <= 0 || n % G != 0) return SQO_ERR_ARG;
    for (long i = 0; i < n; ++i)
        for (int j = 0; j < d; ++j)
            out[i * d + j] = (double)codes[i * d + j] * (double)scale[(i / G) * d + j] + (double)zero[(i / G) * d + j];
    return SQO_OK;
}

/* Values: scale/zero indexed [token][channel / G]. */
int sqo_dequant_values(const uint8_t *codes, const float *scale, const float *zero,
                       long n, int d, int G, double *out)
{
    if (!codes || !scale || !zero || !out || n < 0 || d <= 0 || G <= 0 || d % G != 0) return SQO_ERR_ARG;
    const int ng = d / G;
    for (long i = 0; i < n; ++i)
        for (int j = 0; j < d; ++j)
            out[i * d + j] = (double)codes[i * d + j] * (double)scale[i * ng + j / G] + (double)zero[i * ng + j / G];
    return SQO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* Cache layout of the codes (ours; the paper gives none): token-major, token i owns
 * d*bits/8 consecutive bytes; channel j's code sits at bit (j*bits) mod 8 of byte
 * floor(j*bits/8), low bits first.  bits must divide 8. */
int sqo_pack(const uint8_t *codes, long n, int d, int bits, uint8_t *packed)
{
    if (!codes || !packed || n < 0 || d <= 0 || (bits != 1 && bits != 2 && bits != 4 && bits != 8) || (d * bits) % 8 != 0)
        return SQO_ERR_ARG;
    const int row = d * bits / 8;
    memset(packed, 0, (size_t)n * row);
    for (long i = 0; i < n; ++i)
        for (int j = 0; j < d; ++j) {
            const int bit = j * bits;
            packed[i * row + bit / 8] |= (uint8_t)((codes[i * d + j] & ((1 << bits) - 1)) << (bit % 8));
        }
    return SQO_OK;
}

int sqo_unpack(const uint8_t *packed, long n, int d, int bits, uint8_t *codes)
{
    if (!codes || !packed || n < 0 || d <= 0 || (bits != 1 && bits != 2 && bits != 4 && bits != 8) || (d * bits) % 8 != 0)
        return SQO_ERR_ARG;
    const int row = d * bits / 8;
    for (long i = 0; i < n; ++i)
        for (int j = 0; j < d; ++j) {
            const int bit = j * bits;
            codes[i * d + j] = (uint8_t)((packed[i * row + bit / 8] >> (bit % 8)) & ((1 << bits) - 1));
        }
    return SQO_OK;
}

/* Appendix B: memory = 2 x b x (l_prompt + l_response) x L x h x d x p bytes. */
long long sqo_kv_cache_bytes(long long batch, long long seq_len, long long layers, long long heads,
                             long long head_dim, long long bytes_per_param)
{
    return 2LL * batch * seq_len * layers * heads * head_dim * bytes_per_param;
}

/* ------------------------------------------------------------------------------------ */
/* One decode step of attention (Section 2): for each of the nq query vectors (the query heads
 * that share this KV head), w_i = <q, k_i> / sqrt(d) over the n cached tokens, p = softmax(w),
 * out = sum_i p_i v_i.  K and V are what a reader of the cache sees: dequantized rows followed
 * by the full-precision rows of the residual buffer.  The largest score is subtracted before
 * exponentiation; that leaves softmax unchanged and keeps exp() in range. */
int sqo_attention_decode(const double *q, int nq, const double *K, const double *V, long n, int d, double *out)
{
    if (!q || !K || !V || !out || nq <= 0 || n <= 0 || d <= 0) return SQO_ERR_ARG;
    double *w = (double *)malloc((size_t)n * sizeof(double));
    if (!w) return SQO_ERR_ALLOC;
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    for (int h = 0; h < nq; ++h) {
        double wmax = -INFINITY;
        for (long i = 0; i < n; ++i) {
            double s = 0.0;
            for (int j = 0; j < d; ++j) s += q[h * d + j] * K[i * d + j];
            w[i] = s * inv_sqrt_d;
            if (w[i] > wmax) wmax = w[i];
        }
        double denom = 0.0;
        for (long i = 0; i < n; ++i) {
            w[i] = exp(w[i] - wmax);
            denom += w[i];
        }
        for (int j = 0; j < d; ++j) {
            double s = 0.0;
            for (long i = 0; i < n; ++i) s += w[i] * V[i * d + j];
            out[h * d + j] = s / denom;
        }
    }
    free(w);
    return SQO_OK;
}

/* ------------------------------------------------------------------------------------ */
/* Rotary position embedding of n rows X [n, d] (d even), in place: for row t at position
 * pos[t] and every i < d/2, with angle a = pos[t] * base^(-2 i / d),
 *     (x_i, x_{i + d/2})  <-  (x_i cos a - x_{i + d/2} sin a,  x_i sin a + x_{i + d/2} cos a).
 * The variant of Section 4 that quantizes keys before the embedding stores un-rotated rows; a
 * reader applies this to each dequantized (and each residual) key row at that row's position
 * before the scores of sqo_attention_decode are formed. */
int sqo_rope_rows(double *X, long n, int d, const long *pos, double base)
{
    if (!X || !pos || n < 0 || d <= 0 || (d & 1) || !(base > 0.0)) return SQO_ERR_ARG;
    const int half = d / 2;
    for (long t = 0; t < n; ++t) {
        for (int i = 0; i < half; ++i) {
            const double theta = pow(base, -2.0 * (double)i / (double)d);
            const double a = (double)pos[t] * theta;
            const double c = cos(a), sn = sin(a);
            const double x0 = X[t * d + i], x1 = X[t * d + i + half];
            X[t * d + i] = x0 * c - x1 * sn;
            X[t * d + i + half] = x0 * sn + x1 * c;
        }
    }
    return SQO_OK;
}
