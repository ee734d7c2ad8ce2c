/*
 * LoCoCo chunk-step oracle: TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, float64 CPU statement of what the per-chunk KV-cache update
 * and the chunk attention compute, written from the paper's definitions:
 *   Eq. 1          causal softmax attention
 *   Eq. 3          cache <- C([cache, chunk])
 *   Eq. 4, Eq. 5   slot i = weighted blend of all cache and chunk tokens,
 *                  same weights for keys and values
 *   Eq. 6          W = 1-D multi-channel convolution over the concatenation
 *   Eq. 7          w_ij = W_ij / sum_k W_ik
 *   Algorithm 2    attention with the old cache, then fill or compress
 * One (sequence, head) unit at a time, positions as rows ([tokens, d], d
 * contiguous).  No blocking, no fusion, no reordering beyond those formulas.
 * It shares no code with the CUDA library and must only be used by tests, the
 * smoke check and the CPU-baseline leg of the benchmark.
 *
 * Readings taken where the paper is silent or inconsistent (all stated again
 * in the design notes):
 *   - conv: stride 1, zero "same" padding p=(k-1)/2, no kernel flip
 *     (cross-correlation), k odd, optional bias;
 *   - conv input channels c_in = d (keys only) or 2d (keys stacked on values
 *     channel-wise, as Eq. 6 writes it);
 *   - concatenation order: cache first, then chunk (Eq. 3, Algorithm 2);
 *     flag LOCOCO_ORACLE_CHUNK_FIRST gives Eq. 6's order instead;
 *   - the ReLU of Section 3.2.1 acts on the conv output, before Eq. 7;
 *     flag LOCOCO_ORACLE_RELU_ON_INPUT applies it to the conv input instead;
 *   - Eq. 7's denominator is sum_k W_ik + eps;
 *   - a compress step with a partly filled cache (c < M, c + b > M) sees only
 *     the S = c + b real entries;
 *   - the mask of Eq. 1 is the usual additive -inf mask;
 *   - protected slots (Section 5.2, Table 6: the compressor next to an eviction
 *     policy that always keeps some tokens, e.g. the initial "sink" tokens):
 *     the paper gives no formula; here rows i < protected_slots of the weight
 *     matrix w are the unit rows e_i, so slot i keeps entry i of [cache; chunk]
 *     unchanged (the tokens that filled those slots first), the conv still reads
 *     every entry, and no gradient reaches the conv weights of those rows.
 *     Cache-first order only.
 *
 * Parity status: every function below is pinned by tests/test_oracle_*.py
 * (textbook correlation, closed forms, hand-worked fixtures, one-hot gather,
 * full attention for short sequences, finite differences).  That these
 * readings are the ones the authors' own code used is unpinned: the paper
 * prints no worked numeric example.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define LOCOCO_ORACLE_CHUNK_FIRST   1
#define LOCOCO_ORACLE_RELU_ON_INPUT 2

typedef struct {
    int32_t d;       /* head dimension */
    int32_t M;       /* cache slots */
    int32_t k;       /* conv kernel width (odd) */
    int32_t c_in;    /* conv input channels: d or 2d */
    int32_t flags;   /* LOCOCO_ORACLE_* */
    int32_t protected_slots; /* first slots kept verbatim (Section 5.2); 0 = plain method */
    double eps;      /* added to Eq. 7's denominator */
    double scale;    /* softmax scale, 1/sqrt(d) in Eq. 1 */
} oracle_params;

static double* dalloc(size_t n) {
    double* p = (double*)calloc(n ? n : 1, sizeof(double));
    return p;
}

/* Eq. 6: A[i,j] = bias_i + sum_ch sum_t G[i,ch,t] * Z[j+t-p, ch], zero outside [0,S). */
void lococo_oracle_conv_logits(const double* Z, int S, int C, const double* G, const double* bias,
                               int M, int k, double* A) {
    const int p = (k - 1) / 2;
#pragma omp parallel for schedule(static)   /* rows of A are independent of each other */
    for (int i = 0; i < M; ++i) {
        for (int j = 0; j < S; ++j) {
            double acc = bias ? bias[i] : 0.0;
            for (int ch = 0; ch < C; ++ch) {
                for (int t = 0; t < k; ++t) {
                    const int jj = j + t - p;
                    if (jj >= 0 && jj < S) acc += G[((size_t)i * C + ch) * k + t] * Z[(size_t)jj * C + ch];
                }
            }
            A[(size_t)i * S + j] = acc;
        }
    }
}

/* Conv input of Eq. 6: keys, or keys stacked on values along the channel axis. */
static void build_conv_input(const oracle_params* P, const double* XK, const double* XV, int S, double* Z) {
    const int d = P->d, C = P->c_in;
    for (int j = 0; j < S; ++j) {
        for (int ch = 0; ch < C; ++ch) {
            double z = ch < d ? XK[(size_t)j * d + ch] : XV[(size_t)j * d + (ch - d)];
            if ((P->flags & LOCOCO_ORACLE_RELU_ON_INPUT) && z < 0.0) z = 0.0;
            Z[(size_t)j * C + ch] = z;
        }
    }
}

/*
 * Eq. 6 -> ReLU -> Eq. 7 -> Eq. 4, Eq. 5 on one concatenated sequence XK, XV [S,d].
 * Outputs: Knew, Vnew [M,d]; optionally w [M,S], the pre-activation logits A [M,S]
 * and the denominators s [M].
 */
void lococo_oracle_compress(const oracle_params* P, const double* XK, const double* XV, int S,
                            const double* G, const double* bias, double* Knew, double* Vnew,
                            double* w_out, double* A_out, double* s_out) {
    const int d = P->d, M = P->M, C = P->c_in;
    double* Z = dalloc((size_t)S * C);
    double* A = dalloc((size_t)M * S);
    build_conv_input(P, XK, XV, S, Z);
    lococo_oracle_conv_logits(Z, S, C, G, bias, M, P->k, A);
#pragma omp parallel for schedule(static)   /* every slot is built from its own row of A */
    for (int i = 0; i < M; ++i) {
        if (i < P->protected_slots) {
            /* Section 5.2: w_i = e_i, the slot keeps entry i as it is */
            if (s_out) s_out[i] = 1.0;
            for (int j = 0; j < S && w_out; ++j) w_out[(size_t)i * S + j] = j == i ? 1.0 : 0.0;
            for (int c = 0; c < d; ++c) {
                Knew[(size_t)i * d + c] = XK[(size_t)i * d + c];
                Vnew[(size_t)i * d + c] = XV[(size_t)i * d + c];
            }
            continue;
        }
        double s = 0.0;
        for (int j = 0; j < S; ++j) {
            double r = A[(size_t)i * S + j];
            if (!(P->flags & LOCOCO_ORACLE_RELU_ON_INPUT) && r < 0.0) r = 0.0;
            s += r;
        }
        s += P->eps;
        if (s_out) s_out[i] = s;
        for (int c = 0; c < d; ++c) { Knew[(size_t)i * d + c] = 0.0; Vnew[(size_t)i * d + c] = 0.0; }
        for (int j = 0; j < S; ++j) {
            double r = A[(size_t)i * S + j];
            if (!(P->flags & LOCOCO_ORACLE_RELU_ON_INPUT) && r < 0.0) r = 0.0;
            const double w = r / s;
            if (w_out) w_out[(size_t)i * S + j] = w;
            for (int c = 0; c < d; ++c) {
                Knew[(size_t)i * d + c] += w * XK[(size_t)j * d + c];
                Vnew[(size_t)i * d + c] += w * XV[(size_t)j * d + c];
            }
        }
    }
    if (A_out) memcpy(A_out, A, sizeof(double) * (size_t)M * S);
    free(Z); free(A);
}

/*
 * Eq. 1 for one chunk (Algorithm 2, Step 3).  XK, XV are [c+b, d] with the c cache
 * entries first; query r sees the whole cache and chunk keys 0..r.
 * O [b,d]; lse [b] (log-sum-exp of the scaled logits) optional; prob [b, c+b] optional.
 */
void lococo_oracle_attention(const double* Q, int b, const double* XK, const double* XV, int c, int d,
                             double scale, double* O, double* lse, double* prob) {
    const int S = c + b;
#pragma omp parallel for schedule(dynamic, 16)   /* queries are independent of each other */
    for (int r = 0; r < b; ++r) {
        double* logit = dalloc((size_t)S);
        const int n = c + r + 1;
        double mx = -INFINITY;
        for (int j = 0; j < n; ++j) {
            double acc = 0.0;
            for (int e = 0; e < d; ++e) acc += Q[(size_t)r * d + e] * XK[(size_t)j * d + e];
            logit[j] = acc * scale;
            if (logit[j] > mx) mx = logit[j];
        }
        double den = 0.0;
        for (int j = 0; j < n; ++j) den += exp(logit[j] - mx);
        for (int e = 0; e < d; ++e) O[(size_t)r * d + e] = 0.0;
        for (int j = 0; j < S; ++j) {
            const double pj = j < n ? exp(logit[j] - mx) / den : 0.0;
            if (prob) prob[(size_t)r * S + j] = pj;
            if (j < n)
                for (int e = 0; e < d; ++e) O[(size_t)r * d + e] += pj * XV[(size_t)j * d + e];
        }
        if (lse) lse[r] = mx + log(den);
        free(logit);
    }
}

/* Concatenate cache and chunk in the configured order. Returns offset of the chunk rows. */
static int concat(const oracle_params* P, const double* cache, int c, const double* chunk, int b, double* X) {
    const int d = P->d;
    if (P->flags & LOCOCO_ORACLE_CHUNK_FIRST) {
        memcpy(X, chunk, sizeof(double) * (size_t)b * d);
        memcpy(X + (size_t)b * d, cache, sizeof(double) * (size_t)c * d);
        return 0;
    }
    memcpy(X, cache, sizeof(double) * (size_t)c * d);
    memcpy(X + (size_t)c * d, chunk, sizeof(double) * (size_t)b * d);
    return c;
}

/*
 * One update of the cache (Algorithm 2, the if/else after Step 3): fill when
 * c + b <= M, otherwise Steps 4 and 5.  Kc, Vc are [M,d] buffers updated in place.
 */
void lococo_oracle_update_cache(const oracle_params* P, double* Kc, double* Vc, int* c_inout,
                                const double* Kn, const double* Vn, int b, const double* G,
                                const double* bias) {
    const int d = P->d, M = P->M, c = *c_inout;
    if (c + b <= M) {
        memcpy(Kc + (size_t)c * d, Kn, sizeof(double) * (size_t)b * d);
        memcpy(Vc + (size_t)c * d, Vn, sizeof(double) * (size_t)b * d);
        *c_inout = c + b;
        return;
    }
    const int S = c + b;
    double* XK = dalloc((size_t)S * d);
    double* XV = dalloc((size_t)S * d);
    concat(P, Kc, c, Kn, b, XK);
    concat(P, Vc, c, Vn, b, XV);
    lococo_oracle_compress(P, XK, XV, S, G, bias, Kc, Vc, NULL, NULL, NULL);
    *c_inout = M;
    free(XK); free(XV);
}

/*
 * Algorithm 2 over L tokens in chunks of B (last chunk may be short).
 * Q, K, V, O are [L,d].  Kc, Vc [M,d] and *c_inout are the cache state, in and out.
 * snap_K / snap_V (optional) receive the cache as it was BEFORE each step:
 * [n_chunks, M, d]; snap_c [n_chunks] the fill counts.
 */
void lococo_oracle_process_sequence(const oracle_params* P, const double* Q, const double* K,
                                    const double* V, int L, int B, const double* G, const double* bias,
                                    double* O, double* Kc, double* Vc, int* c_inout, double* lse,
                                    double* snap_K, double* snap_V, int32_t* snap_c) {
    const int d = P->d, M = P->M;
    int c = *c_inout;
    double* XK = dalloc((size_t)(M + B) * d);
    double* XV = dalloc((size_t)(M + B) * d);
    int step = 0;
    for (int t0 = 0; t0 < L; t0 += B, ++step) {
        const int b = (L - t0 < B) ? (L - t0) : B;
        const double* Qn = Q + (size_t)t0 * d;
        const double* Kn = K + (size_t)t0 * d;
        const double* Vn = V + (size_t)t0 * d;
        if (snap_K) memcpy(snap_K + (size_t)step * M * d, Kc, sizeof(double) * (size_t)M * d);
        if (snap_V) memcpy(snap_V + (size_t)step * M * d, Vc, sizeof(double) * (size_t)M * d);
        if (snap_c) snap_c[step] = c;
        /* Step 3: attention over [old cache, chunk]; attention always sees cache first. */
        memcpy(XK, Kc, sizeof(double) * (size_t)c * d);
        memcpy(XK + (size_t)c * d, Kn, sizeof(double) * (size_t)b * d);
        memcpy(XV, Vc, sizeof(double) * (size_t)c * d);
        memcpy(XV + (size_t)c * d, Vn, sizeof(double) * (size_t)b * d);
        lococo_oracle_attention(Qn, b, XK, XV, c, d, P->scale, O + (size_t)t0 * d,
                                lse ? lse + t0 : NULL, NULL);
        /* fill, or Steps 4-5 */
        lococo_oracle_update_cache(P, Kc, Vc, &c, Kn, Vn, b, G, bias);
    }
    *c_inout = c;
    free(XK); free(XV);
}

/* Gradient of Eq. 1 for one chunk: given dO [b,d], accumulate dQ [b,d], dXK, dXV [c+b,d].
 * With P the softmax probabilities: dP_rj = <dO_r, V_j>, dS_rj = scale * P_rj (dP_rj - sum_l P_rl dP_rl)
 * (the row term equals <dO_r, O_r>), then dQ = dS XK, dXK = dS^T Q, dXV = P^T dO.  The first loop runs over
 * queries and the second over keys, so that each may be shared out among threads without two of them
 * adding to the same entry. */
static void attention_backward(const double* Q, int b, const double* XK, const double* XV, int c, int d,
                               double scale, const double* dO, double* dQ, double* dXK, double* dXV) {
    const int S = c + b;
    double* O = dalloc((size_t)b * d);
    double* prob = dalloc((size_t)b * S);
    double* dS = dalloc((size_t)b * S);
    lococo_oracle_attention(Q, b, XK, XV, c, d, scale, O, NULL, prob);
#pragma omp parallel for schedule(dynamic, 16)
    for (int r = 0; r < b; ++r) {
        const int n = c + r + 1;
        double dot = 0.0;
        for (int e = 0; e < d; ++e) dot += dO[(size_t)r * d + e] * O[(size_t)r * d + e];
        for (int j = 0; j < n; ++j) {
            const double pj = prob[(size_t)r * S + j];
            double dp = 0.0;
            for (int e = 0; e < d; ++e) dp += dO[(size_t)r * d + e] * XV[(size_t)j * d + e];
            const double dl = pj * (dp - dot) * scale;
            dS[(size_t)r * S + j] = dl;
            for (int e = 0; e < d; ++e) dQ[(size_t)r * d + e] += dl * XK[(size_t)j * d + e];
        }
    }
#pragma omp parallel for schedule(dynamic, 16)
    for (int j = 0; j < S; ++j) {
        /* key j is seen by the queries r with c + r >= j */
        for (int r = (j > c ? j - c : 0); r < b; ++r) {
            const double pj = prob[(size_t)r * S + j], dl = dS[(size_t)r * S + j];
            for (int e = 0; e < d; ++e) {
                dXV[(size_t)j * d + e] += pj * dO[(size_t)r * d + e];
                dXK[(size_t)j * d + e] += dl * Q[(size_t)r * d + e];
            }
        }
    }
    free(O); free(prob); free(dS);
}

/*
 * Gradient of lococo_oracle_compress (output-ReLU reading only): given dKnew, dVnew [M,d],
 * accumulate dXK, dXV [S,d], dG [M,c_in,k], dbias [M] (optional).
 */
static void compress_backward(const oracle_params* P, const double* XK, const double* XV, int S,
                              const double* G, const double* bias, const double* dKnew,
                              const double* dVnew, double* dXK, double* dXV, double* dG, double* dbias) {
    const int d = P->d, M = P->M, C = P->c_in, k = P->k, p = (k - 1) / 2;
    double* Kn = dalloc((size_t)M * d);
    double* Vn = dalloc((size_t)M * d);
    double* w = dalloc((size_t)M * S);
    double* A = dalloc((size_t)M * S);
    double* s = dalloc((size_t)M);
    double* Z = dalloc((size_t)S * C);
    double* dA = dalloc((size_t)M * S);
    build_conv_input(P, XK, XV, S, Z);
    lococo_oracle_compress(P, XK, XV, S, G, bias, Kn, Vn, w, A, s);
    for (int i = 0; i < M; ++i) {
        /* dw_ij = <dKnew_i, XK_j> + <dVnew_i, XV_j>;  blend's own input gradient */
        double inner = 0.0;
        for (int j = 0; j < S; ++j) {
            double dw = 0.0;
            for (int e = 0; e < d; ++e) {
                dw += dKnew[(size_t)i * d + e] * XK[(size_t)j * d + e] + dVnew[(size_t)i * d + e] * XV[(size_t)j * d + e];
                dXK[(size_t)j * d + e] += w[(size_t)i * S + j] * dKnew[(size_t)i * d + e];
                dXV[(size_t)j * d + e] += w[(size_t)i * S + j] * dVnew[(size_t)i * d + e];
            }
            dA[(size_t)i * S + j] = dw;
            inner += dw * w[(size_t)i * S + j];
        }
        /* through w = R / s, s = sum R + eps, R = max(A, 0) */
        for (int j = 0; j < S; ++j) {
            const double dR = (dA[(size_t)i * S + j] - inner) / s[i];
            dA[(size_t)i * S + j] = A[(size_t)i * S + j] > 0.0 ? dR : 0.0;
            if (i < P->protected_slots) dA[(size_t)i * S + j] = 0.0;   /* constant row: nothing flows to Eq. 6 */
        }
    }
    /* through Eq. 6: A[i,j] = bias_i + sum_ch sum_t G[i,ch,t] Z[j+t-p,ch].  The channel loop is the outer
     * one so that channels can be shared out among threads: an input channel owns its entries of dG and of
     * dXK / dXV, and each of them still receives its terms in the order (i, j, t). */
    if (dbias)
        for (int i = 0; i < M; ++i)
            for (int j = 0; j < S; ++j) dbias[i] += dA[(size_t)i * S + j];
#pragma omp parallel for schedule(static)
    for (int ch = 0; ch < C; ++ch) {
        for (int i = 0; i < M; ++i) {
            for (int j = 0; j < S; ++j) {
                const double g = dA[(size_t)i * S + j];
                if (g == 0.0) continue;
                for (int t = 0; t < k; ++t) {
                    const int jj = j + t - p;
                    if (jj < 0 || jj >= S) continue;
                    dG[((size_t)i * C + ch) * k + t] += g * Z[(size_t)jj * C + ch];
                    const double dz = g * G[((size_t)i * C + ch) * k + t];
                    if (ch < d) dXK[(size_t)jj * d + ch] += dz;
                    else dXV[(size_t)jj * d + (ch - d)] += dz;
                }
            }
        }
    }
    free(Kn); free(Vn); free(w); free(A); free(s); free(Z); free(dA);
}

/*
 * Gradients of  loss = <dO, O> + <dKc_final, Kc_final> + <dVc_final, Vc_final>
 * through Algorithm 2 (cache-first order, output ReLU) started from the cache Kc_in, Vc_in [M,d] with
 * c_in valid rows (NULL, NULL, 0: an empty cache).  A sequence processed in several calls of the loop
 * is differentiated call by call, last call first: the cache gradient a call returns in dKc_in, dVc_in
 * [M,d] (optional; rows >= c_in are zero) is the dKc_final, dVc_final of the call before it.
 * Accumulates into dQ, dK, dV [L,d], dG [M,c_in,k], dbias [M] (optional): callers zero them.
 * Returns 0, or -1 if a flag selects a reading the backward does not cover.
 */
int lococo_oracle_process_sequence_grad_from(const oracle_params* P, const double* Q, const double* K,
                                             const double* V, int L, int B, const double* G, const double* bias,
                                             const double* Kc_in, const double* Vc_in, int c_in,
                                             const double* dO, const double* dKc_final, const double* dVc_final,
                                             double* dQ, double* dK, double* dV, double* dG, double* dbias,
                                             double* dKc_in, double* dVc_in) {
    if (P->flags != 0) return -1;
    const int d = P->d, M = P->M;
    const int N = (L + B - 1) / B;
    double* O = dalloc((size_t)L * d);
    double* Kc = dalloc((size_t)M * d);
    double* Vc = dalloc((size_t)M * d);
    double* snapK = dalloc((size_t)N * M * d);
    double* snapV = dalloc((size_t)N * M * d);
    int32_t* snapc = (int32_t*)calloc((size_t)N, sizeof(int32_t));
    int c_final = c_in;
    if (c_in > 0) {
        memcpy(Kc, Kc_in, sizeof(double) * (size_t)c_in * d);
        memcpy(Vc, Vc_in, sizeof(double) * (size_t)c_in * d);
    }
    lococo_oracle_process_sequence(P, Q, K, V, L, B, G, bias, O, Kc, Vc, &c_final, NULL, snapK, snapV, snapc);

    /* gradient w.r.t. the cache as it stands after step n (starts as the loss's own term) */
    double* gKc = dalloc((size_t)M * d);
    double* gVc = dalloc((size_t)M * d);
    memcpy(gKc, dKc_final, sizeof(double) * (size_t)M * d);
    memcpy(gVc, dVc_final, sizeof(double) * (size_t)M * d);
    double* XK = dalloc((size_t)(M + B) * d);
    double* XV = dalloc((size_t)(M + B) * d);
    double* dXK = dalloc((size_t)(M + B) * d);
    double* dXV = dalloc((size_t)(M + B) * d);

    for (int n = N - 1; n >= 0; --n) {
        const int t0 = n * B;
        const int b = (L - t0 < B) ? (L - t0) : B;
        const int c = snapc[n];
        const int S = c + b;
        const double* Kold = snapK + (size_t)n * M * d;
        const double* Vold = snapV + (size_t)n * M * d;
        memcpy(XK, Kold, sizeof(double) * (size_t)c * d);
        memcpy(XK + (size_t)c * d, K + (size_t)t0 * d, sizeof(double) * (size_t)b * d);
        memcpy(XV, Vold, sizeof(double) * (size_t)c * d);
        memcpy(XV + (size_t)c * d, V + (size_t)t0 * d, sizeof(double) * (size_t)b * d);
        memset(dXK, 0, sizeof(double) * (size_t)S * d);
        memset(dXV, 0, sizeof(double) * (size_t)S * d);
        /* cache update of step n: fill copies rows, compress goes through Eq. 4-7 */
        if (c + b <= M) {
            memcpy(dXK, gKc, sizeof(double) * (size_t)S * d);
            memcpy(dXV, gVc, sizeof(double) * (size_t)S * d);
        } else {
            compress_backward(P, XK, XV, S, G, bias, gKc, gVc, dXK, dXV, dG, dbias);
        }
        /* attention of step n read the same [old cache, chunk] */
        attention_backward(Q + (size_t)t0 * d, b, XK, XV, c, d, P->scale, dO + (size_t)t0 * d,
                           dQ + (size_t)t0 * d, dXK, dXV);
        /* split: first c rows flow to the cache of step n-1, last b rows are this chunk's K, V */
        memset(gKc, 0, sizeof(double) * (size_t)M * d);
        memset(gVc, 0, sizeof(double) * (size_t)M * d);
        memcpy(gKc, dXK, sizeof(double) * (size_t)c * d);
        memcpy(gVc, dXV, sizeof(double) * (size_t)c * d);
        for (size_t x = 0; x < (size_t)b * d; ++x) {
            dK[(size_t)t0 * d + x] += dXK[(size_t)c * d + x];
            dV[(size_t)t0 * d + x] += dXV[(size_t)c * d + x];
        }
    }
    /* what is left is the gradient w.r.t. the cache the loop started from */
    if (dKc_in) memcpy(dKc_in, gKc, sizeof(double) * (size_t)M * d);
    if (dVc_in) memcpy(dVc_in, gVc, sizeof(double) * (size_t)M * d);
    free(O); free(Kc); free(Vc); free(snapK); free(snapV); free(snapc);
    free(gKc); free(gVc); free(XK); free(XV); free(dXK); free(dXV);
    return 0;
}

/* The same from an empty cache. */
int lococo_oracle_process_sequence_grad(const oracle_params* P, const double* Q, const double* K,
                                        const double* V, int L, int B, const double* G, const double* bias,
                                        const double* dO, const double* dKc_final, const double* dVc_final,
                                        double* dQ, double* dK, double* dV, double* dG, double* dbias) {
    return lococo_oracle_process_sequence_grad_from(P, Q, K, V, L, B, G, bias, NULL, NULL, 0, dO, dKc_final, dVc_final,
                                                    dQ, dK, dV, dG, dbias, NULL, NULL);
}

/*
 * Batched drivers: units = batch*heads independent (sequence, head) problems, contiguous
 * [units, L, d] arrays.  g_unit_stride is 0 for weights shared by all heads, else M*c_in*k
 * with unit u using head u % heads.  OpenMP only across units.
 */
void lococo_oracle_process_batch(const oracle_params* P, int units, int heads, const double* Q,
                                 const double* K, const double* V, int L, int B, const double* G,
                                 long g_head_stride, const double* bias, long bias_head_stride,
                                 double* O, double* Kc, double* Vc, int32_t* c_inout, double* lse) {
    const int d = P->d, M = P->M;
#pragma omp parallel for schedule(dynamic, 1) if (units > 1)   /* one unit: the loops inside it take the threads */
    for (int u = 0; u < units; ++u) {
        const int h = u % heads;
        int c = c_inout[u];
        lococo_oracle_process_sequence(P, Q + (size_t)u * L * d, K + (size_t)u * L * d, V + (size_t)u * L * d,
                                       L, B, G + (size_t)h * g_head_stride,
                                       bias ? bias + (size_t)h * bias_head_stride : NULL,
                                       O + (size_t)u * L * d, Kc + (size_t)u * M * d, Vc + (size_t)u * M * d,
                                       &c, lse ? lse + (size_t)u * L : NULL, NULL, NULL, NULL);
        c_inout[u] = c;
    }
}

/* dG / dbias are summed over the units that share a weight set (g_head_stride == 0: all). */
int lococo_oracle_grad_batch(const oracle_params* P, int units, int heads, const double* Q,
                             const double* K, const double* V, int L, int B, const double* G,
                             long g_head_stride, const double* bias, long bias_head_stride,
                             const double* dO, const double* dKc_final, const double* dVc_final,
                             double* dQ, double* dK, double* dV, double* dG, double* dbias) {
    const int d = P->d, M = P->M;
    const size_t gsz = (size_t)M * P->c_in * P->k;
    int rc = 0;
#pragma omp parallel for schedule(dynamic, 1) if (units > 1)   /* one unit: the loops inside it take the threads */
    for (int u = 0; u < units; ++u) {
        const int h = u % heads;
        double* dG_u = dalloc(gsz);
        double* db_u = dalloc((size_t)M);
        int r = lococo_oracle_process_sequence_grad(
            P, Q + (size_t)u * L * d, K + (size_t)u * L * d, V + (size_t)u * L * d, L, B,
            G + (size_t)h * g_head_stride, bias ? bias + (size_t)h * bias_head_stride : NULL,
            dO + (size_t)u * L * d, dKc_final + (size_t)u * M * d, dVc_final + (size_t)u * M * d,
            dQ + (size_t)u * L * d, dK + (size_t)u * L * d, dV + (size_t)u * L * d, dG_u,
            dbias ? db_u : NULL);
#pragma omp critical
        {
            if (r) rc = r;
            double* dst = dG + (size_t)h * g_head_stride;
            for (size_t x = 0; x < gsz; ++x) dst[x] += dG_u[x];
            if (dbias) {
                double* bd = dbias + (size_t)h * bias_head_stride;
                for (int i = 0; i < M; ++i) bd[i] += db_u[i];
            }
        }
        free(dG_u); free(db_u);
    }
    return rc;
}

int lococo_oracle_threads(void) {
    int n = 1;
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    n = omp_get_max_threads();
#endif
    return n;
}
