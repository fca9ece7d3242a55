/*
 * fp64 CPU oracle for scaled-dot-product attention, forward and backward.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
 * CUDA path is checked against.  Only the tests, the smoke check and the
 * bench's cpu_baseline / reference legs may call it; the product path never
 * does.  It shares no code, header, table or helper with the CUDA sources.
 *
 * What it computes is the textbook definition, written out: the whole score
 * row is materialised, the softmax is taken in two passes (max, then
 * exp/sum), and the gradients are the exact derivatives of
 *     Loss = sum(dO * O(Q, K, V)).
 * There is no tiling, no online rescaling and no recomputation trick, so the
 * tiled/online evaluation order of the GPU kernels (the consumer loop of the
 * corrected Algorithm 2 in the paper's appendix "Published and corrected
 * FlashAttention-3 pseudocode") is checked against an independent order.
 *
 * Operator definition: paper, appendix "Workloads" (forward returns O and an
 * fp32 log-sum-exp per (head, query); the causal variants apply a
 * lower-triangular mask; backward consumes Q, K, V, O, dO, LSE and returns
 * dQ, dK, dV) and "Generalization attention workloads" (GQA, ragged/packed
 * batches).  LSE = m + log(l): epilogue of the corrected Algorithm 2, read as
 * the natural log of the scaled, masked scores.
 *
 * Layout (all double, contiguous, token-major / packed):
 *   q, o, dout, dq : [T, Hq,  D]        k, v, dk, dv : [T, Hkv, D]
 *   lse            : [Hq, T]
 *   cu_seqlens     : int32 [B+1], sequence b owns token rows cu[b] .. cu[b+1]-1
 * GQA: query head h reads kv head h / (Hq / Hkv).
 * Causal: query i of a sequence sees keys 0..i of the same sequence.
 *
 * Parity pins (tests, CPU only): softmax row sums, constant-V, causal row 0,
 * Q = 0 closed forms, key-permutation and score-shift invariance,
 * rowsum(dS) = 0, sum(dQ*Q) = sum(dK*K), central finite differences, GQA ==
 * repeated-KV MHA, packed == per-sequence, torch CPU float64 SDPA + autograd,
 * a second brute-force numpy restatement, online == materialised.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double dot(const double* a, const double* b, int n) {
    double acc = 0.0;
#pragma omp simd reduction(+ : acc)
    for (int d = 0; d < n; ++d) acc += a[d] * b[d];
    return acc;
}

static void axpy(double alpha, const double* x, double* y, int n) {
#pragma omp simd
    for (int d = 0; d < n; ++d) y[d] += alpha * x[d];
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* One query row: scores over the allowed keys, softmax, output row, lse.
 * p[0..n) receives the probabilities.  Returns n, the number of allowed keys. */
static int fwd_row(const double* qrow, const double* k, const double* v, int ldkv, int L, int i,
                   int D, int causal, double scale, double* p, double* orow, double* lse_out) {
    int n = causal ? (i + 1) : L; /* lower-triangular mask: keys 0..i */
    double m = -INFINITY;
    for (int j = 0; j < n; ++j) {
        p[j] = scale * dot(qrow, k + (size_t)j * ldkv, D); /* s_ij = scale * q_i . k_j */
        if (p[j] > m) m = p[j];
    }
    double l = 0.0;
    for (int j = 0; j < n; ++j) {
        p[j] = exp(p[j] - m);
        l += p[j];
    }
    for (int j = 0; j < n; ++j) p[j] /= l;
    for (int d = 0; d < D; ++d) orow[d] = 0.0;
    for (int j = 0; j < n; ++j) axpy(p[j], v + (size_t)j * ldkv, orow, D); /* o_i = sum_j p_ij v_j */
    *lse_out = m + log(l);
    return n;
}

/* Forward: O = softmax(scale * Q K^T + mask) V, LSE = log sum exp of the scaled masked scores. */
int oracle_sdpa_fwd(const double* q, const double* k, const double* v, double* o, double* lse,
                    const int32_t* cu_seqlens, int B, int Hq, int Hkv, int D, int causal,
                    double scale) {
    if (B < 0 || Hq < 1 || Hkv < 1 || D < 1 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    const int T = cu_seqlens[B];
    int maxL = 0;
    for (int b = 0; b < B; ++b) {
        int L = cu_seqlens[b + 1] - cu_seqlens[b];
        if (L < 0) return -2;
        if (L > maxL) maxL = L;
    }
    const int ldq = Hq * D, ldkv = Hkv * D;
    int err = 0;
#pragma omp parallel
    {
        double* p = (double*)malloc(sizeof(double) * (size_t)(maxL > 0 ? maxL : 1));
        if (!p) {
#pragma omp atomic write
            err = 1;
        }
        for (int b = 0; b < B && p; ++b) {
            const int r0 = cu_seqlens[b], L = cu_seqlens[b + 1] - r0;
#pragma omp for collapse(2) schedule(dynamic, 4) nowait
            for (int h = 0; h < Hq; ++h) {
                for (int i = 0; i < L; ++i) {
                    const int g = h / G;
                    const double* kb = k + (size_t)r0 * ldkv + (size_t)g * D;
                    const double* vb = v + (size_t)r0 * ldkv + (size_t)g * D;
                    const size_t qo = (size_t)(r0 + i) * ldq + (size_t)h * D;
                    fwd_row(q + qo, kb, vb, ldkv, L, i, D, causal, scale, p, o + qo,
                            lse + (size_t)h * T + r0 + i);
                }
            }
        }
        free(p);
    }
    return err ? -3 : 0;
}

/* Backward of Loss = sum(dO * O).  With P the softmax probabilities:
 *   dP_ij = dO_i . v_j          D_i = dO_i . o_i         dS_ij = P_ij (dP_ij - D_i)
 *   dQ_i = scale * sum_j dS_ij k_j
 *   dK_j = scale * sum_{h in group} sum_i dS_ij q_i
 *   dV_j =         sum_{h in group} sum_i P_ij dO_i
 * The forward is recomputed here in fp64 (the oracle's own O); o and lse are
 * also written when the pointers are non-null. */
int oracle_sdpa_bwd(const double* q, const double* k, const double* v, const double* dout,
                    double* dq, double* dk, double* dv, double* o, double* lse,
                    const int32_t* cu_seqlens, int B, int Hq, int Hkv, int D, int causal,
                    double scale) {
    if (B < 0 || Hq < 1 || Hkv < 1 || D < 1 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    const int T = cu_seqlens[B];
    int maxL = 0;
    for (int b = 0; b < B; ++b) {
        int L = cu_seqlens[b + 1] - cu_seqlens[b];
        if (L < 0) return -2;
        if (L > maxL) maxL = L;
    }
    const int ldq = Hq * D, ldkv = Hkv * D;
    memset(dk, 0, sizeof(double) * (size_t)T * ldkv);
    memset(dv, 0, sizeof(double) * (size_t)T * ldkv);
    int err = 0;
#pragma omp parallel
    {
        const size_t nl = (size_t)(maxL > 0 ? maxL : 1);
        double* p = (double*)malloc(sizeof(double) * nl);
        double* ds = (double*)malloc(sizeof(double) * nl);
        double* orow = (double*)malloc(sizeof(double) * (size_t)D);
        /* thread-private dK/dV of one (sequence, kv head), summed after the row loop */
        double* dk_acc = (double*)malloc(sizeof(double) * nl * D);
        double* dv_acc = (double*)malloc(sizeof(double) * nl * D);
        if (!p || !ds || !orow || !dk_acc || !dv_acc) {
#pragma omp atomic write
            err = 1;
        }
#pragma omp barrier
        int bad;
#pragma omp atomic read
        bad = err;
        for (int b = 0; b < B && !bad; ++b) {
            const int r0 = cu_seqlens[b], L = cu_seqlens[b + 1] - r0;
            for (int g = 0; g < Hkv; ++g) {
                const double* kb = k + (size_t)r0 * ldkv + (size_t)g * D;
                const double* vb = v + (size_t)r0 * ldkv + (size_t)g * D;
                memset(dk_acc, 0, sizeof(double) * (size_t)L * D);
                memset(dv_acc, 0, sizeof(double) * (size_t)L * D);
#pragma omp for collapse(2) schedule(dynamic, 4) nowait
                for (int hh = 0; hh < G; ++hh) {
                    for (int i = 0; i < L; ++i) {
                        const int h = g * G + hh;
                        const size_t qo = (size_t)(r0 + i) * ldq + (size_t)h * D;
                        const double* qrow = q + qo;
                        const double* dorow = dout + qo;
                        double lse_i;
                        const int n =
                            fwd_row(qrow, kb, vb, ldkv, L, i, D, causal, scale, p, orow, &lse_i);
                        if (o) memcpy(o + qo, orow, sizeof(double) * (size_t)D);
                        if (lse) lse[(size_t)h * T + r0 + i] = lse_i;
                        const double Di = dot(dorow, orow, D);
                        double* dqrow = dq + qo;
                        for (int d = 0; d < D; ++d) dqrow[d] = 0.0;
                        for (int j = 0; j < n; ++j) {
                            const double dp = dot(dorow, vb + (size_t)j * ldkv, D);
                            ds[j] = p[j] * (dp - Di);
                        }
                        for (int j = 0; j < n; ++j) {
                            axpy(scale * ds[j], kb + (size_t)j * ldkv, dqrow, D);
                            axpy(scale * ds[j], qrow, dk_acc + (size_t)j * D, D);
                            axpy(p[j], dorow, dv_acc + (size_t)j * D, D);
                        }
                    }
                }
#pragma omp critical
                {
                    for (int j = 0; j < L; ++j) {
                        axpy(1.0, dk_acc + (size_t)j * D, dk + (size_t)(r0 + j) * ldkv + (size_t)g * D, D);
                        axpy(1.0, dv_acc + (size_t)j * D, dv + (size_t)(r0 + j) * ldkv + (size_t)g * D, D);
                    }
                }
#pragma omp barrier
            }
        }
        free(p);
        free(ds);
        free(orow);
        free(dk_acc);
        free(dv_acc);
    }
    return err ? -3 : 0;
}
