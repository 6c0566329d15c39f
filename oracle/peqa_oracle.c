/*
 * PEQA reference oracle -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow CPU statement of what the PEQA quantized linear layer computes
 * (arXiv 2305.14152).  Only tests, the smoke check and the benchmark's CPU
 * baseline may call it.  It shares no code, header, table or helper with the
 * CUDA library; it is written directly from the paper's equations:
 *
 *   Eq. 1  (Sec. 3.2)  W_hat0 = s0 * (clamp(round(W0/s0) + z0, 0, 2^b-1) - z0)
 *   Eq. 2  (Sec. 3.2)  W_hat  = (s0 + ds) * W_bar0,   W_bar0 = Q - z  frozen
 *   Sec. 4.2 "Group-wise Quantization": one (s, z) per run of g input columns
 *   App. A: AdamW is the optimizer acting on s
 *
 * Conventions: W is [N out, K in] row-major; group gi of row i covers columns
 * [gi*g, (gi+1)*g); per-channel is g == K.  Activations arrive as bf16 bit
 * patterns (uint16) and are widened exactly to double.  All contractions
 * accumulate in double, in the index order of the defining sum.  OpenMP splits
 * only the outermost independent loop; nothing is blocked, fused or reordered.
 *
 * Pins (tests/test_oracle_*.py): exact worked examples for Eq. 1, hand-packed
 * words, brute-force Python loops on tiny shapes, s=1,z=0 integer matmul,
 * g=K == per-channel, linearity of <dY,Y> in s (finite difference == dS),
 * the adjoint identity <dY,fwd(X)> == <dX,X>, and the closed form of the
 * first AdamW step; for the searched quantizer: candidate 0 == plain RTN, a
 * brute-force search on tiny groups, never worse than RTN; for the real-valued
 * zero-point: equality with the integer functions on integral z, exact rational
 * brute force, and finite differences of <dY,Y> in z.  No function here is
 * "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t h) {
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static int n_groups(int K, int g) { return K / g; }

/* ---------------------------------------------------------------- Eq. 1 ---
 * Asymmetric round-to-nearest quantization of one [N,K] matrix, one (s,z) per
 * (row, group).  The arithmetic is IEEE binary32 with round-half-to-even at
 * every operation (compile with -ffp-contract=off, no fast-math), because a
 * code is an integer decision and both sides must take it in one precision:
 *     mn, mx = min/max over the group
 *     s  = (mx - mn) / (2^b - 1)            (s := 1 when mx == mn)
 *     z  = clamp(rint(-mn / s), 0, 2^b-1)
 *     q  = clamp(rint(w / s) + z, 0, 2^b-1)
 * The paper's Eq. 1 has no clamp on z and does not name the rounding mode;
 * the readings are listed in the design notes.
 */
void oracle_quantize_rtn(const float* W, int N, int K, int bits, int g,
                         uint8_t* codes, uint8_t* zeros, float* scales) {
    const float qmax = (float)((1 << bits) - 1);
    const int G = n_groups(K, g);
#pragma omp parallel for schedule(static)
    for (int i = 0; i < N; ++i) {
        for (int gi = 0; gi < G; ++gi) {
            const float* w = W + (size_t)i * K + (size_t)gi * g;
            float mn = w[0], mx = w[0];
            for (int j = 1; j < g; ++j) {
                if (w[j] < mn) mn = w[j];
                if (w[j] > mx) mx = w[j];
            }
            volatile float range = mx - mn;
            volatile float s = range / qmax;
            if (mx == mn) s = 1.0f;
            volatile float zq = (-mn) / s;
            float z = rintf(zq);
            if (z < 0.0f) z = 0.0f;
            if (z > qmax) z = qmax;
            scales[(size_t)i * G + gi] = s;
            zeros[(size_t)i * G + gi] = (uint8_t)z;
            for (int j = 0; j < g; ++j) {
                volatile float r = w[j] / s;
                volatile float q = rintf(r) + z;
                float qc = q;
                if (qc < 0.0f) qc = 0.0f;
                if (qc > qmax) qc = qmax;
                codes[(size_t)i * K + (size_t)gi * g + j] = (uint8_t)qc;
            }
        }
    }
}

/* Same steps with every division and rounding taken in binary64.  Used only to
 * count how many codes depend on the precision of the quotient (near-ties). */
void oracle_quantize_rtn_f64(const float* W, int N, int K, int bits, int g,
                             uint8_t* codes, uint8_t* zeros, double* scales) {
    const double qmax = (double)((1 << bits) - 1);
    const int G = n_groups(K, g);
#pragma omp parallel for schedule(static)
    for (int i = 0; i < N; ++i) {
        for (int gi = 0; gi < G; ++gi) {
            const float* w = W + (size_t)i * K + (size_t)gi * g;
            double mn = w[0], mx = w[0];
            for (int j = 1; j < g; ++j) {
                if (w[j] < mn) mn = w[j];
                if (w[j] > mx) mx = w[j];
            }
            double s = (mx - mn) / qmax;
            if (mx == mn) s = 1.0;
            double z = rint((-mn) / s);
            if (z < 0.0) z = 0.0;
            if (z > qmax) z = qmax;
            scales[(size_t)i * G + gi] = s;
            zeros[(size_t)i * G + gi] = (uint8_t)z;
            for (int j = 0; j < g; ++j) {
                double q = rint((double)w[j] / s) + z;
                if (q < 0.0) q = 0.0;
                if (q > qmax) q = qmax;
                codes[(size_t)i * K + (size_t)gi * g + j] = (uint8_t)q;
            }
        }
    }
}

/* ------------------------------------------------------- packed layout ----
 * The paper only says the weights are a b-bit integer matrix (Sec. 3.3); the
 * interchange layout is this library's: each row is a little-endian bit string
 * in which column j occupies bits [b*j, b*j + b).  Cut into uint32 words this
 * gives 8 columns per word for b=4 and 32 columns per 3 words for b=3 (columns
 * 10 and 21 of every 32 straddle a word boundary).  The oracle writes and
 * reads one bit at a time so that no shift/mask shortcut can hide a mistake.
 */
void oracle_pack(const uint8_t* codes, int N, int K, int bits, uint32_t* words) {
    const size_t wpr = (size_t)K * bits / 32;
    memset(words, 0, (size_t)N * wpr * sizeof(uint32_t));
    for (int i = 0; i < N; ++i)
        for (int j = 0; j < K; ++j)
            for (int t = 0; t < bits; ++t) {
                size_t bit = (size_t)j * bits + t;
                uint32_t v = (codes[(size_t)i * K + j] >> t) & 1u;
                words[(size_t)i * wpr + bit / 32] |= v << (bit % 32);
            }
}

void oracle_unpack(const uint32_t* words, int N, int K, int bits, uint8_t* codes) {
    const size_t wpr = (size_t)K * bits / 32;
    for (int i = 0; i < N; ++i)
        for (int j = 0; j < K; ++j) {
            uint8_t c = 0;
            for (int t = 0; t < bits; ++t) {
                size_t bit = (size_t)j * bits + t;
                uint32_t v = (words[(size_t)i * wpr + bit / 32] >> (bit % 32)) & 1u;
                c |= (uint8_t)(v << t);
            }
            codes[(size_t)i * K + j] = c;
        }
}

/* Row i of W_hat = s * (Q - z) (Eq. 2), widened to double. */
static void what_row(const uint8_t* codes, const uint8_t* zeros, const float* scales,
                     int K, int g, int i, double* out) {
    const int G = n_groups(K, g);
    for (int j = 0; j < K; ++j) {
        int gi = j / g;
        double s = (double)scales[(size_t)i * G + gi];
        double wbar = (double)codes[(size_t)i * K + j] - (double)zeros[(size_t)i * G + gi];
        out[j] = s * wbar;
    }
}

/* ------------------------------------------------------------ forward -----
 * Y[t,i] = sum_j X[t,j] * W_hat[i,j]   (the layer y = x W_hat^T with Eq. 2).
 * tok_sel (length n_sel) lists the token rows to evaluate; NULL means all T
 * rows in order.  Y is [n_sel, N] double.
 */
void oracle_fwd(const uint16_t* X, int T, const uint8_t* codes, const uint8_t* zeros,
                const float* scales, int N, int K, int g,
                const int32_t* tok_sel, int n_sel, double* Y) {
    if (!tok_sel) n_sel = T;
    double* Xd = (double*)malloc((size_t)n_sel * K * sizeof(double));
    for (int r = 0; r < n_sel; ++r) {
        int t = tok_sel ? tok_sel[r] : r;
        for (int j = 0; j < K; ++j) Xd[(size_t)r * K + j] = bf16_to_double(X[(size_t)t * K + j]);
    }
#pragma omp parallel
    {
        double* w = (double*)malloc((size_t)K * sizeof(double));
#pragma omp for schedule(static)
        for (int i = 0; i < N; ++i) {
            what_row(codes, zeros, scales, K, g, i, w);
            for (int r = 0; r < n_sel; ++r) {
                const double* x = Xd + (size_t)r * K;
                double acc = 0.0;
                for (int j = 0; j < K; ++j) acc += x[j] * w[j];
                Y[(size_t)r * N + i] = acc;
            }
        }
        free(w);
    }
    free(Xd);
}

/* ------------------------------------------------------ backward: dX ------
 * dX[t,j] = sum_i dY[t,i] * W_hat[i,j]   (chain rule through y = x W_hat^T).
 * tok_sel as in oracle_fwd.  dX is [n_sel, K] double.
 */
void oracle_bwd_dx(const uint16_t* dY, int T, const uint8_t* codes, const uint8_t* zeros,
                   const float* scales, int N, int K, int g,
                   const int32_t* tok_sel, int n_sel, double* dX) {
    if (!tok_sel) n_sel = T;
    double* What = (double*)malloc((size_t)N * K * sizeof(double));
#pragma omp parallel for schedule(static)
    for (int i = 0; i < N; ++i) what_row(codes, zeros, scales, K, g, i, What + (size_t)i * K);
#pragma omp parallel for schedule(static)
    for (int r = 0; r < n_sel; ++r) {
        int t = tok_sel ? tok_sel[r] : r;
        double* out = dX + (size_t)r * K;
        for (int j = 0; j < K; ++j) out[j] = 0.0;
        for (int i = 0; i < N; ++i) {
            double d = bf16_to_double(dY[(size_t)t * N + i]);
            const double* w = What + (size_t)i * K;
            for (int j = 0; j < K; ++j) out[j] += d * w[j];
        }
    }
    free(What);
}

/* ------------------------------------------------------ backward: dS ------
 * Since dW_hat[i,j]/ds[i,gi] = (Q[i,j] - z[i,gi]) for j in group gi (Eq. 2):
 *   dS[i,gi] = sum_{j in gi} (Q[i,j] - z[i,gi]) * dW[i,j],
 *   dW[i,j]  = sum_t dY[t,i] * X[t,j].
 * row_sel (length n_sel) lists the output channels i to evaluate; NULL = all.
 * dS is [n_sel, G] double.
 */
void oracle_bwd_ds(const uint16_t* X, const uint16_t* dY, int T, const uint8_t* codes,
                   const uint8_t* zeros, int N, int K, int g,
                   const int32_t* row_sel, int n_sel, double* dS) {
    const int G = n_groups(K, g);
    if (!row_sel) n_sel = N;
    double* Xd = (double*)malloc((size_t)T * K * sizeof(double));
#pragma omp parallel for schedule(static)
    for (int t = 0; t < T; ++t)
        for (int j = 0; j < K; ++j) Xd[(size_t)t * K + j] = bf16_to_double(X[(size_t)t * K + j]);
#pragma omp parallel
    {
        double* dw = (double*)malloc((size_t)K * sizeof(double));
#pragma omp for schedule(static)
        for (int r = 0; r < n_sel; ++r) {
            int i = row_sel ? row_sel[r] : r;
            for (int j = 0; j < K; ++j) dw[j] = 0.0;
            for (int t = 0; t < T; ++t) {
                double d = bf16_to_double(dY[(size_t)t * N + i]);
                const double* x = Xd + (size_t)t * K;
                for (int j = 0; j < K; ++j) dw[j] += d * x[j];
            }
            for (int gi = 0; gi < G; ++gi) {
                double acc = 0.0;
                double z = (double)zeros[(size_t)i * G + gi];
                for (int j = gi * g; j < (gi + 1) * g; ++j)
                    acc += ((double)codes[(size_t)i * K + j] - z) * dw[j];
                dS[(size_t)r * G + gi] = acc;
            }
        }
        free(dw);
    }
    free(Xd);
}

/* ------------------------------------------------- zero-point gradient -----
 * App. K trains the zero-points as well; by the chain rule on Eq. 2,
 * d W_hat[i,j] / d z[i,g] = -s[i,g] for the columns j of group g, so
 *   dZ[i,g] = -s[i,g] * sum_{j in g} (dY^T X)[i,j].
 * X [T,K], dY [T,N] bf16 bit patterns; scales fp32 [N,G]; row_sel as in oracle_bwd_ds;
 * dZ is [n_sel, G] double.
 */
void oracle_bwd_dz(const uint16_t* X, const uint16_t* dY, int T, const float* scales, int N,
                   int K, int g, const int32_t* row_sel, int n_sel, double* dZ) {
    const int G = n_groups(K, g);
    if (!row_sel) n_sel = N;
#pragma omp parallel for schedule(static)
    for (int r = 0; r < n_sel; ++r) {
        int i = row_sel ? row_sel[r] : r;
        for (int gi = 0; gi < G; ++gi) {
            double acc = 0.0;
            for (int j = gi * g; j < (gi + 1) * g; ++j) {
                double dw = 0.0;
                for (int t = 0; t < T; ++t)
                    dw += bf16_to_double(dY[(size_t)t * N + i]) * bf16_to_double(X[(size_t)t * K + j]);
                acc += dw;
            }
            dZ[(size_t)r * G + gi] = -(double)scales[(size_t)i * G + gi] * acc;
        }
    }
}

/* ---------------------------------------- per-channel dS from the saved Y ---
 * With one scale per output channel (G = 1), Eq. 2 gives Y[t,i] = s[i] * u[t,i] with
 * u[t,i] = sum_j X[t,j] (Q[i,j] - z[i]), and the chain rule gives
 * dS[i] = sum_t dY[t,i] u[t,i].  Hence, written out with the stored output,
 *   dS[i] = ( sum_t dY[t,i] * Y[t,i] ) / s[i].
 * Y is the bf16 tensor the forward pass stored (its rounding is part of the input here).
 * dY, Y are bf16 bit patterns [T, N]; scales is fp32 [N]; dS is double [N].
 */
void oracle_bwd_ds_from_y(const uint16_t* dY, const uint16_t* Y, const float* scales, int T,
                          int N, double* dS) {
#pragma omp parallel for schedule(static)
    for (int i = 0; i < N; ++i) {
        double acc = 0.0;
        for (int t = 0; t < T; ++t)
            acc += bf16_to_double(dY[(size_t)t * N + i]) * bf16_to_double(Y[(size_t)t * N + i]);
        dS[i] = acc / (double)scales[i];
    }
}

/* ------------------------------------- Eq. 1 with a searched clipping range --
 * Sec. 3.2 says that s0 and z0 "are initialized to minimize" the Frobenius error
 * of Eq. 1 and gives no procedure (Sec. 4.1 names plain round-to-nearest).  The
 * reading taken: per (row, group), try n_cand shrunken ranges and keep the one
 * whose reconstruction error is smallest.  Candidate k = 0 .. n_cand-1 scales the
 * group's extremes by p_k = 1 - k/64 (k = 0 is the plain min/max range of
 * oracle_quantize_rtn) and then follows Eq. 1 exactly as above, in binary32:
 *     lo = p*mn, hi = p*mx;  s = (hi - lo)/(2^b-1)  (s := 1 when hi == lo)
 *     z = clamp(rint(-lo/s), 0, 2^b-1);  q_j = clamp(rint(w_j/s) + z, 0, 2^b-1)
 *     r_j = s*(q_j - z);  e_j = w_j - r_j                       (binary32 each)
 *     err = sum_j e_j^2    in binary64, columns in ascending order
 * The first candidate with the smallest err wins (a later one must be strictly
 * better), so the result is never worse than plain round-to-nearest.
 * chosen[i*G+gi] receives the winning k; err_out (may be NULL) its error.
 * n_cand <= 64.
 */
void oracle_quantize_search(const float* W, int N, int K, int bits, int g, int n_cand,
                            uint8_t* codes, uint8_t* zeros, float* scales, uint8_t* chosen,
                            double* err_out) {
    const float qmax = (float)((1 << bits) - 1);
    const int G = n_groups(K, g);
#pragma omp parallel for schedule(static)
    for (int i = 0; i < N; ++i) {
        uint8_t* tmp = (uint8_t*)malloc((size_t)g);
        for (int gi = 0; gi < G; ++gi) {
            const float* w = W + (size_t)i * K + (size_t)gi * g;
            uint8_t* out = codes + (size_t)i * K + (size_t)gi * g;
            float mn = w[0], mx = w[0];
            for (int j = 1; j < g; ++j) {
                if (w[j] < mn) mn = w[j];
                if (w[j] > mx) mx = w[j];
            }
            double best = 0.0;
            int best_k = -1;
            for (int k = 0; k < n_cand; ++k) {
                volatile float p = 1.0f - (float)k / 64.0f;
                volatile float lo = p * mn;
                volatile float hi = p * mx;
                volatile float range = hi - lo;
                volatile float s = range / qmax;
                if (hi == lo) s = 1.0f;
                volatile float zq = (-lo) / s;
                float z = rintf(zq);
                if (z < 0.0f) z = 0.0f;
                if (z > qmax) z = qmax;
                double err = 0.0;
                for (int j = 0; j < g; ++j) {
                    volatile float r = w[j] / s;
                    volatile float q = rintf(r) + z;
                    float qc = q;
                    if (qc < 0.0f) qc = 0.0f;
                    if (qc > qmax) qc = qmax;
                    volatile float d = qc - z;
                    volatile float rec = s * d;
                    volatile float e = w[j] - rec;
                    err += (double)e * (double)e;
                    tmp[j] = (uint8_t)qc;
                }
                if (best_k < 0 || err < best) {
                    best = err;
                    best_k = k;
                    scales[(size_t)i * G + gi] = s;
                    zeros[(size_t)i * G + gi] = (uint8_t)z;
                    memcpy(out, tmp, (size_t)g);
                }
            }
            chosen[(size_t)i * G + gi] = (uint8_t)best_k;
            if (err_out) err_out[(size_t)i * G + gi] = best;
        }
        free(tmp);
    }
}

/* --------------------------------------- the layer with a real-valued z -----
 * App. K also trains the zero-points ("zero-points only", "both"); z then leaves
 * the integer grid and Eq. 2's weight is W_hat[i,j] = s[i,g] * (Q[i,j] - z[i,g])
 * with z a binary32 number.  The three functions below are oracle_fwd,
 * oracle_bwd_dx and oracle_bwd_ds with that z; the zero-point gradient
 * (oracle_bwd_dz) does not depend on z.
 */
static void what_row_zf(const uint8_t* codes, const float* zeros_f, const float* scales,
                        int K, int g, int i, double* out) {
    const int G = n_groups(K, g);
    for (int j = 0; j < K; ++j) {
        int gi = j / g;
        double s = (double)scales[(size_t)i * G + gi];
        double wbar = (double)codes[(size_t)i * K + j] - (double)zeros_f[(size_t)i * G + gi];
        out[j] = s * wbar;
    }
}

void oracle_fwd_zf(const uint16_t* X, int T, const uint8_t* codes, const float* zeros_f,
                   const float* scales, int N, int K, int g,
                   const int32_t* tok_sel, int n_sel, double* Y) {
    if (!tok_sel) n_sel = T;
#pragma omp parallel
    {
        double* w = (double*)malloc((size_t)K * sizeof(double));
#pragma omp for schedule(static)
        for (int i = 0; i < N; ++i) {
            what_row_zf(codes, zeros_f, scales, K, g, i, w);
            for (int r = 0; r < n_sel; ++r) {
                int t = tok_sel ? tok_sel[r] : r;
                double acc = 0.0;
                for (int j = 0; j < K; ++j) acc += bf16_to_double(X[(size_t)t * K + j]) * w[j];
                Y[(size_t)r * N + i] = acc;
            }
        }
        free(w);
    }
}

void oracle_bwd_dx_zf(const uint16_t* dY, int T, const uint8_t* codes, const float* zeros_f,
                      const float* scales, int N, int K, int g,
                      const int32_t* tok_sel, int n_sel, double* dX) {
    if (!tok_sel) n_sel = T;
    double* What = (double*)malloc((size_t)N * K * sizeof(double));
#pragma omp parallel for schedule(static)
    for (int i = 0; i < N; ++i) what_row_zf(codes, zeros_f, scales, K, g, i, What + (size_t)i * K);
#pragma omp parallel for schedule(static)
    for (int r = 0; r < n_sel; ++r) {
        int t = tok_sel ? tok_sel[r] : r;
        double* out = dX + (size_t)r * K;
        for (int j = 0; j < K; ++j) out[j] = 0.0;
        for (int i = 0; i < N; ++i) {
            double d = bf16_to_double(dY[(size_t)t * N + i]);
            const double* w = What + (size_t)i * K;
            for (int j = 0; j < K; ++j) out[j] += d * w[j];
        }
    }
    free(What);
}

void oracle_bwd_ds_zf(const uint16_t* X, const uint16_t* dY, int T, const uint8_t* codes,
                      const float* zeros_f, int N, int K, int g,
                      const int32_t* row_sel, int n_sel, double* dS) {
    const int G = n_groups(K, g);
    if (!row_sel) n_sel = N;
#pragma omp parallel
    {
        double* dw = (double*)malloc((size_t)K * sizeof(double));
#pragma omp for schedule(static)
        for (int r = 0; r < n_sel; ++r) {
            int i = row_sel ? row_sel[r] : r;
            for (int j = 0; j < K; ++j) dw[j] = 0.0;
            for (int t = 0; t < T; ++t) {
                double d = bf16_to_double(dY[(size_t)t * N + i]);
                for (int j = 0; j < K; ++j) dw[j] += d * bf16_to_double(X[(size_t)t * K + j]);
            }
            for (int gi = 0; gi < G; ++gi) {
                double acc = 0.0;
                double z = (double)zeros_f[(size_t)i * G + gi];
                for (int j = gi * g; j < (gi + 1) * g; ++j)
                    acc += ((double)codes[(size_t)i * K + j] - z) * dw[j];
                dS[(size_t)r * G + gi] = acc;
            }
        }
        free(dw);
    }
}

/* -------------------------------------------------------------- AdamW -----
 * One step of AdamW (decoupled weight decay, bias-corrected moments, step
 * counted from 1) on the scales -- App. A names the optimizer, none of its
 * constants:
 *   s <- s * (1 - lr*wd)
 *   m <- b1*m + (1-b1)*grad ;  v <- b2*v + (1-b2)*grad^2
 *   s <- s - lr * (m / (1-b1^t)) / (sqrt(v / (1-b2^t)) + eps)
 * Inputs are the fp32 state; all arithmetic and outputs are double.
 */
void oracle_adamw(const float* s, const float* grad, const float* m, const float* v,
                  int64_t n, double lr, double b1, double b2, double eps, double wd,
                  int64_t step, double* s_out, double* m_out, double* v_out) {
    const double c1 = 1.0 - pow(b1, (double)step);
    const double c2 = 1.0 - pow(b2, (double)step);
    for (int64_t e = 0; e < n; ++e) {
        double gr = (double)grad[e];
        double sn = (double)s[e] * (1.0 - lr * wd);
        double mn = b1 * (double)m[e] + (1.0 - b1) * gr;
        double vn = b2 * (double)v[e] + (1.0 - b2) * gr * gr;
        double mhat = mn / c1;
        double vhat = vn / c2;
        s_out[e] = sn - lr * mhat / (sqrt(vhat) + eps);
        m_out[e] = mn;
        v_out[e] = vn;
    }
}

int oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    n = omp_get_max_threads();
#endif
    return n;
}
