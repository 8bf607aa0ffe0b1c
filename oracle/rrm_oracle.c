/*
 * CPU oracle for the Recurrent Residual Module hot path.  TEST INFRASTRUCTURE ONLY:
 * it defines what the CUDA library must compute and is never called by the product.
 * It shares no code with the CUDA path.
 *
 * Layouts: activations [N][C][H][W], filters [C_out][C_in][kh][kw], all row-major.
 * Element types: double (used for fp32 layers: fp32 data promoted exactly to fp64)
 * and int64_t (used for int8 and binary layers: exact integer arithmetic; binary
 * values are the integers +1 / -1, padding is 0).
 *
 * "Convolution" is cross-correlation with zero padding:
 *   P[n,co,oy,ox] = b[co] + sum_{ci,ky,kx} F[co,ci,ky,kx] * I[n,ci,oy*s+ky-p,ox*s+kx-p].
 */
#include <stdint.h>
#include <stdlib.h>
#include <math.h>

#define OUT_DIM(in, k, s, p) (((in) + 2 * (p) - (k)) / (s) + 1)

/* ---- Eq. 3 (projection layer), convolution case: P = F * I + b, plain definition ---- */
#define DEFINE_CONV(NAME, T)                                                              \
void NAME(const T* I, const T* F, const T* b, T* P, int N, int C, int H, int W, int K,    \
          int kh, int kw, int s, int p)                                                   \
{                                                                                         \
    const int OH = OUT_DIM(H, kh, s, p), OW = OUT_DIM(W, kw, s, p);                       \
    _Pragma("omp parallel for collapse(2) schedule(static)")                              \
    for (int n = 0; n < N; ++n)                                                           \
        for (int co = 0; co < K; ++co)                                                    \
            for (int oy = 0; oy < OH; ++oy)                                               \
                for (int ox = 0; ox < OW; ++ox) {                                         \
                    T acc = b ? b[co] : (T)0;                                             \
                    for (int ci = 0; ci < C; ++ci)                                        \
                        for (int ky = 0; ky < kh; ++ky) {                                 \
                            const int iy = oy * s + ky - p;                               \
                            if (iy < 0 || iy >= H) continue;                              \
                            for (int kx = 0; kx < kw; ++kx) {                             \
                                const int ix = ox * s + kx - p;                           \
                                if (ix < 0 || ix >= W) continue;                          \
                                acc += F[(((size_t)co * C + ci) * kh + ky) * kw + kx] *   \
                                       I[(((size_t)n * C + ci) * H + iy) * W + ix];       \
                            }                                                             \
                        }                                                                 \
                    P[(((size_t)n * K + co) * OH + oy) * OW + ox] = acc;                  \
                }                                                                         \
}
DEFINE_CONV(rrm_oracle_conv_f64, double)
DEFINE_CONV(rrm_oracle_conv_i64, int64_t)

/* ---- Eq. 3, fully-connected case: P = W I + b, W is [C_out][C_in] ---- */
#define DEFINE_FC(NAME, T)                                                                \
void NAME(const T* I, const T* Wm, const T* b, T* P, int N, int C, int K)                 \
{                                                                                         \
    _Pragma("omp parallel for collapse(2) schedule(static)")                              \
    for (int n = 0; n < N; ++n)                                                           \
        for (int o = 0; o < K; ++o) {                                                     \
            T acc = b ? b[o] : (T)0;                                                      \
            for (int j = 0; j < C; ++j) acc += Wm[(size_t)o * C + j] * I[(size_t)n * C + j]; \
            P[(size_t)n * K + o] = acc;                                                   \
        }                                                                                 \
}
DEFINE_FC(rrm_oracle_fc_f64, double)
DEFINE_FC(rrm_oracle_fc_i64, int64_t)

/*
 * ---- Algorithm 1, the update P_t = P_{t-1} + F * dI, evaluated the way Sec. 3.5
 * describes a dynamic-sparse product: scan dI for its non-zero entries, and for each
 * one multiply the weights that touch it and add into the output accumulators.
 * No bias (it cancels in Eq. 4).  Returns the multiply-accumulates executed, which is
 * the exact count behind the rho-scaled complexity of Table 1.
 */
#define DEFINE_CONV_DELTA(NAME, T)                                                        \
int64_t NAME(const T* D, const T* F, T* P, int N, int C, int H, int W, int K,             \
             int kh, int kw, int s, int p)                                                \
{                                                                                         \
    const int OH = OUT_DIM(H, kh, s, p), OW = OUT_DIM(W, kw, s, p);                       \
    const size_t total = (size_t)N * C * H * W;                                           \
    size_t nnz = 0;                                                                       \
    for (size_t i = 0; i < total; ++i) nnz += (D[i] != (T)0);                             \
    size_t* idx = (size_t*)malloc((nnz ? nnz : 1) * sizeof(size_t));                      \
    size_t m = 0;                                                                         \
    for (size_t i = 0; i < total; ++i) if (D[i] != (T)0) idx[m++] = i;                    \
    int64_t taps = 0;                                                                     \
    _Pragma("omp parallel for schedule(static) reduction(+:taps)")                        \
    for (int co = 0; co < K; ++co) {                                                      \
        for (size_t e = 0; e < nnz; ++e) {                                                \
            const size_t i = idx[e];                                                      \
            const int x = (int)(i % W), y = (int)((i / W) % H);                           \
            const int ci = (int)((i / ((size_t)W * H)) % C), n = (int)(i / ((size_t)W * H * C)); \
            const T d = D[i];                                                             \
            for (int ky = 0; ky < kh; ++ky) {                                             \
                const int ty = y + p - ky;                                                \
                if (ty < 0 || ty % s) continue;                                           \
                const int oy = ty / s;                                                    \
                if (oy >= OH) continue;                                                   \
                for (int kx = 0; kx < kw; ++kx) {                                         \
                    const int tx = x + p - kx;                                            \
                    if (tx < 0 || tx % s) continue;                                       \
                    const int ox = tx / s;                                                \
                    if (ox >= OW) continue;                                               \
                    P[(((size_t)n * K + co) * OH + oy) * OW + ox] +=                      \
                        F[(((size_t)co * C + ci) * kh + ky) * kw + kx] * d;               \
                    ++taps;                                                               \
                }                                                                         \
            }                                                                             \
        }                                                                                 \
    }                                                                                     \
    free(idx);                                                                            \
    return taps;                                                                          \
}
DEFINE_CONV_DELTA(rrm_oracle_conv_delta_f64, double)
DEFINE_CONV_DELTA(rrm_oracle_conv_delta_i64, int64_t)

/* FC case of the same update: for each non-zero dI_j add column j of W scaled by dI_j. */
#define DEFINE_FC_DELTA(NAME, T)                                                          \
int64_t NAME(const T* D, const T* Wm, T* P, int N, int C, int K)                          \
{                                                                                         \
    int64_t macs = 0;                                                                     \
    for (int n = 0; n < N; ++n)                                                           \
        for (int j = 0; j < C; ++j) {                                                     \
            const T d = D[(size_t)n * C + j];                                             \
            if (d == (T)0) continue;                                                      \
            _Pragma("omp parallel for schedule(static)")                                  \
            for (int o = 0; o < K; ++o) P[(size_t)n * K + o] += Wm[(size_t)o * C + j] * d; \
            macs += K;                                                                    \
        }                                                                                 \
    return macs;                                                                          \
}
DEFINE_FC_DELTA(rrm_oracle_fc_delta_f64, double)
DEFINE_FC_DELTA(rrm_oracle_fc_delta_i64, int64_t)

/* ---- max pooling, window k, stride s, padding p; padded cells never win ---- */
#define DEFINE_POOL(NAME, T, LOWEST)                                                      \
void NAME(const T* X, T* Y, int N, int C, int H, int W, int k, int s, int p)              \
{                                                                                         \
    const int OH = OUT_DIM(H, k, s, p), OW = OUT_DIM(W, k, s, p);                         \
    _Pragma("omp parallel for schedule(static)")                                          \
    for (int nc = 0; nc < N * C; ++nc)                                                    \
        for (int oy = 0; oy < OH; ++oy)                                                   \
            for (int ox = 0; ox < OW; ++ox) {                                             \
                T best = LOWEST;                                                          \
                for (int ky = 0; ky < k; ++ky) {                                          \
                    const int iy = oy * s + ky - p;                                       \
                    if (iy < 0 || iy >= H) continue;                                      \
                    for (int kx = 0; kx < k; ++kx) {                                      \
                        const int ix = ox * s + kx - p;                                   \
                        if (ix < 0 || ix >= W) continue;                                  \
                        const T v = X[((size_t)nc * H + iy) * W + ix];                    \
                        if (v > best) best = v;                                           \
                    }                                                                     \
                }                                                                         \
                Y[((size_t)nc * OH + oy) * OW + ox] = best;                               \
            }                                                                             \
}
DEFINE_POOL(rrm_oracle_maxpool_f64, double, -INFINITY)
DEFINE_POOL(rrm_oracle_maxpool_i64, int64_t, INT64_MIN)
