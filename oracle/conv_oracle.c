/*
 * fp64 CPU oracle for the stride-1, pad-1, 3x3 2-D convolution and for its
 * Winograd evaluation.  TEST INFRASTRUCTURE ONLY: it exists so that the CUDA
 * library can be checked against something written independently of it.  It
 * shares no code, header, table or constant with the CUDA sources.
 *
 * What each function follows:
 *  - oracle_direct*: the definition of the operator the paper replaces
 *    (ggml_conv_2d with a 3x3 filter; Abstract and Section "Techniques";
 *    tensor layouts from the header of Table 1: Filter = [KW,KH,IC,OC],
 *    Activation = [IW,IH,IC,N], fastest dimension first, i.e. contiguous
 *    w[OC][IC][KH][KW] and x[N][IC][IH][IW]).  Cross-correlation (no filter
 *    flip), zero padding of one pixel, stride 1.
 *  - oracle_winograd: the three steps of Section "Techniques": (i) preprocess
 *    the filter and the activation, (ii) element-wise multiplication of the
 *    preprocessed tensors (summed over input channels), (iii) postprocess the
 *    intermediate result.  The transform matrices are arguments: the paper
 *    prints none, so the caller (oracle/__init__.py) supplies the Toom-Cook
 *    matrices of the Lavin & Gray construction the paper cites.
 *
 * No blocking, fusion or reordering beyond the definitions: every loop nest is
 * the formula written out.  OpenMP only splits independent output planes.
 */
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define IDX4(a, b, c, d, B, C, D) ((((size_t)(a) * (B) + (b)) * (C) + (c)) * (D) + (d))

/* Zero-extended read of x[n][c][i][j]. */
static double x_at(const double *x, int C, int H, int W, int n, int c, int i, int j)
{
    if (i < 0 || i >= H || j < 0 || j >= W) return 0.0;
    return x[IDX4(n, c, i, j, C, H, W)];
}

/* y[n][k][i][j] = b[k] + sum_c sum_u sum_v xhat[n][c][i+u-1][j+v-1] * w[k][c][u][v]
 * for the output channels listed in ks[0..nk) (ks == NULL: all K channels, nk
 * ignored).  y has shape [N][nk][H][W] (or [N][K][H][W] when ks == NULL). */
int oracle_direct_channels(const double *x, const double *w, const double *bias, double *y,
                           int N, int C, int H, int W, int K, const int *ks, int nk)
{
    if (!x || !w || !y || N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0) return 1;
    int KO = ks ? nk : K;
    long long planes = (long long)N * KO;
#pragma omp parallel for schedule(dynamic, 1)
    for (long long pl = 0; pl < planes; ++pl) {
        int n = (int)(pl / KO), ko = (int)(pl % KO);
        int k = ks ? ks[ko] : ko;
        double *yp = y + ((size_t)n * KO + ko) * H * W;
        double b = bias ? bias[k] : 0.0;
        for (int i = 0; i < H; ++i)
            for (int j = 0; j < W; ++j) {
                double acc = 0.0;
                for (int c = 0; c < C; ++c)
                    for (int u = 0; u < 3; ++u)
                        for (int v = 0; v < 3; ++v)
                            acc += x_at(x, C, H, W, n, c, i + u - 1, j + v - 1) *
                                   w[IDX4(k, c, u, v, C, 3, 3)];
                yp[(size_t)i * W + j] = b + acc;
            }
    }
    return 0;
}

/* The same sum sampled with stride s (the downsampling convolutions of the UNet, stride 2, pad 1):
 * y[n][k][i][j] = b[k] + sum_c sum_u sum_v xhat[n][c][s*i+u-1][s*j+v-1] * w[k][c][u][v],
 * i < Ho = (H - 1) / s + 1, j < Wo = (W - 1) / s + 1.  y has shape [N][K][Ho][Wo]. */
int oracle_direct_strided(const double *x, const double *w, const double *bias, double *y,
                          int N, int C, int H, int W, int K, int s)
{
    if (!x || !w || !y || N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0 || s <= 0) return 1;
    int Ho = (H - 1) / s + 1, Wo = (W - 1) / s + 1;
    long long planes = (long long)N * K;
#pragma omp parallel for schedule(dynamic, 1)
    for (long long pl = 0; pl < planes; ++pl) {
        int n = (int)(pl / K), k = (int)(pl % K);
        double *yp = y + (size_t)pl * Ho * Wo;
        double b = bias ? bias[k] : 0.0;
        for (int i = 0; i < Ho; ++i)
            for (int j = 0; j < Wo; ++j) {
                double acc = 0.0;
                for (int c = 0; c < C; ++c)
                    for (int u = 0; u < 3; ++u)
                        for (int v = 0; v < 3; ++v)
                            acc += x_at(x, C, H, W, n, c, s * i + u - 1, s * j + v - 1) *
                                   w[IDX4(k, c, u, v, C, 3, 3)];
                yp[(size_t)i * Wo + j] = b + acc;
            }
    }
    return 0;
}

int oracle_direct(const double *x, const double *w, const double *bias, double *y,
                  int N, int C, int H, int W, int K)
{
    return oracle_direct_channels(x, w, bias, y, N, C, H, W, K, NULL, 0);
}

/* Number of threads the parallel loops use (reported beside timings). */
int oracle_threads(void)
{
    int t = 1;
#ifdef _OPENMP
#pragma omp parallel
    {
#pragma omp single
        t = omp_get_num_threads();
    }
#endif
    return t;
}

/* Step (i), filter half: U[k][c] = G * w[k][c] * G^T.  G is a x 3 row-major,
 * U is [K][C][a][a]. */
int oracle_filter_transform(const double *w, const double *G, double *U, int K, int C, int a)
{
    if (!w || !G || !U || K <= 0 || C <= 0 || a <= 0) return 1;
    for (long long kc = 0; kc < (long long)K * C; ++kc) {
        const double *g = w + (size_t)kc * 9;
        double *u = U + (size_t)kc * a * a;
        for (int p = 0; p < a; ++p)
            for (int q = 0; q < a; ++q) {
                double s = 0.0;
                for (int r = 0; r < 3; ++r)
                    for (int t = 0; t < 3; ++t)
                        s += G[p * 3 + r] * g[r * 3 + t] * G[q * 3 + t];
                u[p * a + q] = s;
            }
    }
    return 0;
}

/* Step (i), activation half, for one tile: V[c] = B^T * d[c] * B where d[c] is
 * the a x a window of the zero-extended image whose top-left pixel is
 * (m*th - 1, m*tw - 1).  Bt is a x a row-major.  V is [C][a][a]. */
int oracle_input_tile_transform(const double *x, const double *Bt, double *V,
                                int C, int H, int W, int n, int th, int tw, int m, int a)
{
    if (!x || !Bt || !V) return 1;
    double *d = (double *)malloc(sizeof(double) * a * a);
    if (!d) return 2;
    for (int c = 0; c < C; ++c) {
        for (int r = 0; r < a; ++r)
            for (int s = 0; s < a; ++s)
                d[r * a + s] = x_at(x, C, H, W, n, c, m * th - 1 + r, m * tw - 1 + s);
        for (int p = 0; p < a; ++p)
            for (int q = 0; q < a; ++q) {
                double acc = 0.0;
                for (int r = 0; r < a; ++r)
                    for (int s = 0; s < a; ++s)
                        acc += Bt[p * a + r] * d[r * a + s] * Bt[q * a + s];
                V[((size_t)c * a + p) * a + q] = acc;
            }
    }
    free(d);
    return 0;
}

/* The whole Winograd evaluation F(m x m, 3 x 3), a = m + 2:
 *   (i)   U[k][c] = G w[k][c] G^T ;  V[c] = B^T d[c] B per tile
 *   (ii)  M[k]    = sum_c U[k][c] (.) V[c]          (element-wise product)
 *   (iii) Y[k]    = A^T M[k] A  (m x m) ; y = Y + b[k] where inside the image.
 * Tiles: TH = ceil(H/m), TW = ceil(W/m); outputs past the image edge are
 * computed and dropped.  At is m x a row-major. */
static int winograd_steps_ii_iii(const double *x, const double *U, const double *bias, double *y,
                                 int N, int C, int H, int W, int K, int m,
                                 const double *Bt, const double *At);

int oracle_winograd(const double *x, const double *w, const double *bias, double *y,
                    int N, int C, int H, int W, int K, int m,
                    const double *G, const double *Bt, const double *At)
{
    if (!x || !w || !y || !G || !Bt || !At) return 1;
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0 || m <= 0) return 1;
    int a = m + 2, aa = a * a;
    double *U = (double *)malloc(sizeof(double) * (size_t)K * C * aa);
    if (!U) return 2;
    oracle_filter_transform(w, G, U, K, C, a);
    int rc = winograd_steps_ii_iii(x, U, bias, y, N, C, H, W, K, m, Bt, At);
    free(U);
    return rc;
}

/* The same evaluation for a transformed filter U[K][C][a][a] handed in by the caller (a filter that was
 * rounded or quantised after step (i)): the activation half of (i), then (ii) and (iii). */
int oracle_winograd_with_filter(const double *x, const double *U, const double *bias, double *y,
                                int N, int C, int H, int W, int K, int m,
                                const double *Bt, const double *At)
{
    if (!x || !U || !y || !Bt || !At) return 1;
    if (N <= 0 || C <= 0 || H <= 0 || W <= 0 || K <= 0 || m <= 0) return 1;
    return winograd_steps_ii_iii(x, U, bias, y, N, C, H, W, K, m, Bt, At);
}

static int winograd_steps_ii_iii(const double *x, const double *U, const double *bias, double *y,
                                 int N, int C, int H, int W, int K, int m,
                                 const double *Bt, const double *At)
{
    int a = m + 2, aa = a * a;
    int TH = (H + m - 1) / m, TW = (W + m - 1) / m;
    int err = 0;
    long long tiles = (long long)N * TH * TW;
#pragma omp parallel for schedule(dynamic, 1)
    for (long long t = 0; t < tiles; ++t) {
        int n = (int)(t / ((long long)TH * TW));
        int th = (int)((t / TW) % TH), tw = (int)(t % TW);
        double *V = (double *)malloc(sizeof(double) * (size_t)C * aa);
        double *Mk = (double *)malloc(sizeof(double) * aa);
        if (!V || !Mk) {
#pragma omp atomic write
            err = 2;
            free(V); free(Mk); continue;
        }
        oracle_input_tile_transform(x, Bt, V, C, H, W, n, th, tw, m, a);
        for (int k = 0; k < K; ++k) {
            for (int e = 0; e < aa; ++e) {
                double s = 0.0;
                for (int c = 0; c < C; ++c)
                    s += U[((size_t)k * C + c) * aa + e] * V[(size_t)c * aa + e];
                Mk[e] = s;
            }
            double b = bias ? bias[k] : 0.0;
            for (int i = 0; i < m; ++i)
                for (int j = 0; j < m; ++j) {
                    int oi = m * th + i, oj = m * tw + j;
                    if (oi >= H || oj >= W) continue;
                    double s = 0.0;
                    for (int p = 0; p < a; ++p)
                        for (int q = 0; q < a; ++q)
                            s += At[i * a + p] * Mk[p * a + q] * At[j * a + q];
                    y[IDX4(n, k, oi, oj, K, H, W)] = s + b;
                }
        }
        free(V);
        free(Mk);
    }
    return err;
}
