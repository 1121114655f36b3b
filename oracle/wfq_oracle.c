/*
 * CPU oracle for the group-wise int8-quantized Winograd convolution F(m,3).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, step-by-step statement of
 * what the method computes.  It shares no code, table or helper with the CUDA path
 * and is never called from it; only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may load it.
 *
 * Conventions (all arrays dense, row-major, last index fastest):
 *   n = m + 2 (input-tile edge), P = n*n Winograd positions, position p = i*n + j,
 *   TH = ceil(H/m), TW = ceil(W/m), tile id t = (img*TH + th)*TW + tw,
 *   groups of `gs` consecutive input channels, G = C/gs.
 * The transform matrices arrive as arguments (the Python side rebuilds them in exact
 * rationals from the paper's interpolation points):
 *   VB[n][n] = V_{n x n}^{-T},  VG[n][3] = V_{n x 3},  VA[m][n] = V_{n x m}^T
 * (Section 4.1's short-hands), with the diagonal scales sB[n], sG[n], sA[n].
 *
 * Floating point: fp64 everywhere except where the quantizer is pinned to fp32
 * (see wfq_oracle_quantize_groups).  Compile with -ffp-contract=off.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int wfq_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * (a) Direct convolution, the plain definition the Winograd identity
 * y = A^T[(G w G^T) .* (B^T x B)]A reproduces (Section 3.1, first equation):
 *   y[n][k][h][w] = sum_c sum_a sum_b x[n][c][h+a-1][w+b-1] * w[k][c][a][b],
 * stride 1, zero padding 1, cross-correlation form, no bias.
 */
void wfq_oracle_direct(const double *x, const double *w, double *y,
                       int N, int C, int K, int H, int W)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < N; ++n)
        for (int k = 0; k < K; ++k) {
            double *yo = y + ((size_t)n * K + k) * H * W;
            for (int i = 0; i < H * W; ++i) yo[i] = 0.0;
            for (int c = 0; c < C; ++c) {
                const double *xi = x + ((size_t)n * C + c) * H * W;
                const double *wf = w + ((size_t)k * C + c) * 9;
                for (int h = 0; h < H; ++h)
                    for (int v = 0; v < W; ++v) {
                        double s = 0.0;
                        for (int a = 0; a < 3; ++a) {
                            int hh = h + a - 1;
                            if (hh < 0 || hh >= H) continue;
                            for (int b = 0; b < 3; ++b) {
                                int ww = v + b - 1;
                                if (ww < 0 || ww >= W) continue;
                                s += xi[(size_t)hh * W + ww] * wf[a * 3 + b];
                            }
                        }
                        yo[(size_t)h * W + v] += s;
                    }
            }
        }
}

/*
 * Filter transform, W = S_G V_G w V_G^T S_G (Section 4.1, first rewritten equation):
 *   U = VG w VG^T (n x n),  Wt[p=(i,j)][k][c] = sG[i]*sG[j]*U[i][j].
 * Output Wt[P][K][C] in fp64 (the caller rounds to fp32 before quantizing).
 */
void wfq_oracle_filter_transform(const double *w, const double *VG, const double *sG,
                                 int K, int C, int n, double *Wt)
{
#pragma omp parallel for schedule(static)
    for (int k = 0; k < K; ++k)
        for (int c = 0; c < C; ++c) {
            const double *f = w + ((size_t)k * C + c) * 9;
            double tmp[8][3]; /* VG w */
            for (int i = 0; i < n; ++i)
                for (int b = 0; b < 3; ++b) {
                    double s = 0.0;
                    for (int a = 0; a < 3; ++a) s += VG[i * 3 + a] * f[a * 3 + b];
                    tmp[i][b] = s;
                }
            for (int i = 0; i < n; ++i)
                for (int j = 0; j < n; ++j) {
                    double s = 0.0;
                    for (int b = 0; b < 3; ++b) s += tmp[i][b] * VG[j * 3 + b];
                    Wt[((size_t)(i * n + j) * K + k) * C + c] = sG[i] * sG[j] * s;
                }
        }
}

/*
 * Input transform, X = S_B V_B x V_B^T S_B (Section 4.1, second rewritten equation).
 * For each listed tile t and channel c the n x n patch d starts at image row th*m-1
 * and column tw*m-1, with zeros outside the image (padding 1; ragged right/bottom
 * edges when m does not divide H or W).
 *   Z = VB d VB^T,  Xt[p=(i,j)][tt][c] = sB[i]*sB[j]*Z[i][j],
 * where tt indexes the list `tiles` (ntiles entries; tiles == NULL means all tiles
 * 0..ntiles-1).  Output Xt[P][ntiles][C] in fp64.
 */
void wfq_oracle_input_transform(const double *x, const double *VB, const double *sB,
                                int N, int C, int H, int W, int m,
                                const int64_t *tiles, int64_t ntiles, double *Xt)
{
    const int n = m + 2;
    const int TH = (H + m - 1) / m, TW = (W + m - 1) / m;
    (void)N;
#pragma omp parallel for schedule(static)
    for (int64_t tt = 0; tt < ntiles; ++tt) {
        const int64_t t = tiles ? tiles[tt] : tt;
        const int tw = (int)(t % TW), th = (int)((t / TW) % TH);
        const int64_t img = t / ((int64_t)TW * TH);
        for (int c = 0; c < C; ++c) {
            const double *xi = x + ((size_t)img * C + c) * H * W;
            double d[8][8], e[8][8];
            for (int a = 0; a < n; ++a)
                for (int b = 0; b < n; ++b) {
                    int hh = th * m - 1 + a, ww = tw * m - 1 + b;
                    d[a][b] = (hh >= 0 && hh < H && ww >= 0 && ww < W)
                                  ? xi[(size_t)hh * W + ww] : 0.0;
                }
            for (int i = 0; i < n; ++i) /* e = VB d */
                for (int b = 0; b < n; ++b) {
                    double s = 0.0;
                    for (int a = 0; a < n; ++a) s += VB[i * n + a] * d[a][b];
                    e[i][b] = s;
                }
            for (int i = 0; i < n; ++i) /* Z = e VB^T */
                for (int j = 0; j < n; ++j) {
                    double s = 0.0;
                    for (int b = 0; b < n; ++b) s += e[i][b] * VB[j * n + b];
                    Xt[((size_t)(i * n + j) * ntiles + tt) * C + c] = sB[i] * sB[j] * s;
                }
        }
    }
}

/*
 * Group-wise symmetric quantizer (Section 2, the uniform-quantization equation, with
 * one scale per group of `gs` consecutive values, Section 3.2; dynamic "min-max" of
 * Section 4.1 read as symmetric abs-max).  Pinned fp32 arithmetic, per group:
 *   amax = max |v|;  if amax < 1e-30: s = 0, codes 0;
 *   else s = fl32(amax / qmax), inv = fl32(qmax / amax),
 *        q = clamp(rint_half_even(fl32(v * inv)), -qmax, +qmax).
 * v[rows][C] -> q[rows][C] (int8), s[rows][C/gs].
 */
void wfq_oracle_quantize_groups(const float *v, int64_t rows, int C, int gs, int qmax,
                                int8_t *q, float *s)
{
    const int G = C / gs;
    const float fq = (float)qmax;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r)
        for (int g = 0; g < G; ++g) {
            const float *vg = v + (size_t)r * C + (size_t)g * gs;
            int8_t *qg = q + (size_t)r * C + (size_t)g * gs;
            float amax = 0.0f;
            for (int e = 0; e < gs; ++e) {
                float a = fabsf(vg[e]);
                if (a > amax) amax = a;
            }
            if (amax < 1e-30f) {
                s[(size_t)r * G + g] = 0.0f;
                for (int e = 0; e < gs; ++e) qg[e] = 0;
                continue;
            }
            volatile float scale = amax / fq;
            volatile float inv = fq / amax;
            s[(size_t)r * G + g] = scale;
            for (int e = 0; e < gs; ++e) {
                volatile float prod = vg[e] * inv;
                float rr = nearbyintf(prod); /* default rounding mode: half to even */
                if (rr > fq) rr = fq;
                if (rr < -fq) rr = -fq;
                qg[e] = (int8_t)rr;
            }
        }
}

/*
 * Integer Hadamard/contraction stage of Eq. `quant-Y`: for every position the
 * element-wise product summed over input channels is a matrix product; the sum is
 * kept separately for every channel group because each group has its own scales.
 *   acc[p][t][k][g] = sum_{c in g} Xq[p][t][c] * Wq[p][k][c]     (exact integers)
 */
void wfq_oracle_contract(const int8_t *Xq, const int8_t *Wq, int P, int64_t T, int K,
                         int C, int gs, int32_t *acc)
{
    const int G = C / gs;
#pragma omp parallel for collapse(2) schedule(static)
    for (int p = 0; p < P; ++p)
        for (int64_t t = 0; t < T; ++t) {
            const int8_t *xr = Xq + ((size_t)p * T + t) * C;
            for (int k = 0; k < K; ++k) {
                const int8_t *wr = Wq + ((size_t)p * K + k) * C;
                for (int g = 0; g < G; ++g) {
                    int64_t s = 0;
                    for (int c = g * gs; c < (g + 1) * gs; ++c)
                        s += (int64_t)xr[c] * (int64_t)wr[c];
                    acc[(((size_t)p * T + t) * K + k) * G + g] = (int32_t)s;
                }
            }
        }
}

/*
 * Dequantization of Eq. `quant-Y`: the factors s_qW s_qX applied per group,
 *   Y[p][t][k] = sum_g acc[p][t][k][g] * sX[p][t][g] * sW[p][k][g]   (fp64).
 */
void wfq_oracle_dequantize(const int32_t *acc, const float *sX, const float *sW, int P,
                           int64_t T, int K, int G, double *Y)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int p = 0; p < P; ++p)
        for (int64_t t = 0; t < T; ++t)
            for (int k = 0; k < K; ++k) {
                double s = 0.0;
                for (int g = 0; g < G; ++g)
                    s += (double)acc[(((size_t)p * T + t) * K + k) * G + g] *
                         (double)sX[((size_t)p * T + t) * G + g] *
                         (double)sW[((size_t)p * K + k) * G + g];
                Y[((size_t)p * T + t) * K + k] = s;
            }
}

/*
 * Unquantized Hadamard stage (Eq. `Hadamard` summed over input channels), used to pin
 * the transforms against the direct convolution:
 *   Y[p][t][k] = sum_c Xt[p][t][c] * Wt[p][k][c]    (fp64).
 */
void wfq_oracle_hadamard_f64(const double *Xt, const double *Wt, int P, int64_t T, int K,
                             int C, double *Y)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int p = 0; p < P; ++p)
        for (int64_t t = 0; t < T; ++t)
            for (int k = 0; k < K; ++k) {
                const double *xr = Xt + ((size_t)p * T + t) * C;
                const double *wr = Wt + ((size_t)p * K + k) * C;
                double s = 0.0;
                for (int c = 0; c < C; ++c) s += xr[c] * wr[c];
                Y[((size_t)p * T + t) * K + k] = s;
            }
}

/*
 * Output transform, y = V_A S_A Y S_A V_A^T (Section 4.1, third rewritten equation):
 * for every listed tile tt and output channel k, with Yt[i][j] = Y[i*n+j][tt][k],
 *   ytile[tt][k][u][v] = sum_i sum_j VA[u][i]*sA[i]*Yt[i][j]*sA[j]*VA[v][j].
 * Output ytile[T][K][m][m] in fp64.
 */
void wfq_oracle_output_transform(const double *Y, const double *VA, const double *sA,
                                 int64_t T, int K, int m, double *ytile)
{
    const int n = m + 2;
#pragma omp parallel for schedule(static)
    for (int64_t tt = 0; tt < T; ++tt)
        for (int k = 0; k < K; ++k) {
            double Ys[8][8], tmp[6][8];
            for (int i = 0; i < n; ++i)
                for (int j = 0; j < n; ++j)
                    Ys[i][j] = sA[i] * Y[((size_t)(i * n + j) * T + tt) * K + k] * sA[j];
            for (int u = 0; u < m; ++u)
                for (int j = 0; j < n; ++j) {
                    double s = 0.0;
                    for (int i = 0; i < n; ++i) s += VA[u * n + i] * Ys[i][j];
                    tmp[u][j] = s;
                }
            for (int u = 0; u < m; ++u)
                for (int v = 0; v < m; ++v) {
                    double s = 0.0;
                    for (int j = 0; j < n; ++j) s += tmp[u][j] * VA[v * n + j];
                    ytile[(((size_t)tt * K + k) * m + u) * m + v] = s;
                }
        }
}

/*
 * Place output tiles into the image, dropping rows/columns beyond H x W (ragged
 * edges).  ytile[ntiles][K][m][m] for the listed tiles -> y[N][K][H][W].
 * Pixels of tiles that are not listed are left untouched.
 */
void wfq_oracle_scatter_tiles(const double *ytile, const int64_t *tiles, int64_t ntiles,
                              int N, int K, int H, int W, int m, double *y)
{
    const int TH = (H + m - 1) / m, TW = (W + m - 1) / m;
    (void)N;
    for (int64_t tt = 0; tt < ntiles; ++tt) {
        const int64_t t = tiles ? tiles[tt] : tt;
        const int tw = (int)(t % TW), th = (int)((t / TW) % TH);
        const int64_t img = t / ((int64_t)TW * TH);
        for (int k = 0; k < K; ++k)
            for (int u = 0; u < m; ++u)
                for (int v = 0; v < m; ++v) {
                    int hh = th * m + u, ww = tw * m + v;
                    if (hh < H && ww < W)
                        y[(((size_t)img * K + k) * H + hh) * W + ww] =
                            ytile[(((size_t)tt * K + k) * m + u) * m + v];
                }
    }
}
