// The paper's fully quantized transforms (Section 4.1), as an optional mode of the plan:
//   input   X~ = s_qB^2 s_qx  Q(S_B V_B / s_qB)  Q(x / s_qx)  Q(V_B^T S_B / s_qB)      (Eq. quant-B)
//   output  y~ = s_qA^2 s_qY  Q(V_A S_A / s_qA)  Q(Y~ / s_qY) Q(S_A V_A^T / s_qA)      (Eq. quant-y)
// with Q the symmetric 8-bit abs-max quantizer of Section 2 (codes in [-127, 127], round half to
// even, scale = abs-max / 127).  The matrix products run on integer codes in int32 (exact); the
// quantizers decide in fp64 (scale = amax / 127, code = rint(v / scale)), which makes every code a
// function of the input values alone, not of an instruction order.  The contraction between the
// two transforms (Eq. quant-Y) is the same kernel as in the floating-point-transform mode: the
// input kernel hands it int8 codes and group scales of fp32(X~), the output kernel reads its fp32 Y.
//
// Readings where the paper is silent: s_qB and s_qA are one scale per matrix (they appear squared);
// s_qx is one scale per (tile, group of `group size` input channels), shared by the n x n patches of
// those channels; s_qY is one scale per (tile, output channel) ("tile") or one per row of the n x n
// matrix for the product with the right-hand matrix, whose result is quantized again per column for
// the left-hand product ("row": Section 3.2 asks for per-tile or per-row/column scales of Y).
//
// These kernels are written for clarity, not speed: one thread per (tile, channel), integer
// matrix products as plain multiply-adds with the codes of the matrices as kernel parameters.
#include <cmath>

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "wfq_internal.h"
#include "wfq_ptx.cuh"

namespace wfq {

namespace {

constexpr double kQmax = 127.0;

// Q(v / s) for s = amax / 127 > 0: fp64 division, round half to even, clipped.
__device__ __noinline__ int code_by_division(double v, double s)
{
    const double q = rint(__ddiv_rn(v, s));
    return (int)fmin(fmax(q, -kQmax), kQmax);
}
// The same code without the division in all but rare cases: a candidate from the reciprocal
// (rinv = 1 / s, one division per scale instead of one per element), its remainder v - q s by one
// fused multiply-add, a step to the neighbour if the remainder says so, and the division itself
// where the remainder is within 1e-9 s of half a step (there the rounding of the quotient
// decides, and the definition is the division).
__device__ __forceinline__ int code_of(double v, double s, double rinv)
{
    double q = rint(__dmul_rn(v, rinv));
    const double r = __fma_rn(-q, s, v);
    const double h = 0.5 * s, ar = fabs(r);
    if (fabs(ar - h) <= 1e-9 * s) return code_by_division(v, s);
    if (ar > h) q += r > 0.0 ? 1.0 : -1.0;
    return (int)fmin(fmax(q, -kQmax), kQmax);
}

// The group quantizer of the contraction's operand (the same rule as the floating-point input
// transform): fp32 scale = amax / 127, codes = rint(fl32(v * fl32(127 / amax))).
__device__ __forceinline__ void group_scale(float amax, float &scale, float &inv)
{
    const bool nz = amax >= 1e-30f;
    scale = nz ? __fdiv_rn(amax, 127.f) : 0.f;
    inv = nz ? __fdiv_rn(127.f, amax) : 0.f;
}
__device__ __forceinline__ int code_bits(float v, float inv)
{
    return (int)__float_as_uint(__fadd_rn(__fmul_rn(v, inv), 12582912.f)) - 0x4B400000;
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__half v) { return __half2float(v); }

// ---- input: one CTA per (tile, channel group), one thread per channel ---------------------------
template <int M, typename Tin>
__global__ void input_transform_int_kernel(const Tin *__restrict__ x, int8_t *__restrict__ Xq,
                                           float *__restrict__ sX, Geometry g, FullQuantTables tab)
{
    constexpr int NN = M + 2, P = NN * NN;
    extern __shared__ float buf[];             // [P][gs + 1] fp32(X~), then one float per warp
    const int gs = blockDim.x, pitch = gs + 1;
    float *red = buf + P * pitch;
    const int t = blockIdx.x, grp = blockIdx.y;
    const int cl = threadIdx.x, c = grp * gs + cl;
    const int tw = t % g.TW, th = (t / g.TW) % g.TH, img = t / (g.TW * g.TH);

    // the channel's n x n patch (zeros outside the image) and the abs-max of the group's patches
    float d[NN][NN];
    float amax = 0.f;
    const Tin *plane = x + ((size_t)img * g.C + c) * g.H * g.W;
#pragma unroll
    for (int a = 0; a < NN; ++a) {
        const int h = th * M - 1 + a;
#pragma unroll
        for (int b = 0; b < NN; ++b) {
            const int w = tw * M - 1 + b;
            const bool in = h >= 0 && h < g.H && w >= 0 && w < g.W;
            d[a][b] = in ? to_float(plane[(size_t)h * g.W + w]) : 0.f;
            amax = fmaxf(amax, fabsf(d[a][b]));
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if ((cl & 31) == 0) red[cl >> 5] = amax;
    __syncthreads();
    amax = 0.f;
    for (int w = 0; w < (gs + 31) / 32; ++w) amax = fmaxf(amax, red[w]);

    // Q(x / s_qx), then the two integer products with the codes of S_B V_B
    const double sqx = __ddiv_rn((double)amax, kQmax);
    const double rqx = amax > 0.f ? __ddiv_rn(1.0, sqx) : 0.0;
    int q[NN][NN];
#pragma unroll
    for (int a = 0; a < NN; ++a)
#pragma unroll
        for (int b = 0; b < NN; ++b) q[a][b] = amax > 0.f ? code_of((double)d[a][b], sqx, rqx) : 0;
    int tmp[NN][NN];
#pragma unroll
    for (int i = 0; i < NN; ++i)
#pragma unroll
        for (int b = 0; b < NN; ++b) {
            int s = 0;
#pragma unroll
            for (int a = 0; a < NN; ++a) s += tab.BTq[i * NN + a] * q[a][b];
            tmp[i][b] = s;
        }
    const double scale = __dmul_rn(tab.sqB2, sqx);
#pragma unroll
    for (int i = 0; i < NN; ++i)
#pragma unroll
        for (int j = 0; j < NN; ++j) {
            int s = 0;
#pragma unroll
            for (int b = 0; b < NN; ++b) s += tmp[i][b] * tab.BTq[j * NN + b];
            buf[(i * NN + j) * pitch + cl] = (float)__dmul_rn((double)s, scale);
        }
    __syncthreads();

    // group quantization of fp32(X~) along the channels: one thread per position
    for (int p = cl; p < P; p += gs) {
        const float *row = buf + p * pitch;
        float m = 0.f;
        for (int k = 0; k < gs; ++k) m = fmaxf(m, fabsf(row[k]));
        float sc, inv;
        group_scale(m, sc, inv);
        uint32_t *dst = reinterpret_cast<uint32_t *>(Xq + ((size_t)p * g.T + t) * g.C + grp * gs);
        for (int k = 0; k < gs; k += 4) {
            uint32_t word = 0;
#pragma unroll
            for (int e = 0; e < 4; ++e) word |= (uint32_t)(code_bits(row[k + e], inv) & 0xff) << (8 * e);
            dst[k / 4] = word;
        }
        sX[((size_t)p * g.G + grp) * g.Ts + t] = sc;
    }
}

// ---- output: one thread per (tile, output channel) ------------------------------------------------
// MODE 1: one scale per tile; MODE 2: one scale per row, then one per column.
template <int M, int MODE>
__global__ void __launch_bounds__(128)
output_transform_int_kernel(const float *__restrict__ Y, float *__restrict__ y, Geometry g,
                            FullQuantTables tab, const float *__restrict__ bias, int act, int out_half)
{
    constexpr int NN = M + 2;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int k = blockIdx.y;
    if (t >= g.T) return;
    const size_t plane = (size_t)g.K * g.Tp;
    const float *src = Y + (size_t)k * g.Tp + t;
    float v[NN][NN];
#pragma unroll
    for (int i = 0; i < NN; ++i)
#pragma unroll
        for (int j = 0; j < NN; ++j) v[i][j] = src[(size_t)(i * NN + j) * plane];

    double out[M][M];
    if constexpr (MODE == 1) {
        float amax = 0.f;
#pragma unroll
        for (int i = 0; i < NN; ++i)
#pragma unroll
            for (int j = 0; j < NN; ++j) amax = fmaxf(amax, fabsf(v[i][j]));
        const double sqY = __ddiv_rn((double)amax, kQmax);
        const double rqY = amax > 0.f ? __ddiv_rn(1.0, sqY) : 0.0;
        int tmp[NN][M];         // Q(Y) Q(S_A V_A^T): [i][v]
#pragma unroll
        for (int i = 0; i < NN; ++i) {
            int q[NN];
#pragma unroll
            for (int j = 0; j < NN; ++j) q[j] = amax > 0.f ? code_of((double)v[i][j], sqY, rqY) : 0;
#pragma unroll
            for (int c = 0; c < M; ++c) {
                int s = 0;
#pragma unroll
                for (int j = 0; j < NN; ++j) s += q[j] * tab.ATq[c * NN + j];
                tmp[i][c] = s;
            }
        }
        const double sA2 = __dmul_rn(tab.sqA, tab.sqA);
#pragma unroll
        for (int u = 0; u < M; ++u)
#pragma unroll
            for (int c = 0; c < M; ++c) {
                int s = 0;
#pragma unroll
                for (int i = 0; i < NN; ++i) s += tab.ATq[u * NN + i] * tmp[i][c];
                out[u][c] = __dmul_rn(__dmul_rn((double)s, sA2), sqY);
            }
    } else {
        double Z[NN][M];        // rows keep their scale: Q(Y_i) Q(S_A V_A^T) s_qA s_row(i)
#pragma unroll
        for (int i = 0; i < NN; ++i) {
            float amax = 0.f;
#pragma unroll
            for (int j = 0; j < NN; ++j) amax = fmaxf(amax, fabsf(v[i][j]));
            const double sr = __ddiv_rn((double)amax, kQmax);
            const double rr = amax > 0.f ? __ddiv_rn(1.0, sr) : 0.0;
            int q[NN];
#pragma unroll
            for (int j = 0; j < NN; ++j) q[j] = amax > 0.f ? code_of((double)v[i][j], sr, rr) : 0;
#pragma unroll
            for (int c = 0; c < M; ++c) {
                int s = 0;
#pragma unroll
                for (int j = 0; j < NN; ++j) s += q[j] * tab.ATq[c * NN + j];
                Z[i][c] = __dmul_rn(__dmul_rn((double)s, tab.sqA), sr);
            }
        }
#pragma unroll
        for (int c = 0; c < M; ++c) {
            double amax = 0.0;
#pragma unroll
            for (int i = 0; i < NN; ++i) amax = fmax(amax, fabs(Z[i][c]));
            const double sc = __ddiv_rn(amax, kQmax);
            const double rc = amax > 0.0 ? __ddiv_rn(1.0, sc) : 0.0;
            int q[NN];
#pragma unroll
            for (int i = 0; i < NN; ++i) q[i] = amax > 0.0 ? code_of(Z[i][c], sc, rc) : 0;
#pragma unroll
            for (int u = 0; u < M; ++u) {
                int s = 0;
#pragma unroll
                for (int i = 0; i < NN; ++i) s += tab.ATq[u * NN + i] * q[i];
                out[u][c] = __dmul_rn(__dmul_rn((double)s, tab.sqA), sc);
            }
        }
    }

    const int tw = t % g.TW, th = (t / g.TW) % g.TH, img = t / (g.TW * g.TH);
    const int h0 = th * M, w0 = tw * M;
    const float bk = bias ? bias[k] : 0.f;
    float *dst = y + (((size_t)img * g.K + k) * g.H + h0) * g.W + w0;
#pragma unroll
    for (int u = 0; u < M; ++u)
#pragma unroll
        for (int c = 0; c < M; ++c)
            if (h0 + u < g.H && w0 + c < g.W) {
                float r = (float)out[u][c] + bk;
                if (act == 1) r = fmaxf(r, 0.f);
                else if (act == 2) r = r * __frcp_rn(1.f + __expf(-r));
                if (out_half == 2) reinterpret_cast<__nv_bfloat16 *>(y)[(dst - y) + (size_t)u * g.W + c] = __float2bfloat16_rn(r);
                else if (out_half) reinterpret_cast<__half *>(y)[(dst - y) + (size_t)u * g.W + c] = __float2half_rn(r);
                else dst[(size_t)u * g.W + c] = r;
            }
}

// Points of F(4,3) and F(6,3) (Section 3.1), the last one at infinity.
const double kPoints2[3] = {0.0, 1.0, -1.0};
const double kPoints4[5] = {0.0, 1.0, -1.0, 2.0, -2.0};
const double kPoints6[7] = {0.0, 1.0, -1.0, 2.0, -2.0, 0.5, -0.5};
// Standard-scaled B^T of the paper's supplementary and its row scales: V_B = diag(1 / s) B^T.
const double kStdBT2[16] = {1, 0, -1, 0,   0, 1, 1, 0,   0, -1, 1, 0,   0, 1, 0, -1};
const double kStdRow2[4] = {1.0, 2.0, 2.0, -1.0};
const double kStdBT4[36] = {4, 0, -5, 0, 1, 0,   0, -4, -4, 1, 1, 0,   0, 4, -4, -1, 1, 0,
                            0, -2, -1, 2, 1, 0,  0, 2, -1, -2, 1, 0,   0, 4, 0, -5, 0, 1};
const double kStdRow4[6] = {4.0, -6.0, -6.0, 24.0, 24.0, 1.0};
const double kStdBT6[64] = {
    1, 0, -5.25, 0, 5.25, 0, -1, 0,        0, 1, 1, -4.25, -4.25, 1, 1, 0,
    0, -1, 1, 4.25, -4.25, -1, 1, 0,       0, 0.5, 0.25, -2.5, -1.25, 2, 1, 0,
    0, -0.5, 0.25, 2.5, -1.25, -2, 1, 0,   0, 2, 4, -2.5, -5, 0.5, 1, 0,
    0, -2, 4, 2.5, -5, -0.5, 1, 0,         0, -1, 0, 5.25, 0, -5.25, 0, 1};
const double kStdRow6[8] = {1.0, -4.5, -4.5, 90.0, 90.0, 45.0 / 32, 45.0 / 32, 1.0};

// Q of a whole matrix: one scale, codes rint(v / scale).
double quantize_matrix(const double *mat, int count, int *codes)
{
    double amax = 0.0;
    for (int i = 0; i < count; ++i) amax = std::fmax(amax, std::fabs(mat[i]));
    const double s = amax / kQmax;
    for (int i = 0; i < count; ++i) {
        double q = s > 0.0 ? std::nearbyint(mat[i] / s) : 0.0;     // round half to even (default mode)
        q = std::fmin(std::fmax(q, -kQmax), kQmax);
        codes[i] = (int)q;
    }
    return s;
}

}  // namespace

// Codes and scales of the two transform matrices for the plan's current scale vectors.
void build_full_quant_tables(wfq_plan &plan)
{
    const Geometry &g = plan.geo;
    const int n = g.n, m = g.m;
    FullQuantTables &tab = plan.fq;
    const double *bt = m == 2 ? kStdBT2 : m == 4 ? kStdBT4 : kStdBT6;
    const double *row = m == 2 ? kStdRow2 : m == 4 ? kStdRow4 : kStdRow6;
    const double *pts = m == 2 ? kPoints2 : m == 4 ? kPoints4 : kPoints6;
    double BT[kMaxN * kMaxN], AT[kMaxN * kMaxN];
    // S_B V_B: V_B = V^{-T}, each entry the correctly rounded quotient of two exact numbers
    for (int i = 0; i < n; ++i)
        for (int a = 0; a < n; ++a) BT[i * n + a] = plan.sB[i] * (bt[i * n + a] / row[i]);
    // V_A S_A: V_A[u][i] = point_i^u, the point at infinity contributes to the last row only
    for (int u = 0; u < m; ++u)
        for (int i = 0; i < n; ++i) {
            double va = i < n - 1 ? 1.0 : (u == m - 1 ? 1.0 : 0.0);
            if (i < n - 1)
                for (int e = 0; e < u; ++e) va *= pts[i];          // exact: small powers of 0, 1, 2, 1/2
            AT[u * n + i] = va * plan.sA[i];
        }
    for (int i = 0; i < kMaxN * kMaxN; ++i) tab.BTq[i] = tab.ATq[i] = 0;
    const double sqB = quantize_matrix(BT, n * n, tab.BTq);
    tab.sqB2 = sqB * sqB;
    tab.sqA = quantize_matrix(AT, m * n, tab.ATq);
}

cudaError_t setup_full_quant()
{
    cudaError_t e = cudaFuncSetAttribute(input_transform_int_kernel<6, __half>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, 80 * 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(input_transform_int_kernel<6, float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 80 * 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(input_transform_int_kernel<4, __half>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 80 * 1024);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(input_transform_int_kernel<4, float>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 80 * 1024);
    return e;
}

cudaError_t launch_input_transform_int(const wfq_plan &plan, const void *x_dev, cudaStream_t stream)
{
    const Geometry &g = plan.geo;
    if (g.gs % 32 != 0 || g.gs > 256) return cudaErrorInvalidValue;
    const dim3 grid((unsigned)g.T, (unsigned)g.G), block((unsigned)g.gs);
    const size_t smem = ((size_t)g.P * (g.gs + 1) + 8) * sizeof(float);
    int8_t *Xq = plan.ws.Xq;
    float *sX = plan.ws.sX;
    if (plan.in_dtype == WFQ_F16) {
        const __half *x = static_cast<const __half *>(x_dev);
        if (g.m == 2) input_transform_int_kernel<2, __half><<<grid, block, smem, stream>>>(x, Xq, sX, g, plan.fq);
        else if (g.m == 4) input_transform_int_kernel<4, __half><<<grid, block, smem, stream>>>(x, Xq, sX, g, plan.fq);
        else input_transform_int_kernel<6, __half><<<grid, block, smem, stream>>>(x, Xq, sX, g, plan.fq);
    } else {
        const float *x = static_cast<const float *>(x_dev);
        if (g.m == 2) input_transform_int_kernel<2, float><<<grid, block, smem, stream>>>(x, Xq, sX, g, plan.fq);
        else if (g.m == 4) input_transform_int_kernel<4, float><<<grid, block, smem, stream>>>(x, Xq, sX, g, plan.fq);
        else input_transform_int_kernel<6, float><<<grid, block, smem, stream>>>(x, Xq, sX, g, plan.fq);
    }
    return cudaGetLastError();
}

cudaError_t launch_output_transform_int(const wfq_plan &plan, float *y_dev, cudaStream_t stream)
{
    const Geometry &g = plan.geo;
    const dim3 grid((unsigned)((g.T + 127) / 128), (unsigned)g.K), block(128);
    const float *Y = plan.ws.Y;
    if (plan.fq_output == 1) {
        if (g.m == 2) output_transform_int_kernel<2, 1><<<grid, block, 0, stream>>>(Y, y_dev, g, plan.fq, plan.bias, plan.act, plan.out_half);
        else if (g.m == 4) output_transform_int_kernel<4, 1><<<grid, block, 0, stream>>>(Y, y_dev, g, plan.fq, plan.bias, plan.act, plan.out_half);
        else output_transform_int_kernel<6, 1><<<grid, block, 0, stream>>>(Y, y_dev, g, plan.fq, plan.bias, plan.act, plan.out_half);
    } else {
        if (g.m == 2) output_transform_int_kernel<2, 2><<<grid, block, 0, stream>>>(Y, y_dev, g, plan.fq, plan.bias, plan.act, plan.out_half);
        else if (g.m == 4) output_transform_int_kernel<4, 2><<<grid, block, 0, stream>>>(Y, y_dev, g, plan.fq, plan.bias, plan.act, plan.out_half);
        else output_transform_int_kernel<6, 2><<<grid, block, 0, stream>>>(Y, y_dev, g, plan.fq, plan.bias, plan.act, plan.out_half);
    }
    return cudaGetLastError();
}

}  // namespace wfq
