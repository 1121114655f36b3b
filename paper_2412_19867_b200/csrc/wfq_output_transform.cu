// Output transform y = V_A S_A Y S_A V_A^T (Section 4.1): one thread per
// (output channel, tile).  Lanes run along the tile index, so the P plane reads of
// Y[P][K][Tp] are 128-byte coalesced and the m-float row segments written by
// neighbouring lanes are contiguous in y[N][K][H][W].  Memory-bound: P*4 bytes read
// and m*m*4 bytes written per thread against ~150 flops.
#include "wfq_internal.h"
#include "wfq_ptx.cuh"

namespace wfq {
namespace {

// 1-D output transform with V_A = V_{n x m}^T for the points 0, 1, -1, 2, -2, inf:
//   o_u = sum_i f_i^u y_i (i < 5) + [u == 3] y_5
__device__ __forceinline__ void at_f43(const float (&v)[6], float (&o)[4])
{
    const float s1 = v[1] + v[2], d1 = v[1] - v[2];
    const float s2 = v[3] + v[4], d2 = v[3] - v[4];
    o[0] = v[0] + s1 + s2;
    o[1] = fmaf(2.f, d2, d1);
    o[2] = fmaf(4.f, s2, s1);
    o[3] = fmaf(8.f, d2, d1) + v[5];
}

// Points 0, 1, -1, 2, -2, 1/2, -1/2, inf.
__device__ __forceinline__ void at_f63(const float (&v)[8], float (&o)[6])
{
    const float s1 = v[1] + v[2], d1 = v[1] - v[2];
    const float s2 = v[3] + v[4], d2 = v[3] - v[4];
    const float s3 = v[5] + v[6], d3 = v[5] - v[6];
    o[0] = v[0] + s1 + s2 + s3;
    o[1] = fmaf(2.f, d2, d1) + 0.5f * d3;
    o[2] = fmaf(4.f, s2, s1) + 0.25f * s3;
    o[3] = fmaf(8.f, d2, d1) + 0.125f * d3;
    o[4] = fmaf(16.f, s2, s1) + 0.0625f * s3;
    o[5] = fmaf(32.f, d2, d1) + 0.03125f * d3 + v[7];
}

template <int M>
__device__ __forceinline__ void at_1d(const float (&v)[M + 2], float (&o)[M])
{
    if constexpr (M == 4) at_f43(v, o); else at_f63(v, o);
}

// STORE: 0 = element-wise with bounds checks (any W), 1 = 8-byte stores (W even),
// 2 = 16-byte stores (F(4,3), W a multiple of 4).  With W a multiple of the store width
// a tile row is either completely inside the image or completely outside.
template <int M, int STORE>
__global__ void __launch_bounds__(128)
output_transform_kernel(const float *__restrict__ Y, float *__restrict__ y, Geometry g,
                        ScaleTables tab)
{
    constexpr int NN = M + 2;
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int k = blockIdx.y;
    ptx::grid_dependency_wait();   // Y comes from the kernel launched before this one
    if (t >= g.T) return;

    const size_t plane = (size_t)g.K * g.Tp;
    const float *src = Y + (size_t)k * g.Tp + t;
    float v[NN][NN];
#pragma unroll
    for (int i = 0; i < NN; ++i)
#pragma unroll
        for (int j = 0; j < NN; ++j) {
            v[i][j] = __ldg(src);
            src += plane;
        }
#pragma unroll
    for (int i = 0; i < NN; ++i)
#pragma unroll
        for (int j = 0; j < NN; ++j) v[i][j] *= tab.out_scale[i * NN + j];

    // columns: tmp[u][j] = sum_i VA[u][i] v[i][j]
    float tmp[M][NN];
#pragma unroll
    for (int j = 0; j < NN; ++j) {
        float col[NN], o[M];
#pragma unroll
        for (int i = 0; i < NN; ++i) col[i] = v[i][j];
        at_1d<M>(col, o);
#pragma unroll
        for (int u = 0; u < M; ++u) tmp[u][j] = o[u];
    }

    const int tw = t % g.TW;
    const int tq = t / g.TW;
    const int th = tq % g.TH;
    const int img = tq / g.TH;
    const int h0 = th * M, w0 = tw * M;
    float *row = y + (((size_t)img * g.K + k) * g.H + h0) * g.W + w0;
    const bool full_w = (w0 + M <= g.W);
#pragma unroll
    for (int u = 0; u < M; ++u) {
        float o[M];
        at_1d<M>(tmp[u], o);
        if (h0 + u < g.H) {
            if (STORE == 2 && full_w) {
                *reinterpret_cast<float4 *>(row) = make_float4(o[0], o[1], o[2], o[3]);
            } else if (STORE >= 1 && full_w) {
#pragma unroll
                for (int v2 = 0; v2 < M; v2 += 2)
                    *reinterpret_cast<float2 *>(row + v2) = make_float2(o[v2], o[v2 + 1]);
            } else {
#pragma unroll
                for (int v2 = 0; v2 < M; ++v2)
                    if (w0 + v2 < g.W) row[v2] = o[v2];
            }
        }
        row += g.W;
    }
}

}  // namespace

cudaError_t launch_output_transform(const wfq_plan &plan, float *y_dev, cudaStream_t stream, bool pdl)
{
    const Geometry &g = plan.geo;
    const int threads = 128;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((g.T + threads - 1) / threads, g.K);
    cfg.blockDim = dim3(threads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    const float *Y = plan.ws.Y;
    // y_dev is 16-byte aligned; rows of an even W keep 8-byte alignment for every tile
    if (g.m == 4) {
        if (g.W % 4 == 0)
            return cudaLaunchKernelEx(&cfg, output_transform_kernel<4, 2>, Y, y_dev, g, plan.tables);
        if (g.W % 2 == 0)
            return cudaLaunchKernelEx(&cfg, output_transform_kernel<4, 1>, Y, y_dev, g, plan.tables);
        return cudaLaunchKernelEx(&cfg, output_transform_kernel<4, 0>, Y, y_dev, g, plan.tables);
    }
    if (g.W % 2 == 0)
        return cudaLaunchKernelEx(&cfg, output_transform_kernel<6, 1>, Y, y_dev, g, plan.tables);
    return cudaLaunchKernelEx(&cfg, output_transform_kernel<6, 0>, Y, y_dev, g, plan.tables);
}

}  // namespace wfq
