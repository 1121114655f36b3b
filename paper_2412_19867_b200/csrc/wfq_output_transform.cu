// Output transform y = V_A S_A Y S_A V_A^T (Section 4.1): one thread per
// (output channel, tile).  Lanes run along the tile index, so the P plane reads of
// Y[P][K][Tp] are 128-byte coalesced; the m-float row segments of neighbouring tiles are
// contiguous in y[N][K][H][W] and are written in whole sectors.  P*4 bytes read
// and m*m*4 bytes written per thread against ~150 flops.
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "wfq_internal.h"
#include "wfq_ptx.cuh"

namespace wfq {
namespace {

// One rounding to the 16-bit output type: kind 1 = fp16, 2 = bf16 (round to nearest even).
__device__ __forceinline__ uint16_t to_bits16(float v, int kind)
{
    return kind == 2 ? __bfloat16_as_ushort(__float2bfloat16_rn(v)) : __half_as_ushort(__float2half_rn(v));
}
__device__ __forceinline__ uint32_t to_bits16x2(float lo, float hi, int kind)
{
    return (uint32_t)to_bits16(lo, kind) | ((uint32_t)to_bits16(hi, kind) << 16);
}

// F(2,3), points 0, 1, -1, inf: V_A = [1,1,1,0; 0,1,-1,1] (the sign of the textbook's last column is
// in the standard S_A).
__device__ __forceinline__ void at_f23(const float (&v)[4], float (&o)[2])
{
    o[0] = v[0] + v[1] + v[2];
    o[1] = v[1] - v[2] + v[3];
}

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
    if constexpr (M == 2) at_f23(v, o);
    else if constexpr (M == 4) at_f43(v, o);
    else at_f63(v, o);
}

// Optional epilogue on the spatial-domain outputs of one row segment: per-output-channel
// bias, then ReLU or SiLU (act: 0 none, 1 ReLU, 2 SiLU).
template <int M>
__device__ __forceinline__ void epilogue(float (&o)[M], float bias, int act)
{
#pragma unroll
    for (int v = 0; v < M; ++v) {
        float t = o[v] + bias;
        if (act == 1) t = fmaxf(t, 0.f);
        else if (act == 2) t = t * __frcp_rn(1.f + __expf(-t));   // exp overflow: t * 0
        o[v] = t;
    }
}

// STORE: 2 = 16-byte stores straight from the
// registers (F(4,3), W a multiple of 4: neighbouring lanes then write neighbouring 16 bytes
// and a warp fills whole sectors), 1 = every other even W, 0 = odd W: the m-float row
// segments of a tile are 24 (or 16) bytes apart, so that direct stores would write every
// 32-byte sector of y in several pieces, and the L2 takes a piece as long as a whole sector
// (measured for F(6,3) with 8-byte stores: 2.3 sector writes per sector of y, and the
// kernel bound by them).  The CTA therefore collects its tiles' outputs in shared memory,
// one array per output row u with the tiles side by side exactly as they lie in the image
// row, and copies them out with consecutive lanes on consecutive 8 bytes (even W) or
// consecutive floats (odd W).
template <int M, int STORE, bool EPI>
__global__ void __launch_bounds__(128, M == 6 ? (EPI ? 6 : 7) : 8)
output_transform_kernel(const float *__restrict__ Y, float *__restrict__ y, Geometry g,
                        ScaleTables tab, const float *__restrict__ bias, int act, int out_half)
{
    // 16-bit output (epilogue variants only; out_half 1 = fp16, 2 = bf16): y points at 2-byte storage
    // of the same shape
    [[maybe_unused]] uint16_t *yh = reinterpret_cast<uint16_t *>(y);
    constexpr int NN = M + 2;
    constexpr int TT = 128;                       // tiles per CTA
    __shared__ __align__(16) float out_s[STORE != 2 ? M * TT * M : 1];   // [u][tile][v]
    __shared__ int tile_base[STORE != 2 ? TT : 1];                       // offset of the tile's y[.][.][h0][w0]
    __shared__ int tile_lim[STORE != 2 ? TT : 1];                        // valid rows * 16 + valid columns
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    const int k = blockIdx.y;
    ptx::grid_dependency_wait();   // Y comes from the kernel launched before this one
    const bool live = t < g.T;
    if (STORE == 2 && !live) return;

    float tmp[M][NN];
    int h0 = 0, w0 = 0;
    size_t base = 0;
    if (live) {
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
        h0 = th * M;
        w0 = tw * M;
        base = (((size_t)img * g.K + k) * g.H + h0) * g.W + w0;
    }

    if constexpr (STORE != 2) {
        const int j = threadIdx.x;
        if (live) {
            const float bk = (EPI && bias) ? __ldg(bias + k) : 0.f;
#pragma unroll
            for (int u = 0; u < M; ++u) {
                float o[M];
                at_1d<M>(tmp[u], o);
                if constexpr (EPI) epilogue<M>(o, bk, act);
                float2 *dst = reinterpret_cast<float2 *>(out_s + (u * TT + j) * M);
#pragma unroll
                for (int v2 = 0; v2 < M; v2 += 2) dst[v2 / 2] = make_float2(o[v2], o[v2 + 1]);
            }
        }
        tile_base[j] = (int)base;
        tile_lim[j] = live ? (min(M, g.H - h0) * 16 + min(M, g.W - w0)) : 0;
        __syncthreads();
        if constexpr (STORE == 0) {
            // float f of row u: tile f / M, column f % M
#pragma unroll
            for (int u = 0; u < M; ++u) {
                const float *row = out_s + u * TT * M;
#pragma unroll
                for (int i = 0; i < M; ++i) {
                    const int f = threadIdx.x + i * TT;
                    const int tj = f / M, v1 = f - tj * M;
                    const int lim = tile_lim[tj];
                    if (u < (lim >> 4) && v1 < (lim & 15)) {
                        const size_t off = (size_t)tile_base[tj] + (size_t)u * g.W + v1;
                        if (EPI && out_half) yh[off] = to_bits16(row[f], out_half);
                        else y[off] = row[f];
                    }
                }
            }
            return;
        }
        // pair q of row u: tile q / (M/2), columns 2 * (q % (M/2)) and the next
        constexpr int PPT = M / 2;                // pairs per tile row
#pragma unroll
        for (int u = 0; u < M; ++u) {
            const float2 *row = reinterpret_cast<const float2 *>(out_s + u * TT * M);
#pragma unroll
            for (int i = 0; i < PPT; ++i) {
                const int q = threadIdx.x + i * TT;
                const int tj = q / PPT, v2 = 2 * (q - tj * PPT);
                const int lim = tile_lim[tj];
                if (u < (lim >> 4) && v2 < (lim & 15)) {    // W even: both columns or none
                    const size_t off = (size_t)tile_base[tj] + (size_t)u * g.W + v2;
                    if (EPI && out_half) *reinterpret_cast<uint32_t *>(yh + off) = to_bits16x2(row[q].x, row[q].y, out_half);
                    else *reinterpret_cast<float2 *>(y + off) = row[q];
                }
            }
        }
    } else {
        float *row = y + base;
        uint16_t *rowh = yh + base;
        const bool full_w = (w0 + M <= g.W);
        const float bk = (EPI && bias) ? __ldg(bias + k) : 0.f;
#pragma unroll
        for (int u = 0; u < M; ++u) {
            float o[M];
            at_1d<M>(tmp[u], o);
            if constexpr (EPI) epilogue<M>(o, bk, act);
            if (h0 + u < g.H) {
                if (EPI && out_half) {
                    if (full_w) {
                        *reinterpret_cast<uint2 *>(rowh) = make_uint2(to_bits16x2(o[0], o[1], out_half),
                                                                      to_bits16x2(o[2], o[3], out_half));
                    } else {
#pragma unroll
                        for (int v2 = 0; v2 < M; ++v2)
                            if (w0 + v2 < g.W) rowh[v2] = to_bits16(o[v2], out_half);
                    }
                } else if (full_w) {
                    *reinterpret_cast<float4 *>(row) = make_float4(o[0], o[1], o[2], o[3]);
                } else {
#pragma unroll
                    for (int v2 = 0; v2 < M; ++v2)
                        if (w0 + v2 < g.W) row[v2] = o[v2];
                }
            }
            row += g.W;
            rowh += g.W;
        }
    }
}

}  // namespace

namespace {

template <int M, int STORE, bool EPI>
cudaError_t carveout()
{
    return cudaFuncSetAttribute(output_transform_kernel<M, STORE, EPI>,
                                cudaFuncAttributePreferredSharedMemoryCarveout, (int)cudaSharedmemCarveoutMaxShared);
}

template <int M, int STORE>
cudaError_t launch_variant(const cudaLaunchConfig_t &cfg, const wfq_plan &plan, float *y_dev)
{
    const float *Y = plan.ws.Y;
    const int out_half = plan.out_half;
    if (plan.bias || plan.act || out_half)
        return cudaLaunchKernelEx(&cfg, output_transform_kernel<M, STORE, true>, Y, y_dev, plan.geo, plan.tables,
                                  plan.bias, plan.act, out_half);
    return cudaLaunchKernelEx(&cfg, output_transform_kernel<M, STORE, false>, Y, y_dev, plan.geo, plan.tables,
                              plan.bias, plan.act, out_half);
}

}  // namespace

// One-time attribute setting (per device): the staged variants want six or more CTAs of
// 10-19 KB of shared memory per SM.
cudaError_t setup_output_transform()
{
    cudaError_t e = carveout<2, 1, false>();
    if (e == cudaSuccess) e = carveout<2, 0, false>();
    if (e == cudaSuccess) e = carveout<2, 1, true>();
    if (e == cudaSuccess) e = carveout<2, 0, true>();
    if (e == cudaSuccess) e = carveout<4, 1, false>();
    if (e == cudaSuccess) e = carveout<6, 1, false>();
    if (e == cudaSuccess) e = carveout<4, 0, false>();
    if (e == cudaSuccess) e = carveout<6, 0, false>();
    if (e == cudaSuccess) e = carveout<4, 1, true>();
    if (e == cudaSuccess) e = carveout<6, 1, true>();
    if (e == cudaSuccess) e = carveout<4, 0, true>();
    if (e == cudaSuccess) e = carveout<6, 0, true>();
    return e;
}

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
    // y_dev is 16-byte aligned; rows of an even W keep 8-byte alignment for every tile
    if (g.m == 2) {
        if (g.W % 2 == 0) return launch_variant<2, 1>(cfg, plan, y_dev);
        return launch_variant<2, 0>(cfg, plan, y_dev);
    }
    if (g.m == 4) {
        if (g.W % 4 == 0) return launch_variant<4, 2>(cfg, plan, y_dev);
        if (g.W % 2 == 0) return launch_variant<4, 1>(cfg, plan, y_dev);
        return launch_variant<4, 0>(cfg, plan, y_dev);
    }
    if (g.W % 2 == 0) return launch_variant<6, 1>(cfg, plan, y_dev);
    return launch_variant<6, 0>(cfg, plan, y_dev);
}

}  // namespace wfq
