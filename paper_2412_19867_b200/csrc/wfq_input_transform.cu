// Fused input transform + group-wise int8 quantization.
//
//   X = S_B V_B x V_B^T S_B   (Section 4.1), fp32, never stored
//   per (position, tile, channel group): amax -> scale, codes (Section 2 quantizer,
//   one scale per group, dynamic abs-max)
//
// A CTA stages a strip of the NCHW input (n rows x a chunk of tile columns x CB
// channels, zero halo) in shared memory with coalesced row loads.  Work is then
// handed out per (tile, channel group): L lanes cooperate on one group, each lane
// owning CPL consecutive channels (gs = CPL*L*NSB), so the codes of a lane pack into
// one 8/16/32-bit store and the group abs-max is a warp-level reduction
// (group_absmax: redux.sync over the whole warp, or a shuffle butterfly over L lanes).
// The 2-D transform uses the standard-scaled matrix B^T (small integers / dyadic
// rationals, hard-coded as add/fma chains); the caller's scales enter as one
// per-position factor.
#include <cuda_fp16.h>

#include "wfq_internal.h"

namespace wfq {
namespace {

struct K1Params {
    int TWC;      // tiles per column chunk
    int NCH;      // chunks per strip
    int CB;       // channels per CTA
    int Wp;       // smem row pitch (elements)
    int CS;       // smem channel stride (elements)
    int NSB;      // channel sub-blocks per group (gs = CPL*L*NSB)
};

// ---- 1-D input transforms with the standard B^T ------------------------------------

// F(4,3): rows [4,0,-5,0,1,0] [0,-4,-4,1,1,0] [0,4,-4,-1,1,0] [0,-2,-1,2,1,0]
//              [0,2,-1,-2,1,0] [0,4,0,-5,0,1]
__device__ __forceinline__ void bt_1d(const float (&d)[6], float (&r)[6])
{
    r[0] = fmaf(4.f, d[0], fmaf(-5.f, d[2], d[4]));
    const float a = fmaf(-4.f, d[2], d[4]);
    const float b = fmaf(-4.f, d[1], d[3]);
    r[1] = a + b;
    r[2] = a - b;
    const float c = d[4] - d[2];
    const float t = d[3] - d[1];
    r[3] = fmaf(2.f, t, c);
    r[4] = fmaf(-2.f, t, c);
    r[5] = fmaf(4.f, d[1], fmaf(-5.f, d[3], d[5]));
}

// F(6,3): rows [1,0,-21/4,0,21/4,0,-1,0] [0,1,1,-17/4,-17/4,1,1,0]
//   [0,-1,1,17/4,-17/4,-1,1,0] [0,1/2,1/4,-5/2,-5/4,2,1,0] [0,-1/2,1/4,5/2,-5/4,-2,1,0]
//   [0,2,4,-5/2,-5,1/2,1,0] [0,-2,4,5/2,-5,-1/2,1,0] [0,-1,0,21/4,0,-21/4,0,1]
__device__ __forceinline__ void bt_1d(const float (&d)[8], float (&r)[8])
{
    r[0] = fmaf(5.25f, d[4] - d[2], d[0] - d[6]);
    r[7] = fmaf(5.25f, d[3] - d[5], d[7] - d[1]);
    const float a = fmaf(-4.25f, d[4], d[2] + d[6]);
    const float b = fmaf(-4.25f, d[3], d[1] + d[5]);
    r[1] = a + b;
    r[2] = a - b;
    const float c = fmaf(-1.25f, d[4], fmaf(0.25f, d[2], d[6]));
    const float e = fmaf(2.f, d[5], fmaf(-2.5f, d[3], 0.5f * d[1]));
    r[3] = c + e;
    r[4] = c - e;
    const float f = fmaf(-5.f, d[4], fmaf(4.f, d[2], d[6]));
    const float g = fmaf(0.5f, d[5], fmaf(-2.5f, d[3], 2.f * d[1]));
    r[5] = f + g;
    r[6] = f - g;
}

// ---- group abs-max over L lanes (L a power of two, lanes of a group adjacent) -------
template <int L>
__device__ __forceinline__ float group_absmax(float v)   // v >= 0
{
    if constexpr (L == 32) {
        // non-negative floats order like their bit patterns
        return __uint_as_float(__reduce_max_sync(0xffffffffu, __float_as_uint(v)));
    } else {
#pragma unroll
        for (int o = L / 2; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
        return v;
    }
}

// ---- patch load from the staged strip ---------------------------------------------
// `ch` points at the channel's plane in smem; `col0` is the (even) smem column whose
// successor is the tile's first input column.
template <int NN>
__device__ __forceinline__ void load_patch(const __half *ch, int col0, int Wp, float (&d)[NN][NN])
{
#pragma unroll
    for (int a = 0; a < NN; ++a) {
        const __half2 *row = reinterpret_cast<const __half2 *>(ch + a * Wp + col0);
        float v[NN + 2];
#pragma unroll
        for (int w = 0; w < (NN + 2) / 2; ++w) {
            const float2 f = __half22float2(row[w]);
            v[2 * w] = f.x;
            v[2 * w + 1] = f.y;
        }
#pragma unroll
        for (int b = 0; b < NN; ++b) d[a][b] = v[b + 1];
    }
}

template <int NN>
__device__ __forceinline__ void load_patch(const float *ch, int col0, int Wp, float (&d)[NN][NN])
{
#pragma unroll
    for (int a = 0; a < NN; ++a)
#pragma unroll
        for (int b = 0; b < NN; ++b) d[a][b] = ch[a * Wp + col0 + 1 + b];
}

// Z = B^T d B with the standard B^T, then the caller's per-position factor.
template <int NN>
__device__ __forceinline__ void transform_patch(float (&d)[NN][NN], const ScaleTables &tab,
                                                float (&X)[NN * NN])
{
#pragma unroll
    for (int b = 0; b < NN; ++b) {   // columns: d <- B^T d
        float col[NN], r[NN];
#pragma unroll
        for (int a = 0; a < NN; ++a) col[a] = d[a][b];
        bt_1d(col, r);
#pragma unroll
        for (int a = 0; a < NN; ++a) d[a][b] = r[a];
    }
#pragma unroll
    for (int i = 0; i < NN; ++i) {   // rows: Z[i][:] = (B^T d)[i][:] B
        float r[NN];
        bt_1d(d[i], r);
#pragma unroll
        for (int j = 0; j < NN; ++j) X[i * NN + j] = __fmul_rn(r[j], tab.in_scale[i * NN + j]);
    }
}

__device__ __forceinline__ int quantize_code(float v, float inv)
{
    const int q = __float2int_rn(__fmul_rn(v, inv));   // round half to even
    return max(-127, min(127, q));
}

template <int CPL>
__device__ __forceinline__ void store_codes(int8_t *dst, const int (&q)[CPL])
{
    if constexpr (CPL == 4) {
        const uint32_t w = (uint32_t)(q[0] & 0xff) | ((uint32_t)(q[1] & 0xff) << 8) |
                           ((uint32_t)(q[2] & 0xff) << 16) | ((uint32_t)(q[3] & 0xff) << 24);
        *reinterpret_cast<uint32_t *>(dst) = w;
    } else if constexpr (CPL == 2) {
        *reinterpret_cast<uint16_t *>(dst) = (uint16_t)((q[0] & 0xff) | ((q[1] & 0xff) << 8));
    } else {
        dst[0] = (int8_t)q[0];
    }
}

// ---- strip staging -----------------------------------------------------------------
// smem column j of the strip holds image column w_base + j (w_base even); rows are
// image rows h_base .. h_base + NN - 1; anything outside the image is zero.
template <typename Tin>
__device__ __forceinline__ void stage_strip(Tin *sm, const Tin *__restrict__ x, const Geometry &g,
                                            const K1Params &prm, int NN, int img, int c_base,
                                            int h_base, int w_base, int cols)
{
    const size_t HW = (size_t)g.H * g.W;
    const Tin *ximg = x + (size_t)img * g.C * HW;
    if ((g.W & 1) == 0 && sizeof(Tin) == 2) {
        // pairs of halves: 4-byte global loads and shared stores
        const int pairs = cols / 2;
        const int total = prm.CB * NN * pairs;
        for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
            const int jp = idx % pairs;
            const int a = (idx / pairs) % NN;
            const int c = idx / (pairs * NN);
            const int h = h_base + a, w = w_base + 2 * jp;
            uint32_t v = 0u;
            if (h >= 0 && h < g.H && w >= 0 && w < g.W)
                v = __ldg(reinterpret_cast<const uint32_t *>(ximg + (size_t)(c_base + c) * HW +
                                                             (size_t)h * g.W + w));
            *reinterpret_cast<uint32_t *>(sm + (size_t)c * prm.CS + a * prm.Wp + 2 * jp) = v;
        }
    } else {
        const int total = prm.CB * NN * cols;
        for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
            const int j = idx % cols;
            const int a = (idx / cols) % NN;
            const int c = idx / (cols * NN);
            const int h = h_base + a, w = w_base + j;
            Tin v = Tin(0);
            if (h >= 0 && h < g.H && w >= 0 && w < g.W)
                v = __ldg(ximg + (size_t)(c_base + c) * HW + (size_t)h * g.W + w);
            sm[(size_t)c * prm.CS + a * prm.Wp + j] = v;
        }
    }
}

// ---- the kernel ----------------------------------------------------------------------
template <int M, typename Tin, int CPL, int L>
__global__ void __launch_bounds__(256)
input_transform_kernel(const Tin *__restrict__ x, int8_t *__restrict__ Xq,
                       float *__restrict__ sX, Geometry g, ScaleTables tab, K1Params prm)
{
    constexpr int NN = M + 2;
    constexpr int P = NN * NN;
    constexpr int TPW = 32 / L;          // tiles per warp step
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Tin *sm = reinterpret_cast<Tin *>(smem_raw);

    const int strip = blockIdx.x / prm.NCH;       // img*TH + th
    const int chunk = blockIdx.x % prm.NCH;
    const int img = strip / g.TH, th = strip % g.TH;
    const int tw0 = chunk * prm.TWC;
    const int ntile = min(prm.TWC, g.TW - tw0);
    const int c_base = blockIdx.y * prm.CB;
    const int h_base = th * M - 1;
    const int w_base = tw0 * M - 2;
    const int cols = prm.Wp;                      // every staged column is initialised

    stage_strip<Tin>(sm, x, g, prm, NN, img, c_base, h_base, w_base, cols);
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nwarps = blockDim.x >> 5;
    const int q = lane % L, ti = lane / L;
    const int groups = prm.CB / g.gs;
    const int tblocks = (ntile + TPW - 1) / TPW;
    const int items = tblocks * groups;

    for (int it = warp; it < items; it += nwarps) {
        const int grp = it % groups, tb = it / groups;
        const int tl = tb * TPW + ti;             // tile within the chunk
        const bool valid = tl < ntile;
        const int tlc = valid ? tl : ntile - 1;   // clamp: idle lanes recompute a real tile
        const int col0 = tlc * M;                 // smem column before the tile's first one
        const int t = (strip * g.TW) + tw0 + tlc; // global tile id
        const int gglob = c_base / g.gs + grp;
        const int c_grp = grp * g.gs;             // first channel of the group within CB

        float amax[P];
#pragma unroll
        for (int p = 0; p < P; ++p) amax[p] = 0.f;

        if (prm.NSB == 1) {
            // single pass: transformed values stay in registers
            float X[CPL][P];
#pragma unroll
            for (int j = 0; j < CPL; ++j) {
                float d[NN][NN];
                load_patch<NN>(sm + (size_t)(c_grp + q * CPL + j) * prm.CS, col0, prm.Wp, d);
                transform_patch<NN>(d, tab, X[j]);
#pragma unroll
                for (int p = 0; p < P; ++p) amax[p] = fmaxf(amax[p], fabsf(X[j][p]));
            }
            const int c_out = c_base + c_grp + q * CPL;
#pragma unroll
            for (int p = 0; p < P; ++p) {
                const float am = group_absmax<L>(amax[p]);
                const bool nz = am >= 1e-30f;
                const float scale = nz ? __fdiv_rn(am, 127.f) : 0.f;
                const float inv = nz ? __fdiv_rn(127.f, am) : 0.f;
                int code[CPL];
#pragma unroll
                for (int j = 0; j < CPL; ++j) code[j] = quantize_code(X[j][p], inv);
                if (valid) {
                    store_codes<CPL>(Xq + ((size_t)p * g.T + t) * g.C + c_out, code);
                    if (q == 0) sX[((size_t)p * g.G + gglob) * g.T + t] = scale;
                }
            }
        } else {
            // two passes over the group's sub-blocks: maxima first, then recompute
            for (int sb = 0; sb < prm.NSB; ++sb) {
#pragma unroll
                for (int j = 0; j < CPL; ++j) {
                    float d[NN][NN], X[P];
                    const int cl = c_grp + (sb * L + q) * CPL + j;
                    load_patch<NN>(sm + (size_t)cl * prm.CS, col0, prm.Wp, d);
                    transform_patch<NN>(d, tab, X);
#pragma unroll
                    for (int p = 0; p < P; ++p) amax[p] = fmaxf(amax[p], fabsf(X[p]));
                }
            }
#pragma unroll
            for (int p = 0; p < P; ++p) {
                const float am = group_absmax<L>(amax[p]);
                const bool nz = am >= 1e-30f;
                if (valid && q == 0)
                    sX[((size_t)p * g.G + gglob) * g.T + t] = nz ? __fdiv_rn(am, 127.f) : 0.f;
                amax[p] = nz ? __fdiv_rn(127.f, am) : 0.f;   // now holds inv
            }
            for (int sb = 0; sb < prm.NSB; ++sb) {
                float X[CPL][P];
#pragma unroll
                for (int j = 0; j < CPL; ++j) {
                    float d[NN][NN];
                    const int cl = c_grp + (sb * L + q) * CPL + j;
                    load_patch<NN>(sm + (size_t)cl * prm.CS, col0, prm.Wp, d);
                    transform_patch<NN>(d, tab, X[j]);
                }
                const int c_out = c_base + c_grp + (sb * L + q) * CPL;
#pragma unroll
                for (int p = 0; p < P; ++p) {
                    int code[CPL];
#pragma unroll
                    for (int j = 0; j < CPL; ++j) code[j] = quantize_code(X[j][p], amax[p]);
                    if (valid) store_codes<CPL>(Xq + ((size_t)p * g.T + t) * g.C + c_out, code);
                }
            }
        }
    }
}

template <int M, typename Tin, int CPL, int L>
cudaError_t launch_k1(const wfq_plan &plan, const void *x_dev, cudaStream_t stream)
{
    const Geometry &g = plan.geo;
    constexpr int NN = M + 2;
    K1Params prm;
    prm.NSB = g.gs / (CPL * L);
    prm.CB = g.gs;                         // one group per CTA row keeps the strip small
    if (g.gs < 64 && g.C % 64 == 0) prm.CB = 64;
    // tiles per chunk: a multiple of 4 (so chunk starts stay 16-byte friendly), sized
    // so the strip stays below ~48 KB
    const int esz = (int)sizeof(Tin);
    int twc = g.TW;
    auto strip_bytes = [&](int tiles, int &Wp, int &CS) {
        Wp = (tiles * M + 4 + 7) / 8 * 8;          // 2 left pad + tiles*M + 1 halo + slack
        CS = NN * Wp;
        // channel stride: an odd number of 32-bit words (bank-conflict-free lane stride)
        if (esz == 2) { CS += 2; if ((CS / 2) % 2 == 0) CS += 2; }
        else { if (CS % 2 == 0) CS += 1; }
        return (size_t)prm.CB * CS * esz;
    };
    int Wp = 0, CS = 0;
    while (twc > 4 && strip_bytes(twc, Wp, CS) > 48 * 1024) twc = (twc / 2 + 3) / 4 * 4;
    const size_t smem = strip_bytes(twc, Wp, CS);
    prm.TWC = twc;
    prm.NCH = (g.TW + twc - 1) / twc;
    prm.Wp = Wp;
    prm.CS = CS;

    auto kern = input_transform_kernel<M, Tin, CPL, L>;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    dim3 grid((unsigned)(g.N * g.TH * prm.NCH), (unsigned)(g.C / prm.CB));
    kern<<<grid, 256, smem, stream>>>(static_cast<const Tin *>(x_dev), plan.ws.Xq, plan.ws.sX, g,
                                      plan.tables, prm);
    return cudaGetLastError();
}

template <int M, typename Tin>
cudaError_t dispatch_gs(const wfq_plan &plan, const void *x, cudaStream_t s)
{
    const int gs = plan.geo.gs;
    if constexpr (M == 4) {
        if (gs == 32) return launch_k1<4, Tin, 4, 8>(plan, x, s);
        if (gs == 64) return launch_k1<4, Tin, 4, 16>(plan, x, s);
        if (gs % 128 == 0) return launch_k1<4, Tin, 4, 32>(plan, x, s);
        return launch_k1<4, Tin, 4, 8>(plan, x, s);      // 96, 160, 192, 224: sub-blocks of 32
    } else {
        if (gs == 32) return launch_k1<6, Tin, 2, 16>(plan, x, s);
        if (gs % 64 == 0) return launch_k1<6, Tin, 2, 32>(plan, x, s);
        return launch_k1<6, Tin, 2, 16>(plan, x, s);
    }
}

}  // namespace

cudaError_t launch_input_transform(const wfq_plan &plan, const void *x_dev, cudaStream_t stream)
{
    const bool f16 = plan.in_dtype == WFQ_F16;
    if (plan.geo.m == 4)
        return f16 ? dispatch_gs<4, __half>(plan, x_dev, stream)
                   : dispatch_gs<4, float>(plan, x_dev, stream);
    return f16 ? dispatch_gs<6, __half>(plan, x_dev, stream)
               : dispatch_gs<6, float>(plan, x_dev, stream);
}

}  // namespace wfq
