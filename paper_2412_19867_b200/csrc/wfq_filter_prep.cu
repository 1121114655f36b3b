// Offline filter path: W = S_G V_G w V_G^T S_G (Section 4.1) in fp64, one rounding to
// fp32, then group-wise int8 quantization along the input channels, stored
// position-major Wq[P][K][C] with scales sW[P][G][K].  Not on the timed path.
#include <cmath>
#include <mutex>

#include "wfq_internal.h"

namespace wfq {
namespace {

struct GScales {
    double s[kMaxN];
};

// Rows of V_{n x 3}: (f^0 g^2, f^1 g^1, f^2 g^0) for the points
// 0, 1, -1, 2, -2, [1/2, -1/2,] infinity.
__device__ __forceinline__ void vg_row(int m, int i, double &a, double &b, double &c)
{
    const int n = m + 2;
    if (i == n - 1) { a = 0.0; b = 0.0; c = 1.0; return; }
    double f;
    switch (i) {
        case 0: f = 0.0; break;
        case 1: f = 1.0; break;
        case 2: f = -1.0; break;
        case 3: f = 2.0; break;
        case 4: f = -2.0; break;
        case 5: f = 0.5; break;
        default: f = -0.5; break;
    }
    a = 1.0; b = f; c = f * f;
}

// One thread per (k, c): all P transformed values, rounded to fp32.
__global__ void filter_transform_kernel(const float *__restrict__ w, float *__restrict__ w32,
                                        int K, int C, int m, GScales sg)
{
    const int n = m + 2;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)K * C) return;
    const int c = (int)(idx % C), k = (int)(idx / C);
    double f[9];
    for (int i = 0; i < 9; ++i) f[i] = (double)w[idx * 9 + i];
    double tmp[kMaxN][3];  // V_G w
    for (int i = 0; i < n; ++i) {
        double a, b, cc;
        vg_row(m, i, a, b, cc);
        for (int col = 0; col < 3; ++col)
            tmp[i][col] = a * f[col] + b * f[3 + col] + cc * f[6 + col];
    }
    for (int i = 0; i < n; ++i)
        for (int j = 0; j < n; ++j) {
            double a, b, cc;
            vg_row(m, j, a, b, cc);
            const double u = tmp[i][0] * a + tmp[i][1] * b + tmp[i][2] * cc;
            w32[((size_t)(i * n + j) * K + k) * C + c] = (float)(sg.s[i] * sg.s[j] * u);
        }
}

// One thread per (p, k, g): abs-max of the group, scale, codes in [-qmax, qmax] (127 for 8-bit
// weights, 7 for 4-bit weights; the codes are stored one per byte either way, which is what the
// int8 tensor-core contraction reads).  sW rows are k_pitch floats apart.
__global__ void filter_quantize_kernel(const float *__restrict__ w32, int8_t *__restrict__ Wq,
                                       float *__restrict__ sW, int P, int K, int C, int gs,
                                       int k_pitch, int qmax)
{
    const float fq = (float)qmax;
    const int G = C / gs;
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long long)P * K * G) return;
    const int g = (int)(idx % G);
    const int k = (int)((idx / G) % K);
    const int p = (int)(idx / ((long long)G * K));
    const float *src = w32 + ((size_t)p * K + k) * C + (size_t)g * gs;
    int8_t *dst = Wq + ((size_t)p * K + k) * C + (size_t)g * gs;
    float amax = 0.f;
    for (int e = 0; e < gs; ++e) amax = fmaxf(amax, fabsf(src[e]));
    float scale = 0.f, inv = 0.f;
    if (amax >= 1e-30f) {
        scale = __fdiv_rn(amax, fq);
        inv = __fdiv_rn(fq, amax);
    }
    sW[((size_t)p * G + g) * k_pitch + k] = scale;
    for (int e = 0; e < gs; ++e) {
        int q = __float2int_rn(__fmul_rn(src[e], inv));
        q = max(-qmax, min(qmax, q));
        dst[e] = (int8_t)q;
    }
}

}  // namespace

cudaError_t launch_filter_prep(const wfq_plan &plan, const float *w_dev, float *scratch_w32,
                               cudaStream_t stream)
{
    const Geometry &g = plan.geo;
    GScales sg;
    for (int i = 0; i < kMaxN; ++i) sg.s[i] = i < g.n ? plan.sG[i] : 0.0;
    {
        const long long total = (long long)g.K * g.C;
        const int threads = 128;
        const unsigned blocks = (unsigned)((total + threads - 1) / threads);
        filter_transform_kernel<<<blocks, threads, 0, stream>>>(w_dev, scratch_w32, g.K, g.C, g.m, sg);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    {
        const long long total = (long long)g.P * g.K * g.G;
        const int threads = 128;
        const unsigned blocks = (unsigned)((total + threads - 1) / threads);
        filter_quantize_kernel<<<blocks, threads, 0, stream>>>(scratch_w32, plan.Wq, plan.sW, g.P,
                                                               g.K, g.C, g.gs, g.Kp,
                                                               plan.w_bits == 4 ? 7 : 127);
        return cudaGetLastError();
    }
}

// 4-bit filter codes of the exported blob: byte j = code 2j in the low nibble, code 2j+1 in the
// high nibble, two's complement.  One thread per 8 codes (two words in, one word out).
namespace {
__global__ void pack_nibbles_kernel(const uint2 *__restrict__ codes, uint32_t *__restrict__ packed, size_t words)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= words) return;
    const uint2 c = codes[i];
    uint32_t out = 0;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        out |= ((c.x >> (8 * e)) & 0xfu) << (4 * e);
        out |= ((c.y >> (8 * e)) & 0xfu) << (16 + 4 * e);
    }
    packed[i] = out;
}

__global__ void unpack_nibbles_kernel(const uint32_t *__restrict__ packed, uint2 *__restrict__ codes, size_t words)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= words) return;
    const uint32_t w = packed[i];
    uint2 c = make_uint2(0u, 0u);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        // sign extension of a nibble: shift it to the top of an int, arithmetic shift back
        const int lo = ((int)(w << (28 - 4 * e))) >> 28;
        const int hi = ((int)(w << (12 - 4 * e))) >> 28;
        c.x |= ((uint32_t)lo & 0xffu) << (8 * e);
        c.y |= ((uint32_t)hi & 0xffu) << (8 * e);
    }
    codes[i] = c;
}
}  // namespace

cudaError_t launch_pack_nibbles(const int8_t *codes, void *packed, size_t n_codes, cudaStream_t stream)
{
    const size_t words = n_codes / 8;
    if (words == 0) return cudaSuccess;
    pack_nibbles_kernel<<<(unsigned)((words + 255) / 256), 256, 0, stream>>>(
        reinterpret_cast<const uint2 *>(codes), static_cast<uint32_t *>(packed), words);
    return cudaGetLastError();
}

cudaError_t launch_unpack_nibbles(const void *packed, int8_t *codes, size_t n_codes, cudaStream_t stream)
{
    const size_t words = n_codes / 8;
    if (words == 0) return cudaSuccess;
    unpack_nibbles_kernel<<<(unsigned)((words + 255) / 256), 256, 0, stream>>>(
        static_cast<const uint32_t *>(packed), reinterpret_cast<uint2 *>(codes), words);
    return cudaGetLastError();
}

}  // namespace wfq

// ---- filter quantization without any allocation -----------------------------------
//
// The fp32 transformed filters that sit between the two kernels above normally live in
// a temporary device buffer.  Here they live in one fixed array inside the library's
// device image, so the whole call needs no allocator at all.
namespace wfq {
namespace {

constexpr size_t kStaticScratchFloats = WFQ_STATIC_SCRATCH_FLOATS;
static __device__ __align__(256) float g_static_w32[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mutex;
float *g_scratch_ptr[kMaxDevices];   // device address of g_static_w32, per device ordinal

// `g_static_w32` is only a host-side handle in host code; the address a kernel can use
// has to be asked for, with the device it is meant for current.
cudaError_t static_scratch_address(int device, float **out)
{
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[device]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_w32);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[device] = static_cast<float *>(p);
    }
    *out = g_scratch_ptr[device];
    return cudaSuccess;
}

}  // namespace
}  // namespace wfq

extern "C" wfq_status_t wfq_quantize_filters_static(const float *w_dev, int K, int C, int m,
                                                    int group_size, const float *sG_host,
                                                    int8_t *wq_dev, float *sw_dev, void *stream)
{
    using namespace wfq;
    if (!w_dev || !wq_dev || !sw_dev) return WFQ_ERR_INVALID_ARG;
    if (K < 1 || C < 1 || m < 1 || group_size < 1) return WFQ_ERR_INVALID_ARG;
    if ((m != 2 && m != 4 && m != 6) || group_size % 32 != 0 || group_size > 256 || C % group_size != 0)
        return WFQ_ERR_UNSUPPORTED;
    const int n = m + 2, P = n * n;
    const unsigned long long need = (unsigned long long)P * (unsigned long long)K * (unsigned long long)C;
    if (need > kStaticScratchFloats) return WFQ_ERR_SCRATCH_TOO_SMALL;

    static const double std2[4] = {1.0, 0.5, 0.5, 1.0};
    static const double std4[6] = {1.0 / 4, -1.0 / 6, -1.0 / 6, 1.0 / 24, 1.0 / 24, 1.0};
    static const double std6[8] = {1.0, -2.0 / 9, -2.0 / 9, 1.0 / 90, 1.0 / 90, 32.0 / 45, 32.0 / 45, 1.0};
    GScales sg;
    for (int i = 0; i < kMaxN; ++i) {
        double v = 0.0;
        if (i < n) {
            v = sG_host ? (double)sG_host[i] : (m == 2 ? std2[i] : m == 4 ? std4[i] : std6[i]);
            if (!std::isfinite(v) || v == 0.0) return WFQ_ERR_INVALID_ARG;
        }
        sg.s[i] = v;
    }

    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return WFQ_ERR_CUDA;
    if (device < 0 || device >= kMaxDevices) return WFQ_ERR_UNSUPPORTED;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess)
        return WFQ_ERR_CUDA;
    if (major != 10) return WFQ_ERR_UNSUPPORTED;
    float *w32 = nullptr;
    if (static_scratch_address(device, &w32) != cudaSuccess || !w32) return WFQ_ERR_CUDA;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int threads = 128;
    {
        const long long total = (long long)K * C;
        const unsigned blocks = (unsigned)((total + threads - 1) / threads);
        filter_transform_kernel<<<blocks, threads, 0, st>>>(w_dev, w32, K, C, m, sg);
        if (cudaGetLastError() != cudaSuccess) return WFQ_ERR_CUDA;
    }
    {
        const long long total = (long long)P * K * (C / group_size);
        const unsigned blocks = (unsigned)((total + threads - 1) / threads);
        filter_quantize_kernel<<<blocks, threads, 0, st>>>(w32, wq_dev, sw_dev, P, K, C, group_size, K, 127);
        if (cudaGetLastError() != cudaSuccess) return WFQ_ERR_CUDA;
    }
    return WFQ_OK;
}
