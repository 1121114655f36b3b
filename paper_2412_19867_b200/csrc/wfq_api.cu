// C ABI of libwfq.so: plan management, argument checks, workspace layout, launch order.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>

#include "wfq_internal.h"

namespace {

// Standard scale vectors of the paper's supplementary ("Standard Winograd
// transforms"): used when the caller passes NULL, and as the reference the kernels'
// hard-coded integer/rational transform matrices are scaled by.
const double kStdSB2[4] = {1.0, 2.0, 2.0, -1.0};          // F(2,3): the textbook matrices
const double kStdSG2[4] = {1.0, 0.5, 0.5, 1.0};
const double kStdSB4[6] = {4.0, -6.0, -6.0, 24.0, 24.0, 1.0};
const double kStdSG4[6] = {1.0 / 4, -1.0 / 6, -1.0 / 6, 1.0 / 24, 1.0 / 24, 1.0};
const double kStdSB6[8] = {1.0, -4.5, -4.5, 90.0, 90.0, 45.0 / 32, 45.0 / 32, 1.0};
const double kStdSG6[8] = {1.0, -2.0 / 9, -2.0 / 9, 1.0 / 90, 1.0 / 90, 32.0 / 45, 32.0 / 45, 1.0};

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

cudaStream_t as_stream(void *s) { return reinterpret_cast<cudaStream_t>(s); }

wfq_status_t cuda_status(cudaError_t e)
{
    if (e == cudaSuccess) return WFQ_OK;
    if (e == cudaErrorMemoryAllocation) return WFQ_ERR_ALLOC;
    return WFQ_ERR_CUDA;
}

wfq_status_t ready_to_run(const wfq_plan *plan)
{
    if (!plan) return WFQ_ERR_INVALID_ARG;
    if (!plan->has_workspace || !plan->prepared) return WFQ_ERR_NOT_PREPARED;
    return WFQ_OK;
}

size_t in_elem_bytes(const wfq_plan *plan) { return plan->in_dtype == WFQ_F16 ? 2 : 4; }

// Kernel attributes (dynamic shared-memory limits, carveouts) are per device and are set
// the first time a plan meets the device; launches then make no other runtime call.
constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
bool g_device_ready[kMaxDevices];

wfq_status_t bind_device(wfq_plan *plan)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return WFQ_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return WFQ_ERR_UNSUPPORTED;
    if (plan->device == dev && plan->sm_count > 0) return WFQ_OK;
    int major = 0, sms = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return WFQ_ERR_CUDA;
    if (major != 10) return WFQ_ERR_UNSUPPORTED;
    {
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_device_ready[dev]) {
            if (wfq::setup_input_transform() != cudaSuccess || wfq::setup_input_transform_tc() != cudaSuccess ||
                wfq::setup_gemm() != cudaSuccess || wfq::setup_output_transform() != cudaSuccess ||
                wfq::setup_full_quant() != cudaSuccess || wfq::setup_input_transform_tcn() != cudaSuccess)
                return WFQ_ERR_CUDA;
            g_device_ready[dev] = true;
        }
    }
    plan->device = dev;
    plan->sm_count = sms;
    wfq::plan_input_transform(*plan);
    wfq::plan_input_transform_tc(*plan);
    return WFQ_OK;
}

}  // namespace

namespace wfq {

bool encode_tmap(CUtensorMap *map, CUtensorMapDataType dtype, int rank, const void *base,
                 const unsigned long long *dims, const unsigned long long *strides,
                 const unsigned *box, CUtensorMapSwizzle swizzle)
{
    typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *,
                                 const cuuint64_t *, const cuuint64_t *, const cuuint32_t *,
                                 const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) !=
                cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
            return false;
        encode = reinterpret_cast<EncodeFn>(fn);
    }
    if (rank < 1 || rank > 4) return false;
    cuuint64_t d[4], st[3];
    cuuint32_t bx[4], estr[4] = {1u, 1u, 1u, 1u};
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; bx[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) st[i] = strides[i];
    CUresult r = encode(map, dtype, (cuuint32_t)rank, const_cast<void *>(base), d, st, bx, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

bool encode_tmap_bytes3d(CUtensorMap *map, const void *base, int inner, int rows, int planes,
                         int box_rows)
{
    const unsigned long long dims[3] = {(unsigned long long)inner, (unsigned long long)rows,
                                        (unsigned long long)planes};
    const unsigned long long strides[2] = {(unsigned long long)inner,
                                           (unsigned long long)inner * (unsigned long long)rows};
    const unsigned box[3] = {128u, (unsigned)box_rows, 1u};
    return encode_tmap(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, base, dims, strides, box,
                       CU_TENSOR_MAP_SWIZZLE_128B);
}

}  // namespace wfq

extern "C" {

int wfq_version(void) { return 100; }

const char *wfq_status_string(wfq_status_t s)
{
    switch (s) {
        case WFQ_OK: return "ok";
        case WFQ_ERR_INVALID_ARG: return "invalid argument";
        case WFQ_ERR_UNSUPPORTED: return "unsupported configuration";
        case WFQ_ERR_ALLOC: return "allocation failed";
        case WFQ_ERR_NOT_PREPARED: return "plan has no workspace or no prepared filters";
        case WFQ_ERR_CUDA: return "CUDA call failed";
        case WFQ_ERR_TIMEOUT: return "device-side wait timed out";
        case WFQ_ERR_SCRATCH_TOO_SMALL:
            return "problem exceeds the library's built-in scratch array";
    }
    return "unknown status";
}

wfq_status_t wfq_plan_create(wfq_plan_t **out, int N, int C, int K, int H, int W, int m, int r,
                             int group_size, int bits)
{
    if (!out) return WFQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (N < 1 || C < 1 || K < 1 || H < 1 || W < 1 || m < 1 || r < 1 || group_size < 1 || bits < 1)
        return WFQ_ERR_INVALID_ARG;
    if (r != 3 || (m != 2 && m != 4 && m != 6) || bits != 8) return WFQ_ERR_UNSUPPORTED;
    if (group_size % 32 != 0 || group_size > 256 || C % group_size != 0)
        return WFQ_ERR_UNSUPPORTED;

    wfq_plan *p = new (std::nothrow) wfq_plan();
    if (!p) return WFQ_ERR_ALLOC;
    wfq::Geometry &g = p->geo;
    g.N = N; g.C = C; g.K = K; g.H = H; g.W = W;
    g.m = m; g.n = m + 2; g.P = g.n * g.n;
    g.TH = (H + m - 1) / m; g.TW = (W + m - 1) / m;
    const long long T = (long long)N * g.TH * g.TW;
    const long long lim = (1LL << 31) - 1;
    if (T > lim || (long long)g.P * T * C > lim || (long long)g.P * K * C > lim ||
        (long long)N * K * H * W > lim || (long long)N * C * H * W > lim ||
        (long long)g.P * K * ((T + 31) / 32 * 32) > lim) {
        delete p;
        return WFQ_ERR_UNSUPPORTED;
    }
    g.T = (int)T; g.Tp = (g.T + 31) / 32 * 32;
    g.Ts = (g.T + 127) / 128 * 128; g.Kp = (K + 127) / 128 * 128;
    g.gs = group_size; g.G = C / group_size;
    wfq::gemm_choose(g, &p->gemm_swap, &p->gemm_bn);

    wfq::Workspace &ws = p->ws;
    ws.xq_bytes = align_up((size_t)g.P * g.T * g.C, 1024);
    ws.sx_bytes = align_up((size_t)g.P * g.G * g.Ts * sizeof(float), 1024);
    ws.y_bytes = align_up((size_t)g.P * g.K * g.Tp * sizeof(float), 1024);
    ws.total = ws.xq_bytes + ws.sx_bytes + ws.y_bytes;
    *out = p;
    return WFQ_OK;
}

wfq_status_t wfq_plan_set_input_dtype(wfq_plan_t *plan, wfq_dtype_t dtype)
{
    if (!plan) return WFQ_ERR_INVALID_ARG;
    if (dtype != WFQ_F32 && dtype != WFQ_F16) return WFQ_ERR_INVALID_ARG;
    plan->in_dtype = dtype;
    plan->host_chunks = 0;            // chunk starts are aligned for the element size
    plan->tmap_x_base = nullptr;
    if (plan->sm_count > 0) {
        wfq::plan_input_transform(*plan);
        wfq::plan_input_transform_tc(*plan);
    }
    return WFQ_OK;
}

wfq_status_t wfq_plan_set_input_layout(wfq_plan_t *plan, wfq_layout_t layout)
{
    if (!plan || (layout != WFQ_NCHW && layout != WFQ_NHWC)) return WFQ_ERR_INVALID_ARG;
    if (layout == WFQ_NHWC && plan->fq_input) return WFQ_ERR_UNSUPPORTED;   // integer input transform: NCHW only
    plan->in_nhwc = layout == WFQ_NHWC;
    plan->tmap_xn_base = nullptr;
    plan->tmap_xn_tc_base = nullptr;
    for (int i = 0; i < 2; ++i)
        if (plan->sub[i]) {
            plan->sub[i]->in_nhwc = plan->in_nhwc;
            plan->sub[i]->tmap_xn_base = nullptr;
            plan->sub[i]->tmap_xn_tc_base = nullptr;
        }
    return WFQ_OK;
}

wfq_status_t wfq_plan_set_epilogue(wfq_plan_t *plan, const float *bias_dev, wfq_activation_t act)
{
    if (!plan) return WFQ_ERR_INVALID_ARG;
    if (act != WFQ_ACT_NONE && act != WFQ_ACT_RELU && act != WFQ_ACT_SILU) return WFQ_ERR_INVALID_ARG;
    if (bias_dev && (reinterpret_cast<uintptr_t>(bias_dev) & 3u)) return WFQ_ERR_INVALID_ARG;
    plan->bias = bias_dev;
    plan->act = (int)act;
    for (int i = 0; i < 2; ++i)
        if (plan->sub[i]) { plan->sub[i]->bias = bias_dev; plan->sub[i]->act = (int)act; }
    return WFQ_OK;
}

size_t wfq_plan_workspace_bytes(const wfq_plan_t *plan) { return plan ? plan->ws.total : 0; }

wfq_status_t wfq_plan_set_output_dtype(wfq_plan_t *plan, wfq_dtype_t dtype)
{
    if (!plan || (dtype != WFQ_F32 && dtype != WFQ_F16 && dtype != WFQ_BF16)) return WFQ_ERR_INVALID_ARG;
    plan->out_half = dtype == WFQ_F16 ? 1 : dtype == WFQ_BF16 ? 2 : 0;
    plan->host_chunks = 0;         // chunk sizes of the host-buffer path depend on the output bytes
    for (int i = 0; i < 2; ++i)
        if (plan->sub[i]) plan->sub[i]->out_half = plan->out_half;
    return WFQ_OK;
}

wfq_status_t wfq_plan_set_weight_bits(wfq_plan_t *plan, int bits)
{
    if (!plan) return WFQ_ERR_INVALID_ARG;
    if (bits != 8 && bits != 4) return WFQ_ERR_UNSUPPORTED;
    if (bits != plan->w_bits) {
        plan->w_bits = bits;
        plan->prepared = false;    // filters quantized at the other width are not valid any more
        for (int i = 0; i < 2; ++i)
            if (plan->sub[i]) plan->sub[i]->prepared = false;
    }
    return WFQ_OK;
}

wfq_status_t wfq_plan_set_full_quant(wfq_plan_t *plan, int quant_input, wfq_y_quant_t y_mode)
{
    if (!plan) return WFQ_ERR_INVALID_ARG;
    if (quant_input != 0 && quant_input != 1) return WFQ_ERR_INVALID_ARG;
    if (y_mode != WFQ_Y_FP32 && y_mode != WFQ_Y_TILE && y_mode != WFQ_Y_ROW) return WFQ_ERR_INVALID_ARG;
    if (quant_input && (plan->geo.gs % 32 != 0 || plan->geo.gs > 256 || plan->in_nhwc)) return WFQ_ERR_UNSUPPORTED;
    plan->fq_input = quant_input != 0;
    plan->fq_output = (int)y_mode;
    for (int i = 0; i < 2; ++i)
        if (plan->sub[i]) { plan->sub[i]->fq_input = plan->fq_input; plan->sub[i]->fq_output = plan->fq_output; }
    return WFQ_OK;
}

wfq_status_t wfq_plan_set_workspace(wfq_plan_t *plan, void *dev_ptr, size_t bytes)
{
    if (!plan || !dev_ptr) return WFQ_ERR_INVALID_ARG;
    if (bytes < plan->ws.total || (reinterpret_cast<uintptr_t>(dev_ptr) & 1023u) != 0)
        return WFQ_ERR_INVALID_ARG;
    wfq_status_t bs = bind_device(plan);
    if (bs != WFQ_OK) return bs;
    wfq::Workspace &ws = plan->ws;
    char *base = static_cast<char *>(dev_ptr);
    ws.Xq = reinterpret_cast<int8_t *>(base);
    ws.sX = reinterpret_cast<float *>(base + ws.xq_bytes);
    ws.Y = reinterpret_cast<float *>(base + ws.xq_bytes + ws.sx_bytes);
    const wfq::Geometry &g = plan->geo;
    plan->tmap_xq_ok = wfq::encode_tmap_bytes3d(&plan->tmap_xq, ws.Xq, g.C, g.T, g.P,
                                               plan->gemm_swap ? plan->gemm_bn : wfq::gemm_block_m());
    if (!plan->tmap_xq_ok) return WFQ_ERR_CUDA;
    plan->has_workspace = true;
    return WFQ_OK;
}

// The per-position products of the plan's scale vectors (rounded once from fp64).
static void fill_scale_tables(wfq_plan *plan)
{
    const wfq::Geometry &g = plan->geo;
    const double *stdB = g.m == 2 ? kStdSB2 : g.m == 4 ? kStdSB4 : kStdSB6;
    for (int i = 0; i < g.n; ++i)
        for (int j = 0; j < g.n; ++j) {
            const double f = (plan->sB[i] / stdB[i]) * (plan->sB[j] / stdB[j]);
            plan->tables.in_scale[i * g.n + j] = (float)f;
            plan->tables.in_scale_lo[i * g.n + j] = (float)(f - (double)(float)f);
            plan->tables.out_scale[i * g.n + j] = (float)(plan->sA[i] * plan->sA[j]);
        }
}

// Device buffers of the prepared filters and the status word (allocated once per plan).
static wfq_status_t ensure_filter_buffers(wfq_plan *plan, cudaStream_t stream)
{
    const wfq::Geometry &g = plan->geo;
    wfq_status_t bs = bind_device(plan);
    if (bs != WFQ_OK) return bs;
    cudaError_t e;
    const size_t wq_bytes = (size_t)g.P * g.K * g.C;
    const size_t sw_bytes = (size_t)g.P * g.G * g.Kp * sizeof(float);
    if (!plan->Wq && (e = cudaMalloc(&plan->Wq, wq_bytes)) != cudaSuccess) return cuda_status(e);
    if (!plan->sW) {
        if ((e = cudaMalloc(&plan->sW, sw_bytes)) != cudaSuccess) return cuda_status(e);
        // the padding columns k >= K stay zero
        if ((e = cudaMemsetAsync(plan->sW, 0, sw_bytes, stream)) != cudaSuccess) return WFQ_ERR_CUDA;
    }
    if (!plan->status) {
        if ((e = cudaMalloc(&plan->status, 4 * sizeof(int))) != cudaSuccess) return cuda_status(e);
        if ((e = cudaMemsetAsync(plan->status, 0, 4 * sizeof(int), stream)) != cudaSuccess) return WFQ_ERR_CUDA;
    }
    return WFQ_OK;
}

// What follows once Wq and sW are in place.
static wfq_status_t finish_filters(wfq_plan *plan)
{
    const wfq::Geometry &g = plan->geo;
    plan->tmap_wq_ok = wfq::encode_tmap_bytes3d(&plan->tmap_wq, plan->Wq, g.C, g.K, g.P,
                                               plan->gemm_swap ? wfq::gemm_block_m() : plan->gemm_bn);
    if (!plan->tmap_wq_ok) return WFQ_ERR_CUDA;
    wfq::build_full_quant_tables(*plan);
    plan->prepared = true;
    return WFQ_OK;
}

wfq_status_t wfq_prepare_filters(wfq_plan_t *plan, const float *w_dev, const float *sB_host,
                                 const float *sG_host, const float *sA_host, void *stream)
{
    if (!plan || !w_dev) return WFQ_ERR_INVALID_ARG;
    const wfq::Geometry &g = plan->geo;
    const double *stdB = g.m == 2 ? kStdSB2 : g.m == 4 ? kStdSB4 : kStdSB6;
    const double *stdG = g.m == 2 ? kStdSG2 : g.m == 4 ? kStdSG4 : kStdSG6;
    for (int i = 0; i < g.n; ++i) {
        const double b = sB_host ? (double)sB_host[i] : stdB[i];
        const double s = sG_host ? (double)sG_host[i] : stdG[i];
        if (!std::isfinite(b) || !std::isfinite(s) || b == 0.0 || s == 0.0)
            return WFQ_ERR_INVALID_ARG;
        double a;
        if (sA_host) {
            a = (double)sA_host[i];
            if (!std::isfinite(a) || a == 0.0) return WFQ_ERR_INVALID_ARG;
        } else {
            a = (double)(float)(1.0 / (b * s));
        }
        plan->sB[i] = b; plan->sG[i] = s; plan->sA[i] = a;
    }
    fill_scale_tables(plan);

    wfq_status_t bs = ensure_filter_buffers(plan, as_stream(stream));
    if (bs != WFQ_OK) return bs;
    cudaError_t e;
    const size_t wq_bytes = (size_t)g.P * g.K * g.C;
    // fp32 transformed filters between the two kernels: stream-ordered allocation, released
    // in stream order after the quantization kernel, so the call neither blocks nor holds
    // the temporary (four times the size of Wq) any longer than the kernels need it
    void *w32 = nullptr;
    if ((e = cudaMallocAsync(&w32, wq_bytes * sizeof(float), as_stream(stream))) != cudaSuccess)
        return cuda_status(e);
    e = wfq::launch_filter_prep(*plan, w_dev, static_cast<float *>(w32), as_stream(stream));
    cudaError_t e2 = cudaFreeAsync(w32, as_stream(stream));
    if (e != cudaSuccess || e2 != cudaSuccess) return WFQ_ERR_CUDA;
    return finish_filters(plan);
}

// ---- prepared filters as a host blob ------------------------------------------------------
namespace {
struct FilterBlobHeader {
    char magic[8];                       // "WFQFILT1"
    int32_t m, C, K, gs, P, G, Kp, w_bits;   // w_bits: 8, 4, or 0 (= 8, blobs written before the field existed)
    double sB[wfq::kMaxN], sG[wfq::kMaxN], sA[wfq::kMaxN];
    char pad[256 - 8 - 8 * 4 - 3 * 8 * wfq::kMaxN];
};
static_assert(sizeof(FilterBlobHeader) == 256, "header is 256 bytes");
const char kBlobMagic[8] = {'W', 'F', 'Q', 'F', 'I', 'L', 'T', '1'};
}  // namespace

// bytes of the code section: one code per byte, or two per byte for 4-bit weights
static size_t blob_wq_bytes(const wfq::Geometry &g, int w_bits)
{
    const size_t codes = (size_t)g.P * g.K * g.C;
    return w_bits == 4 ? codes / 2 : codes;
}

size_t wfq_filters_bytes(const wfq_plan_t *plan)
{
    if (!plan) return 0;
    const wfq::Geometry &g = plan->geo;
    return sizeof(FilterBlobHeader) + blob_wq_bytes(g, plan->w_bits) + (size_t)g.P * g.G * g.Kp * sizeof(float);
}

wfq_status_t wfq_filters_export(wfq_plan_t *plan, void *host_buf, size_t bytes, void *stream)
{
    if (!plan || !host_buf) return WFQ_ERR_INVALID_ARG;
    if (!plan->prepared) return WFQ_ERR_NOT_PREPARED;
    if (bytes < wfq_filters_bytes(plan)) return WFQ_ERR_INVALID_ARG;
    const wfq::Geometry &g = plan->geo;
    FilterBlobHeader h;
    memset(&h, 0, sizeof(h));
    memcpy(h.magic, kBlobMagic, 8);
    h.m = g.m; h.C = g.C; h.K = g.K; h.gs = g.gs; h.P = g.P; h.G = g.G; h.Kp = g.Kp; h.w_bits = plan->w_bits;
    for (int i = 0; i < g.n; ++i) { h.sB[i] = plan->sB[i]; h.sG[i] = plan->sG[i]; h.sA[i] = plan->sA[i]; }
    memcpy(host_buf, &h, sizeof(h));
    char *dst = static_cast<char *>(host_buf) + sizeof(h);
    const size_t codes = (size_t)g.P * g.K * g.C, wq_bytes = blob_wq_bytes(g, plan->w_bits);
    const size_t sw_bytes = (size_t)g.P * g.G * g.Kp * sizeof(float);
    cudaStream_t st = as_stream(stream);
    void *packed = nullptr;
    const void *src = plan->Wq;
    if (plan->w_bits == 4) {
        // two codes per byte, packed on the device into a stream-ordered temporary
        if (cudaMallocAsync(&packed, wq_bytes, st) != cudaSuccess) return WFQ_ERR_CUDA;
        if (wfq::launch_pack_nibbles(plan->Wq, packed, codes, st) != cudaSuccess) {
            cudaFreeAsync(packed, st);
            return WFQ_ERR_CUDA;
        }
        src = packed;
    }
    bool ok = cudaMemcpyAsync(dst, src, wq_bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess &&
              cudaMemcpyAsync(dst + wq_bytes, plan->sW, sw_bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    if (packed) ok = (cudaFreeAsync(packed, st) == cudaSuccess) && ok;
    if (!ok) return WFQ_ERR_CUDA;
    return cuda_status(cudaStreamSynchronize(st));
}

wfq_status_t wfq_filters_import(wfq_plan_t *plan, const void *host_buf, size_t bytes, void *stream)
{
    if (!plan || !host_buf || bytes < sizeof(FilterBlobHeader)) return WFQ_ERR_INVALID_ARG;
    const wfq::Geometry &g = plan->geo;
    FilterBlobHeader h;
    memcpy(&h, host_buf, sizeof(h));
    if (memcmp(h.magic, kBlobMagic, 8) != 0 || h.m != g.m || h.C != g.C || h.K != g.K || h.gs != g.gs ||
        h.P != g.P || h.G != g.G || h.Kp != g.Kp || (h.w_bits != 0 && h.w_bits != 8 && h.w_bits != 4))
        return WFQ_ERR_INVALID_ARG;
    const int w_bits = h.w_bits == 4 ? 4 : 8;
    const size_t codes = (size_t)g.P * g.K * g.C, wq_bytes = blob_wq_bytes(g, w_bits);
    const size_t sw_bytes = (size_t)g.P * g.G * g.Kp * sizeof(float);
    if (bytes < sizeof(FilterBlobHeader) + wq_bytes + sw_bytes) return WFQ_ERR_INVALID_ARG;
    for (int i = 0; i < g.n; ++i)
        if (!std::isfinite(h.sB[i]) || !std::isfinite(h.sG[i]) || !std::isfinite(h.sA[i]) || h.sB[i] == 0.0 ||
            h.sG[i] == 0.0 || h.sA[i] == 0.0)
            return WFQ_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    wfq_status_t bs = ensure_filter_buffers(plan, st);
    if (bs != WFQ_OK) return bs;
    // from here on the plan's filters are being replaced: a CUDA error below leaves it unprepared
    plan->prepared = false;
    for (int i = 0; i < g.n; ++i) { plan->sB[i] = h.sB[i]; plan->sG[i] = h.sG[i]; plan->sA[i] = h.sA[i]; }
    fill_scale_tables(plan);
    plan->w_bits = w_bits;
    const char *src = static_cast<const char *>(host_buf) + sizeof(h);
    if (w_bits == 4) {
        void *packed = nullptr;
        if (cudaMallocAsync(&packed, wq_bytes, st) != cudaSuccess) return WFQ_ERR_CUDA;
        const bool ok = cudaMemcpyAsync(packed, src, wq_bytes, cudaMemcpyHostToDevice, st) == cudaSuccess &&
                        wfq::launch_unpack_nibbles(packed, plan->Wq, codes, st) == cudaSuccess;
        if (cudaFreeAsync(packed, st) != cudaSuccess || !ok) return WFQ_ERR_CUDA;
    } else if (cudaMemcpyAsync(plan->Wq, src, wq_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
        return WFQ_ERR_CUDA;
    }
    if (cudaMemcpyAsync(plan->sW, src + wq_bytes, sw_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return WFQ_ERR_CUDA;
    // the caller may free or change the blob when this returns
    if (cudaStreamSynchronize(st) != cudaSuccess) return WFQ_ERR_CUDA;
    return finish_filters(plan);
}

wfq_status_t wfq_input_transform_quantize(wfq_plan_t *plan, const void *x_dev, void *stream)
{
    wfq_status_t s = ready_to_run(plan);
    if (s != WFQ_OK) return s;
    if (!x_dev || (reinterpret_cast<uintptr_t>(x_dev) & 3u)) return WFQ_ERR_INVALID_ARG;
    if (plan->fq_input) return cuda_status(wfq::launch_input_transform_int(*plan, x_dev, as_stream(stream)));
    return cuda_status(wfq::launch_input_transform(*plan, x_dev, as_stream(stream)));
}

wfq_status_t wfq_gemm_dequantize(wfq_plan_t *plan, void *stream)
{
    wfq_status_t s = ready_to_run(plan);
    if (s != WFQ_OK) return s;
    return cuda_status(wfq::launch_gemm(*plan, nullptr, as_stream(stream), false));
}

wfq_status_t wfq_debug_gemm_acc32(wfq_plan_t *plan, int32_t *acc_dev, void *stream)
{
    wfq_status_t s = ready_to_run(plan);
    if (s != WFQ_OK) return s;
    if (!acc_dev) return WFQ_ERR_INVALID_ARG;
    return cuda_status(wfq::launch_gemm(*plan, acc_dev, as_stream(stream), false));
}

wfq_status_t wfq_debug_int8_mma_rate(wfq_plan_t *plan, int n_cols, int mmas_per_sm, long long *ops,
                                     void *stream)
{
    if (!plan || !ops) return WFQ_ERR_INVALID_ARG;
    if (!plan->prepared) return WFQ_ERR_NOT_PREPARED;       // needs the status word and the device
    if ((n_cols != 64 && n_cols != 128 && n_cols != 256) || mmas_per_sm < 4 || mmas_per_sm > (1 << 24) ||
        mmas_per_sm % 4 != 0)
        return WFQ_ERR_INVALID_ARG;
    *ops = (long long)plan->sm_count * mmas_per_sm * 2LL * 128 * n_cols * 32;
    return cuda_status(wfq::launch_mma_peak(*plan, n_cols, mmas_per_sm, as_stream(stream)));
}

wfq_status_t wfq_output_transform(wfq_plan_t *plan, float *y_dev, void *stream)
{
    wfq_status_t s = ready_to_run(plan);
    if (s != WFQ_OK) return s;
    if (!y_dev || (reinterpret_cast<uintptr_t>(y_dev) & 15u)) return WFQ_ERR_INVALID_ARG;
    if (plan->fq_output) return cuda_status(wfq::launch_output_transform_int(*plan, y_dev, as_stream(stream)));
    return cuda_status(wfq::launch_output_transform(*plan, y_dev, as_stream(stream), false));
}

wfq_status_t wfq_conv_forward(wfq_plan_t *plan, const void *x_dev, float *y_dev, void *stream)
{
    wfq_status_t s = ready_to_run(plan);
    if (s != WFQ_OK) return s;
    if (!x_dev || !y_dev || (reinterpret_cast<uintptr_t>(x_dev) & 3u) ||
        (reinterpret_cast<uintptr_t>(y_dev) & 15u))
        return WFQ_ERR_INVALID_ARG;
    cudaStream_t st = as_stream(stream);
    cudaError_t e = plan->fq_input ? wfq::launch_input_transform_int(*plan, x_dev, st)
                                   : wfq::launch_input_transform(*plan, x_dev, st);
    if (e == cudaSuccess) e = wfq::launch_gemm(*plan, nullptr, st, true);
    if (e == cudaSuccess)
        e = plan->fq_output ? wfq::launch_output_transform_int(*plan, y_dev, st)
                            : wfq::launch_output_transform(*plan, y_dev, st, true);
    return cuda_status(e);
}

// Number of chunks for the pipelined host path: a divisor of N (whole images per chunk,
// all chunks alike), at least three so that two chunks fit the caller's workspace, and
// only for transfers large enough to pay for the extra launches.
static int pick_host_chunks(const wfq_plan *plan, size_t xb, size_t yb)
{
    const int N = plan->geo.N;
    if (N < 3 || xb + yb < ((size_t)12 << 20)) return 1;
    const int prefer[] = {4, 3, 5, 6, 7, 8};
    for (int c : prefer)
        if (N % c == 0 && (xb / c) % 16 == 0 && (yb / c) % 16 == 0) return c;   // aligned chunk starts
    return 1;
}

// (Re)builds the two chunk plans from the parent's current state.  Cheap: no device work
// except, the first time, the creation of two streams and three events.
static wfq_status_t setup_host_pipeline(wfq_plan *plan)
{
    const wfq::Geometry &g = plan->geo;
    const int nc = g.N / plan->host_chunks;
    for (int s = 0; s < 2; ++s) {
        if (!plan->sub[s]) {
            wfq_status_t st = wfq_plan_create(&plan->sub[s], nc, g.C, g.K, g.H, g.W, g.m, 3, g.gs, 8);
            if (st != WFQ_OK) return st;
            plan->sub[s]->borrowed = true;
        }
        wfq_plan *q = plan->sub[s];
        wfq_plan_set_input_dtype(q, plan->in_dtype);
        q->k1_choice = plan->k1_choice;
        q->in_nhwc = plan->in_nhwc;
        // same orientation of the contraction as the whole batch: identical arithmetic
        q->gemm_swap = plan->gemm_swap;
        q->gemm_bn = plan->gemm_bn;
        const size_t slice = align_up(q->ws.total, 1024);
        if (2 * slice > plan->ws.total) return WFQ_ERR_UNSUPPORTED;
        wfq_status_t st = wfq_plan_set_workspace(q, reinterpret_cast<char *>(plan->ws.Xq) + s * slice, slice);
        if (st != WFQ_OK) return st;
        q->Wq = plan->Wq; q->sW = plan->sW; q->status = plan->status;
        q->tables = plan->tables;
        q->tmap_wq = plan->tmap_wq; q->tmap_wq_ok = plan->tmap_wq_ok;
        q->wait_cycles = plan->wait_cycles;
        q->bias = plan->bias; q->act = plan->act; q->out_half = plan->out_half;
        q->fq_input = plan->fq_input; q->fq_output = plan->fq_output; q->fq = plan->fq;
        q->prepared = true;
        if (!plan->host_stream[s] &&
            cudaStreamCreateWithFlags(&plan->host_stream[s], cudaStreamNonBlocking) != cudaSuccess)
            return WFQ_ERR_CUDA;
    }
    for (int i = 0; i < 3; ++i)
        if (!plan->host_event[i] &&
            cudaEventCreateWithFlags(&plan->host_event[i], cudaEventDisableTiming) != cudaSuccess)
            return WFQ_ERR_CUDA;
    return WFQ_OK;
}

static wfq_status_t forward_host(wfq_plan_t *plan, const void *x_host, float *y_host, void *stream, bool wait)
{
    wfq_status_t s = ready_to_run(plan);
    if (s != WFQ_OK) return s;
    if (!x_host || !y_host) return WFQ_ERR_INVALID_ARG;
    const wfq::Geometry &g = plan->geo;
    const size_t xb = (size_t)g.N * g.C * g.H * g.W * in_elem_bytes(plan);
    const size_t yb = (size_t)g.N * g.K * g.H * g.W * (plan->out_half ? 2 : sizeof(float));
    cudaError_t e;
    if (!plan->x_stage && (e = cudaMalloc(&plan->x_stage, (size_t)g.N * g.C * g.H * g.W * 4)) != cudaSuccess)
        return cuda_status(e);
    if (!plan->y_stage && (e = cudaMalloc(&plan->y_stage, (size_t)g.N * g.K * g.H * g.W * sizeof(float))) != cudaSuccess)
        return cuda_status(e);
    cudaStream_t st = as_stream(stream);

    if (plan->host_chunks == 0) plan->host_chunks = pick_host_chunks(plan, xb, yb);
    if (plan->host_chunks > 1 && setup_host_pipeline(plan) != WFQ_OK) plan->host_chunks = 1;

    if (plan->host_chunks > 1) {
        const int chunks = plan->host_chunks;
        const size_t xc = xb / chunks, yc = yb / chunks;
        // the internal streams start after the work already queued on the caller's stream
        if (cudaEventRecord(plan->host_event[2], st) != cudaSuccess) return WFQ_ERR_CUDA;
        for (int i = 0; i < 2; ++i)
            if (cudaStreamWaitEvent(plan->host_stream[i], plan->host_event[2], 0) != cudaSuccess)
                return WFQ_ERR_CUDA;
        wfq_status_t err = WFQ_OK;
        for (int c = 0; c < chunks && err == WFQ_OK; ++c) {
            cudaStream_t cs = plan->host_stream[c & 1];
            char *xd = static_cast<char *>(plan->x_stage) + (size_t)c * xc;
            float *yd = reinterpret_cast<float *>(reinterpret_cast<char *>(plan->y_stage) + (size_t)c * yc);
            if (cudaMemcpyAsync(xd, static_cast<const char *>(x_host) + (size_t)c * xc, xc,
                                cudaMemcpyHostToDevice, cs) != cudaSuccess) {
                err = WFQ_ERR_CUDA;
                break;
            }
            err = wfq_conv_forward(plan->sub[c & 1], xd, yd, cs);
            if (err == WFQ_OK &&
                cudaMemcpyAsync(reinterpret_cast<char *>(y_host) + (size_t)c * yc, yd, yc,
                                cudaMemcpyDeviceToHost, cs) != cudaSuccess)
                err = WFQ_ERR_CUDA;
        }
        // The caller's stream continues after both internal streams; on an error the
        // copies already queued are waited for as well, so that nothing writes y_host
        // after this (synchronous) call has returned.
        for (int i = 0; i < 2; ++i) {
            if (cudaEventRecord(plan->host_event[i], plan->host_stream[i]) != cudaSuccess ||
                cudaStreamWaitEvent(st, plan->host_event[i], 0) != cudaSuccess) {
                cudaStreamSynchronize(plan->host_stream[i]);
                if (err == WFQ_OK) err = WFQ_ERR_CUDA;
            }
        }
        // an error leaves copies queued that must not outlive the call: wait for them either way
        const cudaError_t se = (wait || err != WFQ_OK) ? cudaStreamSynchronize(st) : cudaSuccess;
        return err != WFQ_OK ? err : cuda_status(se);
    }

    if ((e = cudaMemcpyAsync(plan->x_stage, x_host, xb, cudaMemcpyHostToDevice, st)) != cudaSuccess)
        return WFQ_ERR_CUDA;
    s = wfq_conv_forward(plan, plan->x_stage, plan->y_stage, stream);
    if (s != WFQ_OK) return s;
    if ((e = cudaMemcpyAsync(y_host, plan->y_stage, yb, cudaMemcpyDeviceToHost, st)) != cudaSuccess)
        return WFQ_ERR_CUDA;
    return wait ? cuda_status(cudaStreamSynchronize(st)) : WFQ_OK;
}

wfq_status_t wfq_conv_forward_host(wfq_plan_t *plan, const void *x_host, float *y_host, void *stream)
{
    return forward_host(plan, x_host, y_host, stream, true);
}

wfq_status_t wfq_conv_forward_host_async(wfq_plan_t *plan, const void *x_host, float *y_host, void *stream)
{
    return forward_host(plan, x_host, y_host, stream, false);
}

wfq_status_t wfq_plan_set_debug_option(wfq_plan_t *plan, wfq_debug_option_t option, long long value)
{
    if (!plan) return WFQ_ERR_INVALID_ARG;
    switch (option) {
        case WFQ_DEBUG_WAIT_CYCLES:
            if (value < 1000) return WFQ_ERR_INVALID_ARG;
            plan->wait_cycles = value;
            break;
        case WFQ_DEBUG_SKIP_INPUT_ITEM:
            if (value < -1 || value > 0x7fffffff) return WFQ_ERR_INVALID_ARG;
            plan->debug_skip_item = (int)value;
            break;
        case WFQ_DEBUG_INPUT_TRANSFORM_KERNEL:
            if (value < 0 || value > 3) return WFQ_ERR_INVALID_ARG;
            plan->k1_choice = (int)value;
            break;
        case WFQ_DEBUG_SKIP_GEMM_STAGE:
            if (value < -1 || value > 0x7fffffff) return WFQ_ERR_INVALID_ARG;
            plan->debug_skip_gemm_stage = (int)value;
            break;
        case WFQ_DEBUG_GEMM_SHAPE: {
            // 0: the library's choice; else 100 * orientation (1 rows = tiles, 2 rows = output
            // channels) + columns per unit (rows = tiles: 16 or 64; rows = channels: 16, 32, 48, 64)
            bool swap;
            int bn;
            if (value == 0) {
                wfq::gemm_choose(plan->geo, &swap, &bn);
            } else {
                const int orient = (int)(value / 100);
                bn = (int)(value % 100);
                if (orient == 1 && (bn == 16 || bn == 64)) swap = false;
                else if (orient == 2 && (bn == 16 || bn == 32 || bn == 48 || bn == 64)) swap = true;
                else return WFQ_ERR_INVALID_ARG;
            }
            plan->gemm_swap = swap;
            plan->gemm_bn = bn;
            const wfq::Geometry &g = plan->geo;
            if (plan->has_workspace)
                plan->tmap_xq_ok = wfq::encode_tmap_bytes3d(&plan->tmap_xq, plan->ws.Xq, g.C, g.T, g.P,
                                                           swap ? bn : wfq::gemm_block_m());
            if (plan->Wq)
                plan->tmap_wq_ok = wfq::encode_tmap_bytes3d(&plan->tmap_wq, plan->Wq, g.C, g.K, g.P,
                                                           swap ? wfq::gemm_block_m() : bn);
            if ((plan->has_workspace && !plan->tmap_xq_ok) || (plan->Wq && !plan->tmap_wq_ok)) return WFQ_ERR_CUDA;
            plan->host_chunks = 0;      // the sub-plans of the host-buffer path copy the shape when rebuilt
            break;
        }
        default:
            return WFQ_ERR_INVALID_ARG;
    }
    for (int i = 0; i < 2; ++i)
        if (plan->sub[i]) {
            plan->sub[i]->wait_cycles = plan->wait_cycles;
            plan->sub[i]->k1_choice = plan->k1_choice;
        }
    return WFQ_OK;
}

wfq_status_t wfq_debug_get(wfq_plan_t *plan, wfq_buffer_t which, void **dev_ptr, size_t *bytes)
{
    if (!plan || !dev_ptr || !bytes) return WFQ_ERR_INVALID_ARG;
    const wfq::Geometry &g = plan->geo;
    *dev_ptr = nullptr;
    *bytes = 0;
    switch (which) {
        case WFQ_BUF_XQ:
            if (!plan->has_workspace) return WFQ_ERR_NOT_PREPARED;
            *dev_ptr = plan->ws.Xq; *bytes = (size_t)g.P * g.T * g.C; return WFQ_OK;
        case WFQ_BUF_SX:
            if (!plan->has_workspace) return WFQ_ERR_NOT_PREPARED;
            *dev_ptr = plan->ws.sX; *bytes = (size_t)g.P * g.G * g.Ts * sizeof(float); return WFQ_OK;
        case WFQ_BUF_Y:
            if (!plan->has_workspace) return WFQ_ERR_NOT_PREPARED;
            *dev_ptr = plan->ws.Y; *bytes = (size_t)g.P * g.K * g.Tp * sizeof(float); return WFQ_OK;
        case WFQ_BUF_WQ:
            if (!plan->prepared) return WFQ_ERR_NOT_PREPARED;
            *dev_ptr = plan->Wq; *bytes = (size_t)g.P * g.K * g.C; return WFQ_OK;
        case WFQ_BUF_SW:
            if (!plan->prepared) return WFQ_ERR_NOT_PREPARED;
            *dev_ptr = plan->sW; *bytes = (size_t)g.P * g.G * g.Kp * sizeof(float); return WFQ_OK;
        case WFQ_BUF_STATUS:
            if (!plan->status) return WFQ_ERR_NOT_PREPARED;
            *dev_ptr = plan->status; *bytes = 4 * sizeof(int); return WFQ_OK;
    }
    return WFQ_ERR_INVALID_ARG;
}

wfq_status_t wfq_check_device_status(wfq_plan_t *plan, void *stream, int *where)
{
    if (!plan) return WFQ_ERR_INVALID_ARG;
    if (!plan->status) return WFQ_ERR_NOT_PREPARED;
    int host[4] = {0, 0, 0, 0};
    cudaStream_t st = as_stream(stream);
    if (cudaMemcpyAsync(host, plan->status, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return WFQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return WFQ_ERR_CUDA;
    if (where) *where = host[1];
    return host[0] == 0 ? WFQ_OK : WFQ_ERR_TIMEOUT;
}

wfq_status_t wfq_plan_destroy(wfq_plan_t *plan)
{
    if (!plan) return WFQ_OK;
    for (int i = 0; i < 2; ++i) {
        if (plan->sub[i]) delete plan->sub[i];       // borrowed device memory: nothing to free
        if (plan->host_stream[i]) cudaStreamDestroy(plan->host_stream[i]);
    }
    for (int i = 0; i < 3; ++i)
        if (plan->host_event[i]) cudaEventDestroy(plan->host_event[i]);
    if (plan->borrowed) { delete plan; return WFQ_OK; }
    if (plan->Wq) cudaFree(plan->Wq);
    if (plan->sW) cudaFree(plan->sW);
    if (plan->status) cudaFree(plan->status);
    if (plan->x_stage) cudaFree(plan->x_stage);
    if (plan->y_stage) cudaFree(plan->y_stage);
    delete plan;
    return WFQ_OK;
}

}  // extern "C"
