// Internal declarations shared by the translation units of libwfq.so.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "wfq.h"

namespace wfq {

constexpr int kMaxN = 8;          // n = m + 2 <= 8
constexpr int kMaxP = kMaxN * kMaxN;

// Identifiers stored in the device status word when a bounded wait expires.
enum WaitId : int {
    kWaitSmemEmpty = 1,   // TMA producer waiting for a free pipeline stage
    kWaitSmemFull = 2,    // MMA issuer waiting for TMA data
    kWaitTmemEmpty = 3,   // MMA issuer waiting for a drained accumulator
    kWaitTmemFull = 4,    // epilogue waiting for a finished accumulator
    kWaitDrain = 5,       // teardown waiting for copies in flight
    kWaitScaleEmpty = 6,  // scale loader waiting for a free ring slot
    kWaitScaleFull = 7,   // epilogue waiting for a group's scales
    kWaitStripEmpty = 8,  // input transform: TMA producer waiting for a free strip buffer
    kWaitStripFull = 9,   // input transform: im2col warps waiting for a strip
    kWaitPairEmpty = 10,  // input transform: im2col warps waiting for a free operand tile
    kWaitPairFull = 11,   // input transform: MMA issuer waiting for operand tiles
    kWaitAccEmpty = 12,   // input transform: MMA issuer waiting for a drained accumulator
    kWaitAccFull = 13     // input transform: quantizer waiting for an accumulator
};

// Geometry and scale tables handed to the kernels by value.
struct Geometry {
    int N, C, K, H, W;
    int m, n, P;          // output tile, input tile, positions
    int TH, TW, T, Tp;    // tiles per column/row, total, T rounded up to 32 (row pitch of Y)
    int Ts, Kp;           // T and K rounded up to 128: row pitches of sX and sW
    int gs, G;            // channels per group, groups
};

// Per-position scale products, filled by the host in fp64 and rounded once.
struct ScaleTables {
    float in_scale[kMaxP];   // (sB_i/sBstd_i)*(sB_j/sBstd_j): applied after the
                             // standard-scaled integer/rational input transform
    float in_scale_lo[kMaxP];  // the part of that factor that in_scale lost to rounding: the
                             // kernels form X = fma(Z, in_scale, Z * in_scale_lo), which is the
                             // correctly rounded product with the unrounded factor in all but
                             // rare double-rounding cases (the quantizer's codes are sensitive
                             // to the last bit of X where a group holds an outlier)
    float out_scale[kMaxP];  // sA_i*sA_j: applied before the output transform
};

// Codes and scales of the two transform matrices for the fully quantized transforms
// (Eqs. quant-B and quant-y), built on the host from the plan's scale vectors.
struct FullQuantTables {
    int BTq[kMaxN * kMaxN];   // Q(S_B V_B / s_qB), [i][a], n x n
    int ATq[kMaxN * kMaxN];   // Q(V_A S_A / s_qA), [u][i], m x n at row pitch n
    double sqB2;              // s_qB^2
    double sqA;               // s_qA
};

// Launch parameters of the cp.async input-transform kernel (any dtype, any shape),
// computed once per plan.
struct K1Params {
    int TB;            // tiles per work item
    int NCH;           // chunks of TB tiles per tile row
    int NCB;           // channel blocks (C / CB)
    int items;         // work items: N * TH * NCH * NCB
    int CB;            // channels per work item (a multiple of the group size)
    int CS;            // shared-memory channel stride of the strip (elements)
    int strip_bytes;   // bytes of the strip, rounded up to 16
    int pair;          // 1: rows can be copied as aligned element pairs
    int vec16;         // 1: rows are copied as aligned 16-byte pieces (fp16, W a multiple of 8, x 16-byte aligned)
    int dbuf;          // 1: two strip buffers, the next item is staged during this one
    int smem, grid;    // dynamic shared memory and CTAs of the launch
};

// Launch parameters of the tensor-core input-transform kernel (fp16 inputs, groups of 32
// or 64 channels, C a multiple of 64, shapes a TMA or bulk copy can stage).
struct K1TcPlan {
    bool use = false;
    int mode = 0;            // 0: 3-D tiled TMA (W, H, N*C); 1: 2-D tiled TMA (H*W, N*C); 2: bulk copy
    int TBW = 0, NCHUNK = 0, NCB = 0, items = 0;
    int CS = 0, RS = 0;      // strip strides in elements: channel, patch row
    int strip_bytes = 0, nstrip = 0, nbp = 0;
    int smem = 0, grid = 0;
    unsigned box[3] = {0, 0, 0};
};

struct Workspace {
    int8_t *Xq = nullptr;   // [P][T][C]
    float *sX = nullptr;    // [P][G][Ts]
    float *Y = nullptr;     // [P][K][Tp]
    size_t xq_bytes = 0, sx_bytes = 0, y_bytes = 0, total = 0;
};

}  // namespace wfq

struct wfq_plan {
    wfq::Geometry geo;
    wfq_dtype_t in_dtype = WFQ_F32;
    wfq::Workspace ws;
    bool has_workspace = false;
    bool prepared = false;
    int w_bits = 8;            // bit width of the filter codes (8 or 4); the stored codes are int8 either way
    int device = -1;
    int sm_count = 0;

    // plan-owned device memory
    int8_t *Wq = nullptr;      // [P][K][C]
    float *sW = nullptr;       // [P][G][Kp]
    int *status = nullptr;     // int32[4]
    const float *bias = nullptr;   // caller-owned fp32[K] added in the output transform, or null
    int act = 0;               // activation after the bias: 0 none, 1 ReLU, 2 SiLU
    int out_half = 0;          // y is written as fp32 (0), fp16 (1) or bf16 (2)
    void *x_stage = nullptr;   // staging for wfq_conv_forward_host
    float *y_stage = nullptr;

    double sB[wfq::kMaxN], sG[wfq::kMaxN], sA[wfq::kMaxN];
    wfq::ScaleTables tables;

    // launch parameters derived from the geometry, the dtype and the device (plan_launches)
    wfq::K1Params k1;          // 4-byte (or 2-byte) copies: any x
    wfq::K1Params k1v;         // 16-byte copies where the layer allows them (vec16 set), else a copy of k1
    wfq::K1Params k1n;         // NHWC input: one TMA box per work item
    bool in_nhwc = false;      // x is [N][H][W][C] instead of [N][C][H][W]
    CUtensorMap tmap_xn;       // the NHWC input as (C, W, H, N)
    const void *tmap_xn_base = nullptr;   // x pointer tmap_xn was encoded for
    CUtensorMap tmap_xn_tc;    // the same with the boxes of the tensor-core NHWC input transform
    const void *tmap_xn_tc_base = nullptr;
    wfq::K1TcPlan k1tc;
    CUtensorMap tmap_x;        // the input tensor as the tensor-core input transform stages it
    const void *tmap_x_base = nullptr;   // x pointer tmap_x was encoded for
    long long wait_cycles = 2000000000LL;   // limit of every device-side wait (~1 s)
    int debug_skip_item = -1;  // >= 0: the input transform's producer skips this work item
    int debug_skip_gemm_stage = -1;   // >= 0: the contraction's producer (CTA 0) skips this stage
    bool fq_input = false;     // input transform on integer codes (Eq. quant-B)
    int fq_output = 0;         // output transform: 0 fp32, 1 integer with one scale of Y per tile, 2 per row / column
    wfq::FullQuantTables fq;   // valid once the filters are prepared
    int k1_choice = 0;         // input-transform kernel: 0 automatic, 1 cp.async, 2 tensor cores where they apply,
                               // 3 cp.async without 16-byte copies

    CUtensorMap tmap_xq;       // Xq as (C, T, P) bytes, 128B-swizzled boxes
    CUtensorMap tmap_wq;       // Wq as (C, K, P)
    bool tmap_xq_ok = false, tmap_wq_ok = false;
    bool gemm_swap = false;    // contraction rows are output channels instead of tiles
    int gemm_bn = 64;          // columns per unit of the contraction

    // wfq_conv_forward_host on batches of several images: the batch is cut into chunks
    // of whole images that alternate between two internal streams, so that the copy in
    // of one chunk, the kernels of another and the copy out of a third overlap.  The two
    // sub-plans describe one chunk each; they borrow this plan's filters, scale tables,
    // status word and halves of its workspace.
    wfq_plan *sub[2] = {nullptr, nullptr};
    int host_chunks = 0;                     // 0: not decided yet, 1: no chunking
    cudaStream_t host_stream[2] = {nullptr, nullptr};
    cudaEvent_t host_event[3] = {nullptr, nullptr, nullptr};
    bool borrowed = false;                   // this is a sub-plan: it owns no device memory
};

namespace wfq {

// Kernel launchers (one per translation unit).  Each returns a cudaError_t from the
// launch; none synchronises.
cudaError_t launch_filter_prep(const wfq_plan &plan, const float *w_dev, float *scratch_w32,
                               cudaStream_t stream);
// 4-bit filter codes <-> two codes per byte (the exported blob's storage); n_codes a multiple of 8
cudaError_t launch_pack_nibbles(const int8_t *codes, void *packed, size_t n_codes, cudaStream_t stream);
cudaError_t launch_unpack_nibbles(const void *packed, int8_t *codes, size_t n_codes, cudaStream_t stream);
cudaError_t launch_input_transform(wfq_plan &plan, const void *x_dev, cudaStream_t stream);
cudaError_t launch_input_transform_tc(const wfq_plan &plan, const void *x_dev, cudaStream_t stream);
bool input_transform_tcn_applies(const wfq_plan &plan);
void input_transform_tcn_box(const wfq_plan &plan, unsigned (&box)[4]);
cudaError_t setup_input_transform_tcn();
cudaError_t launch_input_transform_tcn(const wfq_plan &plan, cudaStream_t stream);

// Per-plan launch parameters (host only, no device work) and per-device one-time kernel
// attributes (shared-memory sizes and carveouts).
void plan_input_transform(wfq_plan &plan);
void plan_input_transform_tc(wfq_plan &plan);
cudaError_t setup_input_transform();
cudaError_t setup_input_transform_tc();
cudaError_t setup_gemm();
cudaError_t setup_output_transform();

// General tiled tensor map (rank 2 or 3, no interleave, zero fill outside the tensor).
// `strides` are in bytes for dimensions 1.. (rank - 1 entries).
bool encode_tmap(CUtensorMap *map, CUtensorMapDataType dtype, int rank, const void *base,
                 const unsigned long long *dims, const unsigned long long *strides,
                 const unsigned *box, CUtensorMapSwizzle swizzle);
cudaError_t launch_gemm(const wfq_plan &plan, int32_t *acc_dump, cudaStream_t stream, bool pdl);
cudaError_t launch_output_transform(const wfq_plan &plan, float *y_dev, cudaStream_t stream, bool pdl);
void build_full_quant_tables(wfq_plan &plan);
cudaError_t setup_full_quant();
cudaError_t launch_input_transform_int(const wfq_plan &plan, const void *x_dev, cudaStream_t stream);
cudaError_t launch_output_transform_int(const wfq_plan &plan, float *y_dev, cudaStream_t stream);
cudaError_t launch_mma_peak(const wfq_plan &plan, int n_cols, int mmas, cudaStream_t stream);

// Builds a 3-D byte tensor map (inner extent `inner`, rows, planes) with a
// (128, box_rows, 1) box and 128-byte swizzle.  Returns false on failure.
bool encode_tmap_bytes3d(CUtensorMap *map, const void *base, int inner, int rows, int planes,
                         int box_rows);


// CTAs of `threads` threads and `smem` bytes of dynamic shared memory that fit on one SM of
// this part (228 KB of shared memory with 1 KB reserved per CTA, 64 K registers allocated in
// units of 256 per warp).  Used to size persistent grids; an overestimate only means that
// some CTAs start later.
template <typename Kernel>
inline int resident_ctas_per_sm(Kernel kern, int threads, size_t smem, int cap)
{
    cudaFuncAttributes fa;
    if (cudaFuncGetAttributes(&fa, kern) != cudaSuccess) return 1;
    const int warps = (threads + 31) / 32;
    const int regs_per_warp = (fa.numRegs * 32 + 255) / 256 * 256;
    int n = 65536 / (regs_per_warp * warps);
    const int by_smem = (int)((228 * 1024) / (smem + fa.sharedSizeBytes + 1024));
    if (by_smem < n) n = by_smem;
    if (2048 / threads < n) n = 2048 / threads;
    if (cap < n) n = cap;
    return n < 1 ? 1 : n;
}

int gemm_block_m();   // rows per unit of the contraction kernel (128)
void gemm_choose(const Geometry &g, bool *swap, int *bn);

}  // namespace wfq
