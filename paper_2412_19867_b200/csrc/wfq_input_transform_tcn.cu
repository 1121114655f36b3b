// Fused input transform + group-wise int8 quantization on the tensor cores for NHWC fp16 input.
//
//   X = S_B V_B x V_B^T S_B   (Section 4.1), then the quantizer of Section 2 with one scale per
//   (position, tile, group of consecutive input channels).
//
// As in wfq_input_transform_tc.cu the 2-D transform of a patch is one contraction with the constant
// matrix BT (x) BT (exact in fp16, products exact in fp32).  With the channels innermost in memory
// the patch data needs no rearrangement at all: a TMA box {64 channels, 8 columns, n rows} of one
// tile lands in shared memory as n x 8 rows of 128 bytes (one row per patch element, the 64 channels
// along the row, 128-byte swizzle), which is an MN-major B operand of tcgen05.mma kind::f16 with
// K = the patch elements (8 per patch row: for F(4,3) the two extra columns meet zero columns of the
// matrix) and N = the 64 channels.  Accumulator rows (TMEM lanes) = (tile of the work item, Winograd
// position), PL rows per tile: the A operand of tile t's MMAs is the constant matrix [position] x
// [patch element] with its rows at t * PL and zeros elsewhere.  Shared memory holds the matrix once,
// K-major, between (TB - 1) * PL zero rows and 128 - PL zero rows, and tile t's descriptor starts
// t * PL rows before the matrix (PL is a multiple of 8, so the 128-byte swizzle keeps its phase);
// only the matrix itself (5-8 KB) is copied from a global image the host builds.  A quantizer
// thread then owns one (tile, position) and reads its 64 channels with tcgen05.ld: abs-max over
// registers, scale, 64 contiguous codes; no im2col, no fp32 round trip through shared memory.
//
// A work item is TB tiles x one channel group of 64, 128 or 256 channels (or two groups of 32): a group of
// 128 / 256 channels is 2 / 4 boxes per tile whose MMAs fill neighbouring 64-column blocks of the same
// accumulator, and its quantizer threads take the abs-max over all those columns before the codes.
//
// Persistent CTAs, two per SM (one for groups of 256: two accumulators of 256 columns are all of tensor
// memory), 8 warps:
//   warp 0     TMA producer: per work item TB boxes (one per tile; tiles past the end of the tile
//              row are loaded all the same and come back as zeros) into a ring of three strips (two for
//              groups of 128 and 256)
//   warp 1     owns TMEM; one lane issues TB * n / 2 MMAs per box of channels (M = 128, N = 64, K = 16) into
//              one of two accumulators of 64, 128 or 256 columns, commits the accumulator and the strip
//   (warp 0 starts its first boxes right after the barrier initialisation; warps 1-7 meanwhile allocate
//   TMEM and build the A operand and meet at a named barrier of their own)
//   warps 4-7  quantizers: warp % 4 selects the 32 TMEM lanes; per-position factor, abs-max, scale,
//              codes, one 32-byte store per 32 codes
// All waits are bounded; on expiry the CTA records the wait, drains its copies and frees TMEM.
#include <cuda_fp16.h>

#include <cstring>
#include <vector>

#include "wfq_internal.h"
#include "wfq_ptx.cuh"
#include "wfq_quant.cuh"

namespace wfq {
namespace {

constexpr int TN_FIRST_QUANT = 4;   // warps 0-3: producer, MMA issuer, two idle; then the quantizer teams of four warps
constexpr int TN_CB = 64;             // channels per box = N of one MMA
constexpr int TN_MAX_NSTRIP = 3;      // strip ring (at most)
constexpr int TN_MAX_NACC = 4;        // accumulators (at most)

// GS = 0 stands for the tile-size-only constants (the constant matrix).  A work item covers one group
// of 64, 128 or 256 channels (NB boxes of 64 channels per tile, side by side in the accumulator), or
// two groups of 32.
template <int M, int GS = 64>
struct TnCfg {
    static constexpr int NB = GS > 64 ? GS / 64 : 1;          // boxes of 64 channels per tile
    static constexpr int ACC_COLS = NB * TN_CB;               // channels per work item = accumulator columns
    // Two accumulators and one quantizer team of four warps.  The code takes NACC accumulators and TEAMS
    // teams (team k quantizes the CTA's items k, k + TEAMS, ...); four accumulators with two teams and a
    // fourth strip were measured and change nothing: per-CTA timestamps show a box arriving every 1.3 us
    // whatever the number in flight (the boxes of the two CTAs of an SM arrive at about 28 KB/us, 4 TB/s
    // over the chip, three times the unique input bytes because neighbouring tiles' boxes overlap), with
    // the MMA issuer and the quantizers waiting for them.
    static constexpr int NACC = 2;
    static constexpr int TEAMS = 1;
    static constexpr int THREADS = 32 * (TN_FIRST_QUANT + 4 * TEAMS);
    static constexpr int TMEM_COLS = NACC * ACC_COLS;         // 128, 256 or 512
    static constexpr int NSTRIP = NB == 1 ? 3 : 2;
    static constexpr int CTAS_PER_SM = NB == 4 ? 1 : 2;       // by shared memory and (groups of 256) tensor memory
    static constexpr int NN = M + 2;
    static constexpr int P = NN * NN;
    static constexpr int TB = M == 6 ? 2 : 3;                 // tiles per work item
    static constexpr int PL = M == 6 ? 64 : 40;               // accumulator rows per tile (>= P, a multiple of 8)
    static constexpr int KT = NN * 8;                         // K elements per tile (8 columns per patch row), <= 64
    static constexpr int KSTEPS = KT / 16;                    // MMAs per tile
    static constexpr int Z0 = (TB - 1) * PL;                  // zero rows before the matrix
    static constexpr int A_ROWS = Z0 + 128;                   // zero rows, matrix, zero rows
    static constexpr int A_BYTES = (A_ROWS * 128 + 1023) / 1024 * 1024;   // rows of 64 fp16, 128-byte swizzle
    static constexpr int AMAT_BYTES = PL * 128;               // the matrix itself
    static constexpr int BOX_BYTES = NN * 8 * 128;            // one tile's box
    static constexpr int STRIP_BYTES = TB * NB * BOX_BYTES;
    static constexpr size_t SMEM_BYTES = 1024 + A_BYTES + NSTRIP * STRIP_BYTES;
};

struct TnShared {
    uint64_t strip_full[TN_MAX_NSTRIP];
    uint64_t strip_empty[TN_MAX_NSTRIP];
    uint64_t acc_full[TN_MAX_NACC];
    uint64_t acc_empty[TN_MAX_NACC];
    uint32_t tmem_base;
    volatile int abort;
};

struct TnArgs {
    int8_t *Xq;
    float *sX;
    int *status;
    long long wait_cycles;
    const uint4 *amat;        // the constant matrix as it lies in shared memory, AMAT_BYTES
    int NCH, NCB, items;      // chunks of TB tiles per tile row, channel blocks, work items
    int debug_skip_item;      // >= 0: the producer skips this item's copies (exercises the bounded waits)
};

template <int M, int GS>
__global__ void __launch_bounds__((TnCfg<M, GS>::THREADS), 2)
input_transform_tcn_kernel(const __grid_constant__ CUtensorMap tmx, TnArgs a, Geometry g, ScaleTables tab)
{
    using C = TnCfg<M, GS>;
    constexpr int TN_NSTRIP = C::NSTRIP, TN_NACC = C::NACC, TN_TEAMS = C::TEAMS, TN_THREADS = C::THREADS;
    extern __shared__ unsigned char smem_dyn[];
    __shared__ TnShared sh;
    unsigned char *base = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);     // swizzle atoms repeat every 1024 B
    unsigned char *amat_s = base;
    unsigned char *strips = base + C::A_BYTES;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const WaitCtx ctx{&sh.abort, a.status, a.wait_cycles};

    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (threadIdx.x == 0) {
        for (int s = 0; s < TN_NSTRIP; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh.strip_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.strip_empty[s]), 1);
        }
        for (int s = 0; s < TN_NACC; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh.acc_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh.acc_empty[s]), 4);
        }
        sh.abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmx);
    }
    __syncthreads();                    // the barriers exist
    uint32_t tmem_base = 0;
    if (warp == 0) {
        // the producer needs neither the A operand nor TMEM: its first boxes are in flight while the
        // other warps set those up
        asm volatile("griddepcontrol.wait;" ::: "memory");
    } else {
        if (warp == 1) {
            ptx::tmem_alloc(ptx::smem_u32(&sh.tmem_base), C::TMEM_COLS);
            ptx::tmem_relinquish();
        }
        // the A operand: zero rows, the constant matrix (a plain copy; it does not depend on the previous
        // kernel), zero rows
        for (int i = threadIdx.x - 32; i < C::A_BYTES / 16; i += TN_THREADS - 32) {
            const int j = i - C::Z0 * 8;                           // 16-byte pieces: 8 per row
            reinterpret_cast<uint4 *>(amat_s)[i] =
                (j >= 0 && j < C::AMAT_BYTES / 16) ? __ldg(a.amat + j) : make_uint4(0u, 0u, 0u, 0u);
        }
        ptx::fence_proxy_async_smem();      // the tensor cores read it through the async proxy
        ptx::tc_fence_before();
        asm volatile("bar.sync 1, %0;" ::"n"(TN_THREADS - 32) : "memory");      // warps 1 ..: operand and TMEM ready
        ptx::tc_fence_after();
        tmem_base = sh.tmem_base;
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }

    const int stride = (int)gridDim.x;
    if (warp == 0) {
        // ---------------- TMA producer ----------------
        int sb = 0;
        uint32_t phase = 0;
        long long issued = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < a.items && ok; item += stride) {
            ok = __all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh.strip_empty[sb]), phase ^ 1u, ctx,
                                                      kWaitStripEmpty));
            if (!ok) break;
            if (lane == 0 && item != a.debug_skip_item) {
                const int cblk = item % a.NCB, rest = item / a.NCB;
                const int srow = rest / a.NCH, chunk = rest - srow * a.NCH;
                const int img = srow / g.TH, th = srow - img * g.TH;
                const uint32_t bar = ptx::smem_u32(&sh.strip_full[sb]);
                ptx::mbar_arrive_expect_tx(bar, (uint32_t)C::STRIP_BYTES);
#pragma unroll
                for (int tl = 0; tl < C::TB; ++tl)
#pragma unroll
                    for (int nb = 0; nb < C::NB; ++nb)
                        ptx::tma_load_4d(
                            ptx::smem_u32(strips + sb * C::STRIP_BYTES + (tl * C::NB + nb) * C::BOX_BYTES), &tmx, bar,
                            cblk * C::ACC_COLS + nb * TN_CB, (chunk * C::TB + tl) * M - 1, th * M - 1, img);
            }
            __syncwarp();
            ++issued;
            if (++sb == TN_NSTRIP) { sb = 0; phase ^= 1u; }
        }
        if (!ok) {
            int s = sb;
            uint32_t ph = phase;
            const long long n = issued < TN_NSTRIP ? issued : TN_NSTRIP;
            for (long long i = 0; i < n; ++i) {
                if (--s < 0) { s = TN_NSTRIP - 1; ph ^= 1u; }
                drain(ptx::smem_u32(&sh.strip_full[s]), ph, a.wait_cycles / 16);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        constexpr uint32_t idesc = ptx::idesc_f16(128, TN_CB) | (1u << 16);     // B is MN-major
        constexpr uint32_t dhi = ptx::smem_desc_sw128_hi();
        const uint32_t a_lo0 = ptx::smem_desc_sw128_lo(ptx::smem_u32(amat_s));
        const uint32_t s_lo0 = ptx::smem_desc_sw128_lo(ptx::smem_u32(strips));
        int sb = 0, slot = 0;
        uint32_t phase = 0, aphase = 0;
        for (int item = blockIdx.x; item < a.items; item += stride) {
            if (!__all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh.strip_full[sb]), phase, ctx, kWaitStripFull)))
                break;
            if (!__all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh.acc_empty[slot]), aphase ^ 1u, ctx,
                                                      kWaitAccEmpty)))
                break;
            ptx::tc_fence_after();
            if (lane == 0) {
                const uint32_t b_lo = s_lo0 + (uint32_t)((sb * C::STRIP_BYTES) >> 4);
#pragma unroll
                for (int nb = 0; nb < C::NB; ++nb) {              // 64 accumulator columns per box of channels
                    const uint32_t d = tmem_base + (uint32_t)(slot * C::ACC_COLS + nb * TN_CB);
#pragma unroll
                    for (int tl = 0; tl < C::TB; ++tl)
#pragma unroll
                        for (int ks = 0; ks < C::KSTEPS; ++ks) {
                            // the matrix's rows land on accumulator rows tl * PL ...: start tl * PL rows early
                            const uint32_t al = a_lo0 + (uint32_t)(((C::Z0 - tl * C::PL) * 128 + ks * 32) >> 4);
                            const uint32_t bl =
                                b_lo + (uint32_t)(((tl * C::NB + nb) * C::BOX_BYTES + ks * 2048) >> 4);
                            if (tl == 0 && ks == 0) ptx::umma_f16_lo<false>(d, al, bl, dhi, idesc);
                            else ptx::umma_f16_lo<true>(d, al, bl, dhi, idesc);
                        }
                }
                ptx::umma_commit(ptx::smem_u32(&sh.acc_full[slot]));
                ptx::umma_commit(ptx::smem_u32(&sh.strip_empty[sb]));
            }
            __syncwarp();
            if (++sb == TN_NSTRIP) { sb = 0; phase ^= 1u; }
            if (++slot == TN_NACC) { slot = 0; aphase ^= 1u; }
        }
    } else if (warp >= TN_FIRST_QUANT) {
        // ---------------- quantizers ----------------
        const int quarter = warp & 3;
        const int r = quarter * 32 + lane;                    // accumulator row = tile * P + position
        const int tl = r / C::PL, p = r - tl * C::PL;
        const bool row_ok = tl < C::TB && p < C::P;
        const float sp = row_ok ? tab.in_scale[p] : 0.f, sl = row_ok ? tab.in_scale_lo[p] : 0.f;
        const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16);
        // one team: both accumulators in turn; two teams: team k owns accumulator k
        // the CTA's j-th item uses accumulator j % NACC; team k takes j = k, k + TEAMS, ...
        const int team = (warp - TN_FIRST_QUANT) >> 2;
        int j = team;
        for (int item = blockIdx.x + team * stride; item < a.items; item += TN_TEAMS * stride, j += TN_TEAMS) {
            const int slot = j % TN_NACC;
            const uint32_t aphase = (uint32_t)(j / TN_NACC) & 1u;
            if (!wait_bounded(ptx::smem_u32(&sh.acc_full[slot]), aphase, ctx, kWaitAccFull)) break;
            ptx::tc_fence_after();
            const int cblk = item % a.NCB, rest = item / a.NCB;
            const int srow = rest / a.NCH, chunk = rest - srow * a.NCH;
            const int tw = chunk * C::TB + tl;
            const bool valid = row_ok && tw < g.TW;
            const int t = srow * g.TW + tw;
            const uint32_t taddr = taddr0 + (uint32_t)(slot * C::ACC_COLS);
            int8_t *dst = a.Xq + ((size_t)p * g.T + t) * g.C + cblk * C::ACC_COLS;
            uint32_t v[32];
            if (GS == 32) {
                float *sd = a.sX + ((size_t)p * g.G + cblk * 2) * g.Ts + t;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    ptx::tmem_ld_x32(taddr + (uint32_t)(32 * h), v);
                    ptx::tmem_ld_wait();
                    if (h == 1) {          // both halves are in registers or done: release the accumulator
                        ptx::tc_fence_before();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.acc_empty[slot]));
                    }
                    float scale, inv;
                    group_scale_inv(fabsf(scaled(absmax32(v, 0.f), sp, sl)), scale, inv);
                    if (valid) {
                        codes32(v, sp, sl, inv, dst + 32 * h);
                        sd[(size_t)h * g.Ts] = scale;
                    }
                }
            } else if (GS > 64) {
                // a group of 128 or 256 channels: abs-max over all its columns, then every 32 columns
                // again from TMEM for the codes
                float m = 0.f;
#pragma unroll
                for (int c = 0; c < C::ACC_COLS / 32; ++c) {
                    ptx::tmem_ld_x32(taddr + (uint32_t)(32 * c), v);
                    ptx::tmem_ld_wait();
                    m = absmax32(v, m);
                }
                float scale, inv;
                group_scale_inv(fabsf(scaled(m, sp, sl)), scale, inv);
                if (valid) a.sX[((size_t)p * g.G + cblk) * g.Ts + t] = scale;
#pragma unroll
                for (int c = 0; c < C::ACC_COLS / 32; ++c) {
                    ptx::tmem_ld_x32(taddr + (uint32_t)(32 * c), v);
                    ptx::tmem_ld_wait();
                    if (c == C::ACC_COLS / 32 - 1) {
                        ptx::tc_fence_before();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.acc_empty[slot]));
                    }
                    if (valid) codes32(v, sp, sl, inv, dst + 32 * c);
                }
            } else {
                // abs-max over both halves, codes for the second half from the registers, then the
                // first half again from TMEM
                ptx::tmem_ld_x32(taddr, v);
                ptx::tmem_ld_wait();
                const float m = absmax32(v, 0.f);
                ptx::tmem_ld_x32(taddr + 32u, v);
                ptx::tmem_ld_wait();
                float scale, inv;
                group_scale_inv(fabsf(scaled(absmax32(v, m), sp, sl)), scale, inv);
                if (valid) {
                    codes32(v, sp, sl, inv, dst + 32);
                    a.sX[((size_t)p * g.G + cblk) * g.Ts + t] = scale;
                }
                ptx::tmem_ld_x32(taddr, v);
                ptx::tmem_ld_wait();
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh.acc_empty[slot]));
                if (valid) codes32(v, sp, sl, inv, dst);
            }
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

// The standard-scaled B^T of the paper's supplementary ("Standard Winograd transforms").
const float kTnBT4[36] = {4, 0, -5, 0, 1, 0,   0, -4, -4, 1, 1, 0,   0, 4, -4, -1, 1, 0,
                          0, -2, -1, 2, 1, 0,  0, 2, -1, -2, 1, 0,   0, 4, 0, -5, 0, 1};
const float kTnBT6[64] = {
    1, 0, -5.25f, 0, 5.25f, 0, -1, 0,        0, 1, 1, -4.25f, -4.25f, 1, 1, 0,
    0, -1, 1, 4.25f, -4.25f, -1, 1, 0,       0, 0.5f, 0.25f, -2.5f, -1.25f, 2, 1, 0,
    0, -0.5f, 0.25f, 2.5f, -1.25f, -2, 1, 0, 0, 2, 4, -2.5f, -5, 0.5f, 1, 0,
    0, -2, 4, 2.5f, -5, -0.5f, 1, 0,         0, -1, 0, 5.25f, 0, -5.25f, 0, 1};

// The constant matrix as it lies in shared memory: [PL rows][64 fp16], K-major with the 128-byte
// swizzle (16-byte chunk c of row r is stored at chunk c ^ (r & 7); the matrix starts at a multiple of
// 8 rows).  Row (i, j), K element a * 8 + b holds BT[i][a] * BT[j][b] (b < n); everything else is zero.
template <int M>
void build_amat(std::vector<uint16_t> &out)
{
    using C = TnCfg<M>;
    const float *bt = M == 6 ? kTnBT6 : kTnBT4;
    out.assign((size_t)C::AMAT_BYTES / 2, 0);
    for (int p = 0; p < C::P; ++p) {
        const int i = p / C::NN, j = p % C::NN;
        for (int aa = 0; aa < C::NN; ++aa)
            for (int b = 0; b < C::NN; ++b) {
                const int k = aa * 8 + b;
                const int chunk = (k / 8) ^ (p & 7);
                const __half h = __float2half_rn(bt[i * C::NN + aa] * bt[j * C::NN + b]);
                uint16_t bits;
                memcpy(&bits, &h, 2);
                out[(size_t)p * 64 + chunk * 8 + (k % 8)] = bits;
            }
    }
}

constexpr int kTnMaxDevices = 64;
void *g_tn_amat[kTnMaxDevices][2];

template <int M, int GS>
cudaError_t launch_tn(const wfq_plan &plan, cudaStream_t stream)
{
    using C = TnCfg<M, GS>;
    const Geometry &g = plan.geo;
    TnArgs a;
    a.Xq = plan.ws.Xq;
    a.sX = plan.ws.sX;
    a.status = plan.status;
    a.wait_cycles = plan.wait_cycles;
    a.amat = static_cast<const uint4 *>(g_tn_amat[plan.device][M == 6 ? 1 : 0]);
    a.NCH = (g.TW + C::TB - 1) / C::TB;
    a.NCB = g.C / C::ACC_COLS;
    a.items = g.N * g.TH * a.NCH * a.NCB;
    a.debug_skip_item = plan.debug_skip_item;
    if (!a.amat) return cudaErrorInvalidValue;
    const int slots = C::CTAS_PER_SM * plan.sm_count;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(a.items < slots ? a.items : slots));
    cfg.blockDim = dim3(C::THREADS);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, input_transform_tcn_kernel<M, GS>, plan.tmap_xn_tc, a, g, plan.tables);
}

}  // namespace

// Does the tensor-core NHWC kernel serve this plan?  fp16, groups of 32, 64, 128 or 256, channels in blocks
// of 64, the paper's two tile sizes.
bool input_transform_tcn_applies(const wfq_plan &plan)
{
    const Geometry &g = plan.geo;
    return plan.in_dtype == WFQ_F16 && (g.gs == 32 || g.gs == 64 || g.gs == 128 || g.gs == 256) && g.C % TN_CB == 0 && (g.m == 4 || g.m == 6);
}

// Box of the input tensor map for this kernel: {64 channels, 8 columns, n rows, 1 image}, 128-byte swizzle.
void input_transform_tcn_box(const wfq_plan &plan, unsigned (&box)[4])
{
    box[0] = TN_CB; box[1] = 8; box[2] = (unsigned)plan.geo.n; box[3] = 1;
}

// Per-device set-up: kernel attributes and the constant matrices in global memory.
cudaError_t setup_input_transform_tcn()
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kTnMaxDevices) return cudaErrorInvalidDevice;
    auto attr = [](auto kern, size_t smem) {
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    };
    if ((e = attr(input_transform_tcn_kernel<4, 32>, TnCfg<4, 32>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = attr(input_transform_tcn_kernel<4, 64>, TnCfg<4, 64>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = attr(input_transform_tcn_kernel<4, 128>, TnCfg<4, 128>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = attr(input_transform_tcn_kernel<4, 256>, TnCfg<4, 256>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = attr(input_transform_tcn_kernel<6, 32>, TnCfg<6, 32>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = attr(input_transform_tcn_kernel<6, 64>, TnCfg<6, 64>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = attr(input_transform_tcn_kernel<6, 128>, TnCfg<6, 128>::SMEM_BYTES)) != cudaSuccess) return e;
    if ((e = attr(input_transform_tcn_kernel<6, 256>, TnCfg<6, 256>::SMEM_BYTES)) != cudaSuccess) return e;
    if (!g_tn_amat[dev][0]) {
        std::vector<uint16_t> a4, a6;
        build_amat<4>(a4);
        build_amat<6>(a6);
        char *buf = nullptr;
        if ((e = cudaMalloc(&buf, (a4.size() + a6.size()) * 2)) != cudaSuccess) return e;
        if ((e = cudaMemcpy(buf, a4.data(), a4.size() * 2, cudaMemcpyHostToDevice)) != cudaSuccess) return e;
        if ((e = cudaMemcpy(buf + a4.size() * 2, a6.data(), a6.size() * 2, cudaMemcpyHostToDevice)) != cudaSuccess)
            return e;
        g_tn_amat[dev][0] = buf;
        g_tn_amat[dev][1] = buf + a4.size() * 2;
    }
    return cudaSuccess;
}

cudaError_t launch_input_transform_tcn(const wfq_plan &plan, cudaStream_t stream)
{
    const int gs = plan.geo.gs;
    if (plan.geo.m == 4)
        return gs == 32 ? launch_tn<4, 32>(plan, stream) : gs == 64 ? launch_tn<4, 64>(plan, stream)
             : gs == 128 ? launch_tn<4, 128>(plan, stream) : launch_tn<4, 256>(plan, stream);
    return gs == 32 ? launch_tn<6, 32>(plan, stream) : gs == 64 ? launch_tn<6, 64>(plan, stream)
         : gs == 128 ? launch_tn<6, 128>(plan, stream) : launch_tn<6, 256>(plan, stream);
}

}  // namespace wfq
