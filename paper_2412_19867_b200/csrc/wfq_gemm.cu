// Winograd-domain contraction with per-group dequantization (Eq. quant-Y):
//   for every position p:  Y_p[t][k] = sum_g sX[p,g,t] * sW[p,g,k] * acc_g[t][k],
//   acc_g[t][k] = sum_{c in g} Xq_p[t][c] * Wq_p[k][c]     (int8 x int8 -> int32)
//
// Persistent, warp-specialised sm_100a kernel, one CTA per SM.  A unit of work is
// (position p, block of 128 rows, block of BN columns).  "Rows" are the 128 TMEM lanes
// of the accumulator: tiles in the normal orientation, output channels in the swapped
// one (used when there are few tiles, so that all 128 lanes carry real work); columns
// are the other of the two.  Both operands are K-major int8 (channels contiguous).
//   warp 0       TMA producer: 128 x 128 B of the row operand and BN x 128 B of the
//                column operand per stage (128-byte swizzle), ring of NSTAGES mbarriers
//   warp 1       allocates TMEM; one lane issues tcgen05.mma kind::i8 (M=128, N=BN,
//                K=32 per instruction).  Every channel group accumulates into its own
//                TMEM buffer (ring of NBUF) and is committed to an mbarrier when done
//   warp 2       scale loader: per group, 128 row scales and BN column scales go to a
//                shared-memory ring with two bulk copies
//   warps 4-19   epilogue: quarter = warp % 4 selects the 32 TMEM lanes the warp may
//                read, (warp - 4) / 4 selects BN/4 of the columns.  tcgen05.ld the
//                finished int32 group sums, release the buffer, convert and scale
//                into fp32 registers; after the last group write Y[p][k][t]
// The tensor pipe therefore runs groups g+1.. while the ALUs promote group g.
// Every wait is bounded; on expiry the CTA records where, stops, drains and frees TMEM.
#include "wfq_internal.h"
#include "wfq_ptx.cuh"

namespace wfq {

namespace {

constexpr int BM = 128;        // rows per unit (MMA M, TMEM lanes)
constexpr int BK = 128;        // bytes (= int8 channels) per pipeline stage
constexpr int UK = 32;         // channels per MMA instruction
constexpr int NSTAGES = 7;
constexpr int NBUF = 8;        // TMEM accumulator buffers
constexpr int NSC = 16;        // scale ring slots (one group each)
constexpr int A_BYTES = BM * BK;
constexpr int NUM_EPI_WARPS = 16;
constexpr int FIRST_EPI_WARP = 4;
constexpr int NUM_THREADS = 32 * (FIRST_EPI_WARP + NUM_EPI_WARPS);
constexpr long long WAIT_CYCLES = 2000000000LL;   // ~1 s at 2 GHz

struct Shared {
    uint64_t full[NSTAGES];
    uint64_t empty[NSTAGES];
    uint64_t tmem_full[NBUF];
    uint64_t tmem_empty[NBUF];
    uint64_t scale_full[NSC];
    uint64_t scale_empty[NSC];
    uint32_t tmem_base;
    volatile int abort;
};

template <int BN>
struct Cfg {
    static constexpr int B_BYTES = BN * BK;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int SCALE_FLOATS = BM + BN;              // per ring slot
    static constexpr int TMEM_COLS = NBUF * BN;               // 512 or 256: a power of two
    static constexpr int CW = BN / (NUM_EPI_WARPS / 4);       // columns per epilogue warp
    static constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)NSTAGES * STAGE_BYTES +
                                         (size_t)NSC * SCALE_FLOATS * sizeof(float) + sizeof(Shared);
};

// Bounded mbarrier wait.  Returns false (and records `where`) on timeout or when
// another role of this CTA already gave up.
__device__ __forceinline__ bool wait_bounded(uint32_t bar, uint32_t parity, Shared *sh, int *status,
                                             int where)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if (sh->abort) return false;
        if (clock64() - t0 > WAIT_CYCLES) {
            sh->abort = 1;
            if (atomicCAS(status, 0, (int)WFQ_ERR_TIMEOUT) == 0) {
                status[1] = where;
                status[2] = (int)blockIdx.x;
                status[3] = (int)parity;
            }
            return false;
        }
    }
}

template <int N>
__device__ __forceinline__ void tmem_ld_cols(uint32_t taddr, uint32_t (&r)[N])
{
    if constexpr (N == 16) ptx::tmem_ld_x16(taddr, r);
    else ptx::tmem_ld_x8(taddr, r);
}

struct GemmArgs {
    const float *row_scale;   // [P][G][row_pitch]: sX (normal) or sW (swapped)
    const float *col_scale;   // [P][G][col_pitch]: sW (normal) or sX (swapped)
    int row_pitch, col_pitch;
    int rows, cols;           // valid rows / columns: (T, K) normal, (K, T) swapped
    float *Y;                 // [P][K][Tp]
    int32_t *acc_dump;        // [P][T][K][G] or null
    int *status;
};

template <int BN, bool SWAP, bool DUMP>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_dequant_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    GemmArgs a, Geometry g)
{
    using C = Cfg<BN>;
    constexpr int CW = C::CW;
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment: the 128-byte swizzle atoms repeat every 1024 bytes
    unsigned char *tiles = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    float *scales = reinterpret_cast<float *>(tiles + (size_t)NSTAGES * C::STAGE_BYTES);
    Shared *sh = reinterpret_cast<Shared *>(scales + (size_t)NSC * C::SCALE_FLOATS);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int MT = (a.rows + BM - 1) / BM, NT = (a.cols + BN - 1) / BN;
    const int units = g.P * MT * NT;
    const int KB = (g.C + BK - 1) / BK;          // stages per unit
    const int gs_steps = g.gs / UK;              // MMAs per group
    int *status = a.status;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGES; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < NBUF; ++b) {
            ptx::mbar_init(ptx::smem_u32(&sh->tmem_full[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->tmem_empty[b]), NUM_EPI_WARPS);
        }
        for (int s = 0; s < NSC; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh->scale_full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->scale_empty[s]), NUM_EPI_WARPS);
        }
        sh->abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), C::TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    // everything above may overlap the tail of the kernel that produces Xq and sX
    ptx::grid_dependency_wait();

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (lane == 0) {
            ptx::prefetch_tmap(&tmA);
            ptx::prefetch_tmap(&tmB);
            int stage = 0;
            uint32_t phase = 0;
            long long issued = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
                const int nt = u % NT, mt = (u / NT) % MT, p = u / (NT * MT);
                for (int kb = 0; kb < KB; ++kb) {
                    if (!wait_bounded(ptx::smem_u32(&sh->empty[stage]), phase ^ 1u, sh, status,
                                      kWaitSmemEmpty)) { ok = false; break; }
                    const uint32_t bar = ptx::smem_u32(&sh->full[stage]);
                    const uint32_t a_dst = ptx::smem_u32(tiles + (size_t)stage * C::STAGE_BYTES);
                    ptx::mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
                    ptx::tma_load_3d(a_dst, &tmA, bar, kb * BK, mt * BM, p);
                    ptx::tma_load_3d(a_dst + A_BYTES, &tmB, bar, kb * BK, nt * BN, p);
                    ++issued;
                    if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
                }
            }
            if (!ok) {
                // give copies still in flight a bounded time to land before the CTA exits
                int s = stage;
                uint32_t ph = phase;
                const long long n = issued < NSTAGES ? issued : NSTAGES;
                for (long long i = 0; i < n; ++i) {
                    if (--s < 0) { s = NSTAGES - 1; ph ^= 1u; }
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(ptx::smem_u32(&sh->full[s]), ph) &&
                           clock64() - t0 < WAIT_CYCLES / 16) { }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_i8(BM, BN);
            int stage = 0, buf = 0;
            uint32_t phase = 0, tphase = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
                int step_in_group = 0;
                for (int kb = 0; kb < KB && ok; ++kb) {
                    if (!wait_bounded(ptx::smem_u32(&sh->full[stage]), phase, sh, status, kWaitSmemFull)) {
                        ok = false; break;
                    }
                    ptx::tc_fence_after();
                    const uint32_t a_addr = ptx::smem_u32(tiles + (size_t)stage * C::STAGE_BYTES);
                    const uint64_t a_desc = ptx::smem_desc_sw128(a_addr);
                    const uint64_t b_desc = ptx::smem_desc_sw128(a_addr + A_BYTES);
                    const int nslice = min(BK, g.C - kb * BK) / UK;
                    for (int s = 0; s < nslice; ++s) {
                        if (step_in_group == 0) {
                            if (!wait_bounded(ptx::smem_u32(&sh->tmem_empty[buf]), tphase ^ 1u, sh,
                                              status, kWaitTmemEmpty)) { ok = false; break; }
                            ptx::tc_fence_after();
                        }
                        // advancing the start address by 32 bytes (>>4 = 2) walks along K
                        // inside the swizzled 128-byte rows
                        ptx::umma_i8(tmem_base + (uint32_t)(buf * BN), a_desc + (uint64_t)(2 * s),
                                     b_desc + (uint64_t)(2 * s), idesc, step_in_group ? 1u : 0u);
                        if (++step_in_group == gs_steps) {
                            ptx::umma_commit(ptx::smem_u32(&sh->tmem_full[buf]));
                            step_in_group = 0;
                            if (++buf == NBUF) { buf = 0; tphase ^= 1u; }
                        }
                    }
                    ptx::umma_commit(ptx::smem_u32(&sh->empty[stage]));
                    if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
                }
            }
        }
    } else if (warp == 2) {
        // ---------------- scale loader ----------------
        if (lane == 0 && !DUMP) {
            int slot = 0;
            uint32_t sphase = 0;
            long long issued = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
                const int nt = u % NT, mt = (u / NT) % MT, p = u / (NT * MT);
                for (int grp = 0; grp < g.G; ++grp) {
                    if (!wait_bounded(ptx::smem_u32(&sh->scale_empty[slot]), sphase ^ 1u, sh, status,
                                      kWaitScaleEmpty)) { ok = false; break; }
                    const uint32_t bar = ptx::smem_u32(&sh->scale_full[slot]);
                    const uint32_t dst = ptx::smem_u32(scales + (size_t)slot * C::SCALE_FLOATS);
                    ptx::mbar_arrive_expect_tx(bar, C::SCALE_FLOATS * 4);
                    ptx::bulk_load(dst, a.row_scale + ((size_t)p * g.G + grp) * a.row_pitch + mt * BM,
                                   BM * 4, bar);
                    ptx::bulk_load(dst + BM * 4,
                                   a.col_scale + ((size_t)p * g.G + grp) * a.col_pitch + nt * BN,
                                   BN * 4, bar);
                    ++issued;
                    if (++slot == NSC) { slot = 0; sphase ^= 1u; }
                }
            }
            if (!ok) {
                int s = slot;
                uint32_t ph = sphase;
                const long long n = issued < NSC ? issued : NSC;
                for (long long i = 0; i < n; ++i) {
                    if (--s < 0) { s = NSC - 1; ph ^= 1u; }
                    const long long t0 = clock64();
                    while (!ptx::mbar_try_wait(ptx::smem_u32(&sh->scale_full[s]), ph) &&
                           clock64() - t0 < WAIT_CYCLES / 16) { }
                }
            }
        }
    } else if (warp >= FIRST_EPI_WARP) {
        // ---------------- epilogue ----------------
        const int quarter = warp & 3;                         // TMEM lanes this warp may read
        const int c0 = ((warp - FIRST_EPI_WARP) >> 2) * CW;   // first column of this warp
        int buf = 0, slot = 0;
        uint32_t tphase = 0, sphase = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
            const int nt = u % NT, mt = (u / NT) % MT, p = u / (NT * MT);
            const int row = mt * BM + quarter * 32 + lane;    // tile (normal) or channel (swapped)
            const int col0 = nt * BN + c0;
            // warp-uniform: does this warp own any valid row and column of the unit?
            const bool active = (mt * BM + quarter * 32 < a.rows) && (col0 < a.cols);
            const bool row_ok = row < a.rows;
            float acc[CW];
#pragma unroll
            for (int j = 0; j < CW; ++j) acc[j] = 0.f;
            for (int grp = 0; grp < g.G; ++grp) {
                if (!wait_bounded(ptx::smem_u32(&sh->tmem_full[buf]), tphase, sh, status, kWaitTmemFull)) {
                    ok = false; break;
                }
                uint32_t r[CW];
                if (active) {
                    ptx::tc_fence_after();
                    const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) +
                                           (uint32_t)(buf * BN + c0);
                    tmem_ld_cols<CW>(taddr, r);
                    ptx::tmem_ld_wait();
                    ptx::tc_fence_before();
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->tmem_empty[buf]));
                if (++buf == NBUF) { buf = 0; tphase ^= 1u; }

                if constexpr (DUMP) {
                    if (active && row_ok) {
#pragma unroll
                        for (int j = 0; j < CW; ++j) {
                            const int col = col0 + j;
                            if (col < a.cols) {
                                const size_t t = SWAP ? col : row, k = SWAP ? row : col;
                                a.acc_dump[(((size_t)p * g.T + t) * g.K + k) * g.G + grp] = (int32_t)r[j];
                            }
                        }
                    }
                } else {
                    if (!wait_bounded(ptx::smem_u32(&sh->scale_full[slot]), sphase, sh, status,
                                      kWaitScaleFull)) { ok = false; break; }
                    if (active) {
                        const float *sc = scales + (size_t)slot * C::SCALE_FLOATS;
                        const float rs = sc[quarter * 32 + lane];
                        const float4 *cs4 = reinterpret_cast<const float4 *>(sc + BM + c0);
#pragma unroll
                        for (int j4 = 0; j4 < CW / 4; ++j4) {
                            const float4 cs = cs4[j4];
                            acc[4 * j4 + 0] = fmaf(__int2float_rn((int32_t)r[4 * j4 + 0]) * rs, cs.x, acc[4 * j4 + 0]);
                            acc[4 * j4 + 1] = fmaf(__int2float_rn((int32_t)r[4 * j4 + 1]) * rs, cs.y, acc[4 * j4 + 1]);
                            acc[4 * j4 + 2] = fmaf(__int2float_rn((int32_t)r[4 * j4 + 2]) * rs, cs.z, acc[4 * j4 + 2]);
                            acc[4 * j4 + 3] = fmaf(__int2float_rn((int32_t)r[4 * j4 + 3]) * rs, cs.w, acc[4 * j4 + 3]);
                        }
                    }
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->scale_empty[slot]));
                    if (++slot == NSC) { slot = 0; sphase ^= 1u; }
                }
            }
            if constexpr (!DUMP) {
                if (ok && active && row_ok) {
                    if constexpr (SWAP) {
                        // row = output channel, columns = tiles: contiguous in Y[p][k][:]
                        float *dst = a.Y + ((size_t)p * g.K + row) * g.Tp + col0;
#pragma unroll
                        for (int j4 = 0; j4 < CW / 4; ++j4)
                            if (col0 + 4 * j4 + 3 < g.Tp)
                                *reinterpret_cast<float4 *>(dst + 4 * j4) =
                                    make_float4(acc[4 * j4], acc[4 * j4 + 1], acc[4 * j4 + 2], acc[4 * j4 + 3]);
                    } else {
                        // row = tile: lanes write consecutive t of one Y[p][k][:] row
                        float *dst = a.Y + ((size_t)p * g.K + col0) * g.Tp + row;
#pragma unroll
                        for (int j = 0; j < CW; ++j)
                            if (col0 + j < a.cols) dst[(size_t)j * g.Tp] = acc[j];
                    }
                }
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

template <int BN, bool SWAP, bool DUMP>
cudaError_t launch_variant(const wfq_plan &plan, int32_t *acc_dump, cudaStream_t stream, bool pdl)
{
    using C = Cfg<BN>;
    const Geometry &g = plan.geo;
    GemmArgs a;
    a.row_scale = SWAP ? plan.sW : plan.ws.sX;
    a.col_scale = SWAP ? plan.ws.sX : plan.sW;
    a.row_pitch = SWAP ? g.Kp : g.Ts;
    a.col_pitch = SWAP ? g.Ts : g.Kp;
    a.rows = SWAP ? g.K : g.T;
    a.cols = SWAP ? g.T : g.K;
    a.Y = plan.ws.Y;
    a.acc_dump = acc_dump;
    a.status = plan.status;
    const int MT = (a.rows + BM - 1) / BM, NT = (a.cols + BN - 1) / BN;
    const int units = g.P * MT * NT;
    const int grid = units < plan.sm_count ? units : plan.sm_count;
    auto kern = gemm_dequant_kernel<BN, SWAP, DUMP>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)C::SMEM_BYTES);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(NUM_THREADS);
    cfg.dynamicSmemBytes = C::SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    const CUtensorMap &tmA = SWAP ? plan.tmap_wq : plan.tmap_xq;
    const CUtensorMap &tmB = SWAP ? plan.tmap_xq : plan.tmap_wq;
    return cudaLaunchKernelEx(&cfg, kern, tmA, tmB, a, g);
}

}  // namespace

int gemm_block_m() { return BM; }

// Orientation and column block of the contraction for a layer: rows (TMEM lanes) are
// tiles unless the swapped orientation leaves less padded work.
void gemm_choose(const Geometry &g, bool *swap, int *bn)
{
    auto up = [](long long v, int b) { return (v + b - 1) / b * b; };
    const long long normal = up(g.T, BM) * up(g.K, 64);
    const int bn_sw = g.T <= 32 ? 32 : 64;
    const long long swapped = up(g.K, BM) * up(g.T, bn_sw);
    *swap = swapped < normal;
    *bn = *swap ? bn_sw : 64;
}

cudaError_t launch_gemm(const wfq_plan &plan, int32_t *acc_dump, cudaStream_t stream, bool pdl)
{
    const bool dump = acc_dump != nullptr;
    if (plan.gemm_swap) {
        if (plan.gemm_bn == 32)
            return dump ? launch_variant<32, true, true>(plan, acc_dump, stream, pdl)
                        : launch_variant<32, true, false>(plan, acc_dump, stream, pdl);
        return dump ? launch_variant<64, true, true>(plan, acc_dump, stream, pdl)
                    : launch_variant<64, true, false>(plan, acc_dump, stream, pdl);
    }
    return dump ? launch_variant<64, false, true>(plan, acc_dump, stream, pdl)
                : launch_variant<64, false, false>(plan, acc_dump, stream, pdl);
}

}  // namespace wfq
