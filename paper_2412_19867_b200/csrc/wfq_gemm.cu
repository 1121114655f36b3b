// Winograd-domain contraction with per-group dequantization (Eq. quant-Y):
//   for every position p:  Y_p[t][k] = sum_g sX[p,g,t] * sW[p,g,k] * acc_g[t][k],
//   acc_g[t][k] = sum_{c in g} Xq_p[t][c] * Wq_p[k][c]     (int8 x int8 -> int32)
//
// Persistent, warp-specialised sm_100a kernel.  One CTA works through units
// (p, 128-tile block, BN-channel block):
//   warp 0      TMA producer: 128 x 128 B of Xq and BN x 128 B of Wq per stage
//               (128-byte swizzle), NSTAGES-deep ring of mbarriers
//   warp 1      allocates TMEM; one lane issues tcgen05.mma kind::i8 (M=128, N=BN,
//               K=32 per instruction).  Each channel group accumulates into its own
//               TMEM buffer (ring of NBUF), committed to an mbarrier when complete
//   warps 2-5   epilogue: tcgen05.ld the finished int32 group sums (TMEM lane = tile
//               row), release the buffer, convert and scale into fp32 registers;
//               after the last group write Y[p][k][t] (lanes along t: coalesced)
// The tensor pipe therefore runs group g+1.. while the ALUs promote group g.
// Every wait is bounded; on expiry the CTA records where, stops, drains and frees TMEM.
#include "wfq_internal.h"
#include "wfq_ptx.cuh"

namespace wfq {

namespace {

constexpr int BM = 128;        // tiles per unit (MMA M, TMEM lanes)
constexpr int BN = 64;         // output channels per unit (MMA N, TMEM columns per buffer)
constexpr int BK = 128;        // bytes (= int8 channels) per pipeline stage
constexpr int UK = 32;         // channels per MMA instruction
constexpr int NSTAGES = 6;
constexpr int NBUF = 4;        // TMEM accumulator buffers
constexpr int TMEM_COLS = NBUF * BN;   // 256, a power of two >= 32
constexpr int A_BYTES = BM * BK;
constexpr int B_BYTES = BN * BK;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int NUM_EPI_WARPS = 4;
constexpr int NUM_THREADS = 32 * (2 + NUM_EPI_WARPS);
constexpr long long WAIT_CYCLES = 2000000000LL;   // ~1 s at 2 GHz

struct Shared {
    uint64_t full[NSTAGES];
    uint64_t empty[NSTAGES];
    uint64_t tmem_full[NBUF];
    uint64_t tmem_empty[NBUF];
    uint32_t tmem_base;
    volatile int abort;
};

constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)NSTAGES * STAGE_BYTES + sizeof(Shared);

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

template <bool DUMP>
__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_dequant_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                    const float *__restrict__ sX, const float *__restrict__ sW, float *__restrict__ Y,
                    int32_t *__restrict__ acc_dump, int *status, Geometry g)
{
    extern __shared__ unsigned char smem_raw[];
    // 1024-byte alignment: the 128-byte swizzle atoms repeat every 1024 bytes
    unsigned char *tiles = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    Shared *sh = reinterpret_cast<Shared *>(tiles + (size_t)NSTAGES * STAGE_BYTES);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int MT = (g.T + BM - 1) / BM, NT = (g.K + BN - 1) / BN;
    const int units = g.P * MT * NT;
    const int KB = (g.C + BK - 1) / BK;          // stages per unit
    const int gs_steps = g.gs / UK;              // MMAs per group

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGES; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < NBUF; ++b) {
            ptx::mbar_init(ptx::smem_u32(&sh->tmem_full[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->tmem_empty[b]), NUM_EPI_WARPS);
        }
        sh->abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

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
                    const uint32_t a_dst = ptx::smem_u32(tiles + (size_t)stage * STAGE_BYTES);
                    ptx::mbar_arrive_expect_tx(bar, STAGE_BYTES);
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
                    const uint32_t a_addr = ptx::smem_u32(tiles + (size_t)stage * STAGE_BYTES);
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
    } else {
        // ---------------- epilogue ----------------
        const int quarter = warp & 3;                 // TMEM lanes this warp may read
        int buf = 0;
        uint32_t tphase = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
            const int nt = u % NT, mt = (u / NT) % MT, p = u / (NT * MT);
            const int t = mt * BM + quarter * 32 + lane;
            const bool t_ok = t < g.T;
            const int k0 = nt * BN;
            float acc[BN];
#pragma unroll
            for (int j = 0; j < BN; ++j) acc[j] = 0.f;
            for (int grp = 0; grp < g.G; ++grp) {
                if (!wait_bounded(ptx::smem_u32(&sh->tmem_full[buf]), tphase, sh, status, kWaitTmemFull)) {
                    ok = false; break;
                }
                ptx::tc_fence_after();
                uint32_t r[BN];
                const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * BN);
#pragma unroll
                for (int c = 0; c < BN / 32; ++c)
                    ptx::tmem_ld_x32(taddr + (uint32_t)(c * 32), *reinterpret_cast<uint32_t(*)[32]>(&r[c * 32]));
                ptx::tmem_ld_wait();
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->tmem_empty[buf]));
                if (++buf == NBUF) { buf = 0; tphase ^= 1u; }

                if constexpr (DUMP) {
                    if (t_ok) {
#pragma unroll
                        for (int j = 0; j < BN; ++j)
                            if (k0 + j < g.K)
                                acc_dump[(((size_t)p * g.T + t) * g.K + (k0 + j)) * g.G + grp] = (int32_t)r[j];
                    }
                } else {
                    const float sx = t_ok ? __ldg(sX + ((size_t)p * g.G + grp) * g.T + t) : 0.f;
                    const float *swp = sW + ((size_t)p * g.G + grp) * g.K + k0;
#pragma unroll
                    for (int j = 0; j < BN; ++j) {
                        const float sw = (k0 + j < g.K) ? __ldg(swp + j) : 0.f;
                        acc[j] = fmaf(__int2float_rn((int32_t)r[j]) * sx, sw, acc[j]);
                    }
                }
            }
            if constexpr (!DUMP) {
                if (ok && t_ok) {
                    float *dst = Y + ((size_t)p * g.K + k0) * g.Tp + t;
#pragma unroll
                    for (int j = 0; j < BN; ++j)
                        if (k0 + j < g.K) dst[(size_t)j * g.Tp] = acc[j];
                }
            }
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

}  // namespace

int gemm_block_n() { return BN; }
int gemm_block_m() { return BM; }

cudaError_t launch_gemm(const wfq_plan &plan, int32_t *acc_dump, cudaStream_t stream)
{
    const Geometry &g = plan.geo;
    const int MT = (g.T + BM - 1) / BM, NT = (g.K + BN - 1) / BN;
    const int units = g.P * MT * NT;
    const int grid = units < plan.sm_count ? units : plan.sm_count;
    cudaError_t e;
    if (acc_dump) {
        auto kern = gemm_dequant_kernel<true>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
        if (e != cudaSuccess) return e;
        kern<<<grid, NUM_THREADS, SMEM_BYTES, stream>>>(plan.tmap_xq, plan.tmap_wq, plan.ws.sX, plan.sW,
                                                       plan.ws.Y, acc_dump, plan.status, g);
    } else {
        auto kern = gemm_dequant_kernel<false>;
        e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES);
        if (e != cudaSuccess) return e;
        kern<<<grid, NUM_THREADS, SMEM_BYTES, stream>>>(plan.tmap_xq, plan.tmap_wq, plan.ws.sX, plan.sW,
                                                       plan.ws.Y, nullptr, plan.status, g);
    }
    return cudaGetLastError();
}

}  // namespace wfq
