// Winograd-domain contraction with per-group dequantization (Eq. quant-Y):
//   for every position p:  Y_p[t][k] = sum_g sX[p,g,t] * sW[p,g,k] * acc_g[t][k],
//   acc_g[t][k] = sum_{c in g} Xq_p[t][c] * Wq_p[k][c]     (int8 x int8 -> int32)
//
// Persistent, warp-specialised sm_100a kernel, two CTAs per SM.  A unit of work is
// (position p, block of 128 rows, block of BN columns).  "Rows" are the 128 TMEM lanes
// of the accumulator: tiles in the normal orientation, output channels in the swapped
// one (used when there are few tiles, so that all 128 lanes carry real work); columns
// are the other of the two.  Both operands are K-major int8 (channels contiguous).
//
// Every mbarrier hand-over costs the thread that makes it a few hundred cycles, so the
// roles synchronise per *chunk* of up to CG channel groups (128 channels when the group
// size divides 128), not per group.  A chunk owns one TMEM slot of 128 columns (its
// groups side by side, BN columns each) and one slot of the scale ring.
//   warp 0   TMA producer: 128 x 128 B of the row operand and BN x 128 B of the column
//            operand per stage (128-byte swizzle), ring of NSTAGES
//   warp 1   allocates TMEM; one lane issues tcgen05.mma kind::i8 (M=128, N=BN, K=32 per
//            instruction): waits for a stage and, at the start of a chunk, for its TMEM
//            slot; commits the stage back to the producer and the chunk to the epilogue
//   warp 2   scale loader: per chunk, 128 row scales and BN column scales per group into
//            the chunk's scale slot (bulk copies)
//   warps 4-7   epilogue: warp % 4 selects the 32 TMEM lanes the warp may read; each warp
//            handles all BN columns of its lanes.  Per chunk: wait for accumulators and
//            scales, then per group tcgen05.ld the int32 sums, convert and scale into fp32
//            registers (packed f32x2 multiply / fma), release the slot; after the last
//            chunk of a unit write Y[p][k][t].
// The second CTA of the SM runs the same pipeline on other units, which hides the
// hand-over latencies and overlaps one CTA's output stores with the other's arithmetic.
// Only four epilogue warps per CTA on purpose: the warp schedulers share issue slots
// evenly among ready warps, so every additional arithmetic warp slows the three
// single-purpose warps whose few instructions sit on the critical path (measured:
// 8 epilogue warps per CTA were 15-25 % slower).
// Every wait is bounded; on expiry the CTA records where, stops, drains and frees TMEM.
#include "wfq_internal.h"
#include "wfq_ptx.cuh"

namespace wfq {

namespace {

constexpr int BM = 128;        // rows per unit (MMA M, TMEM lanes)
constexpr int BK = 128;        // bytes (= int8 channels) per pipeline stage
constexpr int UK = 32;         // channels per MMA instruction
constexpr int NSTAGES = 4;     // shared-memory operand stages
constexpr int NSLOT = 2;       // TMEM / scale slots (chunks in flight)
constexpr int SLOT_COLS = 128; // TMEM columns per slot
constexpr int TMEM_COLS = NSLOT * SLOT_COLS;
constexpr int A_BYTES = BM * BK;
constexpr int NUM_EPI_WARPS = 4;
constexpr int FIRST_EPI_WARP = 4;
constexpr int NUM_THREADS = 32 * (FIRST_EPI_WARP + NUM_EPI_WARPS);

struct Shared {
    uint64_t full[NSTAGES];        // operands of a stage have landed
    uint64_t empty[NSTAGES];       // the MMAs reading a stage have completed
    uint64_t acc_full[NSLOT];      // the MMAs of a chunk have completed
    uint64_t slot_free[NSLOT];     // all epilogue warps are done with a chunk
    uint64_t scale_full[NSLOT];    // the scales of a chunk have landed
    uint32_t tmem_base;
    volatile int abort;
};

template <int BN>
struct Cfg {
    static constexpr int B_BYTES = BN * BK;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int CG_MAX = SLOT_COLS / BN;             // groups per chunk at most
    static constexpr int GROUP_SCALE_FLOATS = BM + BN;        // row scales, then column scales
    static constexpr int SLOT_SCALE_FLOATS = CG_MAX * GROUP_SCALE_FLOATS;
    static constexpr int CW = BN / (NUM_EPI_WARPS / 4);       // columns per epilogue warp
    static constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + (size_t)NSTAGES * STAGE_BYTES +
                                         (size_t)NSLOT * SLOT_SCALE_FLOATS * sizeof(float) + sizeof(Shared);
};

struct GemmArgs {
    const float *row_scale;   // [P][G][row_pitch]: sX (normal) or sW (swapped)
    const float *col_scale;   // [P][G][col_pitch]: sW (normal) or sX (swapped)
    int row_pitch, col_pitch;
    int rows, cols;           // valid rows / columns: (T, K) normal, (K, T) swapped
    int cg;                   // groups per chunk
    float *Y;                 // [P][K][Tp]
    int32_t *acc_dump;        // [P][T][K][G] or null
    int *status;
    long long wait_cycles;    // limit of every mbarrier wait (about a second by default)
    int debug_skip_stage;     // >= 0: CTA 0's producer skips the loads of this stage (test hook)
    long long l2_prefetch_bytes;   // per CTA: filter bytes it may ask into L2 ahead of the previous kernel's end
};

// MMA issue loop for the common shapes in which the chunks tile a stage exactly
// (GSTEPS MMAs per group, CGT groups per chunk, GSTEPS * CGT in {2, 4} MMAs per chunk):
// per chunk one slot wait, the chunk's MMAs as straight-line code with constant
// descriptor offsets and accumulate flags, one commit.  The generic loop in the kernel
// spends several hundred cycles per MMA on its bookkeeping, which made the issuing
// warp the bottleneck of every layer with more than one chunk per unit.
template <int BN, int GSTEPS, int CGT>
__device__ __forceinline__ void mma_issue_aligned(Shared *sh, uint32_t tiles_lo, uint32_t tmem_base,
                                                  int units, int KB, int last_slices, int lane,
                                                  const WaitCtx &ctx)
{
    using C = Cfg<BN>;
    constexpr int CHUNK_STEPS = GSTEPS * CGT;            // MMAs per chunk
    constexpr int NCH = (BK / UK) / CHUNK_STEPS;         // chunks per stage
    static_assert(NCH >= 1 && NCH * CHUNK_STEPS == BK / UK, "chunks must tile a stage");
    constexpr uint32_t idesc = ptx::idesc_i8(BM, BN);
    constexpr uint32_t dhi = ptx::smem_desc_sw128_hi();
    const uint32_t full0 = ptx::smem_u32(&sh->full[0]), empty0 = ptx::smem_u32(&sh->empty[0]);
    const uint32_t acc0 = ptx::smem_u32(&sh->acc_full[0]), free0 = ptx::smem_u32(&sh->slot_free[0]);
    int stage = 0, slot = 0;
    uint32_t phase = 0, sphase = 0;
    for (int u = blockIdx.x; u < units; u += gridDim.x) {
        for (int kb = 0; kb < KB; ++kb) {
            const int nslice = kb == KB - 1 ? last_slices : BK / UK;
            if (!__all_sync(0xffffffffu, wait_bounded(full0 + 8u * stage, phase, ctx, kWaitSmemFull)))
                return;
            const uint32_t a_lo = tiles_lo + (uint32_t)(stage * (C::STAGE_BYTES >> 4));
            const uint32_t b_lo = a_lo + (uint32_t)(A_BYTES >> 4);
#pragma unroll
            for (int c = 0; c < NCH; ++c) {
                if (c * CHUNK_STEPS < nslice) {           // the chunk has at least one group
                    if (!__all_sync(0xffffffffu, wait_bounded(free0 + 8u * slot, sphase ^ 1u, ctx,
                                                              kWaitTmemEmpty)))
                        return;
                    ptx::tc_fence_after();
                    if (lane == 0) {
                        const uint32_t d = tmem_base + (uint32_t)(slot * SLOT_COLS);
                        if ((c + 1) * CHUNK_STEPS <= nslice) {
#pragma unroll
                            for (int s = 0; s < CHUNK_STEPS; ++s) {
                                const uint32_t off = 2u * (uint32_t)(c * CHUNK_STEPS + s);
                                if (s % GSTEPS) ptx::umma_i8_lo<true>(d + (s / GSTEPS) * BN, a_lo + off, b_lo + off, dhi, idesc);
                                else ptx::umma_i8_lo<false>(d + (s / GSTEPS) * BN, a_lo + off, b_lo + off, dhi, idesc);
                            }
                        } else {
                            // last stage of a unit whose channel count is not a multiple of 128
#pragma unroll
                            for (int s = 0; s < CHUNK_STEPS; ++s) {
                                const uint32_t off = 2u * (uint32_t)(c * CHUNK_STEPS + s);
                                if (c * CHUNK_STEPS + s < nslice) {
                                    if (s % GSTEPS) ptx::umma_i8_lo<true>(d + (s / GSTEPS) * BN, a_lo + off, b_lo + off, dhi, idesc);
                                    else ptx::umma_i8_lo<false>(d + (s / GSTEPS) * BN, a_lo + off, b_lo + off, dhi, idesc);
                                }
                            }
                        }
                        ptx::umma_commit(acc0 + 8u * slot);
                    }
                    __syncwarp();
                    if (++slot == NSLOT) { slot = 0; sphase ^= 1u; }
                }
            }
            if (lane == 0) ptx::umma_commit(empty0 + 8u * stage);
            __syncwarp();
            if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
        }
    }
}

template <int BN, bool SWAP, bool DUMP>
__global__ void __launch_bounds__(NUM_THREADS, 2)
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
    Shared *sh = reinterpret_cast<Shared *>(scales + (size_t)NSLOT * C::SLOT_SCALE_FLOATS);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int MT = (a.rows + BM - 1) / BM, NT = (a.cols + BN - 1) / BN;
    const int units = g.P * MT * NT;
    const int KB = (g.C + BK - 1) / BK;          // stages per unit
    const int gs_steps = g.gs / UK;              // MMAs per group
    const int cg = a.cg;                         // groups per chunk
    const int nchunk = (g.G + cg - 1) / cg;      // chunks per unit
    const WaitCtx ctx{&sh->abort, a.status, a.wait_cycles};

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGES; ++s) {
            ptx::mbar_init(ptx::smem_u32(&sh->full[s]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->empty[s]), 1);
        }
        for (int b = 0; b < NSLOT; ++b) {
            ptx::mbar_init(ptx::smem_u32(&sh->acc_full[b]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->slot_free[b]), NUM_EPI_WARPS);
            ptx::mbar_init(ptx::smem_u32(&sh->scale_full[b]), 1);
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

    // Everything above may overlap the kernel that produces Xq and sX.  So may the filter
    // stream, which does not depend on it: before waiting for that kernel the producer loads
    // the filter half of its first stages and asks for the filter tiles of its first units
    // to be brought into L2 (bounded by a per-CTA share of `l2_prefetch_bytes`).
    constexpr int W_ROWS = SWAP ? BM : BN;                 // filter rows of a stage
    // stages of the first unit whose filter half is loaded early
    const int pre = (a.l2_prefetch_bytes > 0 && (int)blockIdx.x < units) ? (KB < NSTAGES ? KB : NSTAGES) : 0;
    if (warp == 0 && lane == 0) {
        ptx::prefetch_tmap(&tmA);
        ptx::prefetch_tmap(&tmB);
        const CUtensorMap *tmW = SWAP ? &tmA : &tmB;
        long long budget = a.l2_prefetch_bytes;
        for (int u = blockIdx.x, first = 1; u < units && budget > 0; u += gridDim.x, first = 0) {
            const int nt = u % NT, mt = (u / NT) % MT, p = u / (NT * MT);
            const int wrow = SWAP ? mt * BM : nt * BN;
            for (int kb = 0; kb < KB && budget > 0; ++kb) {
                if (first && kb < pre) {
                    if (!(blockIdx.x == 0 && kb == a.debug_skip_stage)) {
                        const uint32_t bar = ptx::smem_u32(&sh->full[kb]);
                        const uint32_t dst = ptx::smem_u32(tiles + (size_t)kb * C::STAGE_BYTES) + (SWAP ? 0 : A_BYTES);
                        ptx::mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
                        ptx::tma_load_3d(dst, tmW, bar, kb * BK, wrow, p);
                    }
                } else {
                    ptx::tma_prefetch_l2_3d(tmW, kb * BK, wrow, p);
                    budget -= W_ROWS * BK;
                }
            }
        }
    }
    if (warp == 0) __syncwarp();
    ptx::grid_dependency_wait();

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        // All 32 lanes walk the loop and wait together; lane 0 alone issues the copies.
        // (A warp whose other lanes sit at the final block barrier while one lane works
        // gets scheduled far too rarely.)
        int stage = 0;
        uint32_t phase = 0;
        long long issued = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
            const int nt = u % NT, mt = (u / NT) % MT, p = u / (NT * MT);
            for (int kb = 0; kb < KB; ++kb) {
                ok = __all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh->empty[stage]), phase ^ 1u, ctx,
                                                          kWaitSmemEmpty));
                if (!ok) break;
                if (lane == 0 && !(blockIdx.x == 0 && issued == a.debug_skip_stage)) {
                    const uint32_t bar = ptx::smem_u32(&sh->full[stage]);
                    const uint32_t a_dst = ptx::smem_u32(tiles + (size_t)stage * C::STAGE_BYTES);
                    if (issued >= pre) {
                        ptx::mbar_arrive_expect_tx(bar, C::STAGE_BYTES);
                        ptx::tma_load_3d(a_dst, &tmA, bar, kb * BK, mt * BM, p);
                        ptx::tma_load_3d(a_dst + A_BYTES, &tmB, bar, kb * BK, nt * BN, p);
                    } else if (SWAP) {      // the filter half of this stage is already on its way
                        ptx::tma_load_3d(a_dst + A_BYTES, &tmB, bar, kb * BK, nt * BN, p);
                    } else {
                        ptx::tma_load_3d(a_dst, &tmA, bar, kb * BK, mt * BM, p);
                    }
                }
                __syncwarp();
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
                drain(ptx::smem_u32(&sh->full[s]), ph, a.wait_cycles / 16);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // The warp stays converged; lane 0 issues every MMA and commit.  Its instructions
        // form one dependent chain, so the descriptors are advanced with 32-bit adds and
        // the accumulate flag is a constant of the instruction.
        constexpr uint32_t idesc = ptx::idesc_i8(BM, BN);
        constexpr uint32_t dhi = ptx::smem_desc_sw128_hi();
        const uint32_t tiles_lo = ptx::smem_desc_sw128_lo(ptx::smem_u32(tiles));
        const int chunk_steps = cg * gs_steps;       // MMAs per full chunk
        const int last_slices = (g.C - (KB - 1) * BK) / UK;
        int stage = 0, slot = 0;
        uint32_t phase = 0, sphase = 0;
        bool ok = true;
        // shapes whose chunks tile a stage exactly take the straight-line issue loop
        if (gs_steps == 2 && cg == 2) {
            mma_issue_aligned<BN, 2, 2>(sh, tiles_lo, tmem_base, units, KB, last_slices, lane, ctx);
            ok = false;
        } else if (gs_steps == 4 && cg == 1) {
            mma_issue_aligned<BN, 4, 1>(sh, tiles_lo, tmem_base, units, KB, last_slices, lane, ctx);
            ok = false;
        } else if (gs_steps == 1 && cg == C::CG_MAX && C::CG_MAX <= 4) {
            mma_issue_aligned<BN, 1, (C::CG_MAX <= 4 ? C::CG_MAX : 4)>(sh, tiles_lo, tmem_base, units, KB,
                                                                    last_slices, lane, ctx);
            ok = false;
        }
        for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
            int step = 0;          // MMA step within the chunk
            int in_group = 0;      // MMA step within the group
            uint32_t dcol = 0;     // TMEM column of the current group
            for (int kb = 0; kb < KB && ok; ++kb) {
                ok = __all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh->full[stage]), phase, ctx,
                                                          kWaitSmemFull));
                if (!ok) break;
                ptx::tc_fence_after();
                // a 32-byte step along K inside the swizzled rows is +2 in the address field
                const uint32_t a_lo = tiles_lo + (uint32_t)(stage * (C::STAGE_BYTES >> 4));
                const uint32_t b_lo = a_lo + (uint32_t)(A_BYTES >> 4);
                const int nslice = min(BK, g.C - kb * BK) / UK;
                for (int s = 0; s < nslice; ++s) {
                    if (step == 0) {
                        // start of a chunk: its TMEM slot must have been drained
                        ok = __all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh->slot_free[slot]),
                                                                  sphase ^ 1u, ctx, kWaitTmemEmpty));
                        if (!ok) break;
                        ptx::tc_fence_after();
                        dcol = tmem_base + (uint32_t)(slot * SLOT_COLS);
                    }
                    if (lane == 0) {
                        if (in_group) ptx::umma_i8_lo<true>(dcol, a_lo + 2 * s, b_lo + 2 * s, dhi, idesc);
                        else ptx::umma_i8_lo<false>(dcol, a_lo + 2 * s, b_lo + 2 * s, dhi, idesc);
                    }
                    ++step;
                    if (++in_group == gs_steps) { in_group = 0; dcol += BN; }
                    if (step == chunk_steps) {
                        if (lane == 0) ptx::umma_commit(ptx::smem_u32(&sh->acc_full[slot]));
                        step = 0;
                        if (++slot == NSLOT) { slot = 0; sphase ^= 1u; }
                    }
                }
                if (!ok) break;
                if (lane == 0) ptx::umma_commit(ptx::smem_u32(&sh->empty[stage]));
                __syncwarp();
                if (++stage == NSTAGES) { stage = 0; phase ^= 1u; }
            }
            if (ok && step != 0) {
                // the last chunk of the unit has fewer groups than a full one
                if (lane == 0) ptx::umma_commit(ptx::smem_u32(&sh->acc_full[slot]));
                __syncwarp();
                if (++slot == NSLOT) { slot = 0; sphase ^= 1u; }
            }
        }
    } else if (warp == 2) {
        // ---------------- scale loader ----------------
        if (!DUMP) {
            int slot = 0;
            uint32_t sphase = 0;
            long long issued = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
                const int nt = u % NT, mt = (u / NT) % MT, p = u / (NT * MT);
                for (int ch = 0; ch < nchunk; ++ch) {
                    const int g0 = ch * cg, ng = min(cg, g.G - g0);
                    ok = __all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh->slot_free[slot]), sphase ^ 1u,
                                                              ctx, kWaitScaleEmpty));
                    if (!ok) break;
                    const uint32_t bar = ptx::smem_u32(&sh->scale_full[slot]);
                    const uint32_t dst = ptx::smem_u32(scales + (size_t)slot * C::SLOT_SCALE_FLOATS);
                    if (lane == 0) ptx::mbar_arrive_expect_tx(bar, (uint32_t)(ng * C::GROUP_SCALE_FLOATS * 4));
                    __syncwarp();
                    // lane j copies the row scales of group j, lane 4 + j its column scales
                    if (lane < 8 && (lane & 3) < ng) {
                        const int j = lane & 3;
                        const size_t pg = (size_t)p * g.G + g0 + j;
                        const uint32_t d = dst + (uint32_t)(j * C::GROUP_SCALE_FLOATS * 4);
                        if (lane < 4)
                            ptx::bulk_load(d, a.row_scale + pg * a.row_pitch + mt * BM, BM * 4, bar);
                        else
                            ptx::bulk_load(d + BM * 4, a.col_scale + pg * a.col_pitch + nt * BN, BN * 4, bar);
                    }
                    __syncwarp();
                    ++issued;
                    if (++slot == NSLOT) { slot = 0; sphase ^= 1u; }
                }
            }
            if (!ok) {
                int s = slot;
                uint32_t ph = sphase;
                const long long n = issued < NSLOT ? issued : NSLOT;
                for (long long i = 0; i < n; ++i) {
                    if (--s < 0) { s = NSLOT - 1; ph ^= 1u; }
                    drain(ptx::smem_u32(&sh->scale_full[s]), ph, a.wait_cycles / 16);
                }
            }
        }
    } else if (warp >= FIRST_EPI_WARP) {
        // ---------------- epilogue ----------------
        const int quarter = warp & 3;                         // TMEM lanes this warp may read
        const int c0 = ((warp - FIRST_EPI_WARP) >> 2) * CW;   // first column of this warp
        const uint32_t tmem_warp = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0;
        int slot = 0;
        uint32_t sphase = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < units && ok; u += gridDim.x) {
            const int nt = u % NT, mt = (u / NT) % MT, p = u / (NT * MT);
            const int row = mt * BM + quarter * 32 + lane;    // tile (normal) or channel (swapped)
            const int col0 = nt * BN + c0;
            // warp-uniform: does this warp own any valid row and column of the unit?
            const bool active = (mt * BM + quarter * 32 < a.rows) && (col0 < a.cols);
            const bool row_ok = row < a.rows;
            float2 acc[CW / 2];
#pragma unroll
            for (int j = 0; j < CW / 2; ++j) acc[j] = make_float2(0.f, 0.f);

            for (int ch = 0; ch < nchunk && ok; ++ch) {
                const int g0 = ch * cg, ng = min(cg, g.G - g0);
                if (!wait_bounded(ptx::smem_u32(&sh->acc_full[slot]), sphase, ctx, kWaitTmemFull)) {
                    ok = false; break;
                }
                if constexpr (!DUMP) {
                    if (!wait_bounded(ptx::smem_u32(&sh->scale_full[slot]), sphase, ctx,
                                      kWaitScaleFull)) { ok = false; break; }
                }
                if (active) {
                    ptx::tc_fence_after();
                    const float *sc = scales + (size_t)slot * C::SLOT_SCALE_FLOATS;
                    for (int j = 0; j < ng; ++j) {
                        const uint32_t taddr = tmem_warp + (uint32_t)(slot * SLOT_COLS + j * BN);
                        const float rs = sc[j * C::GROUP_SCALE_FLOATS + quarter * 32 + lane];
                        const float2 rs2 = make_float2(rs, rs);
                        const float4 *cs4 = reinterpret_cast<const float4 *>(
                            sc + j * C::GROUP_SCALE_FLOATS + BM + c0);
#pragma unroll
                        for (int h = 0; h < CW / 16; ++h) {          // 16 columns at a time
                            uint32_t r[16];
                            ptx::tmem_ld_x16(taddr + (uint32_t)(16 * h), r);
                            ptx::tmem_ld_wait();
                            if constexpr (DUMP) {
                                if (row_ok) {
#pragma unroll
                                    for (int i = 0; i < 16; ++i) {
                                        const int col = col0 + 16 * h + i;
                                        if (col < a.cols) {
                                            const size_t t = SWAP ? col : row, k = SWAP ? row : col;
                                            a.acc_dump[(((size_t)p * g.T + t) * g.K + k) * g.G + g0 + j] =
                                                (int32_t)r[i];
                                        }
                                    }
                                }
                            } else {
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    const float4 cs = cs4[4 * h + q];
                                    float2 f0 = make_float2(__int2float_rn((int32_t)r[4 * q + 0]),
                                                            __int2float_rn((int32_t)r[4 * q + 1]));
                                    float2 f1 = make_float2(__int2float_rn((int32_t)r[4 * q + 2]),
                                                            __int2float_rn((int32_t)r[4 * q + 3]));
                                    f0 = __fmul2_rn(f0, rs2);
                                    f1 = __fmul2_rn(f1, rs2);
                                    acc[8 * h + 2 * q] = __ffma2_rn(f0, make_float2(cs.x, cs.y), acc[8 * h + 2 * q]);
                                    acc[8 * h + 2 * q + 1] =
                                        __ffma2_rn(f1, make_float2(cs.z, cs.w), acc[8 * h + 2 * q + 1]);
                                }
                            }
                        }
                    }
                    ptx::tc_fence_before();
                }
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->slot_free[slot]));
                if (++slot == NSLOT) { slot = 0; sphase ^= 1u; }
            }

            if constexpr (!DUMP) {
                if (ok && active && row_ok) {
                    if constexpr (SWAP) {
                        // row = output channel, columns = tiles: contiguous in Y[p][k][:];
                        // 32-byte stores so that every instruction fills whole sectors
                        float *dst = a.Y + ((size_t)p * g.K + row) * g.Tp + col0;
#pragma unroll
                        for (int j8 = 0; j8 < CW / 8; ++j8)
                            if (col0 + 8 * j8 + 7 < g.Tp)
                                ptx::st_global_v8(dst + 8 * j8, acc[4 * j8].x, acc[4 * j8].y, acc[4 * j8 + 1].x,
                                                  acc[4 * j8 + 1].y, acc[4 * j8 + 2].x, acc[4 * j8 + 2].y,
                                                  acc[4 * j8 + 3].x, acc[4 * j8 + 3].y);
                    } else {
                        // row = tile: lanes write consecutive t of one Y[p][k][:] row
                        float *dst = a.Y + ((size_t)p * g.K + col0) * g.Tp + row;
#pragma unroll
                        for (int j = 0; j < CW / 2; ++j) {
                            if (col0 + 2 * j < a.cols) dst[(size_t)(2 * j) * g.Tp] = acc[j].x;
                            if (col0 + 2 * j + 1 < a.cols) dst[(size_t)(2 * j + 1) * g.Tp] = acc[j].y;
                        }
                    }
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
    // groups per chunk: as many whole groups as fit into 128 channels (one stage) and
    // into one TMEM slot; group sizes that do not divide 128 get one group per chunk
    a.cg = 1;
    if (BK % g.gs == 0) a.cg = BK / g.gs < C::CG_MAX ? BK / g.gs : C::CG_MAX;
    a.Y = plan.ws.Y;
    a.acc_dump = acc_dump;
    a.status = plan.status;
    a.wait_cycles = plan.wait_cycles;
    a.debug_skip_stage = plan.debug_skip_gemm_stage;
    const int MT = (a.rows + BM - 1) / BM, NT = (a.cols + BN - 1) / BN;
    const int units = g.P * MT * NT;
    const int slots = 2 * plan.sm_count;          // two CTAs per SM
    const int grid = units < slots ? units : slots;
    // the filters share L2 (126 MB) with Xq, sX and Y: at most 48 MB of them are asked for early
    a.l2_prefetch_bytes = pdl ? (48LL << 20) / grid : 0;
    auto kern = gemm_dequant_kernel<BN, SWAP, DUMP>;
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

// ---- tensor-pipe rate of tcgen05.mma kind::i8 -----------------------------------------
// One CTA per SM issues `mmas` accumulating 128 x BN x 32 MMAs on operands that stay in
// shared memory (no global traffic), then waits (bounded) for the last one.  Timed by the
// caller with events: grid * mmas * 2 * 128 * BN * 32 operations.
struct PeakShared { uint64_t done; uint32_t tmem_base; volatile int abort; };

template <int BN>
__global__ void __launch_bounds__(128, 1) mma_peak_kernel(int mmas, int *status, long long wait_cycles)
{
    extern __shared__ unsigned char smem_raw[];
    unsigned char *tiles = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int BYTES = (BM + BN) * BK;
    PeakShared *sh = reinterpret_cast<PeakShared *>(tiles + BYTES);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int i = threadIdx.x; i < BYTES / 4; i += blockDim.x) reinterpret_cast<uint32_t *>(tiles)[i] = 0x01010101u;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&sh->done), 1);
        sh->abort = 0;
        ptx::fence_mbar_init();
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), BN < 32 ? 32 : BN);
        ptx::tmem_relinquish();
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem = sh->tmem_base;
    if (warp == 0) {
        const WaitCtx ctx{&sh->abort, status, wait_cycles};
        if (lane == 0) {
            constexpr uint32_t idesc = ptx::idesc_i8(BM, BN);
            constexpr uint32_t dhi = ptx::smem_desc_sw128_hi();
            const uint32_t a_lo = ptx::smem_desc_sw128_lo(ptx::smem_u32(tiles));
            const uint32_t b_lo = a_lo + (uint32_t)(A_BYTES >> 4);
            for (int i = 0; i < mmas; i += 4) {
                ptx::umma_i8_lo<true>(tmem, a_lo, b_lo, dhi, idesc);
                ptx::umma_i8_lo<true>(tmem, a_lo + 2, b_lo + 2, dhi, idesc);
                ptx::umma_i8_lo<true>(tmem, a_lo + 4, b_lo + 4, dhi, idesc);
                ptx::umma_i8_lo<true>(tmem, a_lo + 6, b_lo + 6, dhi, idesc);
            }
            ptx::umma_commit(ptx::smem_u32(&sh->done));
        }
        __syncwarp();
        wait_bounded(ptx::smem_u32(&sh->done), 0, ctx, kWaitTmemFull);
    }
    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem, BN < 32 ? 32 : BN);
    }
}

template <int BN>
cudaError_t launch_peak(int grid, int mmas, int *status, long long wait_cycles, cudaStream_t stream)
{
    const int smem = 1024 + (BM + BN) * BK + (int)sizeof(PeakShared);
    cudaError_t e = cudaFuncSetAttribute(mma_peak_kernel<BN>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    mma_peak_kernel<BN><<<grid, 128, smem, stream>>>(mmas, status, wait_cycles);
    return cudaGetLastError();
}

template <int BN, bool SWAP, bool DUMP>
cudaError_t setup_variant()
{
    return cudaFuncSetAttribute(gemm_dequant_kernel<BN, SWAP, DUMP>,
                                cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<BN>::SMEM_BYTES);
}

}  // namespace

// One-time attribute setting for the kernels of this file (per device).
cudaError_t setup_gemm()
{
    cudaError_t e = setup_variant<16, true, true>();
    if (e == cudaSuccess) e = setup_variant<16, true, false>();
    if (e == cudaSuccess) e = setup_variant<16, false, true>();
    if (e == cudaSuccess) e = setup_variant<16, false, false>();
    if (e == cudaSuccess) e = setup_variant<32, true, true>();
    if (e == cudaSuccess) e = setup_variant<32, true, false>();
    if (e == cudaSuccess) e = setup_variant<48, true, true>();
    if (e == cudaSuccess) e = setup_variant<48, true, false>();
    if (e == cudaSuccess) e = setup_variant<64, true, true>();
    if (e == cudaSuccess) e = setup_variant<64, true, false>();
    if (e == cudaSuccess) e = setup_variant<64, false, true>();
    if (e == cudaSuccess) e = setup_variant<64, false, false>();
    return e;
}

cudaError_t launch_mma_peak(const wfq_plan &plan, int n_cols, int mmas, cudaStream_t stream)
{
    const int grid = plan.sm_count;
    switch (n_cols) {
        case 64: return launch_peak<64>(grid, mmas, plan.status, plan.wait_cycles, stream);
        case 128: return launch_peak<128>(grid, mmas, plan.status, plan.wait_cycles, stream);
        case 256: return launch_peak<256>(grid, mmas, plan.status, plan.wait_cycles, stream);
        default: return cudaErrorInvalidValue;
    }
}

int gemm_block_m() { return BM; }

// Orientation and column block of the contraction for a layer: rows (TMEM lanes) are
// tiles unless the swapped orientation leaves less padded work.
void gemm_choose(const Geometry &g, bool *swap, int *bn)
{
    auto up = [](long long v, int b) { return (v + b - 1) / b * b; };
    const long long normal = up(g.T, BM) * up(g.K, 64);
    // swapped: the tile columns are padded to a multiple of the column block (32, 48 or 64:
    // every padded column is promoted like a real one); the largest block among the least padded
    int bn_sw = 64;
    for (int c : {48, 32})
        if (up(g.T, c) < up(g.T, bn_sw)) bn_sw = c;
    const long long swapped = up(g.K, BM) * up(g.T, bn_sw);
    *swap = 5 * swapped < 4 * normal;   // swapped stores are less efficient: want >= 20 % less work
    *bn = *swap ? bn_sw : 64;
}

cudaError_t launch_gemm(const wfq_plan &plan, int32_t *acc_dump, cudaStream_t stream, bool pdl)
{
    const bool dump = acc_dump != nullptr;
    // 16 columns: never chosen by gemm_choose, only by the debug option (the shape a contraction
    // fused with the output transform would be confined to by its accumulator space)
    if (plan.gemm_bn == 16) {
        if (plan.gemm_swap)
            return dump ? launch_variant<16, true, true>(plan, acc_dump, stream, pdl)
                        : launch_variant<16, true, false>(plan, acc_dump, stream, pdl);
        return dump ? launch_variant<16, false, true>(plan, acc_dump, stream, pdl)
                    : launch_variant<16, false, false>(plan, acc_dump, stream, pdl);
    }
    if (plan.gemm_swap) {
        if (plan.gemm_bn == 32)
            return dump ? launch_variant<32, true, true>(plan, acc_dump, stream, pdl)
                        : launch_variant<32, true, false>(plan, acc_dump, stream, pdl);
        if (plan.gemm_bn == 48)
            return dump ? launch_variant<48, true, true>(plan, acc_dump, stream, pdl)
                        : launch_variant<48, true, false>(plan, acc_dump, stream, pdl);
        return dump ? launch_variant<64, true, true>(plan, acc_dump, stream, pdl)
                    : launch_variant<64, true, false>(plan, acc_dump, stream, pdl);
    }
    return dump ? launch_variant<64, false, true>(plan, acc_dump, stream, pdl)
                : launch_variant<64, false, false>(plan, acc_dump, stream, pdl);
}

}  // namespace wfq
