// Fused input transform + group-wise int8 quantization on the tensor cores (fp16 inputs).
//
//   X = S_B V_B x V_B^T S_B   (Section 4.1), then the quantizer of Section 2 with one
//   scale per (position, tile, group of consecutive input channels).
//
// The 2-D transform of a patch d (n x n, fp16) is one contraction with a constant matrix:
//   Z[p = (i, j)] = sum_{a, b} BT[i][a] BT[j][b] d[a][b],   BT = the standard-scaled B^T,
// whose entries (products of small integers and dyadic rationals, numerators <= 441) are
// exact in fp16 and whose products with fp16 data are exact in fp32.  So the transform is a
// tcgen05.mma kind::f16 with the Winograd positions on the accumulator rows (TMEM lanes)
// and (tile, channel) on its columns: afterwards a thread owns one position of one tile
// and reads a run of 64 channels from TMEM, which is exactly what the group quantizer
// needs: abs-max over registers, one scale, 64 contiguous int8 codes per thread.  There
// is no fp32 round trip through shared memory and no shuffle.
//
// One persistent CTA per SM, 32 warps of at most 64 registers:
//   warp 0      TMA producer: the zero-padded input strip of a work item (tiles of one
//               tile row x 64 channels) into a ring of strip buffers
//   warp 1      owns TMEM; one lane issues the MMAs: per pair of patch tiles KSTEPS
//               instructions of M = 128, N = 128 (2 tiles x 64 channels), K = 16
//   warp 2      turns the completions of the pairs' MMAs, in order, into a counter that the
//               im2col warps poll before they overwrite an operand tile
//   warps 4-15  im2col: copy patch rows (8 halves = 16 bytes) from the strip into the
//               K-major, 128-byte-swizzled operand tiles the MMA reads (row = channel,
//               K = a * 8 + b); a warp takes four tiles x 16 channels, lanes = (tile, patch
//               row)
//   warps 16-31 quantizers, two teams of eight that alternate over the accumulators:
//               warp % 4 selects the 32 TMEM lanes, the next bit the tile of the pair;
//               tcgen05.ld of 32 columns at a time, per-position factor, abs-max, scale,
//               codes, one 32-byte store per 32 codes
// (Few warps with many registers were tried first: every role is a chain of dependent
// instructions and mbarrier hand-overs of a few hundred cycles each, and only many
// resident warps hide them.)
// Accumulator rows: S "slots" of PL lanes (F(6,3): 2 x 64, F(4,3): 3 x 40).  The constant
// matrix is the A operand and lives in tensor memory, one copy per slot with its rows on
// lanes s * PL ... and zeros on all other lanes; the MMAs of a pair use the copy of their
// slot, so one accumulator of 128 columns holds 2 * S tiles, and the tensor cores read only
// the patch tiles from shared memory (whose bandwidth bounds this kernel).  Patch tiles flow through the kernel as one flat
// sequence (pairs, then groups of S pairs), independent of the work items they came from.
//
// Staging modes (chosen on the host):
//   0  3-D tiled TMA over (W, H, N*C): column chunks of a tile row (the whole row where it
//      fits), all padding by zero fill; needs W*2 to be a multiple of 16.  The box width is
//      8 modulo 16 elements, so that the eight patch rows of a channel start in different
//      shared-memory banks for the im2col reads.
//   1  2-D tiled TMA over (H*W, N*C): a strip is a whole tile row, n image rows x full width
//      per channel in one box (<= 256 elements); top/bottom padding by zero fill, left/right
//      by masks.  For widths that are not a multiple of 8 with H*W*2 a multiple of 16.
//   2  one bulk copy of a whole 64-channel block of a (small) image, all padding by masks.
// The constant matrix is built once per device on the host; four warps of every CTA copy it
// from global memory into tensor memory while the first strips are in flight.
#include <cuda_fp16.h>

#include <cstring>
#include <vector>

#include "wfq_internal.h"
#include "wfq_ptx.cuh"
#include "wfq_quant.cuh"

namespace wfq {
namespace {

constexpr int TC_THREADS = 1024;
constexpr int TC_CB = 64;            // channels per work item = rows of an operand tile
constexpr int TC_TILE_BYTES = TC_CB * 128;
constexpr int TC_NACC = 2;           // accumulators of 128 TMEM columns, one per quantizer team
constexpr int TC_TMEM_COLS = 512;    // allocation: accumulators, then the constant matrix
constexpr int TC_AMAT_COL = 128 * TC_NACC;
constexpr int TC_MAX_STRIP = 8;
constexpr int TC_MAX_PAIR = 8;
constexpr int TC_IDS = 64;           // ring of tile ids (operand tiles in flight < 64)
constexpr int TC_CQ = 4;             // channel quarters of an operand tile (16 rows each)
constexpr int TC_READERS = 12;       // im2col warps
constexpr int TC_FIRST_READER = 4;
constexpr int TC_FIRST_QUANT = 16;
constexpr int TC_TEAMS = 2;          // quantizer teams
constexpr int TC_TEAM_WARPS = 8;     // warps per team: 4 lane quarters x 2 tiles of a pair

struct TcShared {
    uint64_t strip_full[TC_MAX_STRIP];    // the strip has landed
    uint64_t strip_empty[TC_MAX_STRIP];   // all im2col warps are done with the strip
    uint64_t pair_full[TC_MAX_PAIR];      // both operand tiles of a pair are written
    uint64_t pair_empty[TC_MAX_PAIR];     // the MMAs reading the pair have completed
    uint64_t acc_full[TC_NACC];           // the MMAs of a group have completed
    uint64_t acc_empty[TC_NACC];          // all quantizer warps have read the accumulator
    uint64_t mma_done;                    // every MMA issued by this CTA has completed
    uint64_t amat_full;                   // the constant matrix has landed
    uint64_t tick;                        // one phase per increment of pairs_consumed
    uint32_t tmem_base;
    volatile int abort;
    volatile int pairs_consumed;          // operand-tile pairs whose MMAs have completed
    int tile_id[TC_IDS];                  // global tile index of an operand tile
    int tile_cb[TC_IDS];                  // its channel block
};

template <int M>
struct TcCfg {
    static constexpr int NN = M + 2;
    static constexpr int P = NN * NN;
    static constexpr int S = M == 6 ? 2 : 3;            // tile slots on the TMEM lanes
    static constexpr int PL = M == 6 ? 64 : 40;         // lanes per slot (a multiple of 8)
    static constexpr int KSTEPS = NN / 2;               // K = 16 = two patch rows per MMA
    static constexpr int KW = KSTEPS * 8;               // 32-bit TMEM columns of the matrix (K / 2)
};

struct TcArgs {
    const __half *x;
    int8_t *Xq;
    float *sX;
    int *status;
    long long wait_cycles;
    int mode, TBW, NCHUNK, NCB, items;
    int CS, RS;              // strip strides in elements: channel, patch row
    int strip_bytes, nstrip, nbp;
    const uint32_t *amat;    // the constant matrix, [P][KW] words (two fp16 K elements each), global
    int debug_skip_item;     // >= 0: the producer skips this item (exercises the bounded waits)
};

// Tiles of work item `item`: (channel block, image, first tile row / column, count).
struct ItemGeo { int cb, img, th, tw0, nb, srow; };

template <int M>
__device__ __forceinline__ ItemGeo item_geo(int item, const TcArgs &a, const Geometry &g)
{
    ItemGeo r;
    r.cb = item % a.NCB;
    const int rest = item / a.NCB;
    if (a.mode == 2) {           // a whole image
        r.img = rest; r.th = 0; r.tw0 = 0; r.nb = g.TH * g.TW; r.srow = rest * g.TH;
    } else {
        r.srow = rest / a.NCHUNK;
        const int chunk = rest - r.srow * a.NCHUNK;
        r.img = r.srow / g.TH;
        r.th = r.srow - r.img * g.TH;
        r.tw0 = chunk * a.TBW;
        r.nb = min(a.TBW, g.TW - r.tw0);
    }
    return r;
}

__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d)
                 : "memory");
}

// Bounded wait until the counter `*ctr` (shared memory, only ever incremented) has reached
// `target`.  Unlike an mbarrier phase a counter can be tested for any future value, so warps
// that work on different parts of the operand ring need not see every phase of every
// buffer.  The waiting itself is not a polling loop (twelve polling warps took two fifths of
// the SM's issue slots): the writer of the counter also arrives on the barrier `tick` once
// per increment, and a waiter that finds the counter at c < target sleeps in a try_wait
// on the phase of tick that the increment to c + 1 completes.  Should the counter move on
// by two between the read and the wait, the try_wait's time hint ends the sleep.
__device__ __noinline__ bool wait_counter(volatile int *ctr, uint32_t tick, int target, const WaitCtx &ctx,
                                          int where)
{
    long long t0 = 0;
    for (;;) {
        const int c = *ctr;
        if (c >= target) return true;
        ptx::mbar_try_wait_ns(tick, (uint32_t)(c & 1), 2000u);
        if (*ctx.abort) return false;
        const long long now = clock64();
        if (t0 == 0) t0 = now;
        if (now - t0 > ctx.limit) {
            *ctx.abort = 1;
            if (atomicCAS(ctx.status, 0, 6 /* WFQ_ERR_TIMEOUT */) == 0) {
                ctx.status[1] = where;
                ctx.status[2] = (int)blockIdx.x;
                ctx.status[3] = target;
            }
            return false;
        }
    }
}

template <int M, int GS, int MODE>
__global__ void __launch_bounds__(TC_THREADS, 1)
input_transform_tc_kernel(const __grid_constant__ CUtensorMap tmx, TcArgs a, Geometry g, ScaleTables tab)
{
    using C = TcCfg<M>;
    constexpr int NN = C::NN, P = C::P, S = C::S, PL = C::PL, KSTEPS = C::KSTEPS;
    extern __shared__ unsigned char smem_raw[];
    unsigned char *base = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    unsigned char *Bring = base;                                 // [2 * nbp][64 rows][128 B]
    unsigned char *strips = Bring + (size_t)2 * a.nbp * TC_TILE_BYTES;
    TcShared *sh = reinterpret_cast<TcShared *>(strips + (size_t)a.nstrip * a.strip_bytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const WaitCtx ctx{&sh->abort, a.status, a.wait_cycles};
    ptx::grid_launch_dependents();   // the next kernel's prologue and filter stream may start

    // One strip load (all lanes call it; lane 0 issues).
    auto issue_strip = [&](int item, int sidx) {
        if (lane != 0 || item == a.debug_skip_item) return;
        const ItemGeo it = item_geo<M>(item, a, g);
        const uint32_t bar = ptx::smem_u32(&sh->strip_full[sidx]);
        const uint32_t dst = ptx::smem_u32(strips + (size_t)sidx * a.strip_bytes);
        ptx::mbar_arrive_expect_tx(bar, (uint32_t)a.strip_bytes);
        const int z = it.img * g.C + it.cb * TC_CB;
        if (MODE == 0) {
            const int first = it.tw0 * M - 1;
            ptx::tma_load_3d(dst, &tmx, bar, ((first + 8) & ~7) - 8, it.th * M - 1, z);
        } else if (MODE == 1) {
            ptx::tma_load_2d(dst, &tmx, bar, ((it.th * M - 1) * g.W) & ~7, z);
        } else {
            ptx::bulk_load(dst, a.x + (size_t)z * g.H * g.W, (uint32_t)a.strip_bytes, bar);
        }
    };

    // ---- set-up: warp 0 initialises the barriers and starts the first loads at once; warp
    // 1 allocates TMEM meanwhile ------------------------------------------------------------
    int prefilled = 0;
    if (warp == 0) {
        if (lane < TC_MAX_STRIP) {
            ptx::mbar_init(ptx::smem_u32(&sh->strip_full[lane]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->strip_empty[lane]), TC_READERS);
        } else if (lane < TC_MAX_STRIP + TC_MAX_PAIR) {
            ptx::mbar_init(ptx::smem_u32(&sh->pair_full[lane - TC_MAX_STRIP]), 2 * TC_CQ);
            ptx::mbar_init(ptx::smem_u32(&sh->pair_empty[lane - TC_MAX_STRIP]), 1);
        } else if (lane < TC_MAX_STRIP + TC_MAX_PAIR + TC_NACC) {
            ptx::mbar_init(ptx::smem_u32(&sh->acc_full[lane - TC_MAX_STRIP - TC_MAX_PAIR]), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->acc_empty[lane - TC_MAX_STRIP - TC_MAX_PAIR]), TC_TEAM_WARPS);
        } else if (lane == 31) {
            ptx::mbar_init(ptx::smem_u32(&sh->mma_done), 1);
            ptx::mbar_init(ptx::smem_u32(&sh->amat_full), 4);
            ptx::mbar_init(ptx::smem_u32(&sh->tick), 1);
            sh->abort = 0;
            sh->pairs_consumed = 0;
        }
        ptx::fence_mbar_init();
        __syncwarp();
        if (lane == 0 && MODE != 2) ptx::prefetch_tmap(&tmx);
        for (int item = blockIdx.x; item < a.items && prefilled < a.nstrip; item += gridDim.x)
            issue_strip(item, prefilled++);
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_u32(&sh->tmem_base), TC_TMEM_COLS);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before();
    __syncthreads();
    ptx::tc_fence_after();
    const uint32_t tmem_base = sh->tmem_base;

    // the number of operand tiles this CTA's items produce
    int nbt = 0;
    if (warp != 0)
        for (int item = blockIdx.x; item < a.items; item += gridDim.x) nbt += item_geo<M>(item, a, g).nb;

    if (warp == 0) {
        // ---------------- TMA producer (the first nstrip loads are already in flight) ------
        int sidx = 0, k = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < a.items && ok; item += gridDim.x, ++k) {
            if (k >= prefilled) {
                ok = __all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh->strip_empty[sidx]), phase ^ 1u, ctx,
                                                          kWaitStripEmpty));
                if (!ok) break;
                issue_strip(item, sidx);
                __syncwarp();
            }
            if (++sidx == a.nstrip) { sidx = 0; phase ^= 1u; }
        }
        if (!ok) {
            // give copies still in flight a bounded time to land before the CTA exits
            const int issued = k > prefilled ? k : prefilled;
            for (int j = issued - 1; j >= 0 && j >= issued - a.nstrip; --j)
                drain(ptx::smem_u32(&sh->strip_full[j % a.nstrip]), (uint32_t)((j / a.nstrip) & 1),
                      a.wait_cycles / 16);
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        constexpr uint32_t idesc = ptx::idesc_f16(128, 128);
        constexpr uint32_t dhi = ptx::smem_desc_sw128_hi();
        const uint32_t b_lo0 = ptx::smem_desc_sw128_lo(ptx::smem_u32(Bring));
        const int npairs = (nbt + 1) >> 1;
        int slot = 0, s = 0, acc = 0;
        uint32_t phase = 0, aphase = 0;
        bool have_a = __all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh->amat_full), 0, ctx, kWaitSmemFull));
        for (int k = 0; k < npairs && have_a; ++k) {
            if (!__all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh->pair_full[slot]), phase, ctx,
                                                      kWaitPairFull)))
                break;
            if (s == 0 && !__all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh->acc_empty[acc]),
                                                                aphase ^ 1u, ctx, kWaitAccEmpty)))
                break;
            ptx::tc_fence_after();
            if (lane == 0) {
                const uint32_t d = tmem_base + (uint32_t)(acc * 128);
                // the copy of the matrix that sits on lanes s * PL ... (zero elsewhere)
                const uint32_t a_t = tmem_base + (uint32_t)(TC_AMAT_COL + s * C::KW);
                const uint32_t b_lo = b_lo0 + (uint32_t)((slot * 2 * TC_TILE_BYTES) >> 4);
#pragma unroll
                for (int ks = 0; ks < KSTEPS; ++ks) {
                    if (ks == 0 && s == 0) ptx::umma_f16_tmem_a<false>(d, a_t, b_lo, dhi, idesc);
                    else ptx::umma_f16_tmem_a<true>(d, a_t + 8 * ks, b_lo + 2 * ks, dhi, idesc);
                }
                ptx::umma_commit(ptx::smem_u32(&sh->pair_empty[slot]));
                if (s == S - 1 || k == npairs - 1) ptx::umma_commit(ptx::smem_u32(&sh->acc_full[acc]));
            }
            __syncwarp();
            if (++slot == a.nbp) { slot = 0; phase ^= 1u; }
            if (++s == S) {
                s = 0;
                if (++acc == TC_NACC) { acc = 0; aphase ^= 1u; }
            }
        }
        // TMEM is released below: no MMA of this CTA may still be running (they all have,
        // unless a wait ran out)
        if (lane == 0) ptx::umma_commit(ptx::smem_u32(&sh->mma_done));
        __syncwarp();
        drain(ptx::smem_u32(&sh->mma_done), 0, a.wait_cycles / 16);
    } else if (warp == 2) {
        // ---------------- retire: completed pairs, in order, as a counter ----------------
        const int npairs = (nbt + 1) >> 1;
        int slot = 0;
        uint32_t phase = 0;
        for (int k = 0; k < npairs; ++k) {
            if (!__all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh->pair_empty[slot]), phase, ctx,
                                                      kWaitPairEmpty)))
                break;
            if (lane == 0) {
                sh->pairs_consumed = k + 1;
                ptx::mbar_arrive(ptx::smem_u32(&sh->tick));
            }
            if (++slot == a.nbp) { slot = 0; phase ^= 1u; }
        }
    } else if (warp >= TC_FIRST_READER && warp < TC_FIRST_READER + TC_READERS) {
        // ---------------- im2col ----------------
        // A task is four neighbouring tiles x 16 channels of an item; the warps take the
        // tasks of an item round robin (twelve warps: items of up to twelve tiles in one go).
        const int rw = warp - TC_FIRST_READER;
        const int pa = lane & 7, tsub = lane >> 3;        // patch row, tile of the quad
        const uint32_t strips_u32 = ptx::smem_u32(strips), bring_u32 = ptx::smem_u32(Bring);
        int sidx = 0, b0 = 0;
        uint32_t sphase = 0;
        bool ok = true;
        for (int item = blockIdx.x; item < a.items && ok; item += gridDim.x) {
            const ItemGeo it = item_geo<M>(item, a, g);
            const int ntask = ((it.nb + 3) >> 2) * TC_CQ;
            // Every im2col warp waits for the strip, also one without a task in this item:
            // its arrival on strip_empty below must not run ahead of the producer, or it
            // would be counted for an earlier use of the same buffer.
            ok = __all_sync(0xffffffffu, wait_bounded(ptx::smem_u32(&sh->strip_full[sidx]), sphase, ctx,
                                                      kWaitStripFull));
            for (int task = rw; task < ntask && ok; task += TC_READERS) {
                const int tq = task / TC_CQ, cq = task - tq * TC_CQ;
                const int bfirst = b0 + tq * 4;
                const int cnt = min(4, it.nb - tq * 4);
                // the buffers of the pairs this task writes are free once the pairs that used
                // them before (nbp pairs earlier) have been consumed
                if (sh->pairs_consumed < ((bfirst + cnt - 1) >> 1) - a.nbp + 1)
                    ok = wait_counter(&sh->pairs_consumed, ptx::smem_u32(&sh->tick), ((bfirst + cnt - 1) >> 1) - a.nbp + 1, ctx,
                                      kWaitPairEmpty);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const uint32_t strip = strips_u32 + (uint32_t)(sidx * a.strip_bytes);
                const int tl = tq * 4 + tsub;             // tile within the item
                if (pa < NN && tsub < cnt) {
                    // first element of this (tile, patch row) in the strip, and which of its
                    // n columns lie inside the image
                    int th = it.th, tw = it.tw0 + tl;
                    if (MODE == 2) { th = tl / g.TW; tw = tl - th * g.TW; }
                    const int col0 = tw * M - 1;
                    int e0;
                    if (MODE == 0) e0 = pa * a.RS + col0 - (((it.tw0 * M - 1 + 8) & ~7) - 8);
                    else if (MODE == 1) e0 = pa * a.RS + col0 + (((it.th * M - 1) * g.W) & 7);
                    else e0 = (th * M - 1 + pa) * a.RS + col0;
                    uint32_t mk[4] = {0xffffffffu, 0xffffffffu, 0xffffffffu, NN == 8 ? 0xffffffffu : 0u};
                    bool masked = false;
                    if (MODE != 0) {
                        const int h = th * M - 1 + pa;
                        const bool rowok = MODE == 1 || (h >= 0 && h < g.H);
                        masked = !rowok || col0 < 0 || col0 + NN > g.W;
                        if (masked) {
#pragma unroll
                            for (int b2 = 0; b2 < NN / 2; ++b2) {
                                const int c = col0 + 2 * b2;
                                mk[b2] = (rowok && c >= 0 && c < g.W ? 0x0000ffffu : 0u) |
                                         (rowok && c + 1 >= 0 && c + 1 < g.W ? 0xffff0000u : 0u);
                            }
                        }
                    }
                    // the element offset may be negative (left / top padding): the words read
                    // there are masked, and the strips are not at the start of shared memory
                    uint32_t src = strip + (uint32_t)(2 * (e0 + cq * 16 * a.CS));
                    const uint32_t src_step = (uint32_t)(2 * a.CS);
                    const uint32_t dst0 = bring_u32 + (uint32_t)(((bfirst + tsub) % (2 * a.nbp)) * TC_TILE_BYTES) +
                                          (uint32_t)(cq * 16 * 128);
                    // four channels per batch: all loads first, so that their latencies overlap
#pragma unroll 1
                    for (int c0 = 0; c0 < 16; c0 += 4) {
                        uint32_t w[4][5], sh16[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const uint32_t sa = src + (uint32_t)q * src_step;
                            const uint32_t wa = sa & ~3u;
                            sh16[q] = (sa & 2u) << 3;
                            w[q][0] = lds32(wa); w[q][1] = lds32(wa + 4); w[q][2] = lds32(wa + 8); w[q][3] = lds32(wa + 12);
                            w[q][4] = NN == 8 ? lds32(wa + 16) : 0u;
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            uint32_t o0 = __funnelshift_r(w[q][0], w[q][1], sh16[q]);
                            uint32_t o1 = __funnelshift_r(w[q][1], w[q][2], sh16[q]);
                            uint32_t o2 = __funnelshift_r(w[q][2], w[q][3], sh16[q]);
                            uint32_t o3 = NN == 8 ? __funnelshift_r(w[q][3], w[q][4], sh16[q]) : 0u;
                            if (MODE != 0 && masked) { o0 &= mk[0]; o1 &= mk[1]; o2 &= mk[2]; o3 &= mk[3]; }
                            const int c = c0 + q;
                            sts128(dst0 + (uint32_t)(c * 128) + (uint32_t)((pa ^ (c & 7)) << 4), o0, o1, o2, o3);
                        }
                        src += 4 * src_step;
                    }
                }
                if (cq == 0 && lane < cnt) {
                    sh->tile_id[(bfirst + lane) % TC_IDS] = it.srow * g.TW + it.tw0 + tq * 4 + lane;
                    sh->tile_cb[(bfirst + lane) % TC_IDS] = it.cb;
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane < cnt) ptx::mbar_arrive(ptx::smem_u32(&sh->pair_full[((bfirst + lane) >> 1) % a.nbp]));
            }
            if (!ok) break;
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->strip_empty[sidx]));
            if (++sidx == a.nstrip) { sidx = 0; sphase ^= 1u; }
            b0 += it.nb;
        }
        // An odd number of operand tiles: the last pair has no second tile.  The MMA still
        // reads those 64 rows, and its zero rows of the constant matrix times whatever the
        // buffer holds (possibly NaN patterns) would reach the columns of the valid tile in
        // the other slot: fill the missing tile with zeros.  (The pair's buffer is free: its
        // first tile was written after a wait for pair_empty.)
        if (ok && (nbt & 1) && rw < TC_CQ)
            ok = __all_sync(0xffffffffu, wait_counter(&sh->pairs_consumed, ptx::smem_u32(&sh->tick), (nbt >> 1) - a.nbp + 1,
                                                      ctx, kWaitPairEmpty));
        if (ok && (nbt & 1) && rw < TC_CQ) {
            const uint32_t dst = bring_u32 + (uint32_t)((nbt % (2 * a.nbp)) * TC_TILE_BYTES) + (uint32_t)(rw * 16 * 128);
#pragma unroll
            for (int i = 0; i < 4; ++i) sts128(dst + (uint32_t)((i * 32 + lane) * 16), 0u, 0u, 0u, 0u);
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->pair_full[(nbt >> 1) % a.nbp]));
        }
    } else if (warp >= TC_FIRST_QUANT) {
        // ---------------- quantizers ----------------
        // Two teams of eight warps take the accumulators alternately; in a team warp % 4
        // selects the 32 TMEM lanes and u the tile of the pair (64 columns).
        const int qw = warp - TC_FIRST_QUANT;
        const int quarter = warp & 3, u = (qw >> 2) & 1, team = qw >> 3;
        const int L = quarter * 32 + lane;                 // TMEM lane = accumulator row
        const int slot = L / PL, p = L - slot * PL;
        const bool lane_ok = slot < S && p < P;
        const float sp = tab.in_scale[lane_ok ? p : 0], sl = tab.in_scale_lo[lane_ok ? p : 0];
        const uint32_t taddr0 = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(u * 64);
        const int ngroups = (nbt + 2 * S - 1) / (2 * S);
        if (qw < 4) {
            // The constant matrix goes to tensor memory once per CTA, one copy per slot: row
            // p of the matrix on lane s * PL + p, zeros on every other lane.
#pragma unroll 1
            for (int sl = 0; sl < S; ++sl) {
                const int pp = L - sl * PL;
                const bool has = pp >= 0 && pp < P;
                const uint32_t *row = a.amat + (size_t)(has ? pp : 0) * C::KW;
#pragma unroll
                for (int kc = 0; kc < C::KW / 8; ++kc) {
                    uint32_t v[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[i] = has ? __ldg(row + kc * 8 + i) : 0u;
                    ptx::tmem_st_x8(tmem_base + ((uint32_t)(quarter * 32) << 16) +
                                    (uint32_t)(TC_AMAT_COL + sl * C::KW + kc * 8), v);
                }
            }
            ptx::tmem_st_wait();
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->amat_full));
        }
        for (int grp = team; grp < ngroups; grp += TC_TEAMS) {
            const int acc = team;                          // TC_NACC == TC_TEAMS
            if (!wait_bounded(ptx::smem_u32(&sh->acc_full[acc]), (uint32_t)((grp / TC_NACC) & 1), ctx, kWaitAccFull))
                break;
            ptx::tc_fence_after();
            const uint32_t taddr = taddr0 + (uint32_t)(acc * 128);
            const int b = grp * 2 * S + 2 * slot + u;      // operand tile of this thread
            const bool valid = lane_ok && b < nbt;
            int t = 0, cb = 0;
            if (valid) { t = sh->tile_id[b % TC_IDS]; cb = sh->tile_cb[b % TC_IDS]; }
            int8_t *dst = a.Xq + ((size_t)p * g.T + t) * g.C + cb * TC_CB;
            uint32_t r[32];
            if (GS == 32) {
                float *sd = a.sX + ((size_t)p * g.G + cb * 2) * g.Ts + t;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    ptx::tmem_ld_x32(taddr + (uint32_t)(32 * h), r);
                    ptx::tmem_ld_wait();
                    if (h == 1) {          // both halves are in registers or done: release
                        ptx::tc_fence_before();
                        __syncwarp();
                        if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->acc_empty[acc]));
                    }
                    float scale, inv;
                    group_scale_inv(fabsf(scaled(absmax32(r, 0.f), sp, sl)), scale, inv);
                    if (valid) {
                        codes32(r, sp, sl, inv, dst + 32 * h);
                        sd[(size_t)h * g.Ts] = scale;
                    }
                }
            } else {
                // abs-max over both halves, codes for the second half from the registers,
                // then the first half again from TMEM
                ptx::tmem_ld_x32(taddr, r);
                ptx::tmem_ld_wait();
                const float m = absmax32(r, 0.f);
                ptx::tmem_ld_x32(taddr + 32u, r);
                ptx::tmem_ld_wait();
                float scale, inv;
                group_scale_inv(fabsf(scaled(absmax32(r, m), sp, sl)), scale, inv);
                if (valid) {
                    codes32(r, sp, sl, inv, dst + 32);
                    a.sX[((size_t)p * g.G + cb) * g.Ts + t] = scale;
                }
                ptx::tmem_ld_x32(taddr, r);
                ptx::tmem_ld_wait();
                ptx::tc_fence_before();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_u32(&sh->acc_empty[acc]));
                if (valid) codes32(r, sp, sl, inv, dst);
            }
        }
    }

    ptx::tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after();
        ptx::tmem_dealloc(tmem_base, TC_TMEM_COLS);
    }
}

// The constant matrix per device ordinal and tile size, built by setup_input_transform_tc.
constexpr int kTcMaxDevices = 64;
void *g_amat[kTcMaxDevices][2];

template <int M, int GS, int MODE>
cudaError_t launch_tc(const wfq_plan &plan, const void *x_dev, cudaStream_t stream)
{
    const K1TcPlan &k = plan.k1tc;
    TcArgs a;
    a.x = static_cast<const __half *>(x_dev);
    a.Xq = plan.ws.Xq;
    a.sX = plan.ws.sX;
    a.status = plan.status;
    a.wait_cycles = plan.wait_cycles;
    a.mode = k.mode; a.TBW = k.TBW; a.NCHUNK = k.NCHUNK; a.NCB = k.NCB; a.items = k.items;
    a.CS = k.CS; a.RS = k.RS;
    a.strip_bytes = k.strip_bytes; a.nstrip = k.nstrip; a.nbp = k.nbp;
    a.amat = static_cast<const uint32_t *>(g_amat[plan.device][M == 6 ? 1 : 0]);
    a.debug_skip_item = plan.debug_skip_item;
    if (!a.amat) return cudaErrorInvalidValue;
    auto kern = input_transform_tc_kernel<M, GS, MODE>;
    kern<<<k.grid, TC_THREADS, k.smem, stream>>>(plan.tmap_x, a, plan.geo, plan.tables);
    return cudaGetLastError();
}

template <int M, int GS>
cudaError_t dispatch_mode(const wfq_plan &plan, const void *x, cudaStream_t s)
{
    switch (plan.k1tc.mode) {
        case 0: return launch_tc<M, GS, 0>(plan, x, s);
        case 1: return launch_tc<M, GS, 1>(plan, x, s);
        default: return launch_tc<M, GS, 2>(plan, x, s);
    }
}

template <typename Kernel>
cudaError_t set_smem(Kernel kern)
{
    return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

// The standard-scaled B^T of the paper's supplementary ("Standard Winograd transforms").
const float kBT4[36] = {4, 0, -5, 0, 1, 0,   0, -4, -4, 1, 1, 0,   0, 4, -4, -1, 1, 0,
                        0, -2, -1, 2, 1, 0,  0, 2, -1, -2, 1, 0,   0, 4, 0, -5, 0, 1};
const float kBT6[64] = {
    1, 0, -5.25f, 0, 5.25f, 0, -1, 0,        0, 1, 1, -4.25f, -4.25f, 1, 1, 0,
    0, -1, 1, 4.25f, -4.25f, -1, 1, 0,       0, 0.5f, 0.25f, -2.5f, -1.25f, 2, 1, 0,
    0, -0.5f, 0.25f, 2.5f, -1.25f, -2, 1, 0, 0, 2, 4, -2.5f, -5, 0.5f, 1, 0,
    0, -2, 4, 2.5f, -5, -0.5f, 1, 0,         0, -1, 0, 5.25f, 0, -5.25f, 0, 1};

// [P][KW] 32-bit words: word (p, a * 4 + b / 2) holds BT[i][a] * BT[j][b] for p = i*n + j and
// two consecutive b (fp16; every product is exact; b >= n gives zero), i.e. K index a*8 + b.
template <int M>
void build_amat(std::vector<uint16_t> &out)
{
    using C = TcCfg<M>;
    const float *bt = M == 6 ? kBT6 : kBT4;
    out.assign((size_t)C::P * C::KW * 2, 0);
    for (int p = 0; p < C::P; ++p) {
        const int i = p / C::NN, j = p % C::NN;
        for (int a = 0; a < C::NN; ++a)
            for (int b = 0; b < C::NN; ++b) {
                const __half h = __float2half_rn(bt[i * C::NN + a] * bt[j * C::NN + b]);
                uint16_t bits;
                memcpy(&bits, &h, 2);
                out[(size_t)p * C::KW * 2 + a * 8 + b] = bits;
            }
    }
}

}  // namespace

// Decides whether the tensor-core kernel serves this layer and sizes its launch.
void plan_input_transform_tc(wfq_plan &plan)
{
    K1TcPlan &k = plan.k1tc;
    const Geometry &g = plan.geo;
    k.use = false;
    if (plan.in_dtype != WFQ_F16 || (g.gs != 32 && g.gs != 64) || g.C % TC_CB != 0 || (g.m != 4 && g.m != 6)) return;
    if (plan.sm_count <= 0) return;
    const int n = g.n, m = g.m;
    const long long hw = (long long)g.H * g.W;
    k.nbp = 4;   // operand-tile ring: pairs in flight
    // shared memory left for the strip ring
    const int budget = 227 * 1024 - 1024 /*alignment*/ - (int)sizeof(TcShared) - k.nbp * 2 * TC_TILE_BYTES;
    const int strip_max = budget / 2;       // at least two strips
    k.NCHUNK = 1;
    int mode = -1;
    if (g.W % 8 == 0) {
        // Column chunks of TBW tiles.  A chunk's first column, tw0 * m - 1, lies up to 7 past
        // the 16-byte boundary the box starts at; the box width is 8 modulo 16 elements (bank
        // spread of the patch rows).  Among the chunk sizes whose strip fits twice, take the
        // one with the least work on the busiest CTA (a strip costs about three tiles).
        long long best = -1;
        for (int nch = 1; nch <= g.TW; ++nch) {
            const int tbw = (g.TW + nch - 1) / nch;
            if ((g.TW + tbw - 1) / tbw != nch) continue;
            int bw = (tbw * m + 2 + 7 + 7) / 8 * 8;
            if (bw % 16 == 0) bw += 8;
            if (bw > 256 || TC_CB * n * bw * 2 > strip_max) continue;
            const long long items = (long long)g.N * g.TH * nch * (g.C / TC_CB);
            const long long cost = ((items + plan.sm_count - 1) / plan.sm_count) * (tbw + 3);
            if (best < 0 || cost < best) {
                best = cost;
                mode = 0;
                k.TBW = tbw; k.NCHUNK = nch;
                k.CS = n * bw; k.RS = bw;
                k.strip_bytes = TC_CB * n * bw * 2;
                k.box[0] = (unsigned)bw; k.box[1] = (unsigned)n; k.box[2] = TC_CB;
            }
        }
    } else if ((hw * 2) % 16 == 0 && n * g.W + 8 <= 256) {
        // one box per strip; it starts at the 16-byte boundary below its first element
        mode = 1;
        const int bw = (n * g.W + 7 + 7) / 8 * 8;
        k.TBW = g.TW;
        k.CS = bw; k.RS = g.W;
        k.strip_bytes = TC_CB * bw * 2;
        k.box[0] = (unsigned)bw; k.box[1] = TC_CB; k.box[2] = 1;
    } else if ((hw * TC_CB * 2) % 128 == 0 && hw * TC_CB * 2 <= strip_max) {
        mode = 2;
        k.TBW = g.TH * g.TW;
        k.CS = (int)hw; k.RS = g.W;
        k.strip_bytes = (int)(hw * TC_CB * 2);
    }
    if (mode < 0 || k.strip_bytes > strip_max || k.strip_bytes % 128 != 0) return;
    k.mode = mode; k.NCB = g.C / TC_CB;
    k.items = g.N * (mode == 2 ? 1 : g.TH * k.NCHUNK) * k.NCB;
    int nstrip = budget / k.strip_bytes;
    if (nstrip > TC_MAX_STRIP) nstrip = TC_MAX_STRIP;
    k.nstrip = nstrip;
    k.smem = 1024 + k.nbp * 2 * TC_TILE_BYTES + nstrip * k.strip_bytes + (int)sizeof(TcShared);
    k.grid = k.items < plan.sm_count ? k.items : plan.sm_count;
    k.use = true;
}

// One-time work for the kernels of this file on the current device: attributes and the
// constant matrices (one small device allocation that lives until the process exits).
cudaError_t setup_input_transform_tc()
{
    cudaError_t e = cudaSuccess;
    auto upd = [&](cudaError_t r) { if (e == cudaSuccess) e = r; };
    upd(set_smem(input_transform_tc_kernel<4, 32, 0>)); upd(set_smem(input_transform_tc_kernel<4, 32, 1>));
    upd(set_smem(input_transform_tc_kernel<4, 32, 2>)); upd(set_smem(input_transform_tc_kernel<4, 64, 0>));
    upd(set_smem(input_transform_tc_kernel<4, 64, 1>)); upd(set_smem(input_transform_tc_kernel<4, 64, 2>));
    upd(set_smem(input_transform_tc_kernel<6, 32, 0>)); upd(set_smem(input_transform_tc_kernel<6, 32, 1>));
    upd(set_smem(input_transform_tc_kernel<6, 32, 2>)); upd(set_smem(input_transform_tc_kernel<6, 64, 0>));
    upd(set_smem(input_transform_tc_kernel<6, 64, 1>)); upd(set_smem(input_transform_tc_kernel<6, 64, 2>));
    if (e != cudaSuccess) return e;
    int dev = -1;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) return e;
    if (dev < 0 || dev >= kTcMaxDevices) return cudaErrorInvalidDevice;
    if (!g_amat[dev][0]) {
        std::vector<uint16_t> a4, a6;
        build_amat<4>(a4);
        build_amat<6>(a6);
        char *buf = nullptr;
        if ((e = cudaMalloc(&buf, (a4.size() + a6.size()) * 2)) != cudaSuccess) return e;
        if ((e = cudaMemcpy(buf, a4.data(), a4.size() * 2, cudaMemcpyHostToDevice)) != cudaSuccess ||
            (e = cudaMemcpy(buf + a4.size() * 2, a6.data(), a6.size() * 2, cudaMemcpyHostToDevice)) != cudaSuccess) {
            cudaFree(buf);
            return e;
        }
        g_amat[dev][0] = buf;
        g_amat[dev][1] = buf + a4.size() * 2;
    }
    return cudaSuccess;
}

cudaError_t launch_input_transform_tc(const wfq_plan &plan, const void *x_dev, cudaStream_t stream)
{
    if (plan.device < 0 || plan.device >= kTcMaxDevices) return cudaErrorInvalidDevice;
    if (plan.geo.m == 4)
        return plan.geo.gs == 32 ? dispatch_mode<4, 32>(plan, x_dev, stream)
                                 : dispatch_mode<4, 64>(plan, x_dev, stream);
    return plan.geo.gs == 32 ? dispatch_mode<6, 32>(plan, x_dev, stream)
                             : dispatch_mode<6, 64>(plan, x_dev, stream);
}

}  // namespace wfq
