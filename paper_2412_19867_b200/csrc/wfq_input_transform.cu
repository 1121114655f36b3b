// Fused input transform + group-wise int8 quantization.
//
//   X = S_B V_B x V_B^T S_B   (Section 4.1), fp32, never stored to global memory
//   per (position, tile, channel group): amax -> scale, codes (Section 2 quantizer,
//   one scale per group, dynamic abs-max)
//
// A work item is TB neighbouring tiles of one tile row and CB input channels (one or two
// whole groups); persistent CTAs walk over the items.  Per item, separated by block
// barriers (where shared memory allows it without costing a resident CTA, the next
// item's strip is staged into a second buffer while this one is processed):
//   stage    the zero-padded input strip (n rows x 16 columns x CB channels) goes to
//            shared memory with 4-byte cp.async copies, all in flight at once
//   phase 1  thread <-> (tile, channel): the n x n patch is transformed with the
//            standard-scaled B^T (small integers / dyadic rationals as add/fma chains)
//            and written as fp32 to a shared [tile][position][channel] array (lanes
//            along the channel: conflict free)
//   phase 2  thread <-> (tile, group, position): it reads the group's values of that
//            position with 16-byte loads (rows 4 floats longer than the channel block:
//            conflict free), multiplies them by the caller's per-position factor, takes
//            the abs-max serially, derives scale and reciprocal once, rounds with the
//            1.5*2^23 trick (same result as mul + round-half-even convert; scalar multiply
//            and add, each rounded) and stores 32 codes per 32-byte store.
// The abs-max over a group of up to 64 channels therefore needs no shuffles; groups of 128
// or 256 channels are shared by two or four neighbouring lanes (64 channels each, one or two
// shuffles for the abs-max); other group sizes read shared memory twice instead of holding
// the group in registers.
#include <cuda_fp16.h>

#include "wfq_internal.h"
#include "wfq_ptx.cuh"

namespace wfq {
namespace {

constexpr int K1_THREADS = 128;
constexpr int K1_WP = 16;        // staged columns per row (image columns w_base .. w_base+15)
constexpr int K1_WPV = 24;       // the same where rows are copied in aligned 16-byte pieces (w_base a multiple of 8)

// ---- 1-D input transforms with the standard B^T ------------------------------------

// F(2,3) (the textbook matrices): rows [1,0,-1,0] [0,1,1,0] [0,-1,1,0] [0,1,0,-1]
__device__ __forceinline__ void bt_1d(const float (&d)[4], float (&r)[4])
{
    r[0] = d[0] - d[2];
    r[1] = d[1] + d[2];
    r[2] = d[2] - d[1];
    r[3] = d[1] - d[3];
}

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

// The same two transforms on two columns at once (packed f32x2 arithmetic: one
// instruction per pair, each component rounded as in the scalar form).
__device__ __forceinline__ float2 f2(float v) { return make_float2(v, v); }

__device__ __forceinline__ void bt_1d(const float2 (&d)[4], float2 (&r)[4])
{
    r[0] = __ffma2_rn(f2(-1.f), d[2], d[0]);
    r[1] = __fadd2_rn(d[1], d[2]);
    r[2] = __ffma2_rn(f2(-1.f), d[1], d[2]);
    r[3] = __ffma2_rn(f2(-1.f), d[3], d[1]);
}

__device__ __forceinline__ void bt_1d(const float2 (&d)[6], float2 (&r)[6])
{
    r[0] = __ffma2_rn(f2(4.f), d[0], __ffma2_rn(f2(-5.f), d[2], d[4]));
    const float2 a = __ffma2_rn(f2(-4.f), d[2], d[4]);
    const float2 b = __ffma2_rn(f2(-4.f), d[1], d[3]);
    r[1] = __fadd2_rn(a, b);
    r[2] = __ffma2_rn(f2(-1.f), b, a);
    const float2 c = __ffma2_rn(f2(-1.f), d[2], d[4]);
    const float2 t = __ffma2_rn(f2(-1.f), d[1], d[3]);
    r[3] = __ffma2_rn(f2(2.f), t, c);
    r[4] = __ffma2_rn(f2(-2.f), t, c);
    r[5] = __ffma2_rn(f2(4.f), d[1], __ffma2_rn(f2(-5.f), d[3], d[5]));
}

__device__ __forceinline__ void bt_1d(const float2 (&d)[8], float2 (&r)[8])
{
    r[0] = __ffma2_rn(f2(5.25f), __ffma2_rn(f2(-1.f), d[2], d[4]), __ffma2_rn(f2(-1.f), d[6], d[0]));
    r[7] = __ffma2_rn(f2(5.25f), __ffma2_rn(f2(-1.f), d[5], d[3]), __ffma2_rn(f2(-1.f), d[1], d[7]));
    const float2 a = __ffma2_rn(f2(-4.25f), d[4], __fadd2_rn(d[2], d[6]));
    const float2 b = __ffma2_rn(f2(-4.25f), d[3], __fadd2_rn(d[1], d[5]));
    r[1] = __fadd2_rn(a, b);
    r[2] = __ffma2_rn(f2(-1.f), b, a);
    const float2 c = __ffma2_rn(f2(-1.25f), d[4], __ffma2_rn(f2(0.25f), d[2], d[6]));
    const float2 e = __ffma2_rn(f2(2.f), d[5], __ffma2_rn(f2(-2.5f), d[3], __fmul2_rn(f2(0.5f), d[1])));
    r[3] = __fadd2_rn(c, e);
    r[4] = __ffma2_rn(f2(-1.f), e, c);
    const float2 f = __ffma2_rn(f2(-5.f), d[4], __ffma2_rn(f2(4.f), d[2], d[6]));
    const float2 g = __ffma2_rn(f2(0.5f), d[5], __ffma2_rn(f2(-2.5f), d[3], __fmul2_rn(f2(2.f), d[1])));
    r[5] = __fadd2_rn(f, g);
    r[6] = __ffma2_rn(f2(-1.f), g, f);
}

__device__ __forceinline__ float to_float32(float v) { return v; }
__device__ __forceinline__ float to_float32(__half v) { return __half2float(v); }

// ---- patch load from the staged strip ---------------------------------------------
// `ch` points at the channel's plane in smem; `col0` is the (even) smem column whose
// successor is the tile's first input column.
template <int NN>
__device__ __forceinline__ void load_patch(const __half *ch, int col0, float (&d)[NN][NN])
{
#pragma unroll
    for (int a = 0; a < NN; ++a) {
        const __half2 *row = reinterpret_cast<const __half2 *>(ch + a * K1_WP + col0);
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

// The same from a strip staged in 16-byte pieces (rows of K1_WPV columns, channel stride a
// multiple of 16 bytes and an odd number of 16-byte units): 16-byte loads, for which the eight
// lanes of a quarter warp then hit eight different groups of four banks.  `k0` is the first of
// the two 16-byte pieces that hold columns col0 .. col0 + NN + 1, WO the 32-bit word of col0
// inside them (col0 is even); both are the same for all lanes of the warp.
template <int NN, int WO>
__device__ __forceinline__ void load_patch_vec(const __half *ch, int k0, float (&d)[NN][NN])
{
#pragma unroll
    for (int a = 0; a < NN; ++a) {
        const uint4 *row = reinterpret_cast<const uint4 *>(ch + a * K1_WPV) + k0;
        const uint4 q0 = row[0], q1 = row[1];
        const uint32_t w[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
        float v[NN + 2];
#pragma unroll
        for (int i = 0; i < (NN + 2) / 2; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[WO + i]));
            v[2 * i] = f.x;
            v[2 * i + 1] = f.y;
        }
#pragma unroll
        for (int b = 0; b < NN; ++b) d[a][b] = v[b + 1];
    }
}
template <int NN>
__device__ __forceinline__ void load_patch_vec(const __half *ch, int col0, float (&d)[NN][NN])
{
    const int k0 = col0 >> 3;
    switch ((col0 & 7) >> 1) {            // warp-uniform
        case 0: load_patch_vec<NN, 0>(ch, k0, d); break;
        case 1: load_patch_vec<NN, 1>(ch, k0, d); break;
        case 2: load_patch_vec<NN, 2>(ch, k0, d); break;
        default: load_patch_vec<NN, 3>(ch, k0, d); break;
    }
}
template <int NN>
__device__ __forceinline__ void load_patch_vec(const float *, int, float (&)[NN][NN]) {}   // fp16 only

template <int NN>
__device__ __forceinline__ void load_patch(const float *ch, int col0, float (&d)[NN][NN])
{
#pragma unroll
    for (int a = 0; a < NN; ++a)
#pragma unroll
        for (int b = 0; b < NN; ++b) d[a][b] = ch[a * K1_WP + col0 + 1 + b];
}

// Codes: round v*inv to the nearest integer (ties to even) and keep the low byte.
// fl32(v*inv) + 1.5*2^23 is exact up to the rounding to an integer, and the sum's bit
// pattern is 0x4B400000 + q for |q| <= 2^22.
// Packed f32x2 multiply (one instruction for two products, each correctly rounded).
__device__ __forceinline__ float2 mul2_rn(float2 a, float2 b)
{
    float2 d;
    asm("{\n\t.reg .b64 ra, rb, rd;\n\t"
        "mov.b64 ra, {%2, %3};\n\tmov.b64 rb, {%4, %5};\n\t"
        "mul.rn.f32x2 rd, ra, rb;\n\t"
        "mov.b64 {%0, %1}, rd;\n\t}"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}

// One code: fl32(v*inv), then + 1.5*2^23; two separately rounded scalar operations, as
// the quantizer is defined.  (A packed multiply followed by a packed add, written as
// intrinsics or as PTX, came out as one fused multiply-add: it rounds once and decides
// near-ties differently, and a single differing code of an outlier-dominated group can
// move the final output by more than the end-to-end tolerance.)
__device__ __forceinline__ uint32_t code_bits(float v, float inv)
{
    return __float_as_uint(__fadd_rn(__fmul_rn(v, inv), 12582912.f));
}
__device__ __forceinline__ uint32_t codes4(float4 v, float inv)
{
    return __byte_perm(__byte_perm(code_bits(v.x, inv), code_bits(v.y, inv), 0x0040),
                       __byte_perm(code_bits(v.z, inv), code_bits(v.w, inv), 0x0040), 0x5410);
}

// X = Z * (s + sl), rounded once: fma(z, s, z * sl) (the factor is held as two floats).
__device__ __forceinline__ float4 scale4(float4 v, float2 s2, float2 sl2)
{
    const float2 a = make_float2(v.x, v.y), b = make_float2(v.z, v.w);
    const float2 lo = __ffma2_rn(a, s2, mul2_rn(a, sl2));
    const float2 hi = __ffma2_rn(b, s2, mul2_rn(b, sl2));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
}

__device__ __forceinline__ float absmax4(float m, float4 v)
{
    return fmaxf(fmaxf(fmaxf(m, fabsf(v.x)), fabsf(v.y)), fmaxf(fabsf(v.z), fabsf(v.w)));
}

// 32-byte store (one full sector); `p` must be 32-byte aligned.
__device__ __forceinline__ void st_global_v8_b32(void *p, uint32_t a, uint32_t b, uint32_t c, uint32_t d,
                                                 uint32_t e, uint32_t f, uint32_t g, uint32_t h)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d), "r"(e), "r"(f), "r"(g), "r"(h)
                 : "memory");
}

__device__ __forceinline__ void cp_async_4(uint32_t dst, const void *src, bool valid)
{
    const int n = valid ? 4 : 0;   // 0 source bytes: the destination is zero filled
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, bool valid)
{
    const int n = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit()
{
    asm volatile("cp.async.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void cp_async_wait_group()   // all but the N newest groups are done
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// ---- strip staging -----------------------------------------------------------------
// smem column j of the strip holds image column w_base + j (w_base even); rows are
// image rows h_base .. h_base + NN - 1; anything outside the image is zero.
template <typename Tin, int NN>
__device__ __forceinline__ void stage_strip(Tin *sm, const Tin *__restrict__ x, const Geometry &g,
                                            const K1Params &prm, int img, int c_base, int h_base,
                                            int w_base)
{
    const size_t HW = (size_t)g.H * g.W;
    const Tin *ximg = x + ((size_t)img * g.C + c_base) * HW;
    // Each thread owns one (row, column) slot of the strip and walks over the channels,
    // so its bounds test and addresses are computed once.
    if (sizeof(Tin) == 2 && prm.vec16) {
        // 16-byte pieces: W and w_base are multiples of 8 and x is 16-byte aligned, so a piece
        // lies inside the image or outside it as a whole
        constexpr int CPR = K1_WPV / 8;                        // copies per row
        constexpr int ROWS = K1_THREADS / CPR;
        constexpr int CSLOTS = ROWS / NN;
        const int jc = threadIdx.x % CPR;
        const int rs = threadIdx.x / CPR;
        const int a = rs % NN, cslot = rs / NN;
        if (cslot < CSLOTS) {
            const int h = h_base + a, w = w_base + 8 * jc;
            const bool ok = h >= 0 && h < g.H && w >= 0 && w < g.W;
            const Tin *src = ok ? ximg + (size_t)cslot * HW + (size_t)h * g.W + w : x;
            const size_t src_step = ok ? (size_t)CSLOTS * HW : 0;
            uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(sm)) +
                           (uint32_t)((cslot * prm.CS + a * K1_WPV + 8 * jc) * sizeof(Tin));
            const uint32_t dst_step = (uint32_t)(CSLOTS * prm.CS * sizeof(Tin));
            for (int c = cslot; c < prm.CB; c += CSLOTS) {
                cp_async_16(dst, src, ok);
                src += src_step;
                dst += dst_step;
            }
        }
    } else if (sizeof(Tin) == 4 || prm.pair) {
        constexpr int EPC = sizeof(Tin) == 4 ? 1 : 2;          // elements per 4-byte copy
        constexpr int CPR = K1_WP / EPC;                       // copies per row
        constexpr int ROWS = K1_THREADS / CPR;                 // rows covered by one pass
        constexpr int CSLOTS = ROWS / NN;                      // channels covered by one pass
        const int jc = threadIdx.x % CPR;
        const int rs = threadIdx.x / CPR;
        const int a = rs % NN, cslot = rs / NN;
        if (cslot < CSLOTS) {
            const int h = h_base + a, w = w_base + EPC * jc;
            const bool ok = h >= 0 && h < g.H && w >= 0 && w < g.W;   // W even for pairs: both or none
            const Tin *src = ok ? ximg + (size_t)cslot * HW + (size_t)h * g.W + w : x;
            const size_t src_step = ok ? (size_t)CSLOTS * HW : 0;
            uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(sm)) +
                           (uint32_t)((cslot * prm.CS + a * K1_WP + EPC * jc) * sizeof(Tin));
            const uint32_t dst_step = (uint32_t)(CSLOTS * prm.CS * sizeof(Tin));
            for (int c = cslot; c < prm.CB; c += CSLOTS) {
                cp_async_4(dst, src, ok);
                src += src_step;
                dst += dst_step;
            }
        }
    } else {
        // fp16 with an odd W or a 2-byte aligned base: plain 2-byte loads, eight channels
        // in flight per thread (these copies are complete when the function returns)
        constexpr int ROWS = K1_THREADS / K1_WP;               // 8 row slots per pass
        constexpr int CSLOTS = ROWS / NN;                      // 1
        const int j = threadIdx.x % K1_WP;
        const int rs = threadIdx.x / K1_WP;
        const int a = rs % NN, cslot = rs / NN;
        if (cslot < CSLOTS) {
            const int h = h_base + a, w = w_base + j;
            const bool ok = h >= 0 && h < g.H && w >= 0 && w < g.W;
            const Tin *src = ximg + (size_t)cslot * HW + (size_t)h * g.W + w;
            Tin *dst = sm + cslot * prm.CS + a * K1_WP + j;
            for (int c = cslot; c < prm.CB; c += 8 * CSLOTS) {     // CB is a multiple of 32
                Tin v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = ok ? __ldg(src + (size_t)u * CSLOTS * HW) : Tin(0);
#pragma unroll
                for (int u = 0; u < 8; ++u) dst[u * CSLOTS * prm.CS] = v[u];
                src += (size_t)8 * CSLOTS * HW;
                dst += 8 * CSLOTS * prm.CS;
            }
        }
    }
}

// Z = B^T d B with the standard B^T, written to out[p * pitch] for p = i*NN + j.
template <int NN>
__device__ __forceinline__ void transform_patch(float (&d)[NN][NN], float *__restrict__ out, int pitch)
{
#pragma unroll
    for (int b = 0; b < NN; b += 2) {   // columns, two at a time: d <- B^T d
        float2 col[NN], r[NN];
#pragma unroll
        for (int a = 0; a < NN; ++a) col[a] = make_float2(d[a][b], d[a][b + 1]);
        bt_1d(col, r);
#pragma unroll
        for (int a = 0; a < NN; ++a) {
            d[a][b] = r[a].x;
            d[a][b + 1] = r[a].y;
        }
    }
#pragma unroll
    for (int i = 0; i < NN; ++i) {   // rows: Z[i][:] = (B^T d)[i][:] B
        float r[NN];
        bt_1d(d[i], r);
#pragma unroll
        for (int j = 0; j < NN; ++j) out[(i * NN + j) * pitch] = r[j];
    }
}

// ---- group abs-max and scale (the quantizer of Section 2, one scale per group) ------
// amax >= 0.  Returns the stored scale and the reciprocal used for the codes.
__device__ __forceinline__ void group_scale(float amax, float &scale, float &inv)
{
    const bool nz = amax >= 1e-30f;
    scale = nz ? __fdiv_rn(amax, 127.f) : 0.f;
    inv = nz ? __fdiv_rn(127.f, amax) : 0.f;
}

// ---- phase 2 of a work item: quantize, one (tile, group, position) per thread -------------
// Zs holds the transformed values of `ntile` tiles as [tile][position][CB + 4] fp32; the item is
// tiles tw0 .. of tile row `srow` (= image * TH + tile row) and channels c_base .. c_base + CB.
template <int P, int GSR, int SPLIT>
__device__ __forceinline__ void quantize_item(const float *__restrict__ Zs, int CBP, int ntile, int ng, int gs,
                                              int srow, int tw0, int c_base, const Geometry &g,
                                              const ScaleTables &tab, int8_t *__restrict__ Xq,
                                              float *__restrict__ sX)
{
    // X = Z * (caller's per-position factor) is formed here, one rounding, as the
    // quantizer's input; then abs-max, scale, reciprocal and codes.
    const int g_base = c_base / gs;
    if constexpr (GSR > 0) {
        // whole warps walk the loop so that the lanes sharing a group can shuffle
        const int tasks = ntile * ng * P * SPLIT;
        for (int base = 0; base < tasks; base += K1_THREADS) {
            const int task = base + (int)threadIdx.x;
            const bool act = task < tasks;          // the lanes of a group are all in or all out
            const int tk = act ? task : 0;
            const int part = tk % SPLIT, rest = tk / SPLIT;
            const int q = rest / P, p = rest - q * P;
            const int tl = q / ng, grp = q - tl * ng;
            const int t = srow * g.TW + tw0 + tl;
            const float4 *src = reinterpret_cast<const float4 *>(Zs + (size_t)(tl * P + p) * CBP + grp * gs +
                                                                 part * GSR);
            int8_t *dst = Xq + ((size_t)p * g.T + t) * g.C + c_base + grp * gs + part * GSR;
            const float sp = tab.in_scale[p], sl = tab.in_scale_lo[p];
            const float2 sp2 = make_float2(sp, sp), sl2 = make_float2(sl, sl);
            float4 v[GSR / 4];
            float amax = 0.f;
#pragma unroll
            for (int k = 0; k < GSR / 4; ++k) {
                v[k] = scale4(src[k], sp2, sl2);
                amax = absmax4(amax, v[k]);
            }
            if constexpr (SPLIT >= 2) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
            if constexpr (SPLIT >= 4) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
            float scale, inv;
            group_scale(amax, scale, inv);
            if (act) {
#pragma unroll
                for (int k = 0; k < GSR / 32; ++k)        // 32 codes = one full sector per store
                    st_global_v8_b32(dst + 32 * k, codes4(v[8 * k], inv), codes4(v[8 * k + 1], inv),
                                     codes4(v[8 * k + 2], inv), codes4(v[8 * k + 3], inv),
                                     codes4(v[8 * k + 4], inv), codes4(v[8 * k + 5], inv),
                                     codes4(v[8 * k + 6], inv), codes4(v[8 * k + 7], inv));
                if (part == 0) sX[((size_t)p * g.G + g_base + grp) * g.Ts + t] = scale;
            }
        }
    } else {
        const int tasks = ntile * ng * P;
        for (int task = threadIdx.x; task < tasks; task += K1_THREADS) {
            const int q = task / P, p = task - q * P;
            const int tl = q / ng, grp = q - tl * ng;
            const int t = srow * g.TW + tw0 + tl;
            const float4 *src = reinterpret_cast<const float4 *>(Zs + (size_t)(tl * P + p) * CBP + grp * gs);
            int8_t *dst = Xq + ((size_t)p * g.T + t) * g.C + c_base + grp * gs;
            const float sp = tab.in_scale[p], sl = tab.in_scale_lo[p];
            const float2 sp2 = make_float2(sp, sp), sl2 = make_float2(sl, sl);
            float scale, inv;
            float amax = 0.f;
            for (int k = 0; k < gs / 4; ++k) amax = absmax4(amax, scale4(src[k], sp2, sl2));
            group_scale(amax, scale, inv);
            for (int k = 0; k < gs / 32; ++k)
                st_global_v8_b32(dst + 32 * k, codes4(scale4(src[8 * k], sp2, sl2), inv),
                                 codes4(scale4(src[8 * k + 1], sp2, sl2), inv), codes4(scale4(src[8 * k + 2], sp2, sl2), inv),
                                 codes4(scale4(src[8 * k + 3], sp2, sl2), inv), codes4(scale4(src[8 * k + 4], sp2, sl2), inv),
                                 codes4(scale4(src[8 * k + 5], sp2, sl2), inv), codes4(scale4(src[8 * k + 6], sp2, sl2), inv),
                                 codes4(scale4(src[8 * k + 7], sp2, sl2), inv));
            sX[((size_t)p * g.G + g_base + grp) * g.Ts + t] = scale;
        }
    }}

// ---- the kernel ----------------------------------------------------------------------
// GSR > 0: channels a thread holds in registers during phase 2 (32 or 64); a group is GSR *
// SPLIT channels, SPLIT neighbouring lanes share it and exchange their abs-max by shuffle.
// GSR == 0: any group size, one thread per group, phase 2 reads shared memory twice.
template <int M, typename Tin, int GSR, int SPLIT>
__global__ void __launch_bounds__(K1_THREADS, 4)
input_transform_kernel(const Tin *__restrict__ x, int8_t *__restrict__ Xq,
                       float *__restrict__ sX, Geometry g, ScaleTables tab, K1Params prm)
{
    constexpr int NN = M + 2;
    constexpr int P = NN * NN;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // The contraction kernel launched behind this one may start its prologue and its filter
    // stream now (it waits for this grid's completion before it touches Xq or sX).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // This kernel itself is launched with programmatic stream serialization: it may become
    // resident while the kernel before it in the stream (normally the previous layer's output
    // transform) drains, and waits here, before its first global access, until that kernel has
    // completed and its writes are visible.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // two strip buffers (the next item is staged while this one is transformed), then Z
    float *Zs = reinterpret_cast<float *>(smem_raw + (1 + prm.dbuf) * prm.strip_bytes);   // [tile][position][CBP]
    const int CBP = prm.CB + 4;   // 16-byte aligned rows an odd number of 16-byte units apart

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int NWARP = K1_THREADS / 32;
    const int cb32 = prm.CB >> 5;
    const int gs = GSR > 0 ? GSR * SPLIT : g.gs;
    const int ng = prm.CB / gs;

    // item -> (tile row, chunk of tiles, channel block); channel blocks vary fastest so
    // that CTAs running side by side read the same image rows
    auto stage_item = [&](int item, int buf) {
        const int cblk = item % prm.NCB, rest = item / prm.NCB;
        const int srow = rest / prm.NCH, chunk = rest - srow * prm.NCH;
        const int img = srow / g.TH, th = srow - img * g.TH;
        // first staged column: two left of the first tile's first output column, or (16-byte
        // pieces) the multiple of 8 at or below the first input column
        const int first = chunk * prm.TB * M - 1;
        const int w_base = prm.vec16 ? ((first + 8) & ~7) - 8 : first - 1;
        stage_strip<Tin, NN>(reinterpret_cast<Tin *>(smem_raw + buf * prm.strip_bytes), x, g, prm, img,
                             cblk * prm.CB, th * M - 1, w_base);
        cp_async_commit();
    };

    int item = blockIdx.x;
    if (prm.dbuf && item < prm.items) stage_item(item, 0);
    for (int it = 0; item < prm.items; ++it, item += gridDim.x) {
        const int buf = prm.dbuf ? (it & 1) : 0;
        const int next = item + gridDim.x;
        if (!prm.dbuf) {
            // one buffer: this item's copies were issued after the previous item's patches had been
            // read (below), and landed while that item was quantized
            if (it == 0) stage_item(item, 0);
            cp_async_wait_group<0>();
        } else if (next < prm.items) {
            stage_item(next, buf ^ 1);
            cp_async_wait_group<1>();          // this item's copies have landed
        } else {
            cp_async_wait_group<0>();
        }
        __syncthreads();

        const Tin *strip = reinterpret_cast<const Tin *>(smem_raw + buf * prm.strip_bytes);
        const int cblk = item % prm.NCB, rest = item / prm.NCB;
        const int srow = rest / prm.NCH, chunk = rest - srow * prm.NCH;   // srow = img*TH + th
        const int tw0 = chunk * prm.TB;
        const int ntile = min(prm.TB, g.TW - tw0);
        const int c_base = cblk * prm.CB;

        // ---- phase 1: transform, one (tile, channel) per thread ----------------------
        const int voff = tw0 * M - 2 - (((tw0 * M - 1 + 8) & ~7) - 8);   // 16-byte pieces: column of tile 0 minus one
        for (int wt = warp; wt < ntile * cb32; wt += NWARP) {
            const int tl = wt / cb32;
            const int c = (wt - tl * cb32) * 32 + lane;
            float d[NN][NN];
            if (sizeof(Tin) == 2 && prm.vec16) load_patch_vec<NN>(strip + c * prm.CS, tl * M + voff, d);
            else load_patch<NN>(strip + c * prm.CS, tl * M, d);
            transform_patch<NN>(d, Zs + (size_t)tl * P * CBP + c, CBP);
        }
        __syncthreads();
        if (!prm.dbuf && next < prm.items) stage_item(next, 0);   // the strip buffer is free: refill it now

        quantize_item<P, GSR, SPLIT>(Zs, CBP, ntile, ng, gs, srow, tw0, c_base, g, tab, Xq, sX);
        __syncthreads();   // Z and this strip buffer are free again
    }
}

// ---- the same for an NHWC input ---------------------------------------------------------
// x[N][H][W][C]: the channels are innermost, so the strip of a work item is one 4-D TMA box
// {CB channels, TB * m + 2 columns, n rows, 1 image} (zero fill outside the image, no alignment
// condition on the row or column it starts at) and lands as [row][column][channel]; a thread
// reads its patch with the lanes along the channels (no bank conflicts, no realignment).  One
// thread issues the copy of an item as soon as the buffer it goes to has been read; everything
// else is the kernel above: transform, [tile][position][channel] array, quantize_item.
struct K1NhwcShared {
    uint64_t full[2];        // the strip of a buffer has landed
    volatile int abort;
};

template <int M, typename Tin, int GSR, int SPLIT>
__global__ void __launch_bounds__(K1_THREADS, 4)
input_transform_nhwc_kernel(const __grid_constant__ CUtensorMap tmx, int8_t *__restrict__ Xq,
                            float *__restrict__ sX, Geometry g, ScaleTables tab, K1Params prm, int *status,
                            long long wait_cycles)
{
    constexpr int NN = M + 2;
    constexpr int P = NN * NN;
    extern __shared__ __align__(16) unsigned char smem_dyn[];
    __shared__ K1NhwcShared sh;
    // a TMA destination must be 128-byte aligned; the dynamic part starts wherever the static part
    // ends, so the strips start at the next multiple of 128 (the launch adds 128 bytes for this)
    unsigned char *smem_raw = reinterpret_cast<unsigned char *>(
        (reinterpret_cast<uintptr_t>(smem_dyn) + 127) & ~(uintptr_t)127);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    float *Zs = reinterpret_cast<float *>(smem_raw + (1 + prm.dbuf) * prm.strip_bytes);   // [tile][position][CBP]
    const int CBP = prm.CB + 4;
    const int WB = prm.TB * M + 2;                     // columns of the box
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    constexpr int NWARP = K1_THREADS / 32;
    const int cb32 = prm.CB >> 5;
    const int gs = GSR > 0 ? GSR * SPLIT : g.gs;
    const int ng = prm.CB / gs;
    const WaitCtx ctx{&sh.abort, status, wait_cycles};
    const uint32_t box_bytes = (uint32_t)(NN * WB * prm.CB * (int)sizeof(Tin));

    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_u32(&sh.full[0]), 1);
        ptx::mbar_init(ptx::smem_u32(&sh.full[1]), 1);
        sh.abort = 0;
        ptx::fence_mbar_init();
        ptx::prefetch_tmap(&tmx);
    }
    __syncthreads();

    // thread 0 only
    auto issue = [&](int item, int buf) {
        const int cblk = item % prm.NCB, rest = item / prm.NCB;
        const int srow = rest / prm.NCH, chunk = rest - srow * prm.NCH;
        const int img = srow / g.TH, th = srow - img * g.TH;
        const uint32_t bar = ptx::smem_u32(&sh.full[buf]);
        ptx::mbar_arrive_expect_tx(bar, box_bytes);
        ptx::tma_load_4d(ptx::smem_u32(smem_raw + buf * prm.strip_bytes), &tmx, bar, cblk * prm.CB,
                         chunk * prm.TB * M - 1, th * M - 1, img);
    };

    const int stride = (int)gridDim.x;
    int item = blockIdx.x;
    int issued = 0;                                     // items whose copy has been issued (thread 0)
    if (threadIdx.x == 0) {
        if (item < prm.items) { issue(item, 0); ++issued; }
        if (prm.dbuf && item + stride < prm.items) { issue(item + stride, 1); ++issued; }
    }
    bool ok = true;
    int it = 0;
    for (; item < prm.items; ++it, item += stride) {
        const int buf = prm.dbuf ? (it & 1) : 0;
        const uint32_t parity = (uint32_t)(prm.dbuf ? (it >> 1) : it) & 1u;
        ok = wait_bounded(ptx::smem_u32(&sh.full[buf]), parity, ctx, kWaitStripFull);
        if (!ok) break;

        const Tin *strip = reinterpret_cast<const Tin *>(smem_raw + buf * prm.strip_bytes);
        const int cblk = item % prm.NCB, rest = item / prm.NCB;
        const int srow = rest / prm.NCH, chunk = rest - srow * prm.NCH;
        const int tw0 = chunk * prm.TB;
        const int ntile = min(prm.TB, g.TW - tw0);
        const int c_base = cblk * prm.CB;

        // ---- phase 1: transform, one (tile, channel) per thread ----------------------
        for (int wt = warp; wt < ntile * cb32; wt += NWARP) {
            const int tl = wt / cb32;
            const int c = (wt - tl * cb32) * 32 + lane;
            float d[NN][NN];
            const Tin *src = strip + (size_t)(tl * M) * prm.CB + c;
#pragma unroll
            for (int a = 0; a < NN; ++a)
#pragma unroll
                for (int b = 0; b < NN; ++b) d[a][b] = to_float32(src[(a * WB + b) * prm.CB]);
            transform_patch<NN>(d, Zs + (size_t)tl * P * CBP + c, CBP);
        }
        __syncthreads();
        // the strip buffer has been read: the item that uses it next may be copied now
        if (threadIdx.x == 0) {
            const int nxt = item + (prm.dbuf ? 2 : 1) * stride;
            if (nxt < prm.items) { issue(nxt, buf); ++issued; }
        }
        quantize_item<P, GSR, SPLIT>(Zs, CBP, ntile, ng, gs, srow, tw0, c_base, g, tab, Xq, sX);
        __syncthreads();   // Z is free again
    }
    if (!ok && threadIdx.x == 0) {
        // a copy never arrived: give the ones still in flight a bounded time to land before the
        // shared memory goes away (copies issued: `issued`, consumed: `it`)
        for (int k = it; k < issued; ++k) {
            const int b = prm.dbuf ? (k & 1) : 0;
            drain(ptx::smem_u32(&sh.full[b]), (uint32_t)(prm.dbuf ? (k >> 1) : k) & 1u, wait_cycles / 16);
        }
    }
}

// Resident CTAs per SM and the attribute calls need the kernel symbol: one entry per
// instantiation.
template <int M, typename Tin, int GSR, int SPLIT>
int k1_resident(size_t smem)
{
    return resident_ctas_per_sm(input_transform_kernel<M, Tin, GSR, SPLIT>, K1_THREADS, smem, 32);
}

template <int M, typename Tin, int GSR, int SPLIT>
cudaError_t k1_setup()
{
    auto kern = input_transform_kernel<M, Tin, GSR, SPLIT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,
                                (int)cudaSharedmemCarveoutMaxShared);
}

template <int M, typename Tin, int GSR, int SPLIT>
cudaError_t launch_k1(const wfq_plan &plan, const void *x_dev, cudaStream_t stream)
{
    // 16-byte pieces need a 16-byte aligned x; the plan holds a second parameter set without them
    const bool vec = plan.k1v.vec16 && plan.k1_choice != 3 && (reinterpret_cast<uintptr_t>(x_dev) & 15u) == 0;
    const K1Params &prm = vec ? plan.k1v : plan.k1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)prm.grid);
    cfg.blockDim = dim3(K1_THREADS);
    cfg.dynamicSmemBytes = prm.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, input_transform_kernel<M, Tin, GSR, SPLIT>, static_cast<const Tin *>(x_dev),
                              plan.ws.Xq, plan.ws.sX, plan.geo, plan.tables, prm);
}

template <int M, typename Tin, int GSR, int SPLIT>
int k1n_resident(size_t smem)
{
    return resident_ctas_per_sm(input_transform_nhwc_kernel<M, Tin, GSR, SPLIT>, K1_THREADS, smem, 32);
}

template <int M, typename Tin, int GSR, int SPLIT>
cudaError_t k1n_setup()
{
    auto kern = input_transform_nhwc_kernel<M, Tin, GSR, SPLIT>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 226 * 1024);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout,
                                (int)cudaSharedmemCarveoutMaxShared);
}

template <int M, typename Tin, int GSR, int SPLIT>
cudaError_t launch_k1n(const wfq_plan &plan, cudaStream_t stream)
{
    const K1Params &prm = plan.k1n;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)prm.grid);
    cfg.blockDim = dim3(K1_THREADS);
    cfg.dynamicSmemBytes = prm.smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, input_transform_nhwc_kernel<M, Tin, GSR, SPLIT>, plan.tmap_xn, plan.ws.Xq,
                              plan.ws.sX, plan.geo, plan.tables, prm, plan.status, plan.wait_cycles);
}

// What to do with the instantiation that serves (m, dtype, group size).
enum K1Op { kK1Launch, kK1Resident, kK1Setup, kK1nLaunch, kK1nResident, kK1nSetup };

template <int M, typename Tin>
long long k1_by_gs(K1Op op, int gs, const wfq_plan *plan, const void *x, cudaStream_t s, size_t smem)
{
#define WFQ_K1_CASE(GSR, SPLIT)                                                        \
    switch (op) {                                                                      \
        case kK1Launch: return (long long)launch_k1<M, Tin, GSR, SPLIT>(*plan, x, s);  \
        case kK1Resident: return k1_resident<M, Tin, GSR, SPLIT>(smem);                \
        case kK1Setup: return (long long)k1_setup<M, Tin, GSR, SPLIT>();               \
        case kK1nLaunch: return (long long)launch_k1n<M, Tin, GSR, SPLIT>(*plan, s);   \
        case kK1nResident: return k1n_resident<M, Tin, GSR, SPLIT>(smem);              \
        default: return (long long)k1n_setup<M, Tin, GSR, SPLIT>();                    \
    }
    if (gs == 32) { WFQ_K1_CASE(32, 1) }
    if (gs == 64) { WFQ_K1_CASE(64, 1) }
    if (gs == 128) { WFQ_K1_CASE(64, 2) }
    if (gs == 256) { WFQ_K1_CASE(64, 4) }
    WFQ_K1_CASE(0, 1)
#undef WFQ_K1_CASE
}

long long k1_op(K1Op op, int m, bool f16, int gs, const wfq_plan *plan, const void *x, cudaStream_t s,
                size_t smem)
{
    if (m == 2)
        return f16 ? k1_by_gs<2, __half>(op, gs, plan, x, s, smem) : k1_by_gs<2, float>(op, gs, plan, x, s, smem);
    if (m == 4)
        return f16 ? k1_by_gs<4, __half>(op, gs, plan, x, s, smem) : k1_by_gs<4, float>(op, gs, plan, x, s, smem);
    return f16 ? k1_by_gs<6, __half>(op, gs, plan, x, s, smem) : k1_by_gs<6, float>(op, gs, plan, x, s, smem);
}

}  // namespace

namespace {

void plan_k1(wfq_plan &plan, K1Params &prm, bool vec16)
{
    const Geometry &g = plan.geo;
    const bool f16 = plan.in_dtype == WFQ_F16;
    const int NN = g.n, P = g.P, M = g.m;
    const int esz = f16 ? 2 : 4;
    prm.vec16 = vec16 ? 1 : 0;
    prm.TB = (K1_WP - 3) / M;                      // 2 tiles for F(6,3), 3 for F(4,3)
    prm.CB = g.gs;
    if (g.gs == 32 && g.C % 64 == 0) prm.CB = 64;  // two groups per CTA
    // channel stride: an odd number of 32-bit words, so lanes that walk over channels
    // hit different banks; with 16-byte pieces an odd number of 16-byte units (16-byte loads)
    int cs = NN * K1_WP;
    if (vec16) { cs = NN * K1_WPV; if ((cs / 8) % 2 == 0) cs += 8; }
    else if (esz == 2) { cs += 2; if ((cs / 2) % 2 == 0) cs += 2; }
    else if (cs % 2 == 0) cs += 1;
    prm.CS = cs;
    prm.strip_bytes = (prm.CB * cs * esz + 15) / 16 * 16;
    prm.pair = (g.W % 2 == 0);                     // x is 4-byte aligned (checked by the entry points)
    auto smem_bytes = [&]() {
        return (1 + prm.dbuf) * (size_t)prm.strip_bytes + (size_t)prm.TB * P * (prm.CB + 4) * sizeof(float);
    };
    // Large groups get fewer tiles per item (aim: two or more CTAs per SM).  The second
    // strip buffer is used only where it does not cost a resident CTA (registers allow four).
    prm.dbuf = 0;
    while (prm.TB > 1 && smem_bytes() > 113 * 1024) --prm.TB;
    // the same number of chunks per tile row with evenly sized chunks (four tiles: 2 + 2, not 3 + 1)
    prm.NCH = (g.TW + prm.TB - 1) / prm.TB;
    prm.TB = (g.TW + prm.NCH - 1) / prm.NCH;
    {
        const size_t per_sm = 227 * 1024, one = smem_bytes() + 1024;
        const size_t two = one + prm.strip_bytes;
        const size_t n1 = per_sm / one < 4 ? per_sm / one : 4, n2 = per_sm / two < 4 ? per_sm / two : 4;
        if (n2 >= 1 && n2 == n1) prm.dbuf = 1;
    }
    prm.smem = (int)smem_bytes();
    prm.NCB = g.C / prm.CB;
    prm.items = g.N * g.TH * prm.NCH * prm.NCB;
    // persistent CTAs: as many as fit on the device at once
    const int per_sm = (int)k1_op(kK1Resident, M, f16, g.gs, nullptr, nullptr, nullptr, (size_t)prm.smem);
    const int resident = per_sm * (plan.sm_count > 0 ? plan.sm_count : 1);
    prm.grid = prm.items < resident ? prm.items : resident;
}

}  // namespace

// The same for the NHWC kernel: the strip is the dense TMA box [n][TB * m + 2][CB].
static void plan_k1_nhwc(wfq_plan &plan)
{
    const Geometry &g = plan.geo;
    const bool f16 = plan.in_dtype == WFQ_F16;
    const int NN = g.n, P = g.P, M = g.m;
    const int esz = f16 ? 2 : 4;
    K1Params &prm = plan.k1n;
    prm = plan.k1;
    prm.vec16 = 0;
    prm.TB = (K1_WP - 3) / M;
    prm.CB = g.gs;
    if (g.gs == 32 && g.C % 64 == 0) prm.CB = 64;
    auto strip = [&]() { return ((NN * (prm.TB * M + 2) * prm.CB * esz + 127) / 128) * 128; };
    auto smem_bytes = [&]() {     // 128 bytes of slack for the alignment of the strips
        return 128 + (1 + prm.dbuf) * (size_t)strip() + (size_t)prm.TB * P * (prm.CB + 4) * sizeof(float);
    };
    prm.dbuf = 0;
    while (prm.TB > 1 && smem_bytes() > 113 * 1024) --prm.TB;
    prm.NCH = (g.TW + prm.TB - 1) / prm.TB;
    prm.TB = (g.TW + prm.NCH - 1) / prm.NCH;
    {
        const size_t per_sm = 226 * 1024, one = smem_bytes() + 1024;
        const size_t two = one + strip();
        const size_t n1 = per_sm / one < 4 ? per_sm / one : 4, n2 = per_sm / two < 4 ? per_sm / two : 4;
        if (n2 >= 1 && n2 == n1) prm.dbuf = 1;
    }
    prm.strip_bytes = strip();
    prm.CS = 0;
    prm.smem = (int)smem_bytes();
    prm.NCB = g.C / prm.CB;
    prm.items = g.N * g.TH * prm.NCH * prm.NCB;
    const int per_sm = (int)k1_op(kK1nResident, M, f16, g.gs, nullptr, nullptr, nullptr, (size_t)prm.smem);
    const int resident = per_sm * (plan.sm_count > 0 ? plan.sm_count : 1);
    prm.grid = prm.items < resident ? prm.items : resident;
}

// Work-item shape, shared-memory layout and grid of the cp.async kernel for this plan: one set
// with 4-byte (or 2-byte) copies for any x, and where fp16 rows are whole 16-byte pieces (W a
// multiple of 8) a second one with 16-byte copies, used when x is 16-byte aligned.
void plan_input_transform(wfq_plan &plan)
{
    plan_k1(plan, plan.k1, false);
    plan.k1v = plan.k1;
    if (plan.in_dtype == WFQ_F16 && plan.geo.W % 8 == 0) plan_k1(plan, plan.k1v, true);
    plan_k1_nhwc(plan);
    plan.tmap_xn_base = nullptr;
    plan.tmap_xn_tc_base = nullptr;
}

cudaError_t setup_input_transform()
{
    const int sizes[5] = {32, 64, 128, 256, 96};
    for (int m = 2; m <= 6; m += 2)
        for (int f16 = 0; f16 < 2; ++f16)
            for (int gs : sizes) {
                cudaError_t e = (cudaError_t)k1_op(kK1Setup, m, f16 != 0, gs, nullptr, nullptr, nullptr, 0);
                if (e != cudaSuccess) return e;
                e = (cudaError_t)k1_op(kK1nSetup, m, f16 != 0, gs, nullptr, nullptr, nullptr, 0);
                if (e != cudaSuccess) return e;
            }
    return cudaSuccess;
}

cudaError_t launch_input_transform(wfq_plan &plan, const void *x_dev, cudaStream_t stream)
{
    const Geometry &g = plan.geo;
    if (plan.in_nhwc) {
        // x[N][H][W][C] as a 4-D tensor (C, W, H, N) with boxes of one work item's strip
        if ((reinterpret_cast<uintptr_t>(x_dev) & 15u) != 0) return cudaErrorInvalidValue;
        const unsigned long long esz0 = plan.in_dtype == WFQ_F16 ? 2 : 4;
        // tensor cores where they apply (fp16, groups of 32 or 64, C a multiple of 64, F(4,3) / F(6,3)),
        // unless the debug option asks for the plain kernel
        if (input_transform_tcn_applies(plan) && plan.k1_choice != 1) {
            if (plan.tmap_xn_tc_base != x_dev) {
                const unsigned long long dims[4] = {(unsigned long long)g.C, (unsigned long long)g.W,
                                                    (unsigned long long)g.H, (unsigned long long)g.N};
                const unsigned long long strides[3] = {(unsigned long long)g.C * esz0,
                                                       (unsigned long long)g.W * g.C * esz0,
                                                       (unsigned long long)g.H * g.W * g.C * esz0};
                unsigned box[4];
                input_transform_tcn_box(plan, box);
                if (!encode_tmap(&plan.tmap_xn_tc, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 4, x_dev, dims, strides, box,
                                 CU_TENSOR_MAP_SWIZZLE_128B))
                    return cudaErrorInvalidValue;
                plan.tmap_xn_tc_base = x_dev;
            }
            return launch_input_transform_tcn(plan, stream);
        }
        if (plan.tmap_xn_base != x_dev) {
            const unsigned long long esz = plan.in_dtype == WFQ_F16 ? 2 : 4;
            const unsigned long long dims[4] = {(unsigned long long)g.C, (unsigned long long)g.W,
                                                (unsigned long long)g.H, (unsigned long long)g.N};
            const unsigned long long strides[3] = {(unsigned long long)g.C * esz, (unsigned long long)g.W * g.C * esz,
                                                   (unsigned long long)g.H * g.W * g.C * esz};
            const unsigned box[4] = {(unsigned)plan.k1n.CB, (unsigned)(plan.k1n.TB * g.m + 2), (unsigned)g.n, 1u};
            if (!encode_tmap(&plan.tmap_xn, plan.in_dtype == WFQ_F16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16
                                                                      : CU_TENSOR_MAP_DATA_TYPE_FLOAT32,
                             4, x_dev, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_NONE))
                return cudaErrorInvalidValue;
            plan.tmap_xn_base = x_dev;
        }
        return (cudaError_t)k1_op(kK1nLaunch, g.m, plan.in_dtype == WFQ_F16, g.gs, &plan, x_dev, stream, 0);
    }
    // tensor-core kernel: fp16 input that a TMA tensor map (16-byte aligned base) can describe
    // (automatic = the cp.async kernel: the tensor-core one measured no faster on any configured layer)
    if (plan.k1tc.use && plan.k1_choice == 2 && (reinterpret_cast<uintptr_t>(x_dev) & 15u) == 0) {
        if (plan.k1tc.mode != 2 && plan.tmap_x_base != x_dev) {
            const unsigned long long hw = (unsigned long long)g.H * g.W;
            bool ok;
            if (plan.k1tc.mode == 0) {
                const unsigned long long dims[3] = {(unsigned long long)g.W, (unsigned long long)g.H,
                                                    (unsigned long long)g.N * g.C};
                const unsigned long long strides[2] = {(unsigned long long)g.W * 2, hw * 2};
                ok = encode_tmap(&plan.tmap_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, x_dev, dims, strides,
                                 plan.k1tc.box, CU_TENSOR_MAP_SWIZZLE_NONE);
            } else {
                const unsigned long long dims[2] = {hw, (unsigned long long)g.N * g.C};
                const unsigned long long strides[1] = {hw * 2};
                ok = encode_tmap(&plan.tmap_x, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, x_dev, dims, strides,
                                 plan.k1tc.box, CU_TENSOR_MAP_SWIZZLE_NONE);
            }
            if (!ok) return cudaErrorInvalidValue;
            plan.tmap_x_base = x_dev;
        }
        return launch_input_transform_tc(plan, x_dev, stream);
    }
    return (cudaError_t)k1_op(kK1Launch, g.m, plan.in_dtype == WFQ_F16, g.gs, &plan, x_dev, stream, 0);
}

}  // namespace wfq
