// Group quantizer on accumulator rows read from tensor memory (shared by the tensor-core input
// transforms): a thread holds the raw transform values z of one (tile, position) for a run of
// consecutive channels as 32-bit patterns and produces the group scale and the int8 codes.
#pragma once

#include <cstdint>

#include <cuda_runtime.h>

namespace wfq {

// One code: fl32(v*inv) + 1.5*2^23 (two separately rounded operations, as the quantizer
// is defined); the low byte of the sum's bit pattern is the code.
__device__ __forceinline__ uint32_t pack4(float a, float b, float c, float d)
{
    const uint32_t ua = __float_as_uint(__fadd_rn(a, 12582912.f)), ub = __float_as_uint(__fadd_rn(b, 12582912.f));
    const uint32_t uc = __float_as_uint(__fadd_rn(c, 12582912.f)), ud = __float_as_uint(__fadd_rn(d, 12582912.f));
    return __byte_perm(__byte_perm(ua, ub, 0x0040), __byte_perm(uc, ud, 0x0040), 0x5410);
}

__device__ __forceinline__ void st_global_v8_u32(void *p, const uint32_t (&w)[8])
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]),
                   "r"(w[7])
                 : "memory");
}

// max |z| of 32 accumulator values folded into m.  (The abs-max of the group is taken on
// the raw transform values: rounding is monotone, so max |fl(z * s)| = |fl(zmax * s)|.)
__device__ __forceinline__ float absmax32(const uint32_t (&r)[32], float m)
{
    float m0 = m, m1 = 0.f, m2 = 0.f, m3 = 0.f;
#pragma unroll
    for (int k = 0; k < 32; k += 4) {
        m0 = fmaxf(m0, fabsf(__uint_as_float(r[k])));
        m1 = fmaxf(m1, fabsf(__uint_as_float(r[k + 1])));
        m2 = fmaxf(m2, fabsf(__uint_as_float(r[k + 2])));
        m3 = fmaxf(m3, fabsf(__uint_as_float(r[k + 3])));
    }
    return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

// x = z * (sp + sl), rounded once: fma(z, sp, z * sl).
__device__ __forceinline__ float scaled(float z, float sp, float sl) { return fmaf(z, sp, __fmul_rn(z, sl)); }

// Scale and reciprocal of a group from its abs-max (the quantizer of Section 2).
__device__ __forceinline__ void group_scale_inv(float amax, float &scale, float &inv)
{
    const bool nz = amax >= 1e-30f;
    scale = nz ? __fdiv_rn(amax, 127.f) : 0.f;
    inv = nz ? __fdiv_rn(127.f, amax) : 0.f;
}

// 32 codes from 32 raw transform values z: x = z * (sp + sl) rounded once, t = fl(x * inv),
// code = low byte of fl(t + 1.5 * 2^23) (round to nearest even); one 32-byte store.
__device__ __forceinline__ void codes32(const uint32_t (&r)[32], float sp, float sl, float inv, int8_t *dst)
{
    const float2 sp2 = make_float2(sp, sp), sl2 = make_float2(sl, sl), inv2 = make_float2(inv, inv);
    uint32_t w[8];
#pragma unroll
    for (int q = 0; q < 8; ++q) {
        const float2 z0 = make_float2(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]));
        const float2 z1 = make_float2(__uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
        const float2 t0 = __fmul2_rn(__ffma2_rn(z0, sp2, __fmul2_rn(z0, sl2)), inv2);
        const float2 t1 = __fmul2_rn(__ffma2_rn(z1, sp2, __fmul2_rn(z1, sl2)), inv2);
        w[q] = pack4(t0.x, t0.y, t1.x, t1.y);
    }
    st_global_v8_u32(dst, w);
}

}  // namespace wfq
