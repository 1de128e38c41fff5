// Shared device helpers of the SFDA kernels (sm_100a).  Nothing here is used by,
// or shared with, the CPU oracle.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sfda {

// ---- element IO in the caller's dtype --------------------------------------------------------
__device__ __forceinline__ float ld_val(const float *p, size_t i) { return p[i]; }
__device__ __forceinline__ float ld_val(const __nv_bfloat16 *p, size_t i) { return __bfloat162float(p[i]); }
__device__ __forceinline__ void st_val(float *p, size_t i, float x) { p[i] = x; }
__device__ __forceinline__ void st_val(__nv_bfloat16 *p, size_t i, float x) { p[i] = __float2bfloat16_rn(x); }

// ---- integer cumulative phase ------------------------------------------------------------------
// A phase is carried as an unsigned 32-bit count of 2*pi/2^32 turns so that the chunk-local prefix
// product Gamma_t = Lambda_t Gamma_{t-1} (Eq. "constructive-Gamma") has, for its unit-modulus part,
// one right answer whatever order a scan adds it in.  theta -> rint((double)theta * 2^32/(2 pi)).
__device__ __forceinline__ uint32_t phase_to_turns(float theta)
{
    const double turns_per_radian = 0x1.45f306dc9c883p+29;  // 2^32 / (2 pi), nearest double
    const double d = __dmul_rn((double)theta, turns_per_radian);
    // |theta| < 1e6 gives |d| < 2^51: adding 1.5 * 2^52 rounds d to an integer (to nearest, ties to even) and
    // leaves that integer, modulo 2^32, in the low word of the sum.  Larger angles take the (slow) conversion
    // instruction instead, under a predicate rather than a branch so that the common case stays straight-line.
    uint32_t u = (uint32_t)__double2loint(__dadd_rn(d, 6755399441055744.0));
    asm("{\n.reg .pred p;\n.reg .s64 t;\nsetp.ge.f32 p, %2, 0f49742400;\n@p cvt.rni.s64.f64 t, %1;\n@p cvt.u32.u64 %0, t;\n}\n"
        : "+r"(u)
        : "d"(d), "f"(fabsf(theta)));
    return u;
}

// cos / sin of a phase given in turns (signed view keeps the float argument in [-1, 1)).
__device__ __forceinline__ void turns_to_cos_sin(uint32_t turns, float *c, float *s)
{
    const float x = (float)(int32_t)turns * 0x1p-31f;  // phase / pi
    sincospif(x, s, c);
}

// log of a decay factor, floored at -30: alpha below e^-30 (alpha = 0 is admissible in the
// recurrence) then acts as e^-30 ~ 9e-14, far below fp32 resolution of anything it multiplies, while
// cumulative sums over a chunk stay small enough that differences of two of them keep fp32 precision.
__device__ __forceinline__ float log_decay(float alpha) { return fmaxf(logf(alpha), -30.0f); }

}  // namespace sfda
