// Per-lane arithmetic of the register machine (vm.h), shared by the interpreter kernels and the
// ahead-of-time compiled programs: one function per opcode family, one rounding per traced op.
#pragma once
#ifndef __CUDACC_RTC__
#include <cuda_runtime.h>
#include <stdint.h>
#endif

#include "vm.h"

#define LT_INF __int_as_float(0x7f800000)

namespace {

// ---------------------------------------------------------------------- math
__device__ __forceinline__ float u2f(uint32_t u) { return __uint_as_float(u); }
__device__ __forceinline__ uint32_t f2u(float f) { return __float_as_uint(f); }

// binary32 -> bfloat16, round to nearest even (the conversion instruction; NaN stays NaN)
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float round_bf16(float x) { return __uint_as_float(pack_bf16x2(0.0f, x) & 0xffff0000u); }

__device__ __forceinline__ float max_nan(float a, float b) {
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ float min_nan(float a, float b) {
    float r;
    asm("min.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ float tanh_approx(float x) {
    float r;
    asm("tanh.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float rcp_approx(float x) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}
__device__ __forceinline__ float sqrt_approx(float x) {
    float r;
    asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(x));
    return r;
}

template <int OP, bool FAST>
__device__ __forceinline__ float f2(float a, float b) {
    if constexpr (OP == F2_ADD) return __fadd_rn(a, b);
    else if constexpr (OP == F2_SUB) return __fsub_rn(a, b);
    else if constexpr (OP == F2_RSUB) return __fsub_rn(b, a);
    else if constexpr (OP == F2_MUL) return __fmul_rn(a, b);
    else if constexpr (OP == F2_DIV) return FAST ? __fdividef(a, b) : __fdiv_rn(a, b);
    else if constexpr (OP == F2_RDIV) return FAST ? __fdividef(b, a) : __fdiv_rn(b, a);
    else if constexpr (OP == F2_MAX) return max_nan(a, b);
    else return min_nan(a, b);
}

template <int OP>
__device__ __forceinline__ float i2(float fa, float fb) {
    uint32_t a = f2u(fa), b = f2u(fb), r;
    if constexpr (OP == I2_ADD) r = a + b;
    else if constexpr (OP == I2_SUB) r = a - b;
    else if constexpr (OP == I2_RSUB) r = b - a;
    else if constexpr (OP == I2_MUL) r = a * b;
    else if constexpr (OP == I2_AND) r = a & b;
    else if constexpr (OP == I2_OR) r = a | b;
    else if constexpr (OP == I2_XOR) r = a ^ b;
    else if constexpr (OP == I2_MAXS) r = (uint32_t)max((int32_t)a, (int32_t)b);
    else if constexpr (OP == I2_MINS) r = (uint32_t)min((int32_t)a, (int32_t)b);
    else if constexpr (OP == I2_MAXU) r = max(a, b);
    else r = min(a, b);
    return u2f(r);
}

template <int CC, class T>
__device__ __forceinline__ bool cmp_t(T a, T b) {
    if constexpr (CC == CC_GT) return a > b;
    else if constexpr (CC == CC_GE) return a >= b;
    else if constexpr (CC == CC_LT) return a < b;
    else if constexpr (CC == CC_LE) return a <= b;
    else if constexpr (CC == CC_EQ) return a == b;
    else return a != b;
}

template <int IDX>
__device__ __forceinline__ float cmp(float a, float b) {
    constexpr int TY = IDX / 6, CC = IDX % 6;
    bool r;
    if constexpr (TY == 0) r = cmp_t<CC, float>(a, b);
    else if constexpr (TY == 1) r = cmp_t<CC, int32_t>((int32_t)f2u(a), (int32_t)f2u(b));
    else r = cmp_t<CC, uint32_t>(f2u(a), f2u(b));
    return u2f(r ? 1u : 0u);
}

template <int OP, bool FAST>
__device__ __forceinline__ float un(float x) {
    if constexpr (OP == OP_U_NEG) return -x;
    else if constexpr (OP == OP_U_ABS) return fabsf(x);
    else if constexpr (OP == OP_U_RELU) return max_nan(x, 0.0f);
    else if constexpr (OP == OP_U_EXP) return FAST ? __expf(x) : expf(x);
    else if constexpr (OP == OP_U_LOG) return FAST ? __logf(x) : logf(x);
    else if constexpr (OP == OP_U_TANH) return FAST ? tanh_approx(x) : tanhf(x);
    else if constexpr (OP == OP_U_SQRT) return FAST ? sqrt_approx(x) : __fsqrt_rn(x);
    else if constexpr (OP == OP_U_RSQRT) return rsqrtf(x);
    else if constexpr (OP == OP_U_RECIP) return FAST ? rcp_approx(x) : __frcp_rn(x);
    else if constexpr (OP == OP_U_SQUARE) return __fmul_rn(x, x);
    else if constexpr (OP == OP_U_SIGMOID)
        return FAST ? rcp_approx(1.0f + __expf(-x)) : __fdiv_rn(1.0f, 1.0f + expf(-x));
    else if constexpr (OP == OP_U_GELU) {
        const float k = 0.7978845608028654f;  // sqrt(2/pi)
        float inner = k * fmaf(0.044715f * x, x * x, x);
        float th = FAST ? tanh_approx(inner) : tanhf(inner);
        return 0.5f * x * (1.0f + th);
    } else if constexpr (OP == OP_U_RBF16) return round_bf16(x);
    else if constexpr (OP == OP_U_INEG) return u2f(0u - f2u(x));
    else if constexpr (OP == OP_U_IABS) return u2f((uint32_t)abs((int32_t)f2u(x)));
    else if constexpr (OP == OP_U_NOT) return u2f(f2u(x) == 0u ? 1u : 0u);
    else if constexpr (OP == OP_C_I2F) return __int2float_rn((int32_t)f2u(x));
    else if constexpr (OP == OP_C_U2F) return __uint2float_rn(f2u(x));
    else if constexpr (OP == OP_C_F2I) return u2f((uint32_t)__float2int_rz(x));
    else if constexpr (OP == OP_C_NZF) return u2f(x != 0.0f ? 1u : 0u);
    else return u2f(f2u(x) != 0u ? 1u : 0u);  // OP_C_NZI
}

// Philox4x32-10 (Salmon et al., SC'11): ten multiply/xor rounds, key bumped by Weyl constants.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t (&out)[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

}  // namespace
