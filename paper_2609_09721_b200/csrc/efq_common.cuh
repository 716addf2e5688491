// Shared device/host helpers of the EFQ-Softmax B200 library (sm_100a only).
#pragma once

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include "efq.h"

namespace efq {

constexpr int kMxBlock = 32;  // keys per microscaling block

// Revision of the fused forward kernel, part of efq_version().  Raise it whenever attention_fwd_kernel changes:
// figures copied from a profiler capture (DRAM bytes per launch in the benchmark) are keyed to it.
#define EFQ_FWD_KERNEL_REVISION "fwd.3"

// Constants of the FP32 code rule, derived on the host in double and rounded once.
// With x = sigma*r - m_s, k the block's scale exponent and z = x - k ln2 - ln6 (Eq. z-def):
//   (z - tau) h + 1  =  r*(sigma h) - h m_s - k (h ln2) + (1 - h (ln6 + tau))
struct ProducerConsts {
    float A;      // sigma * h
    float HL2;    // h * ln 2
    float C1;     // 1 - h * (ln 6 + tau)
    float h;
    float sigma;
    float LOG2E;  // 1 / ln 2
    float L2_29;  // log2(2/9), the constant of the scale rule (Eq. k-rule)
};

inline ProducerConsts make_producer_consts(float sigma, float tau, float h)
{
    ProducerConsts c;
    const double ln2 = 0.693147180559945309417232121458, ln6 = 1.79175946922805500081247735838;
    c.A = static_cast<float>(static_cast<double>(sigma) * static_cast<double>(h));
    c.HL2 = static_cast<float>(static_cast<double>(h) * ln2);
    c.C1 = static_cast<float>(1.0 - static_cast<double>(h) * (ln6 + static_cast<double>(tau)));
    c.h = h;
    c.sigma = sigma;
    c.LOG2E = static_cast<float>(1.0 / ln2);
    c.L2_29 = static_cast<float>(log(2.0 / 9.0) / ln2);
    return c;
}

// LUT variant (Sec. "EFQ-Softmax-LUT Variant"): the same scale rule and the same affine form with the fixed pair
// tau16 = ln(1/24), h16 = 14 / ln 24 (taken in double, the FP32 constants rounded once); the 16-level index then
// goes through the folding table C16 = [0,1,1,1,1,1,2,2,3,3,4,5,5,6,7,7], held as one nibble per entry.
constexpr uint64_t kLutFold16 = 0x7765543322111110ull;

inline ProducerConsts make_producer_consts_lut(float sigma)
{
    ProducerConsts c;
    const double ln2 = 0.693147180559945309417232121458, ln6 = 1.79175946922805500081247735838;
    const double h16 = 14.0 / log(24.0), tau16 = log(1.0 / 24.0);
    c.A = static_cast<float>(static_cast<double>(sigma) * h16);
    c.HL2 = static_cast<float>(h16 * ln2);
    c.C1 = static_cast<float>(1.0 - h16 * (ln6 + tau16));
    c.h = static_cast<float>(h16);
    c.sigma = sigma;
    c.LOG2E = static_cast<float>(1.0 / ln2);
    c.L2_29 = static_cast<float>(log(2.0 / 9.0) / ln2);
    return c;
}

#ifdef __CUDACC__

// Per-block part of Algorithm 1 (steps 1-3): from the block's largest raw score and the
// row maximum m_s (scaled units) to the E8M0 byte and the additive term of the code rule.
// Separate mul and sub (never contracted) so the result equals the reference FP32 order.
struct BlockScale {
    float Bb;       // additive term: v_t = fma(r_t, A, Bb)
    uint32_t byte;  // k_b + 127, or 0 for a block with no finite score
    bool live;
};

__device__ __forceinline__ BlockScale efq_block_scale(float rmax, float m_s, const ProducerConsts& K)
{
    BlockScale s;
    s.live = rmax != -INFINITY;
    const float Mb = __fsub_rn(__fmul_rn(K.sigma, rmax), m_s);
    // k = clamp(floor(t), -127, 127) = floor(clamp(t, -127, 127)); the floor by a round-down add of 1.5 * 2^23
    // (exact for |t| < 2^22), which also leaves k in the low mantissa bits: no conversion instruction needed.
    float t = __fmaf_rn(Mb, K.LOG2E, K.L2_29);
    t = fminf(fmaxf(t, -127.0f), 127.0f);          // a NaN (block and row both without a finite score) becomes -127
    float km;
    asm("add.rm.f32 %0, %1, %2;" : "=f"(km) : "f"(t), "f"(12582912.0f));
    const float kf = __fsub_rn(km, 12582912.0f);
    s.Bb = __fmaf_rn(-K.h, m_s, __fmaf_rn(-K.HL2, kf, K.C1));
    s.byte = s.live ? (__float_as_uint(km) - 0x4B400000u + 127u) : 0u;
    return s;
}

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// LUT variant, one element: 16-level index j = floor(min(max(v, 0), 15)) of v = fma(r, A, Bb), folded to a code.
//   w = fma.rn.sat(r, A/16, Bb/16) = clamp(v, 0, 16) / 16   (scaling by 2^-4 commutes with rounding)
//   fma.rm(w, 16, 2^23) = 2^23 + floor(16 w): the index sits in the low mantissa bits, 16 only when v >= 16
__device__ __forceinline__ uint32_t lut_code(float r, float A16, float B16)
{
    float w, t;
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(w) : "f"(r), "f"(A16), "f"(B16));
    asm("fma.rm.f32 %0, %1, %2, %3;" : "=f"(t) : "f"(w), "f"(16.0f), "f"(8388608.0f));
    const uint32_t j = min(__float_as_uint(t) & 31u, 15u);
    return static_cast<uint32_t>(kLutFold16 >> (4u * j)) & 15u;
}

// exp-then-quantize with the block scale folded into the exponential (the strongest form of the baseline on this
// machine): p 2^-e = 2^(x log2(e) - e), so with t = fma(r, sigma log2(e), -m_s log2(e)) the scaled probability is one
// FMA and one ex2 away from the raw score; the exponential is monotone, so the block maximum of p is ex2 of
// t(rmax) and e = floor(t(rmax)) - 2 (block maximum in [4, 8)) needs no pass over p.  Same mathematics as
// p = exp(x), e = floor(log2 max p) - 2, q = RNE(p 2^-e); rounding differs at knife-edges only.
// The block's exponent is taken from x(rmax) = fl(fl(sigma rmax) - m_s), which is exactly 0 for the row maximum:
// p = 1 sits on a power of two, and the fused form fma(rmax, c1, c0) lands a rounding error below it as often as
// above, which would put the row's largest probability one binade too high and saturate it.
struct FoldedScale {
    float c1;       // sigma * log2(e)
    float c0e;      // -m_s * log2(e) - e
    uint32_t byte;  // e + 127, or 0 for a block without a finite score
    bool live;
};
__device__ __forceinline__ FoldedScale etq_folded_scale(float rmax, float m_s, const ProducerConsts& K)
{
    FoldedScale f;
    f.c1 = __fmul_rn(K.sigma, K.LOG2E);
    const float c0 = __fmul_rn(-m_s, K.LOG2E);
    f.live = rmax != -INFINITY;
    float t = __fmul_rn(__fsub_rn(__fmul_rn(K.sigma, rmax), m_s), K.LOG2E);
    t = fminf(fmaxf(t, -125.0f), 129.0f);            // e = floor(t) - 2 stays in [-127, 127]; NaN (no finite score) -> -125
    float km;
    asm("add.rm.f32 %0, %1, %2;" : "=f"(km) : "f"(t), "f"(12582912.0f));   // floor by a round-down add of 1.5 * 2^23
    const float ef = __fsub_rn(__fsub_rn(km, 12582912.0f), 2.0f);
    f.c0e = __fsub_rn(c0, ef);
    f.byte = f.live ? (__float_as_uint(km) - 0x4B400000u - 2u + 127u) : 0u;
    return f;
}

// 2^t by arithmetic alone, for the part of the exponentials that the FMA pipe takes over from the special-function
// unit (16 ex2 per clock per SM against 128 FMA): floor by a round-down add of 1.5 * 2^23, a cubic on the fraction
// (own minimax fit on [0, 1], relative error 8.6e-5 - two orders below the E2M1 step), the integer part added to
// the exponent field.  t below -127 (masked scores: -inf) gives 0.
__device__ __forceinline__ float ex2_poly3(float t)
{
    t = fmaxf(t, -127.0f);
    float km;
    asm("add.rm.f32 %0, %1, %2;" : "=f"(km) : "f"(t), "f"(12582912.0f));
    const float f = __fsub_rn(t, __fsub_rn(km, 12582912.0f));
    float p = __fmaf_rn(f, 0.07706704f, 0.22764499f);
    p = __fmaf_rn(f, p, 0.69511676f);
    p = __fmaf_rn(f, p, 1.0f);
    return __uint_as_float(__float_as_uint(p) + (__float_as_uint(km) << 23));
}
// which elements of a run of eight take the polynomial: 2 of 8 (3 of 8 was slower everywhere: the polynomial costs
// about 12 issue slots per element and the two paths overlap less than their pipe counts promise)
__device__ __forceinline__ constexpr bool ex2_by_poly(int i) { return (i & 7) == 1 || (i & 7) == 5; }

// Two floats -> one byte of E2M1 (round-to-nearest-even, saturating); `lo` lands in bits 0-3.
__device__ __forceinline__ uint32_t cvt_e2m1x2(float lo, float hi)
{
    uint16_t out;
    asm("{ .reg .b8 t;\n"
        "  cvt.rn.satfinite.e2m1x2.f32 t, %2, %1;\n"
        "  mov.b16 %0, {t, 0}; }\n"
        : "=h"(out)
        : "f"(lo), "f"(hi));
    return out;
}

#endif  // __CUDACC__

}  // namespace efq
