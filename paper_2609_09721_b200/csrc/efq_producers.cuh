// Probability producers for one 32-key microscaling block held in registers: the EFQ rule (Algorithm 1)
// and the exp-then-quantize comparison producer.  Shared by the fused forward and the in-SM microbenchmark.
#pragma once

#include "efq_common.cuh"

namespace efq {

__device__ __forceinline__ float max3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float fma_sat(float a, float b, float c)
{
    float d;
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ uint64_t pack2(float lo, float hi)
{
    uint64_t d;
    asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
    return d;
}

// Largest of 32 scores with 3-input maxima.
__device__ __forceinline__ float block_max32(const float* r)
{
    float m[11];
#pragma unroll
    for (int i = 0; i < 10; ++i) m[i] = max3(r[3 * i], r[3 * i + 1], r[3 * i + 2]);
    m[10] = fmaxf(r[30], r[31]);
    const float a = max3(m[0], m[1], m[2]), b = max3(m[3], m[4], m[5]), c = max3(m[6], m[7], m[8]);
    return max3(max3(a, b, c), m[9], m[10]);
}

// 32 scores of one microscaling block -> 16 bytes of codes + scale byte.
// PRODUCER: 0 = EFQ (affine rule), 1 / 2 = exp-then-quantize with the block maximum in [4, 8) / (3, 6],
// 3 = EFQ-LUT, 4 = exp-then-quantize [4, 8) with the scale folded into the exponential, 5 = the same with 2 of 8
// exponentials computed by a polynomial on the FMA pipe, 6 = producer 1 that also adds its 32 FP32 exponentials to
// *psum (for the baseline whose denominator is the sum of the exponentials instead of the quantised operand).
//
// EFQ (Algorithm 1), three FMA-pipe instructions per element, bit-identical to
// c = floor(min(max(fma(r, A, Bb), 0), 7)):
//   w  = fma.rn.sat(r, A/8, Bb/8)      = clamp(fma(r, A, Bb), 0, 8) / 8   (scaling by 2^-3 commutes with rounding)
//   a' = fma.rm(w, 8, u)               = u + floor(8 w)                   (u an integer in [2^23, 2^24): ulp 1, round down)
//   u' = fma.rn(a', 16, -15 * 2^23)    = 2^23 + 16 X                      (a' = 2^23 + X, exact)
// so four elements accumulate Horner-style into X = c3 c2 c1 c0 (one nibble each) in the mantissa; the two
// chain steps run as packed f32x2 FMAs on the low and high half of a 32-bit word at once.  floor(8 w) = 8 happens
// only when fma(r, A, Bb) >= 8; FIX8 turns that nibble into 7 (needed when (ln 1.5 - tau) h + 1 can reach 8).
template <int PRODUCER, bool FIX8>
__device__ __forceinline__ void produce32(const float* r, float rmax, float m_s, const ProducerConsts& K, uint4& codes,
                                          uint32_t& byte, float* psum = nullptr)
{
    uint32_t w[4];
    if (PRODUCER == 0) {
        BlockScale s = efq_block_scale(rmax, m_s, K);
        byte = s.byte;
        const float A8 = K.A * 0.125f, B8 = s.Bb * 0.125f;
        const uint64_t eight2 = pack2(8.0f, 8.0f), sixteen2 = pack2(16.0f, 16.0f);
        const uint64_t magic2 = pack2(8388608.0f, 8388608.0f), back2 = pack2(-125829120.0f, -125829120.0f);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint64_t a2 = magic2;
#pragma unroll
            for (int i = 3; i >= 0; --i) {
                const uint64_t w2 = pack2(fma_sat(r[q * 8 + i], A8, B8), fma_sat(r[q * 8 + 4 + i], A8, B8));
                uint64_t u2 = magic2;
                if (i != 3) asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(u2) : "l"(a2), "l"(sixteen2), "l"(back2));
                asm("fma.rm.f32x2 %0, %1, %2, %3;" : "=l"(a2) : "l"(w2), "l"(eight2), "l"(u2));
            }
            uint32_t lo, hi;
            asm("mov.b64 {%0, %1}, %2;" : "=r"(lo), "=r"(hi) : "l"(a2));
            uint32_t word = __byte_perm(lo, hi, 0x5410);
            if (FIX8) word -= (word >> 3) & 0x11111111u;
            w[q] = word;   // a block without a finite score has w = 0 everywhere (sat(-inf) and sat(NaN) are 0)
        }
    } else if (PRODUCER == 3) {
        // LUT variant: the same block scale, 16-level index, folding table (one element at a time: the
        // accuracy-oriented comparison point of the paper, not the fast path)
        BlockScale s = efq_block_scale(rmax, m_s, K);
        byte = s.byte;
        const float A16 = K.A * 0.0625f, B16 = s.Bb * 0.0625f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t word = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) word |= lut_code(r[q * 8 + i], A16, B16) << (4 * i);
            w[q] = word;
        }
    } else if (PRODUCER == 4 || PRODUCER == 5) {
        // exp-then-quantize (block maximum in [4, 8)) with the scale folded into the exponential: one FMA, one ex2
        // and half a conversion per element; bound by the exponential unit.  PRODUCER 5 moves 2 of every 8
        // exponentials onto the FMA pipe (cubic polynomial).
        const FoldedScale f = etq_folded_scale(rmax, m_s, K);
        byte = f.byte;
        auto ex2 = [&](const int i) {
            const float t = __fmaf_rn(r[i], f.c1, f.c0e);
            return (PRODUCER == 5 && ex2_by_poly(i)) ? ex2_poly3(t) : ex2_approx(t);
        };
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            uint32_t word = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i)
                word |= (cvt_e2m1x2(ex2(q * 8 + 2 * i), ex2(q * 8 + 2 * i + 1)) & 0xffu) << (8 * i);
            w[q] = f.live ? word : 0u;
        }
    } else {
        float p[32];
        float amax = 0.0f, sum = 0.0f;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
            float x = __fsub_rn(__fmul_rn(K.sigma, r[i]), m_s);
            p[i] = ex2_approx(__fmul_rn(x, K.LOG2E));
            amax = fmaxf(amax, p[i]);
            if (PRODUCER == 6) sum += p[i];       // masked scores (-inf) give exactly 0
        }
        if (PRODUCER == 6) *psum += sum;
        if (amax == 0.0f) {
            byte = 0;
            w[0] = w[1] = w[2] = w[3] = 0;
        } else {
            const uint32_t bits = __float_as_uint(amax);
            const int E = static_cast<int>((bits >> 23) & 0xffu) - 127;
            int e = (PRODUCER == 1 || PRODUCER == 6) ? E - 2 : ((bits & 0x7fffffu) > 0x400000u ? E - 1 : E - 2);
            e = max(e, -127);
            const float s = __uint_as_float(static_cast<uint32_t>(127 - e) << 23);
            byte = static_cast<uint32_t>(e + 127);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                uint32_t word = 0;
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    word |= (cvt_e2m1x2(p[q * 8 + 2 * i] * s, p[q * 8 + 2 * i + 1] * s) & 0xffu) << (8 * i);
                w[q] = word;
            }
        }
    }
    codes = make_uint4(w[0], w[1], w[2], w[3]);
}

}  // namespace efq
