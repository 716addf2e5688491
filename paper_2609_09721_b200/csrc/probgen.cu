// Standalone probability-generation stage (kernel interface of Sec. 4.3): a streaming,
// HBM-bound pass over an fp32 score matrix that emits packed E2M1 codes and one E8M0
// byte per 32-column microscaling block.  Two producers share the data movement:
//   EFQ  - Algorithm 1: exponent-only scale from the block maximum + one affine rule, no exp;
//   ETQ  - exp -> FP32 probabilities -> block abs-max -> scale -> round to E2M1.
//
// Data movement: one warp owns 1024 consecutive columns of a row (32 blocks).  Lane l in
// pass i loads the 8 floats at element (i*32 + l)*8 with one 256-bit load, so every load
// instruction covers 1 KiB of contiguous bytes; a microscaling block is spread over 4
// adjacent lanes and its maximum is a 2-step butterfly.  Each lane then holds 8 codes
// (32 bits) per pass; the words of a pass are contiguous in the packed output (128 bytes
// per warp per pass).
// Algorithmic traffic: 4 B/element in, 0.5 B/element + 1 B/32 elements out.
#include "efq_common.cuh"

namespace efq {

enum Producer : int { kEfq = 0, kEtq4 = 1, kEtq6 = 2, kEfqLut = 3, kEtq4Fold = 4, kEtq4Hybrid = 5 };

constexpr int kSegCols = 1024;       // columns per warp task
constexpr int kWarpsPerCta = 8;

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
__device__ __forceinline__ float fma_rm(float a, float b, float c)
{
    float d;
    asm("fma.rm.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// 8 consecutive scores of one lane (a microscaling block spans 4 adjacent lanes) -> 8 codes (32 bits) + scale byte
template <int PRODUCER>
__device__ __forceinline__ void produce_block(const float (&r)[8], float m_s, const ProducerConsts& K,
                                              uint32_t& code32, uint32_t& byte)
{
    if (PRODUCER == kEfq) {
        float rmax = fmaxf(max3(r[0], r[1], r[2]), max3(r[3], r[4], r[5]));
        rmax = max3(rmax, r[6], r[7]);
        rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, 1));
        rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, 2));
        BlockScale s = efq_block_scale(rmax, m_s, K);
        // Codes Horner-style on the FMA pipe, bit-identical to floor(min(max(fma(r, A, Bb), 0), 7)):
        //   w = fma.rn.sat(r, A/8, Bb/8) = clamp(v, 0, 8)/8;  a = fma.rm(w, 8, u) = u + floor(8w) for an integer
        //   u in [2^23, 2^24);  u' = fma.rn(a, 16, -15*2^23) = 2^23 + 16 X.  Four codes per chain.
        const float A8 = K.A * 0.125f, B8 = s.Bb * 0.125f;
        float lo = fma_rm(fma_sat(r[3], A8, B8), 8.0f, 8388608.0f);
        float hi = fma_rm(fma_sat(r[7], A8, B8), 8.0f, 8388608.0f);
#pragma unroll
        for (int i = 2; i >= 0; --i) {
            lo = fma_rm(fma_sat(r[i], A8, B8), 8.0f, __fmaf_rn(lo, 16.0f, -125829120.0f));
            hi = fma_rm(fma_sat(r[4 + i], A8, B8), 8.0f, __fmaf_rn(hi, 16.0f, -125829120.0f));
        }
        uint32_t c = __byte_perm(__float_as_uint(lo), __float_as_uint(hi), 0x5410);
        c -= (c >> 3) & 0x11111111u;        // floor(8w) = 8 only when v >= 8: that nibble is 7
        code32 = c;                         // a block without a finite score has w = 0 everywhere
        byte = s.byte;
    } else if (PRODUCER == kEtq4Fold || PRODUCER == kEtq4Hybrid) {
        float rmax = fmaxf(max3(r[0], r[1], r[2]), max3(r[3], r[4], r[5]));
        rmax = max3(rmax, r[6], r[7]);
        rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, 1));
        rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, 2));
        const FoldedScale f = etq_folded_scale(rmax, m_s, K);
        uint32_t c = 0;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const float tl = __fmaf_rn(r[2 * u], f.c1, f.c0e), th = __fmaf_rn(r[2 * u + 1], f.c1, f.c0e);
            const float lo = (PRODUCER == kEtq4Hybrid && ex2_by_poly(2 * u)) ? ex2_poly3(tl) : ex2_approx(tl);
            const float hi = (PRODUCER == kEtq4Hybrid && ex2_by_poly(2 * u + 1)) ? ex2_poly3(th) : ex2_approx(th);
            c |= (cvt_e2m1x2(lo, hi) & 0xffu) << (8 * u);
        }
        code32 = f.live ? c : 0u;
        byte = f.byte;
    } else if (PRODUCER == kEfqLut) {
        float rmax = fmaxf(max3(r[0], r[1], r[2]), max3(r[3], r[4], r[5]));
        rmax = max3(rmax, r[6], r[7]);
        rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, 1));
        rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, 2));
        BlockScale s = efq_block_scale(rmax, m_s, K);
        const float A16 = K.A * 0.0625f, B16 = s.Bb * 0.0625f;
        uint32_t c = 0;
#pragma unroll
        for (int u = 0; u < 8; ++u) c |= lut_code(r[u], A16, B16) << (4 * u);
        code32 = c;
        byte = s.byte;
    } else {
        float p[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            float x = __fsub_rn(__fmul_rn(K.sigma, r[u]), m_s);
            p[u] = ex2_approx(__fmul_rn(x, K.LOG2E));   // exp(-inf) = 0 covers masked entries
        }
        float amax = fmaxf(max3(p[0], p[1], p[2]), max3(p[3], p[4], p[5]));
        amax = max3(amax, p[6], p[7]);
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 1));
        amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
        if (amax == 0.0f) {
            code32 = 0u;
            byte = 0u;
            return;
        }
        const uint32_t bits = __float_as_uint(amax);
        const int E = static_cast<int>((bits >> 23) & 0xffu) - 127;
        int e;
        if (PRODUCER == kEtq4) {
            e = E - 2;                                   // maximum lands in [4, 8)
        } else {
            e = (bits & 0x7fffffu) > 0x400000u ? E - 1 : E - 2;   // smallest e with amax <= 6 * 2^e
        }
        e = max(e, -127);
        // 2^-e as a float: e is in [-127, 125], so the exponent field 127 - e is in [2, 254].
        const float s = __uint_as_float(static_cast<uint32_t>(127 - e) << 23);
        uint32_t c = 0;
#pragma unroll
        for (int u = 0; u < 4; ++u) c |= (cvt_e2m1x2(p[2 * u] * s, p[2 * u + 1] * s) & 0xffu) << (8 * u);
        code32 = c;
        byte = static_cast<uint32_t>(e + 127);
    }
}

// 8 consecutive floats with one 256-bit load (address 32-byte aligned), bypassing L1
__device__ __forceinline__ void load8(const float* p, float (&r)[8])
{
    asm volatile("ld.global.L1::no_allocate.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
                 : "l"(p));
}

template <int PRODUCER>
__device__ __forceinline__ void probgen_body(const float* __restrict__ scores, int64_t ld, const float* __restrict__ row_max,
                                             int64_t rows, int64_t cols, const ProducerConsts& K, uint8_t* __restrict__ codes,
                                             uint8_t* __restrict__ scales, int aligned32)
{
    const int lane = threadIdx.x & 31;
    const int64_t segs_per_row = (cols + kSegCols - 1) / kSegCols;
    const int64_t n_tasks = rows * segs_per_row;
    const int64_t nblk = (cols + kMxBlock - 1) / kMxBlock;
    const int64_t warp0 = static_cast<int64_t>(blockIdx.x) * kWarpsPerCta + (threadIdx.x >> 5);
    const int64_t n_warps = static_cast<int64_t>(gridDim.x) * kWarpsPerCta;

    for (int64_t task = warp0; task < n_tasks; task += n_warps) {
        const int64_t row = task / segs_per_row;
        const int64_t c0 = (task - row * segs_per_row) * kSegCols;
        const float* src = scores + row * ld + c0;
        const float m_s = __ldg(row_max + row);
        uint8_t* crow = codes + row * nblk * (kMxBlock / 2) + c0 / 2;
        uint8_t* srow = scales + row * nblk + c0 / kMxBlock;
        const bool full = c0 + kSegCols <= cols;
        const int rem = full ? kSegCols : static_cast<int>(cols - c0);   // valid columns of this segment

        // pass i: lane l holds columns (i*32 + l)*8 .. +7 -> every load instruction covers 1 KiB
        float r[4][8];
        if (full && aligned32) {
#pragma unroll
            for (int i = 0; i < 4; ++i) load8(src + (i * 32 + lane) * 8, r[i]);
        } else if (full) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float4* q = reinterpret_cast<const float4*>(src + (i * 32 + lane) * 8);
                float4 a = __ldcs(q), b = __ldcs(q + 1);
                r[i][0] = a.x; r[i][1] = a.y; r[i][2] = a.z; r[i][3] = a.w;
                r[i][4] = b.x; r[i][5] = b.y; r[i][6] = b.z; r[i][7] = b.w;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int u = 0; u < 8; ++u) {
                    const int c = (i * 32 + lane) * 8 + u;
                    r[i][u] = c < rem ? __ldcs(src + c) : -INFINITY;
                }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t code32, byte;
            produce_block<PRODUCER>(r[i], m_s, K, code32, byte);
            const int blk_col = ((i * 32 + lane) >> 2) * kMxBlock;   // first column of this lane's block, in the segment
            if (full || blk_col < rem) {
                *reinterpret_cast<uint32_t*>(crow + i * 128 + lane * 4) = code32;
                if ((lane & 3) == 0) srow[i * 8 + (lane >> 2)] = static_cast<uint8_t>(byte);
            }
        }
    }
}

template <int PRODUCER>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
probgen_kernel(const float* __restrict__ scores, int64_t ld, const float* __restrict__ row_max, int64_t rows, int64_t cols,
               ProducerConsts K, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales, int aligned32)
{
    probgen_body<PRODUCER>(scores, ld, row_max, rows, cols, K, codes, scales, aligned32);
}

// The LUT producer is issue-bound and register-hungry (one code at a time through a 64-bit shift): it gains more from
// three resident CTAs per SM than from the registers the compiler would otherwise take (69 -> 54 microseconds).
__global__ void __launch_bounds__(kWarpsPerCta * 32, 3)
probgen_lut_kernel(const float* __restrict__ scores, int64_t ld, const float* __restrict__ row_max, int64_t rows,
                   int64_t cols, ProducerConsts K, uint8_t* __restrict__ codes, uint8_t* __restrict__ scales, int aligned32)
{
    probgen_body<kEfqLut>(scores, ld, row_max, rows, cols, K, codes, scales, aligned32);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

efq_status_t launch_probgen(int producer, const float* scores, int64_t ld, const float* row_max, int64_t rows,
                            int64_t cols, float sigma, float tau, float h, uint8_t* codes, uint8_t* scales,
                            cudaStream_t stream)
{
    if (rows < 0 || cols < 0) return EFQ_ERR_INVALID_ARG;
    if (rows == 0 || cols == 0) return EFQ_OK;
    if (!scores || !row_max || !codes || !scales) return EFQ_ERR_INVALID_ARG;
    if (!isfinite(sigma) || !isfinite(tau) || !isfinite(h) || !(h > 0.0f)) return EFQ_ERR_INVALID_ARG;
    if (ld < cols) return EFQ_ERR_INVALID_ARG;
    if (!aligned16(scores) || (ld & 3) != 0 || !aligned16(codes)) return EFQ_ERR_ALIGNMENT;

    int dev = 0, major = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return EFQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return EFQ_ERR_CUDA;
    if (major != 10) return EFQ_ERR_ARCH;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return EFQ_ERR_CUDA;

    ProducerConsts K = producer == kEfqLut ? make_producer_consts_lut(sigma) : make_producer_consts(sigma, tau, h);
    const int64_t n_tasks = rows * ((cols + kSegCols - 1) / kSegCols);
    int64_t ctas = (n_tasks + kWarpsPerCta - 1) / kWarpsPerCta;
    const int64_t cap = static_cast<int64_t>(sms) * 8 * 64;   // whole waves of 8 resident CTAs per SM
    if (ctas > cap) ctas = cap;
    dim3 grid(static_cast<unsigned>(ctas)), block(kWarpsPerCta * 32);
    const int a32 = ((reinterpret_cast<uintptr_t>(scores) & 31u) == 0 && (ld & 7) == 0) ? 1 : 0;   // 256-bit loads allowed
    switch (producer) {
        case kEfq:  probgen_kernel<kEfq><<<grid, block, 0, stream>>>(scores, ld, row_max, rows, cols, K, codes, scales, a32); break;
        case kEtq4: probgen_kernel<kEtq4><<<grid, block, 0, stream>>>(scores, ld, row_max, rows, cols, K, codes, scales, a32); break;
        case kEtq6: probgen_kernel<kEtq6><<<grid, block, 0, stream>>>(scores, ld, row_max, rows, cols, K, codes, scales, a32); break;
        case kEtq4Fold: probgen_kernel<kEtq4Fold><<<grid, block, 0, stream>>>(scores, ld, row_max, rows, cols, K, codes, scales, a32); break;
        case kEtq4Hybrid: probgen_kernel<kEtq4Hybrid><<<grid, block, 0, stream>>>(scores, ld, row_max, rows, cols, K, codes, scales, a32); break;
        case kEfqLut: probgen_lut_kernel<<<grid, block, 0, stream>>>(scores, ld, row_max, rows, cols, K, codes, scales, a32); break;
        default: return EFQ_ERR_INVALID_ARG;
    }
    return cudaGetLastError() == cudaSuccess ? EFQ_OK : EFQ_ERR_CUDA;
}

}  // namespace efq

extern "C" efq_status_t efq_probgen(const float* scores, int64_t ld, const float* row_max, int64_t rows,
                                    int64_t cols, float score_scale, const efq_params_t* params,
                                    uint8_t* codes, uint8_t* scales, void* stream)
{
    float tau = -3.06f, h = 2.30f;
    int producer = efq::kEfq;
    if (params) {
        if (params->variant != 0 && params->variant != 1) return EFQ_ERR_UNSUPPORTED;
        if (params->variant == 1) producer = efq::kEfqLut;   // fixed (tau16, h16): tau and h are not read
        tau = params->variant == 1 ? 0.0f : params->tau;
        h = params->variant == 1 ? 1.0f : params->h;
    }
    return efq::launch_probgen(producer, scores, ld, row_max, rows, cols, score_scale, tau, h, codes, scales,
                               static_cast<cudaStream_t>(stream));
}

extern "C" efq_status_t exp_then_quantize_probgen(const float* scores, int64_t ld, const float* row_max,
                                                  int64_t rows, int64_t cols, float score_scale, int scale_mode,
                                                  uint8_t* codes, uint8_t* scales, void* stream)
{
    if (scale_mode < 0 || scale_mode > 3) return EFQ_ERR_INVALID_ARG;
    return efq::launch_probgen(scale_mode == 0 ? efq::kEtq4 : scale_mode == 1 ? efq::kEtq6 : scale_mode == 2 ? efq::kEtq4Fold : efq::kEtq4Hybrid, scores, ld, row_max, rows, cols,
                               score_scale, 0.0f, 1.0f, codes, scales, static_cast<cudaStream_t>(stream));
}
