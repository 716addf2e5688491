// Offline selection of the affine rule's parameters (Algorithm 3, Sec. "Parameter Calibration") and its helpers:
//   efq_exact_attention_fwd   softmax attention in FP32 on the unquantised bf16 inputs: the reference output O_ref
//                             of the calibration objective, and the "exact" side of every error figure reported;
//   efq_relative_error        rho = ||A - R||_F / ||R||_F, the objective itself (sums kept in double);
//   efq_calibrate             the grid search: operands quantised once, one fused forward per candidate (tau, h),
//                             rho of each, the first minimum in scan order.
// None of this is on the inference path: the selected pair stays fixed afterwards.  The reference kernel is a
// plain tiled CUDA-core kernel (32 queries x 32 keys per step); it is a measuring stick, not a fast path.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <vector>

#include "efq_common.cuh"

namespace efq {
namespace {

constexpr int kRq = 32;   // query rows per CTA
constexpr int kRk = 32;   // keys per step
constexpr int kD = 128;

__global__ void __launch_bounds__(256)
exact_attention_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                       const __nv_bfloat16* __restrict__ v, float* __restrict__ o, int Hq, int Hkv, int64_t Sq,
                       int64_t Sk, int causal, float sigma)
{
    __shared__ float qs[kRq][kD + 1];
    __shared__ __nv_bfloat16 ks[kRk][kD + 8];
    __shared__ __nv_bfloat16 vs[kRk][kD];
    __shared__ float ps[kRq][kRk + 1];
    __shared__ float alpha_s[kRq], m_s[kRq], l_s[kRq];

    const int t = threadIdx.x;
    const int64_t bh = blockIdx.y;
    const int64_t b = bh / Hq, hq = bh % Hq, hkv = hq / (Hq / Hkv);
    const int64_t q0 = static_cast<int64_t>(blockIdx.x) * kRq;
    const __nv_bfloat16* qh = q + (bh * Sq) * kD;
    const __nv_bfloat16* kh = k + ((b * Hkv + hkv) * Sk) * kD;
    const __nv_bfloat16* vh = v + ((b * Hkv + hkv) * Sk) * kD;
    const int64_t shift = Sk - Sq;

    for (int i = t; i < kRq * kD; i += 256) {
        const int r = i / kD, c = i % kD;
        qs[r][c] = q0 + r < Sq ? __bfloat162float(qh[(q0 + r) * kD + c]) : 0.0f;
    }
    if (t < kRq) { m_s[t] = -INFINITY; l_s[t] = 0.0f; }
    const int row = t >> 3;            // score and output row of this thread
    const int kq = t & 7;              // scores: keys kq, kq+8, kq+16, kq+24; output: channels kq*16 .. +15
    float acc[16];
#pragma unroll
    for (int c = 0; c < 16; ++c) acc[c] = 0.0f;

    int64_t last_key = Sk - 1;         // last key any row of this tile sees
    if (causal) {
        const int64_t last_row = q0 + kRq - 1 < Sq ? q0 + kRq - 1 : Sq - 1;
        last_key = last_row + shift < Sk - 1 ? last_row + shift : Sk - 1;
    }
    __syncthreads();

    for (int64_t k0 = 0; k0 <= last_key; k0 += kRk) {
        // K and V tile: 32 keys x 128 channels of bf16 each, 16 bytes per thread and tensor
        {
            const int key = t >> 3, part = t & 7;     // 8 x 16 channels per key
            uint4 kk = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
            uint4 kk2 = kk, vv2 = vv;
            if (k0 + key < Sk) {
                const uint4* ksrc = reinterpret_cast<const uint4*>(kh + (k0 + key) * kD + part * 16);
                const uint4* vsrc = reinterpret_cast<const uint4*>(vh + (k0 + key) * kD + part * 16);
                kk = ksrc[0]; kk2 = ksrc[1]; vv = vsrc[0]; vv2 = vsrc[1];
            }
            *reinterpret_cast<uint4*>(&ks[key][part * 16]) = kk;
            *reinterpret_cast<uint4*>(&ks[key][part * 16 + 8]) = kk2;
            *reinterpret_cast<uint4*>(&vs[key][part * 16]) = vv;
            *reinterpret_cast<uint4*>(&vs[key][part * 16 + 8]) = vv2;
        }
        __syncthreads();
        // scores
        {
            float s[4] = {0.f, 0.f, 0.f, 0.f};
            for (int c = 0; c < kD; c += 2) {
                const float q0f = qs[row][c], q1f = qs[row][c + 1];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 kf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&ks[kq + 8 * i][c]));
                    s[i] = fmaf(q0f, kf.x, s[i]);
                    s[i] = fmaf(q1f, kf.y, s[i]);
                }
            }
            const int64_t limit = causal ? q0 + row + shift : Sk - 1;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int64_t key = k0 + kq + 8 * i;
                ps[row][kq + 8 * i] = (key <= limit && key < Sk && q0 + row < Sq) ? s[i] * sigma : -INFINITY;
            }
        }
        __syncthreads();
        // online softmax of the 32 rows (one thread per row; small next to the two contractions)
        if (t < kRq) {
            float m_old = m_s[t], m_new = m_old;
            for (int i = 0; i < kRk; ++i) m_new = fmaxf(m_new, ps[t][i]);
            float a = 1.0f, sum = 0.0f;
            if (m_new == -INFINITY) {
                for (int i = 0; i < kRk; ++i) ps[t][i] = 0.0f;
            } else {
                a = m_old == -INFINITY ? 0.0f : expf(m_old - m_new);
                for (int i = 0; i < kRk; ++i) {
                    const float p = expf(ps[t][i] - m_new);   // exp(-inf) = 0 for masked keys
                    ps[t][i] = p;
                    sum += p;
                }
            }
            alpha_s[t] = a;
            m_s[t] = m_new;
            l_s[t] = l_s[t] * a + sum;
        }
        __syncthreads();
        // O <- alpha O + P V
        {
            const float a = alpha_s[row];
#pragma unroll
            for (int c = 0; c < 16; ++c) acc[c] *= a;
            for (int i = 0; i < kRk; ++i) {
                const float p = ps[row][i];
#pragma unroll
                for (int c = 0; c < 16; c += 2) {
                    const float2 vf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&vs[i][kq * 16 + c]));
                    acc[c] = fmaf(p, vf.x, acc[c]);
                    acc[c + 1] = fmaf(p, vf.y, acc[c + 1]);
                }
            }
        }
        __syncthreads();
    }
    if (q0 + row < Sq) {
        const float l = l_s[row];
        const float inv = l > 0.0f ? 1.0f / l : 0.0f;
        float* dst = o + ((bh * Sq) + q0 + row) * kD + kq * 16;
#pragma unroll
        for (int c = 0; c < 16; ++c) dst[c] = acc[c] * inv;
    }
}

// sums[0] += sum (a - r)^2, sums[1] += sum r^2, in double
__global__ void __launch_bounds__(256) error_sums_kernel(const float* __restrict__ a, const float* __restrict__ r,
                                                         int64_t n, double* sums)
{
    double d2 = 0.0, r2 = 0.0;
    for (int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; i < n; i += static_cast<int64_t>(gridDim.x) * 256) {
        const double x = static_cast<double>(a[i]), y = static_cast<double>(r[i]);
        d2 += (x - y) * (x - y);
        r2 += y * y;
    }
    for (int off = 16; off > 0; off >>= 1) {
        d2 += __shfl_xor_sync(0xffffffffu, d2, off);
        r2 += __shfl_xor_sync(0xffffffffu, r2, off);
    }
    __shared__ double sd[8], sr[8];
    if ((threadIdx.x & 31) == 0) { sd[threadIdx.x >> 5] = d2; sr[threadIdx.x >> 5] = r2; }
    __syncthreads();
    if (threadIdx.x == 0) {
        double td = 0.0, tr = 0.0;
        for (int w = 0; w < 8; ++w) { td += sd[w]; tr += sr[w]; }
        atomicAdd(&sums[0], td);
        atomicAdd(&sums[1], tr);
    }
}

bool is_sm100()
{
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return false;
    return major == 10;
}

}  // namespace
}  // namespace efq

extern "C" efq_status_t efq_exact_attention_fwd(const void* q, const void* k, const void* v, float* o, int B, int Hq,
                                                int Hkv, int64_t Sq, int64_t Sk, int d, int causal,
                                                float softmax_scale, void* stream)
{
    if (!q || !k || !v || !o) return EFQ_ERR_INVALID_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || Hq % Hkv != 0) return EFQ_ERR_INVALID_ARG;
    if (d != 128) return EFQ_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) | reinterpret_cast<uintptr_t>(v) |
         reinterpret_cast<uintptr_t>(o)) & 15u)
        return EFQ_ERR_ALIGNMENT;
    if (static_cast<int64_t>(B) * Hq > 65535) return EFQ_ERR_UNSUPPORTED;
    if (!efq::is_sm100()) return EFQ_ERR_ARCH;
    const float sigma = softmax_scale > 0.0f ? softmax_scale : 0.08838834764831845f;
    dim3 grid(static_cast<unsigned>((Sq + efq::kRq - 1) / efq::kRq), static_cast<unsigned>(B * Hq));
    efq::exact_attention_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __nv_bfloat16*>(q), static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v), o,
        Hq, Hkv, Sq, Sk, causal ? 1 : 0, sigma);
    return cudaGetLastError() == cudaSuccess ? EFQ_OK : EFQ_ERR_CUDA;
}

extern "C" efq_status_t efq_relative_error(const float* a, const float* ref, int64_t n, double* sums, void* stream)
{
    if (!a || !ref || !sums || n < 0) return EFQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(sums, 0, 2 * sizeof(double), s) != cudaSuccess) return EFQ_ERR_CUDA;
    if (n == 0) return EFQ_OK;
    int64_t blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    efq::error_sums_kernel<<<static_cast<unsigned>(blocks), 256, 0, s>>>(a, ref, n, sums);
    return cudaGetLastError() == cudaSuccess ? EFQ_OK : EFQ_ERR_CUDA;
}

extern "C" efq_status_t efq_calibrate(const void* q, const void* k, const void* v, const float* o_ref, float* o_tmp,
                                      int B, int Hq, int Hkv, int64_t Sq, int64_t Sk, int d, int causal,
                                      float softmax_scale, const float* taus, int n_tau, const float* hs, int n_h,
                                      double* sums, double* rho, float* best_tau, float* best_h, void* workspace,
                                      size_t workspace_bytes, void* stream)
{
    if (!o_ref || !o_tmp || !taus || !hs || !sums || !rho || n_tau <= 0 || n_h <= 0) return EFQ_ERR_INVALID_ARG;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    efq_status_t st = efq_quantize_qkv(q, k, v, B, Hq, Hkv, Sq, Sk, d, workspace, workspace_bytes, stream);
    if (st != EFQ_OK) return st;
    const int64_t n = static_cast<int64_t>(B) * Hq * Sq * d;
    const int n_cand = n_tau * n_h;
    for (int it = 0; it < n_tau; ++it) {
        for (int ih = 0; ih < n_h; ++ih) {
            efq_params_t p;
            p.tau = taus[it];
            p.h = hs[ih];
            p.variant = 0;
            p.kv_tile = 0;
            p.rescale_threshold = 0.0f;
            st = efq_attention_fwd_quantized(o_tmp, B, Hq, Hkv, Sq, Sk, d, causal, softmax_scale, 0, &p, workspace,
                                             workspace_bytes, nullptr, stream);
            if (st != EFQ_OK) return st;
            st = efq_relative_error(o_tmp, o_ref, n, sums + 2 * (it * n_h + ih), stream);
            if (st != EFQ_OK) return st;
        }
    }
    std::vector<double> host(2 * static_cast<size_t>(n_cand));
    if (cudaMemcpyAsync(host.data(), sums, host.size() * sizeof(double), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return EFQ_ERR_CUDA;
    st = efq_poll_status(workspace, stream);          // synchronises the stream; reports an expired device-side wait
    if (st != EFQ_OK) return st;
    double best = INFINITY;
    if (best_tau) *best_tau = taus[0];
    if (best_h) *best_h = hs[0];
    for (int i = 0; i < n_cand; ++i) {
        rho[i] = host[2 * i + 1] > 0.0 ? sqrt(host[2 * i] / host[2 * i + 1]) : (host[2 * i] > 0.0 ? INFINITY : 0.0);
        if (rho[i] < best) {                          // strict: the first minimum in scan order (tau outer, h inner)
            best = rho[i];
            if (best_tau) *best_tau = taus[i / n_h];
            if (best_h) *best_h = hs[i % n_h];
        }
    }
    return EFQ_OK;
}
