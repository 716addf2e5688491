// Two measurement kernels behind the C ABI:
//   efq_fp4_mma_peak_probe   MMA-only loop of kind::mxf4 block-scaled 128x256x64 MMAs on operands resident in
//                            shared memory, one CTA per SM: the dense FP4 rate the tensor pipe reaches here.
//   efq_stage_microbench     the probability producers of the fused forward on register-resident scores, no
//                            memory traffic: elements per clock per SM for EFQ versus exp-then-quantize - the
//                            in-SM form of the paper's "vector stage" comparison (Sec. 5.5).
#include <cuda_runtime.h>

#include "efq_common.cuh"
#include "efq_producers.cuh"
#include "sm100_ptx.cuh"

namespace efq {
namespace {

constexpr uint64_t kProbeTimeoutCycles = 4000000000ull;

__global__ void __launch_bounds__(128) fp4_peak_kernel(int iters, uint32_t* sink)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    __shared__ uint32_t tmem_base_s;
    __shared__ __align__(8) uint64_t mbar;
    const int tid = threadIdx.x, warp = tid >> 5;
    // A: 128 rows x 64 B, B: 256 rows x 64 B of pseudo-random E2M1 codes; unit scale factors
    for (int i = tid; i < (8192 + 16384) / 4; i += 128)
        reinterpret_cast<uint32_t*>(smem)[i] = static_cast<uint32_t>(i * 2654435761u) ^ (static_cast<uint32_t>(i) << 13) ^ (0x5bd1e995u * (blockIdx.x + 1));
    for (int i = tid; i < 1024 / 4; i += 128) reinterpret_cast<uint32_t*>(smem + 8192 + 16384)[i] = 0x7f7f7f7fu;
    ptx::fence_proxy_async_smem();
    if (warp == 0) ptx::tmem_alloc(&tmem_base_s, 512);
    if (tid == 0) {
        ptx::mbar_init(&mbar, 1);
        ptx::mbar_init_fence();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tbase = tmem_base_s;
    if (warp == 0) {
        if (ptx::elect_one()) {
            const uint64_t dsf = ptx::smem_desc(ptx::smem_u32(smem + 8192 + 16384), 16, 128, ptx::kLayoutNone);
            for (int c = 0; c < 3; ++c) ptx::tmem_cp_sf(tbase + 256 + 4 * c, dsf);
            const uint64_t da = ptx::smem_desc(ptx::smem_u32(smem), 16, 512, ptx::kLayoutSw64);
            const uint64_t db = ptx::smem_desc(ptx::smem_u32(smem + 8192), 16, 512, ptx::kLayoutSw64);
            for (int it = 0; it < iters; ++it) {
                const uint32_t k = (it & 1) * 2;   // alternate the two 64-element halves of K
                ptx::mma_mxf4(tbase, da + k, db + k, ptx::mxf4_idesc(256, 0), tbase + 256, tbase + 260, it > 0 ? 1u : 0u);
            }
            ptx::mma_commit(&mbar);
        }
        __syncwarp();
    }
    // bounded wait, all threads
    bool ok = ptx::mbar_try_wait(&mbar, 0);
    const long long t0 = clock64();
    while (!ok) {
        ok = ptx::mbar_try_wait_suspend(&mbar, 0, 20000u);
        if (!ok && static_cast<uint64_t>(clock64() - t0) > kProbeTimeoutCycles) break;
    }
    ok = __all_sync(0xffffffffu, ok);
    ptx::tc_fence_after_sync();
    if (warp == 0) {
        const uint32_t v = ok ? ptx::tmem_ld1(tbase) : 0xffffffffu;
        if (ok) ptx::tmem_wait_ld();
        if (tid == 0) sink[blockIdx.x] = ok ? v : 0xdeadbeefu;
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) ptx::tmem_dealloc(tbase, 512);
}

template <int PRODUCER, bool FIX8>
__global__ void __launch_bounds__(256) stage_kernel(ProducerConsts K, int iters, uint32_t* sink, long long* cycles)
{
    float r[32];
    const uint32_t seed = (blockIdx.x * 256u + threadIdx.x) * 2654435761u;
#pragma unroll
    for (int i = 0; i < 32; ++i) {   // raw scores of a plausible spread (sigma * r of a few units)
        const uint32_t h = (seed + i * 0x9E3779B9u) * 0x85EBCA6Bu;
        r[i] = (static_cast<float>(h >> 8) * (1.0f / 16777216.0f) - 0.5f) * 160.0f;
    }
    float m_s = 7.0f;
    uint32_t acc = 0;
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
        uint4 codes;
        uint32_t byte;
        const float rmax = block_max32(r);
        produce32<PRODUCER, FIX8>(r, rmax, m_s, K, codes, byte);
        acc ^= codes.x ^ codes.y ^ codes.z ^ codes.w ^ byte;
        const float delta = __uint_as_float(0x3a000000u + (acc & 0xffu));   // keeps the loop from being hoisted
#pragma unroll
        for (int i = 0; i < 32; ++i) r[i] += delta;
        m_s += 1e-3f;
    }
    const long long t1 = clock64();
    __syncthreads();
    if (threadIdx.x == 0) cycles[blockIdx.x] = t1 - t0;
    sink[blockIdx.x * 256 + threadIdx.x] = acc;
}

}  // namespace
}  // namespace efq

extern "C" efq_status_t efq_fp4_mma_peak_probe(uint32_t* sink, int num_ctas, int iters, double* flops, void* stream)
{
    if (!sink || num_ctas <= 0 || iters <= 0) return EFQ_ERR_INVALID_ARG;
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return EFQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return EFQ_ERR_CUDA;
    if (major != 10) return EFQ_ERR_ARCH;
    const size_t smem = 8192 + 16384 + 1024 + 1024;
    if (cudaFuncSetAttribute(efq::fp4_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess)
        return EFQ_ERR_CUDA;
    efq::fp4_peak_kernel<<<num_ctas, 128, smem, static_cast<cudaStream_t>(stream)>>>(iters, sink);
    if (flops) *flops = 2.0 * 128.0 * 256.0 * 64.0 * static_cast<double>(iters) * static_cast<double>(num_ctas);
    return cudaGetLastError() == cudaSuccess ? EFQ_OK : EFQ_ERR_CUDA;
}

extern "C" efq_status_t efq_stage_microbench(int producer, const efq_params_t* params, int num_ctas, int iters,
                                             uint32_t* sink, long long* cycles, void* stream)
{
    if (!sink || !cycles || num_ctas <= 0 || iters <= 0) return EFQ_ERR_INVALID_ARG;
    float tau = -3.06f, h = 2.30f;
    if (params) { tau = params->tau; h = params->h; }
    if (!(h > 0.0f)) return EFQ_ERR_INVALID_ARG;
    const efq::ProducerConsts K = efq::make_producer_consts(0.08838834764831845f, tau, h);
    const bool fix8 = (log(1.5) - static_cast<double>(tau)) * static_cast<double>(h) + 1.0 > 7.999;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    switch (producer) {
        case 0:
            if (fix8) efq::stage_kernel<0, true><<<num_ctas, 256, 0, s>>>(K, iters, sink, cycles);
            else efq::stage_kernel<0, false><<<num_ctas, 256, 0, s>>>(K, iters, sink, cycles);
            break;
        case 1: efq::stage_kernel<1, false><<<num_ctas, 256, 0, s>>>(K, iters, sink, cycles); break;
        case 2: efq::stage_kernel<2, false><<<num_ctas, 256, 0, s>>>(K, iters, sink, cycles); break;
        case 5: efq::stage_kernel<5, false><<<num_ctas, 256, 0, s>>>(K, iters, sink, cycles); break;
        case 4: efq::stage_kernel<4, false><<<num_ctas, 256, 0, s>>>(K, iters, sink, cycles); break;
        case 3: efq::stage_kernel<3, false><<<num_ctas, 256, 0, s>>>(efq::make_producer_consts_lut(0.08838834764831845f), iters, sink, cycles); break;
        default: return EFQ_ERR_INVALID_ARG;
    }
    return cudaGetLastError() == cudaSuccess ? EFQ_OK : EFQ_ERR_CUDA;
}
