// Operand preparation for the fused forward: bf16 Q, K, V -> MXFP4 (packed E2M1 codes + one E8M0
// byte per 32 elements) in the layouts the TMA loads and tcgen05 block-scaled MMAs consume.
// This is the surrounding kernel's "existing low-bit path" (Sec. 3.1); EFQ itself does not touch it.
//
// OCP microscaling rule per 32-element block: shared exponent e = floor(log2 amax) - 2 (clamped to
// the E8M0 range), elements rounded to nearest-even E2M1 of x * 2^-e, saturating at +-6; an all-zero
// block gets byte 0 and zero codes.
//
// Layouts written (S_pad = S rounded up to 128; padding rows/keys are zero codes, byte 0):
//   Q, K codes   [B*H, S_pad, 64 B]          row-major, 2 codes per byte, element 2u in the low nibble
//                (few query tokens: the query heads of a KV group packed into one 128-row tile, [B*Hkv, 128, 64 B])
//   V^T codes    [B*Hkv, 128 (channel), S_pad/2 B]   keys contiguous: the P~V contraction runs over keys
//                (packed variable-length batch: [Hkv, 128, sum of S_pad / 2 B], the sequences side by side along the keys)
//   scale tiles  one 512-byte tile per 128 rows (Q, K: rows = tokens, 4 blocks along d;
//                V: rows = channels, 4 key blocks of the 128-key tile); byte of (row r, block b) at
//                (r % 32) * 16 + (r / 32) * 4 + b, the order the scale-factor copy into TMEM expects.
#include <cuda_bf16.h>

#include "efq_common.cuh"
#include "efq_internal.cuh"

namespace efq {

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b) { return __uint_as_float(b << 16); }

// 32 bf16 values (as 16 packed 32-bit words, element 2u in the low half) -> 16 bytes of codes + scale byte
__device__ __forceinline__ void mxfp4_block(const uint32_t (&w)[16], uint4& codes, uint32_t& byte)
{
    uint32_t amax = 0;   // bf16 magnitudes compare like unsigned integers
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        amax = max(amax, w[i] & 0x7fffu);
        amax = max(amax, (w[i] >> 16) & 0x7fffu);
    }
    if (amax == 0) {
        codes = make_uint4(0, 0, 0, 0);
        byte = 0;
        return;
    }
    int e = static_cast<int>(amax >> 7) - 127 - 2;   // exponent field of the largest magnitude, minus 2
    e = max(e, -127);
    const float s = __uint_as_float(static_cast<uint32_t>(127 - e) << 23);   // 2^-e, field in [2, 254]
    uint32_t out[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        uint32_t word = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            uint32_t v = w[q * 4 + i];
            float lo = bf16_bits_to_float(v & 0xffffu) * s;
            float hi = bf16_bits_to_float(v >> 16) * s;
            word |= (cvt_e2m1x2(lo, hi) & 0xffu) << (8 * i);
        }
        out[q] = word;
    }
    codes = make_uint4(out[0], out[1], out[2], out[3]);
    byte = static_cast<uint32_t>(e + 127);
}

__device__ __forceinline__ uint32_t sf_tile_offset(uint32_t r, uint32_t b) { return (r & 31u) * 16u + (r >> 5) * 4u + b; }

// One thread per (row, 32-wide block along d); d = 128.  t counts (padded row, block) pairs of the job.  The four
// scale bytes of a row are gathered by shuffles and stored as one word by the thread of block 0.
template <bool DENSE>
__device__ __forceinline__ void quantize_row_block(const QuantSeg& g, int64_t t)
{
    const bool active = t < g.heads * g.S_pad * 4;
    const int blk = static_cast<int>(t & 3);
    const int64_t prow = t >> 2;               // padded row index over all heads of the job
    uint4 c = make_uint4(0, 0, 0, 0);
    uint32_t byte = 0;
    if (active) {
        const int64_t head = prow / g.S_pad;
        const int64_t row = prow - head * g.S_pad;
        if (row < g.S) {
            int64_t src_head = head, src_row = row;
            if (g.pack_G > 1) {                // packed query tile: rows run over (query head of the group, token)
                const int64_t gq = row / g.pack_lq;
                src_head = head * g.pack_G + gq;
                src_row = row - gq * g.pack_lq;
            }
            const uint4* src = reinterpret_cast<const uint4*>(g.src + src_head * g.head_stride +
                                                              src_row * (DENSE ? 128 : g.row_stride) + blk * 32);
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 v = __ldg(src + i);
                w[4 * i + 0] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
            }
            mxfp4_block(w, c, byte);
        }
        *reinterpret_cast<uint4*>(g.codes + prow * 64 + blk * 16) = c;
    }
    // lanes 4k .. 4k+3 hold the four blocks of one row (the thread count is a multiple of 4, so a row never
    // straddles warps or the end of the range)
    uint32_t word = byte;
    word |= __shfl_down_sync(0xffffffffu, byte, 1) << 8;
    word |= __shfl_down_sync(0xffffffffu, byte, 2) << 16;
    word |= __shfl_down_sync(0xffffffffu, byte, 3) << 24;
    if (active && blk == 0) {
        const int64_t tile = prow >> 7;        // S_pad is a multiple of 128, so tiles never straddle heads
        *reinterpret_cast<uint32_t*>(g.sf + tile * 512 + sf_tile_offset(static_cast<uint32_t>(prow & 127), 0)) = word;
    }
}

// One thread per (32-key block, channel); consecutive threads take consecutive channels.  kb counts the key blocks
// of the job over all heads.
template <bool DENSE>
__device__ __forceinline__ void quantize_v_block(const QuantSeg& g, int64_t kb, int ch)
{
    const int64_t blocks_per_head = g.S_pad / 32;
    if (kb >= g.heads * blocks_per_head) return;
    const int64_t head = kb / blocks_per_head;
    const int64_t kblk = kb - head * blocks_per_head;
    const int64_t rs = DENSE ? 128 : g.row_stride;
    const uint16_t* src = reinterpret_cast<const uint16_t*>(g.src) + head * g.head_stride + kblk * 32 * rs + ch;
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int64_t k0 = kblk * 32 + 2 * i;
        uint32_t lo = k0 < g.S ? __ldg(src + (2 * i) * rs) : 0u;
        uint32_t hi = k0 + 1 < g.S ? __ldg(src + (2 * i + 1) * rs) : 0u;
        w[i] = lo | (hi << 16);
    }
    uint4 c;
    uint32_t byte;
    mxfp4_block(w, c, byte);
    *reinterpret_cast<uint4*>(g.codes + (head * 128 + ch) * g.v_row_bytes + g.v_x0 + kblk * 16) = c;
    const int64_t tile = head * g.v_sf_tiles_per_head + g.v_sf_tile0 + (kblk >> 2);
    g.sf[tile * 512 + sf_tile_offset(static_cast<uint32_t>(ch), static_cast<uint32_t>(kblk & 3))] = static_cast<uint8_t>(byte);
}

struct QuantArgs {
    QuantSeg q, k, v;
    uint32_t* status;           // 256 words, cleared here: the forward that follows starts from a clean status
    int64_t q_ctas, k_ctas;     // the grid: Q rows, then K rows, then V key blocks (two per CTA)
};

// The three operands in one launch.  DENSE: rows of a head are contiguous (row stride 128 known at compile time).
template <bool DENSE>
__global__ void __launch_bounds__(256) quantize_qkv_kernel(const QuantArgs a)
{
    const int64_t cta = blockIdx.x;
    if (cta == 0) a.status[threadIdx.x] = 0u;
    if (cta < a.q_ctas) {
        quantize_row_block<DENSE>(a.q, cta * 256 + threadIdx.x);
    } else if (cta < a.q_ctas + a.k_ctas) {
        quantize_row_block<DENSE>(a.k, (cta - a.q_ctas) * 256 + threadIdx.x);
    } else {
        quantize_v_block<DENSE>(a.v, (cta - a.q_ctas - a.k_ctas) * 2 + (threadIdx.x >> 7), static_cast<int>(threadIdx.x & 127));
    }
}

// The jobs of a packed batch in one launch: a CTA finds its job by bisection of the prefix sums.
__global__ void __launch_bounds__(256) quantize_jobs_kernel(const QuantJob* __restrict__ jobs, const int32_t* __restrict__ first_cta,
                                                            int n_jobs, uint32_t* status)
{
    const int cta = blockIdx.x;
    if (cta == 0) status[threadIdx.x] = 0u;
    int lo = 0, hi = n_jobs;                  // first_cta[lo] <= cta < first_cta[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(first_cta + mid) <= cta) lo = mid; else hi = mid;
    }
    const QuantJob& job = jobs[lo];
    const int64_t local = cta - __ldg(first_cta + lo);
    if (job.kind == kQuantRows) quantize_row_block<false>(job.seg, local * 256 + threadIdx.x);
    else quantize_v_block<false>(job.seg, local * 2 + (threadIdx.x >> 7), static_cast<int>(threadIdx.x & 127));
}

int64_t quantize_job_ctas(const QuantJob& job)
{
    if (job.kind == kQuantRows) return (job.seg.heads * job.seg.S_pad * 4 + 255) / 256;
    return (job.seg.heads * (job.seg.S_pad / 32) + 1) / 2;
}

cudaError_t launch_quantize_qkv(const QuantSeg& q, const QuantSeg& k, const QuantSeg& v, uint32_t* status, cudaStream_t stream)
{
    QuantArgs a;
    a.q = q; a.k = k; a.v = v;
    a.status = status;
    a.q_ctas = (q.heads * q.S_pad * 4 + 255) / 256;
    a.k_ctas = (k.heads * k.S_pad * 4 + 255) / 256;
    const int64_t v_ctas = (v.heads * (v.S_pad / 32) + 1) / 2;
    const int64_t grid = a.q_ctas + a.k_ctas + v_ctas;
    if (grid <= 0 || grid > 0x7fffffffll) return cudaErrorInvalidValue;
    if (q.row_stride == 128 && k.row_stride == 128 && v.row_stride == 128)
        quantize_qkv_kernel<true><<<static_cast<unsigned>(grid), 256, 0, stream>>>(a);
    else
        quantize_qkv_kernel<false><<<static_cast<unsigned>(grid), 256, 0, stream>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_quantize_jobs(const QuantJob* jobs, const int32_t* first_cta, int n_jobs, int64_t total_ctas, uint32_t* status,
                                 cudaStream_t stream)
{
    if (n_jobs <= 0 || total_ctas <= 0 || total_ctas > 0x7fffffffll) return cudaErrorInvalidValue;
    quantize_jobs_kernel<<<static_cast<unsigned>(total_ctas), 256, 0, stream>>>(jobs, first_cta, n_jobs, status);
    return cudaGetLastError();
}

}  // namespace efq
