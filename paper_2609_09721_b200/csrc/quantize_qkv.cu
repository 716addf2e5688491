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
//   V^T codes    [B*Hkv, 128 (channel), S_pad/2 B]   keys contiguous: the P~V contraction runs over keys
//   scale tiles  one 512-byte tile per 128 rows (Q, K: rows = tokens, 4 blocks along d;
//                V: rows = channels, 4 key blocks of the 128-key tile); byte of (row r, block b) at
//                (r % 32) * 16 + (r / 32) * 4 + b, the order the scale-factor copy into TMEM expects.
#include <cuda_bf16.h>

#include "efq_common.cuh"

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

// One thread per (row, 32-wide block along d); d = 128.  The input is addressed by strides in elements:
// element (head, row, c) at x[head * head_stride + row * row_stride + c].  The four scale bytes of a row are
// gathered by shuffles and stored as one word by the thread of block 0.
__device__ __forceinline__ void quantize_row_block(const __nv_bfloat16* __restrict__ x, int64_t t, int64_t S,
                                                   int64_t S_pad, int64_t head_stride, int64_t row_stride,
                                                   uint8_t* __restrict__ codes, uint8_t* __restrict__ sf, bool active)
{
    const int blk = static_cast<int>(t & 3);
    const int64_t prow = t >> 2;               // padded row index over all heads
    uint4 c = make_uint4(0, 0, 0, 0);
    uint32_t byte = 0;
    if (active) {
        const int64_t head = prow / S_pad;
        const int64_t row = prow - head * S_pad;
        if (row < S) {
            const uint4* src = reinterpret_cast<const uint4*>(x + head * head_stride + row * row_stride + blk * 32);
            uint32_t w[16];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                uint4 v = __ldg(src + i);
                w[4 * i + 0] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
            }
            mxfp4_block(w, c, byte);
        }
        *reinterpret_cast<uint4*>(codes + prow * 64 + blk * 16) = c;
    }
    // lanes 4k .. 4k+3 hold the four blocks of one row (the thread count is a multiple of 4, so a row never
    // straddles warps or the end of the range)
    uint32_t word = byte;
    word |= __shfl_down_sync(0xffffffffu, byte, 1) << 8;
    word |= __shfl_down_sync(0xffffffffu, byte, 2) << 16;
    word |= __shfl_down_sync(0xffffffffu, byte, 3) << 24;
    if (active && blk == 0) {
        const int64_t tile = prow >> 7;        // S_pad is a multiple of 128, so tiles never straddle heads
        *reinterpret_cast<uint32_t*>(sf + tile * 512 + sf_tile_offset(static_cast<uint32_t>(prow & 127), 0)) = word;
    }
}

// One thread per (32-key block, channel); consecutive threads take consecutive channels.
__device__ __forceinline__ void quantize_v_block(const __nv_bfloat16* __restrict__ v, int64_t kb, int ch, int64_t S,
                                                 int64_t S_pad, int64_t head_stride, int64_t row_stride,
                                                 uint8_t* __restrict__ vt_codes, uint8_t* __restrict__ sf)
{
    const int64_t blocks_per_head = S_pad / 32;
    const int64_t head = kb / blocks_per_head;
    const int64_t kblk = kb - head * blocks_per_head;
    const uint16_t* src = reinterpret_cast<const uint16_t*>(v) + head * head_stride + kblk * 32 * row_stride + ch;
    uint32_t w[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int64_t k0 = kblk * 32 + 2 * i;
        uint32_t lo = k0 < S ? __ldg(src + (2 * i) * row_stride) : 0u;
        uint32_t hi = k0 + 1 < S ? __ldg(src + (2 * i + 1) * row_stride) : 0u;
        w[i] = lo | (hi << 16);
    }
    uint4 c;
    uint32_t byte;
    mxfp4_block(w, c, byte);
    *reinterpret_cast<uint4*>(vt_codes + (head * 128 + ch) * (S_pad / 2) + kblk * 16) = c;
    const int64_t tile = head * (S_pad / 128) + (kblk >> 2);
    sf[tile * 512 + sf_tile_offset(static_cast<uint32_t>(ch), static_cast<uint32_t>(kblk & 3))] = static_cast<uint8_t>(byte);
}

struct QuantArgs {
    const __nv_bfloat16 *q, *k, *v;
    int64_t q_heads, kv_heads, Sq, Sq_pad, Sk, Sk_pad;
    int64_t q_head_stride, q_row_stride, kv_head_stride, kv_row_stride;     // elements
    uint8_t *q_codes, *q_sf, *k_codes, *k_sf, *vt_codes, *v_sf;
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
        const int64_t t = cta * 256 + threadIdx.x;
        quantize_row_block(a.q, t, a.Sq, a.Sq_pad, a.q_head_stride, DENSE ? 128 : a.q_row_stride, a.q_codes, a.q_sf,
                           t < a.q_heads * a.Sq_pad * 4);
    } else if (cta < a.q_ctas + a.k_ctas) {
        const int64_t t = (cta - a.q_ctas) * 256 + threadIdx.x;
        quantize_row_block(a.k, t, a.Sk, a.Sk_pad, a.kv_head_stride, DENSE ? 128 : a.kv_row_stride, a.k_codes, a.k_sf,
                           t < a.kv_heads * a.Sk_pad * 4);
    } else {
        const int64_t kb = (cta - a.q_ctas - a.k_ctas) * 2 + (threadIdx.x >> 7);
        if (kb < a.kv_heads * (a.Sk_pad / 32))
            quantize_v_block(a.v, kb, static_cast<int>(threadIdx.x & 127), a.Sk, a.Sk_pad, a.kv_head_stride,
                             DENSE ? 128 : a.kv_row_stride, a.vt_codes, a.v_sf);
    }
}

cudaError_t launch_quantize_qkv(const void* q, const void* k, const void* v, int64_t q_heads, int64_t kv_heads, int64_t Sq,
                                int64_t Sq_pad, int64_t Sk, int64_t Sk_pad, int64_t q_head_stride, int64_t q_row_stride,
                                int64_t kv_head_stride, int64_t kv_row_stride, uint8_t* q_codes, uint8_t* q_sf,
                                uint8_t* k_codes, uint8_t* k_sf, uint8_t* vt_codes, uint8_t* v_sf, uint32_t* status,
                                cudaStream_t stream)
{
    QuantArgs a;
    a.q = static_cast<const __nv_bfloat16*>(q); a.k = static_cast<const __nv_bfloat16*>(k); a.v = static_cast<const __nv_bfloat16*>(v);
    a.q_heads = q_heads; a.kv_heads = kv_heads; a.Sq = Sq; a.Sq_pad = Sq_pad; a.Sk = Sk; a.Sk_pad = Sk_pad;
    a.q_head_stride = q_head_stride; a.q_row_stride = q_row_stride;
    a.kv_head_stride = kv_head_stride; a.kv_row_stride = kv_row_stride;
    a.q_codes = q_codes; a.q_sf = q_sf; a.k_codes = k_codes; a.k_sf = k_sf; a.vt_codes = vt_codes; a.v_sf = v_sf;
    a.status = status;
    a.q_ctas = (q_heads * Sq_pad * 4 + 255) / 256;
    a.k_ctas = (kv_heads * Sk_pad * 4 + 255) / 256;
    const int64_t v_ctas = (kv_heads * (Sk_pad / 32) + 1) / 2;
    const int64_t grid = a.q_ctas + a.k_ctas + v_ctas;
    if (grid <= 0 || grid > 0x7fffffffll) return cudaErrorInvalidValue;
    if (q_row_stride == 128 && kv_row_stride == 128)
        quantize_qkv_kernel<true><<<static_cast<unsigned>(grid), 256, 0, stream>>>(a);
    else
        quantize_qkv_kernel<false><<<static_cast<unsigned>(grid), 256, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace efq
