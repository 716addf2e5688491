// Declarations shared by the operand preparation (quantize_qkv.cu) and the fused forward (attention_fwd.cu):
// the job descriptions of the quantiser and the tables a packed variable-length batch hands to the kernels.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace efq {

// One operand of one sequence for the quantiser.  Rows of Q and K are quantised along d (blocks of 32), V along
// the keys (blocks of 32 aligned to the sequence's own key index, per channel) and written transposed.
struct QuantSeg {
    const __nv_bfloat16* src;  // element (head, row, c) at src[head * head_stride + row * row_stride + c]
    int64_t heads;             // heads of the code matrix: query (or KV) heads; KV heads for a packed Q
    int64_t S;                 // valid rows per head (tokens; pack_G * pack_lq rows for a packed Q)
    int64_t S_pad;             // rows per head in the code matrix, a multiple of 128
    int64_t head_stride, row_stride;   // of the source, in elements
    int32_t pack_lq, pack_G;   // Q only; pack_G > 1: row r of KV head h is token r % pack_lq of query head h * pack_G + r / pack_lq
    uint8_t* codes;            // Q, K: [heads * S_pad, 64 B] from here on; V: see v_row_bytes
    uint8_t* sf;               // scale tiles: Q, K one 512-byte tile per 128 rows from here on; V: see v_sf_tile0
    int64_t v_row_bytes;       // V only: bytes of one row (channel) of the transposed code matrix [heads * 128, v_row_bytes]
    int64_t v_x0;              // V only: byte offset of this sequence's first key inside a row
    int64_t v_sf_tiles_per_head, v_sf_tile0;   // V only: tile of (head, 128-key tile t) = head * per_head + tile0 + t
};

enum QuantKind : int32_t { kQuantRows = 0, kQuantV = 1 };

struct QuantJob {
    QuantSeg seg;
    int32_t kind;
    int32_t pad;
};

// Q, K and V of one [B, H, S, d] problem (or one sequence) in one launch; also clears the 256 status words.
cudaError_t launch_quantize_qkv(const QuantSeg& q, const QuantSeg& k, const QuantSeg& v, uint32_t* status, cudaStream_t stream);
// The jobs of a packed batch in one launch: jobs and first_cta (n_jobs + 1 prefix sums of CTAs) live in device memory.
cudaError_t launch_quantize_jobs(const QuantJob* jobs, const int32_t* first_cta, int n_jobs, int64_t total_ctas, uint32_t* status,
                                 cudaStream_t stream);
// CTAs a job needs (256 threads each)
int64_t quantize_job_ctas(const QuantJob& job);

// One sequence of a packed batch as the fused forward sees it.
struct SeqDesc {
    int64_t Sq, Sk;          // query and key tokens of the sequence
    int64_t o_off;           // element offset of the sequence's first output row in o
    int32_t q_row0;          // first row of the sequence in the Q code matrix (head 0, tile 0)
    int32_t Sq_pad;          // rows per head there
    int32_t k_row0, Sk_pad;  // the same for K
    int32_t k_col0;          // first key of the sequence along the key axis of the V^T code matrix (a multiple of 128)
    int32_t packed;          // 1: the query heads of a KV group share one 128-row query tile (few query tokens)
};
// One work item (CTA) of the fused forward over a packed batch.
struct ItemDesc {
    int32_t seq;             // index into the sequence table
    int32_t qt;              // query tile inside the sequence (0 when packed)
    int32_t head;            // query head, or KV head when packed
    int32_t pad;
};

}  // namespace efq
