/*
 * efq.h - C ABI of the B200 (sm_100a) EFQ-Softmax library.
 *
 * EFQ-Softmax replaces the exp-then-quantize producer of a block-scaled FP4 attention
 * forward by direct generation of the low-bit probability operand: per 32-key
 * microscaling block an exponent-only E8M0 scale taken from the block's largest shifted
 * score, and per element a nonnegative E2M1 code from one affine rule.  The same operand
 * feeds the numerator P~V and the denominator P~1; the online-softmax recurrence around
 * it is unchanged.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers unless the parameter name ends in _host.
 *   - The library never allocates or frees device memory on these paths; the caller owns
 *     every buffer, including the workspace, for the duration of the stream work.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Launches
 *     are asynchronous; a returned EFQ_OK means "validated and enqueued".
 *   - Errors are return codes; nothing aborts or traps.  Device-side waits are bounded and
 *     report through the status word read by efq_poll_status().
 *   - Packed E2M1 codes: element 2u sits in bits 0-3 of byte u, element 2u+1 in bits 4-7.
 *     Probability codes are nonnegative (bit 3 of every nibble is 0).
 *   - E8M0 scale byte b means the power of two 2^(b-127).
 *   - Microscaling block: 32 consecutive keys (columns), aligned to absolute index.
 */
#ifndef EFQ_H_
#define EFQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    EFQ_OK = 0,
    EFQ_ERR_INVALID_ARG = 1,    /* null pointer, non-positive size, non-finite parameter, Hq % Hkv != 0 */
    EFQ_ERR_UNSUPPORTED = 2,    /* d != 128, kv_tile not supported, variant not built */
    EFQ_ERR_ALIGNMENT = 3,      /* a pointer or leading dimension breaks the stated alignment */
    EFQ_ERR_WORKSPACE = 4,      /* workspace pointer null or smaller than efq_attention_workspace_bytes() */
    EFQ_ERR_ARCH = 5,           /* current device is not compute capability 10.x */
    EFQ_ERR_CUDA = 6,           /* a CUDA runtime/driver call failed (launch, copy, descriptor encode) */
    EFQ_ERR_DEVICE_TIMEOUT = 7, /* a bounded device-side wait expired; the output is invalid */
    EFQ_ERR_STATIC_LIMIT = 8    /* efq_attention_fwd_static: the problem needs more than EFQ_STATIC_SCRATCH_BYTES */
} efq_status_t;

/* Parameters of the affine code rule c = clip_[0,7](floor((z - tau) h) + 1)
 * (Eq. d8-index).  (tau, h) are global, fixed after calibration; the operating points
 * printed in the paper are EFQ-Mean (-3.06, 2.30), EFQ-MMLU (-2.90, 2.00) and
 * EFQ-Balance (-2.10, 2.70).  Passing NULL for a params pointer selects EFQ-Mean,
 * variant 0, kv_tile 128, rescale_threshold 0. */
typedef struct {
    float tau;
    float h;          /* > 0 */
    int32_t variant;  /* 0 = affine rule (Eq. d8-index).
                         1 = EFQ-Softmax-LUT (Sec. "EFQ-Softmax-LUT Variant"): the same block scale, the index
                         j = clip_[0,15](floor((z - tau16) h16) + 1) with the fixed pair tau16 = ln(1/24),
                         h16 = 14 / ln 24, folded by C16 = [0,1,1,1,1,1,2,2,3,3,4,5,5,6,7,7]; tau and h above
                         are not read.  Accepted by efq_probgen, every efq_attention_fwd* entry point and (as
                         producer 0 + variant 1) by the entry points that take a producer id.  Any other value
                         returns EFQ_ERR_UNSUPPORTED. */
    int32_t kv_tile;  /* Bc, keys per online-softmax step; 0 = default (128).  The shifted score uses the
                         running row maximum that includes the current KV block (Algorithm 2, steps 2-3),
                         so codes depend on this width.  Must be 128 in this build. */
    float rescale_threshold; /* T >= 0 in scaled-score units.  0 (default) is Algorithm 2 as printed: the running
                         maximum shifts the scores and the history is rescaled whenever it grows.  T > 0 (not in
                         the paper) keeps the shifting maximum m from tile to tile while the true running maximum
                         exceeds it by at most T: with cand = max(m, tile maximum), m <- cand if m = -inf or
                         fl(fl(scale cand) - fl(scale m)) > T, else m stays; a tile that keeps m needs no
                         rescaling of the accumulators.  Shifted scores may then reach +T; the scale rule is
                         shift-equivariant, so only block exponents move - but codes differ from T = 0.  Used by
                         the fused forwards only (efq_probgen takes its row maximum from the caller). */
} efq_params_t;

/* Optional debug dump of the fused forward for one head and a range of query rows.
 * Any pointer may be NULL.  Row r of each buffer is query row q_begin + r.
 *   raw_scores  fp32 [q_end-q_begin, Sk]            Q^ K^T before the softmax scale; masked keys hold -inf
 *   row_max     fp32 [q_end-q_begin, ceil(Sk/Bc)]   scaled running maximum m_s used for each KV tile
 *   codes       u8   [q_end-q_begin, ceil(Sk/32)*16] packed probability codes (linear order)
 *   scales      u8   [q_end-q_begin, ceil(Sk/32)]   E8M0 bytes */
typedef struct {
    float* raw_scores;
    float* row_max;
    uint8_t* codes;
    uint8_t* scales;
    int32_t batch;
    int32_t head;
    int64_t q_begin;
    int64_t q_end;
} efq_debug_t;

/* Probability-generation stage on a score matrix (kernel interface of Sec. 4.3:
 * (x, B, tau, h) -> (Q_P, s_P); Algorithm 1 applied to every 32-column block).
 *   scores   fp32 [rows, ld], 16-byte aligned, ld >= cols and ld % 4 == 0; masked entries = -inf
 *   row_max  fp32 [rows], the row maximum in scaled units: the shifted score is
 *            x = score_scale * scores - row_max
 *   codes    u8 [rows, ceil(cols/32)*16], 16-byte aligned; positions past `cols` in the last
 *            block get code 0
 *   scales   u8 [rows, ceil(cols/32)]; a block with no finite entry gets byte 0 and zero codes
 * Returns INVALID_ARG for null pointers, rows/cols < 0, h <= 0 or non-finite parameters,
 * ALIGNMENT as stated above.  rows == 0 or cols == 0 is a valid no-op. */
efq_status_t efq_probgen(const float* scores, int64_t ld, const float* row_max, int64_t rows, int64_t cols,
                         float score_scale, const efq_params_t* params, uint8_t* codes, uint8_t* scales,
                         void* stream);

/* The conventional producer on the same interface (Eq. post-softmax-path):
 * p = exp(x) in FP32, per block e = floor(log2 max p) - 2 (scale_mode 0, block maximum in
 * [4, 8)) or e = ceil(log2(max p / 6)) (scale_mode 1, block maximum in (3, 6]),
 * q = round-to-nearest-even E2M1 of p 2^-e, saturating.  Same layouts and errors.
 * scale_mode 2 is scale_mode 0 in its fastest form on this machine: the same mathematics with the scale folded
 * into the exponential, p 2^-e = 2^(x log2(e) - e), so that no FP32 probability is formed either - one FMA, one
 * ex2 and half a conversion per element, bound by the exponential unit (16 per clock per SM).  Results agree
 * with scale_mode 0 except at rounding knife-edges.
 * scale_mode 3 is scale_mode 2 with 2 of every 8 exponentials computed on the FMA pipe (floor, cubic polynomial
 * of the fraction with relative error 8.6e-5, exponent insertion) to take load off the exponential unit.  Measured
 * on B200 it gains 3 % in the register-resident stage and loses 6 % in the fused forward, where issue slots and
 * not the exponential unit are short; it is kept as the record of that comparison.  Codes differ from
 * scale_mode 0 on a few elements in ten thousand (the polynomial's error against the E2M1 rounding step). */
efq_status_t exp_then_quantize_probgen(const float* scores, int64_t ld, const float* row_max, int64_t rows,
                                       int64_t cols, float score_scale, int scale_mode, uint8_t* codes,
                                       uint8_t* scales, void* stream);

/* Bytes of caller-owned device workspace the fused forward needs for a problem shape
 * (MXFP4 copies of Q, K, V with their scale tiles, and the status word; tensor-map descriptors are built on the
 * host and travel as kernel parameters).
 * Returns 0 for an unsupported shape. */
size_t efq_attention_workspace_bytes(int B, int Hq, int Hkv, int64_t Sq, int64_t Sk, int d);

/* Fused block-scaled FP4 attention forward with EFQ probability generation
 * (Algorithm 2 looped over KV tiles; Algorithm 1 per microscaling block).
 *   q        bf16 [B, Hq, Sq, d] contiguous, 16-byte aligned
 *   k, v     bf16 [B, Hkv, Sk, d] contiguous, 16-byte aligned; query head h reads KV head h / (Hq/Hkv)
 *   o        fp32 [B, Hq, Sq, d]
 *   causal   nonzero: query i sees keys t <= i + Sk - Sq (bottom-right aligned)
 *   softmax_scale  <= 0 selects 1/sqrt(d)
 *   workspace  device, 256-byte aligned, >= efq_attention_workspace_bytes(...)
 * Q, K (blocks of 32 along d) and V (blocks of 32 along keys) are first quantised to MXFP4
 * (shared exponent floor(log2 amax) - 2, round-to-nearest-even, saturating); a query row with
 * no visible key yields zeros.  d must be 128 (UNSUPPORTED otherwise). */
efq_status_t efq_attention_fwd(const void* q, const void* k, const void* v, float* o, int B, int Hq, int Hkv,
                               int64_t Sq, int64_t Sk, int d, int causal, float softmax_scale,
                               const efq_params_t* params, void* workspace, size_t workspace_bytes,
                               const efq_debug_t* debug, void* stream);

/* The MXFP4 comparison path: identical pipeline, the producer replaced by exp-then-quantize
 * (scale_mode 0-3 as in exp_then_quantize_probgen).  The denominator comes from the same
 * quantised operand as the numerator (Eq. denominator-basic applied to the baseline: everything but the
 * producer held equal).
 * scale_mode 4 is scale_mode 0 with the other convention for the denominator, the one of attention kernels that
 * quantise P only for the P V product: l is the sum of the row's FP32 exponentials, carried in registers through
 * the online recurrence (rescaled with the same alpha), and the ones columns of the tensor-core product are
 * ignored.  Numerator and denominator then no longer come from one operand; the paper states the shared-operand
 * rule for its own method only, so both conventions are offered for the baseline. */
efq_status_t exp_then_quantize_attention_fwd(const void* q, const void* k, const void* v, float* o, int B,
                                             int Hq, int Hkv, int64_t Sq, int64_t Sk, int d, int causal,
                                             float softmax_scale, int scale_mode, void* workspace,
                                             size_t workspace_bytes, const efq_debug_t* debug, void* stream);

/* The two halves of efq_attention_fwd as separate calls, for callers that reuse quantised operands
 * (K/V shared by several forwards) or time the stages separately.
 * efq_quantize_qkv: operand preparation only (bf16 -> MXFP4 into the workspace; resets the status word).
 * efq_attention_fwd_quantized: the fused forward on a workspace prepared by efq_quantize_qkv for the
 * same shape; producer 0 = EFQ (with params->variant 1: EFQ-LUT), 1 = exp-then-quantize scale4, 2 = exp-then-quantize
 * scale6, 4 = exp-then-quantize scale4 with the scale folded into the exponential (scale_mode 2), 5 = scale_mode 3,
 * 6 = exp-then-quantize scale4 with the FP32-exponential denominator (scale_mode 4).
 * Arguments, layouts and errors as for efq_attention_fwd. */
efq_status_t efq_quantize_qkv(const void* q, const void* k, const void* v, int B, int Hq, int Hkv, int64_t Sq,
                              int64_t Sk, int d, void* workspace, size_t workspace_bytes, void* stream);
efq_status_t efq_attention_fwd_quantized(float* o, int B, int Hq, int Hkv, int64_t Sq, int64_t Sk, int d, int causal,
                                         float softmax_scale, int producer, const efq_params_t* params,
                                         void* workspace, size_t workspace_bytes, const efq_debug_t* debug,
                                         void* stream);

/* Packed variable-length batch (cross-attention, prefill of mixed lengths, decode steps; Sec. 4 names cross-attention
 * among the places the method applies).  The n_seqs sequences lie one after the other along the token axis:
 *   q [total_q, Hq, d], k and v [total_k, Hkv, d] bf16, o [total_q, Hq, d] fp32, all DEVICE, token-major;
 *   cu_seqlens_q / cu_seqlens_k: HOST arrays of n_seqs + 1 non-decreasing prefix sums starting at 0; sequence i owns
 *   query tokens [cu_q[i], cu_q[i+1]) and key tokens [cu_k[i], cu_k[i+1]).
 * Every sequence is an attention problem of its own (Algorithm 2 over its own keys; with `causal`, query i of a
 * sequence sees its keys <= i + len_k - len_q, the rule of efq_attention_fwd); the operands of a sequence are
 * quantised by themselves, so the result of a sequence equals efq_attention_fwd on that sequence alone, bit for
 * bit.  A sequence without queries is skipped; one without keys gets zero rows.  `producer` as for
 * efq_attention_fwd_quantized.
 * The whole batch takes two kernel launches on `stream` whatever the number of sequences: one operand preparation
 * over all sequences (each quantised on its own: V blocks of 32 keys are aligned to the sequence's own key index)
 * and one fused forward whose work items come from a table in the workspace.  A sequence with so few query tokens
 * that the query heads of a KV group fit into one 128-row tile (Hq / Hkv * len_q <= 128: decode steps, short
 * chunks) is run with those heads sharing a tile, so its K/V tiles are read once per KV head.  The same packing is
 * applied by efq_attention_fwd to a [B, H, S, d] batch with few query tokens; rows never interact, so results do
 * not depend on it.
 * The workspace holds the MXFP4 copies of all sequences side by side plus the tables:
 * efq_attention_varlen_workspace_bytes() gives the size for the given prefix sums (0 for invalid arguments).  The
 * two prefix arrays are read during the call only.
 * Asynchronous; efq_poll_status(workspace, stream) reports a device-side problem of any sequence.
 * Errors: INVALID_ARG (null pointer, n_seqs < 0, prefix sums not starting at 0 or decreasing, bad params),
 * UNSUPPORTED (d != 128, a batch too long for the 32-bit tile coordinates), ALIGNMENT, WORKSPACE, ARCH, CUDA. */
size_t efq_attention_varlen_workspace_bytes(const int64_t* cu_seqlens_q, const int64_t* cu_seqlens_k, int n_seqs, int Hq,
                                            int Hkv, int d);
efq_status_t efq_attention_fwd_varlen(const void* q, const void* k, const void* v, float* o, const int64_t* cu_seqlens_q,
                                      const int64_t* cu_seqlens_k, int n_seqs, int Hq, int Hkv, int d, int causal,
                                      float softmax_scale, int producer, const efq_params_t* params, void* workspace,
                                      size_t workspace_bytes, void* stream);

/* End-to-end form with HOST inputs and output: copies q/k/v from (preferably pinned) host
 * memory into caller-owned device staging buffers, runs the forward selected by `producer`
 * (0 = EFQ, 1 = exp-then-quantize scale4, 2 = exp-then-quantize scale6), copies o back, all on
 * `stream`.  q_dev/k_dev/v_dev/o_dev are device buffers of the same sizes as the host ones. */
efq_status_t efq_attention_fwd_host(const void* q_host, const void* k_host, const void* v_host, float* o_host,
                                    void* q_dev, void* k_dev, void* v_dev, float* o_dev, int B, int Hq, int Hkv,
                                    int64_t Sq, int64_t Sk, int d, int causal, float softmax_scale, int producer,
                                    const efq_params_t* params, void* workspace, size_t workspace_bytes,
                                    void* stream);

/* efq_attention_fwd_host with the copies overlapped: the problem is cut into `n_chunks` runs of KV heads (with
 * their query heads; a run never crosses a batch entry, so at most B * Hkv chunks are used), and chunk i+1's
 * inputs travel on `stream_in` while chunk i is computed on `stream_compute` and chunk i-1's output travels on
 * `stream_out` (three distinct streams; the host buffers should be pinned).  Same arithmetic and results as
 * efq_attention_fwd_host: heads are independent.  All chunks share one workspace slot (they are computed in
 * order): `workspace_bytes` must cover the workspace of one chunk plus 256 bytes, which the size for the whole
 * problem does whenever two or more chunks are used (with a single chunk the call is efq_attention_fwd_host on
 * `stream_compute`).  The call is asynchronous; when the work queued on
 * `stream_compute` has completed, so have the last copies, and efq_poll_status(workspace, stream_compute) reports
 * a device-side timeout of any chunk.  Calls may follow one another with the same staging buffers and workspace:
 * at entry `stream_in` is made to wait for the work `stream_compute` already holds, so the input copies of a call
 * never overtake the forwards of the call before it.  (The host output buffer of the earlier call is complete once
 * `stream_compute` has been synchronised.)  Errors as efq_attention_fwd_host, plus INVALID_ARG for n_chunks <= 0. */
efq_status_t efq_attention_fwd_host_pipelined(const void* q_host, const void* k_host, const void* v_host, float* o_host,
                                              void* q_dev, void* k_dev, void* v_dev, float* o_dev, int B, int Hq,
                                              int Hkv, int64_t Sq, int64_t Sk, int d, int causal, float softmax_scale,
                                              int producer, const efq_params_t* params, void* workspace,
                                              size_t workspace_bytes, int n_chunks, void* stream_in,
                                              void* stream_compute, void* stream_out);

/* Built-in scratch of efq_attention_fwd_static, in bytes (4 MiB).  Enough for, e.g., one head of 8192 tokens or
 * 8 query / 2 KV heads of 2048 tokens; efq_attention_workspace_bytes() gives the need of a shape. */
#define EFQ_STATIC_SCRATCH_BYTES (4u << 20)

/* efq_attention_fwd for callers that have no device memory to hand over as workspace.  (The paper has no
 * counterpart: this is a packaging variant of efq_attention_fwd, same arithmetic, same results.)
 *
 * Who needs it: code that runs where device allocation is off the table - a serving loop that must not call
 * cudaMalloc after start-up because the call synchronises the device and can fail once the memory pool is
 * fully handed out, or a plug-in living inside a host application that owns all device memory and gives
 * none of it to the plug-in.  Such a caller still owns q, k, v and o, but cannot produce the MXFP4 workspace.
 *
 * What it does instead: the MXFP4 copies of Q, K, V, their scale tiles and the status word go into a fixed
 * array of EFQ_STATIC_SCRATCH_BYTES that is part of the library image (so every device that loads the
 * library holds these bytes until the process exits).  The call allocates and frees nothing.
 *   - Shapes whose workspace would exceed the array are refused with EFQ_ERR_STATIC_LIMIT; nothing is
 *     launched.  Other argument rules and error codes are those of efq_attention_fwd (no debug dump).
 *   - The first call on each device looks up the array's device address (a host-side step, done with that
 *     device current, protected by a lock).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the previous call left; each call
 *     rewrites every byte it later reads and clears the status word first.  Two calls whose GPU work
 *     overlaps (different streams, or one stream from several threads without ordering) race on the array:
 *     serialise them.  The status word sits in the same array and this entry point has no poll call: a
 *     caller that must detect a device-side timeout uses efq_attention_fwd with a workspace of its own
 *     and efq_poll_status. */
efq_status_t efq_attention_fwd_static(const void* q, const void* k, const void* v, float* o, int B, int Hq, int Hkv,
                                      int64_t Sq, int64_t Sk, int d, int causal, float softmax_scale,
                                      const efq_params_t* params, void* stream);

/* Softmax attention in FP32 on the unquantised bf16 inputs (the problem statement of Sec. 3.1 with no low-bit
 * operand anywhere): O = softmax(scale Q K^T + mask) V, online over the keys, exponentials by expf.  This is the
 * reference output O_ref of the calibration objective and the "exact" side of the error figures; a plain
 * CUDA-core kernel, not a fast path.  Arguments as for efq_attention_fwd (no workspace); B * Hq <= 65535. */
efq_status_t efq_exact_attention_fwd(const void* q, const void* k, const void* v, float* o, int B, int Hq, int Hkv,
                                     int64_t Sq, int64_t Sk, int d, int causal, float softmax_scale, void* stream);

/* The calibration objective rho = ||a - ref||_F / ||ref||_F (Sec. "Parameter Calibration"), as its two sums:
 * on return of the stream work, sums[0] = sum (a - ref)^2 and sums[1] = sum ref^2 over n elements, both
 * accumulated in double.  a, ref fp32 device; sums double[2] device (overwritten).  Asynchronous. */
efq_status_t efq_relative_error(const float* a, const float* ref, int64_t n, double* sums, void* stream);

/* Offline selection of (tau, h) by grid search (Algorithm 3): the operands are quantised once, then for every
 * tau in taus (outer loop) and h in hs (inner loop) the fused EFQ forward runs on the calibration inputs and
 * rho(tau, h) = ||O~(tau, h) - O_ref||_F / ||O_ref||_F is formed; the pair with the smallest rho wins, the first
 * one in scan order on a tie.  The selected pair is meant to stay fixed at inference.
 *   q, k, v, shape, causal, softmax_scale, workspace   as for efq_attention_fwd
 *   o_ref    fp32 [B, Hq, Sq, d] device: the reference output (e.g. from efq_exact_attention_fwd)
 *   o_tmp    fp32 [B, Hq, Sq, d] device scratch for the candidate outputs
 *   taus, hs HOST arrays of n_tau and n_h candidates (every h > 0)
 *   sums     double [2 * n_tau * n_h] device scratch
 *   rho      HOST double [n_tau * n_h], row-major over (tau, h): the objective of every candidate
 *   best_tau, best_h  HOST outputs (may be NULL)
 * Synchronises `stream` before returning.  Errors: those of efq_attention_fwd, INVALID_ARG for empty candidate
 * sets or null pointers, DEVICE_TIMEOUT if a bounded device-side wait expired in any forward. */
efq_status_t efq_calibrate(const void* q, const void* k, const void* v, const float* o_ref, float* o_tmp, int B,
                           int Hq, int Hkv, int64_t Sq, int64_t Sk, int d, int causal, float softmax_scale,
                           const float* taus, int n_tau, const float* hs, int n_h, double* sums, double* rho,
                           float* best_tau, float* best_h, void* workspace, size_t workspace_bytes, void* stream);

/* Synchronises `stream` and returns the device-side status word of the last forward that
 * used `workspace` (EFQ_OK, or EFQ_ERR_DEVICE_TIMEOUT if a bounded wait expired), or
 * EFQ_ERR_CUDA if the stream reports an error. */
efq_status_t efq_poll_status(void* workspace, void* stream);

/* Dense FP4 tensor-pipe microbenchmark: `iters` back-to-back 128x256x64 block-scaled E2M1 MMAs per CTA on
 * operands resident in shared memory (launch one CTA per SM).  Writes one word per CTA to `sink`
 * (u32 [num_ctas], device; 0xdeadbeef marks a CTA whose bounded wait expired) and the FLOPs of the launch to
 * *flops (host).  The caller times the launch; FLOPs / time is the MMA-only FP4 rate that the fused forward's
 * tensor-pipe fraction can be quoted against. */
efq_status_t efq_fp4_mma_peak_probe(uint32_t* sink, int num_ctas, int iters, double* flops, void* stream);

/* In-SM microbenchmark of the probability producers (Algorithm 1 versus exp-then-quantize) on register-resident
 * scores: 256 threads per CTA, each coding one 32-key block per iteration, no memory traffic.
 *   producer 0 = EFQ (params or EFQ-Mean), 1 = exp-then-quantize scale4, 2 = scale6, 3 = EFQ-LUT, 4 = scale4 folded, 5 = scale4 folded + polynomial
 *   sink    u32 [num_ctas * 256], device (keeps the work alive)
 *   cycles  i64 [num_ctas], device: clock cycles CTA c spent on its `iters` iterations
 * Elements per clock per SM = resident CTAs per SM * 256 * 32 * iters / cycles. */
efq_status_t efq_stage_microbench(int producer, const efq_params_t* params, int num_ctas, int iters, uint32_t* sink,
                                  long long* cycles, void* stream);

/* Test hook for the bounded-wait path (no GPU fault is involved): efq_attention_fwd with the K/V loads left
 * out, so that the first device-side wait on them runs out after its limit (under a second).  Every role then
 * drains, tensor memory is released, the kernel returns normally and the status word reads
 * EFQ_ERR_DEVICE_TIMEOUT through efq_poll_status(); `o` is undefined.  The context stays usable and the next
 * efq_attention_fwd on the same workspace clears the status. */
efq_status_t efq_attention_fwd_inject_timeout(const void* q, const void* k, const void* v, float* o, int B, int Hq,
                                              int Hkv, int64_t Sq, int64_t Sk, int d, void* workspace,
                                              size_t workspace_bytes, void* stream);

const char* efq_status_string(efq_status_t status);

/* Library build tag: "efq-b200 sm_100a <revision of the fused forward kernel>", e.g. "efq-b200 sm_100a fwd.3".
 * Measurement records that were taken from a profiler capture name the revision they saw. */
const char* efq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* EFQ_H_ */
