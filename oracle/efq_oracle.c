/*
 * CPU oracle for the EFQ-Softmax probability-generation path and the attention forward
 * around it.  TEST INFRASTRUCTURE ONLY: plain, slow, written from the paper's definitions;
 * it shares no code with the CUDA path and is never called by the product library.
 *
 * Three paths (paper Sec. 3.1, "Targeted probability path"):
 *   exact   O = softmax(Q K^T / sqrt(d)) V in double on the unquantised inputs;
 *   EFQ     Algorithm 2 (online update per key/value block) with Algorithm 1 (code
 *           generation for one microscaling block) as the probability producer;
 *   ETQ     the same online loop with the exp-then-quantize producer of the
 *           "conventional construction" x -> exp(x) -> P_FP32 -> Quant_E2M1(P).
 *
 * Readings of the paper that this file fixes (the paper gives real-number formulas only):
 *   - microscaling block = 32 consecutive keys, aligned to absolute key index;
 *   - log is the natural logarithm in the scale rule k_b = floor((M_b + log(2/9))/log 2);
 *   - the integer decisions (scale exponent, code) are taken in FP32 with one fixed
 *     operation order, stated at efq_block(); a double-precision evaluation of the same
 *     equations lives in oracle/efq_math.py and must agree except at knife-edges;
 *   - the shifted score uses the running row maximum m_i^j that already includes the
 *     current key/value block (Algorithm 2, steps 2-3), so codes depend on the KV tile
 *     width Bc, which is a parameter here;
 *   - Q, K (blocks of 32 along d) and V (blocks of 32 along keys, per channel) are
 *     quantised to MXFP4 by the OCP rule: shared exponent floor(log2 amax) - 2,
 *     round-to-nearest-even onto E2M1, saturating;
 *   - raw scores are the exact sum of the dequantised products, rounded once to FP32;
 *   - the exp-then-quantize baseline takes its denominator from the same quantised
 *     operand as its numerator (everything but the producer held equal).
 *
 * Pins: tests/test_oracle_*.py (code set, scale interval, threshold form of the affine
 * rule, closed-form special cases, library softmax attention).  The accuracy level of
 * EFQ versus exact attention is "parity unpinned": the paper prints no error figure.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define MXB 32 /* microscaling block size */

/* Nonnegative E2M1 code set C8 (paper Sec. 3.2): value of bit pattern c = 0..7. */
static const double C8[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

int efq_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

double efq_oracle_c8(int c) { return C8[c & 7]; }

/* ---------------------------------------------------------------------------------- */
/* MXFP4 operand quantiser (the "existing low-bit path" the paper leaves to the         */
/* surrounding kernel; OCP microscaling rule).                                         */
/* ---------------------------------------------------------------------------------- */

/* Nearest value of C8 to y >= 0, ties to the code with an even bit pattern, saturating. */
static int e2m1_nearest_even(double y)
{
    int best = 0;
    double bestd = fabs(y - C8[0]);
    for (int c = 1; c < 8; ++c) {
        double dd = fabs(y - C8[c]);
        if (dd < bestd || (dd == bestd && (c & 1) == 0)) {
            best = c;
            bestd = dd;
        }
    }
    return best;
}

/* floor(log2(a)) for finite a > 0 */
static int floor_log2(double a)
{
    int ex;
    (void)frexp(a, &ex); /* a = f * 2^ex, f in [0.5, 1) */
    return ex - 1;
}

/* One block of n <= 32 values with the given element stride.
 * Writes n 4-bit codes (bit 3 = sign) and the E8M0 byte (exponent + 127). */
void efq_oracle_mxfp4_block(const float* v, int n, int64_t stride, uint8_t* code, uint8_t* scale_byte)
{
    double amax = 0.0;
    for (int i = 0; i < n; ++i) {
        double a = fabs((double)v[i * stride]);
        if (a > amax) amax = a;
    }
    if (amax == 0.0) {
        *scale_byte = 0;
        for (int i = 0; i < n; ++i) code[i] = 0;
        return;
    }
    int e = floor_log2(amax) - 2;
    if (e < -127) e = -127;
    if (e > 127) e = 127;
    *scale_byte = (uint8_t)(e + 127);
    for (int i = 0; i < n; ++i) {
        double x = (double)v[i * stride];
        int c = e2m1_nearest_even(ldexp(fabs(x), -e));
        code[i] = (uint8_t)(c | (signbit(x) ? 8 : 0));
    }
}

static double mxfp4_value(uint8_t code, uint8_t scale_byte)
{
    double m = C8[code & 7];
    return ldexp((code & 8) ? -m : m, (int)scale_byte - 127);
}

/* Quantise-dequantise a [n_rows, d] matrix with blocks of 32 along d (Q and K). */
void efq_oracle_mxfp4_rows(const float* x, int64_t n_rows, int d, float* xhat,
                           uint8_t* codes /* [n_rows, d] one code per byte, or NULL */,
                           uint8_t* scales /* [n_rows, d/32], or NULL */)
{
    int nb = (d + MXB - 1) / MXB;
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < n_rows; ++r) {
        uint8_t c[MXB], sb;
        for (int b = 0; b < nb; ++b) {
            int n = d - b * MXB < MXB ? d - b * MXB : MXB;
            efq_oracle_mxfp4_block(x + r * d + b * MXB, n, 1, c, &sb);
            for (int i = 0; i < n; ++i) {
                xhat[r * d + b * MXB + i] = (float)mxfp4_value(c[i], sb);
                if (codes) codes[r * d + b * MXB + i] = c[i];
            }
            if (scales) scales[r * nb + b] = sb;
        }
    }
}

/* Quantise-dequantise V [S, d] with blocks of 32 along the key index, per channel. */
void efq_oracle_mxfp4_cols(const float* x, int64_t S, int d, float* xhat,
                           uint8_t* codes /* [S, d] or NULL */,
                           uint8_t* scales /* [ceil(S/32), d] or NULL */)
{
    int64_t nb = (S + MXB - 1) / MXB;
#pragma omp parallel for schedule(static)
    for (int64_t b = 0; b < nb; ++b) {
        uint8_t c[MXB], sb;
        int n = S - b * MXB < MXB ? (int)(S - b * MXB) : MXB;
        for (int ch = 0; ch < d; ++ch) {
            efq_oracle_mxfp4_block(x + b * MXB * d + ch, n, d, c, &sb);
            for (int i = 0; i < n; ++i) {
                xhat[(b * MXB + i) * d + ch] = (float)mxfp4_value(c[i], sb);
                if (codes) codes[(b * MXB + i) * d + ch] = c[i];
            }
            if (scales) scales[b * d + ch] = sb;
        }
    }
}

/* ---------------------------------------------------------------------------------- */
/* Probability producers for one microscaling block                                    */
/* ---------------------------------------------------------------------------------- */

typedef struct {
    float A;      /* fl32(sigma * h)                 */
    float HL2;    /* fl32(h * ln 2)                  */
    float C1;     /* fl32(1 - h * (ln 6 + tau))      */
    float h;      /* h as given                      */
    float sigma;  /* score scale as given            */
    float LOG2E;  /* fl32(1 / ln 2)                  */
    float L2_29;  /* fl32(log2(2/9))                 */
    int top;      /* largest index of the affine rule: 7 (Eq. d8-index) or 15 (16-level index of the LUT variant) */
    int fold;     /* 1: the index goes through the 16 -> 8 folding table */
} efq_consts;

/* Folding table of the LUT variant (Sec. "EFQ-Softmax-LUT Variant"): 16-level index -> E2M1 code. */
static const uint8_t C16[16] = {0, 1, 1, 1, 1, 1, 2, 2, 3, 3, 4, 5, 5, 6, 7, 7};

static efq_consts make_consts(float sigma, float tau, float h)
{
    efq_consts k;
    k.A = (float)((double)sigma * (double)h);
    k.HL2 = (float)((double)h * log(2.0));
    k.C1 = (float)(1.0 - (double)h * (log(6.0) + (double)tau));
    k.h = h;
    k.sigma = sigma;
    k.LOG2E = (float)(1.0 / log(2.0));
    k.L2_29 = (float)(log(2.0 / 9.0) / log(2.0));
    k.top = 7;
    k.fold = 0;
    return k;
}

/* LUT variant: the same scale rule, the index rule with the fixed pair tau16 = ln(1/24), h16 = 14 / ln 24 and
 * sixteen levels, then the folding table.  tau16 and h16 enter in double; the FP32 constants are rounded once. */
static efq_consts make_consts_lut(float sigma)
{
    const double h16 = 14.0 / log(24.0), tau16 = log(1.0 / 24.0);
    efq_consts k;
    k.A = (float)((double)sigma * h16);
    k.HL2 = (float)(h16 * log(2.0));
    k.C1 = (float)(1.0 - h16 * (log(6.0) + tau16));
    k.h = (float)h16;
    k.sigma = sigma;
    k.LOG2E = (float)(1.0 / log(2.0));
    k.L2_29 = (float)(log(2.0 / 9.0) / log(2.0));
    k.top = 15;
    k.fold = 1;
    return k;
}

/* producer ids: 0 = EFQ, 1 = exp-then-quantize scale4, 2 = exp-then-quantize scale6, 3 = EFQ-LUT,
 * 4 = exp-then-quantize scale4 whose DENOMINATOR is summed from the FP32 exponentials instead of the quantised
 * operand (the convention of attention kernels that quantise P only for the P V product; reported as context,
 * the paper's shared-operand rule is producers 0-3). */
static efq_consts consts_for(int producer, float sigma, float tau, float h)
{
    return producer == 3 ? make_consts_lut(sigma) : make_consts(sigma, tau, h);
}
static int is_efq(int producer) { return producer == 0 || producer == 3; }

/* Algorithm 1 for one block of n <= 32 raw scores r_t (before the score scale sigma),
 * with m_s = the row maximum in scaled units (fl32(sigma * max r) inside attention, the
 * caller's row_max in the standalone stage).  Masked positions carry r = -inf.
 *
 * FP32 order, fixed here and mirrored by the kernels:
 *   M_b  = fl32(fl32(sigma * rmax_b) - m_s)                          step 1
 *   k_b  = clamp(floor(fma(M_b, 1/ln2, log2(2/9))), -127, 127)       step 2 (Eq. k-rule)
 *   B_b  = fma(-h, m_s, fma(-h ln2, (float)k_b, 1 - h (ln6 + tau)))
 *   v_t  = fma(r_t, sigma h, B_b)   == (z_t - tau) h + 1 with z_t of Eq. z-def   step 5
 *   c_t  = floor(min(max(v_t, 0), 7))                                step 6 (Eq. d8-index;
 *          the +1 sits inside the floor, clip and floor commute on [0,7])
 * LUT variant: the same sequence with (tau16, h16), j_t = floor(min(max(v_t, 0), 15)), c_t = C16[j_t].
 * A block whose maximum is -inf (fully masked) gets byte 0 and all-zero codes.
 * Returns the E8M0 byte k_b + 127 and writes n codes (0..7, one per byte). */
static uint8_t efq_block(const float* r, int n, float m_s, const efq_consts* K, uint8_t* code)
{
    float rmax = -INFINITY;
    for (int t = 0; t < n; ++t)
        if (r[t] > rmax) rmax = r[t];
    if (rmax == -INFINITY) {
        for (int t = 0; t < n; ++t) code[t] = 0;
        return 0;
    }
    float sr = K->sigma * rmax;
    float Mb = sr - m_s;
    float kf = floorf(fmaf(Mb, K->LOG2E, K->L2_29));
    if (kf < -127.0f) kf = -127.0f;
    if (kf > 127.0f) kf = 127.0f;
    float Bb = fmaf(-K->h, m_s, fmaf(-K->HL2, kf, K->C1));
    for (int t = 0; t < n; ++t) {
        float v = fmaf(r[t], K->A, Bb);
        if (!(v > 0.0f)) v = 0.0f; /* also catches -inf */
        if (v > (float)K->top) v = (float)K->top;
        int idx = (int)floorf(v);
        code[t] = K->fold ? C16[idx] : (uint8_t)idx;
    }
    return (uint8_t)((int)kf + 127);
}

/* exp-then-quantize producer for one block:
 *   p_t = exp(fl32(fl32(sigma r_t) - m_s)) rounded to FP32, e_b = floor(log2 max p) - 2
 *   (scale_mode 0, "scale4": block maximum lands in [4, 8)) or ceil(log2(max p / 6))
 *   (scale_mode 1, "scale6": block maximum lands in (3, 6], no saturation),
 *   q_t = nearest-even E2M1 of p_t 2^-e_b, saturating. */
static uint8_t etq_block(const float* r, int n, float m_s, float sigma, int scale_mode, uint8_t* code)
{
    float p[MXB];
    float amax = 0.0f;
    for (int t = 0; t < n; ++t) {
        if (r[t] == -INFINITY) {
            p[t] = 0.0f;
        } else {
            float x = sigma * r[t];
            x = x - m_s;
            p[t] = (float)exp((double)x);
        }
        if (p[t] > amax) amax = p[t];
    }
    if (amax == 0.0f) {
        for (int t = 0; t < n; ++t) code[t] = 0;
        return 0;
    }
    int e;
    if (scale_mode == 0) {
        e = floor_log2((double)amax) - 2;
    } else {
        e = (int)ceil(log2((double)amax / 6.0));
    }
    if (e < -127) e = -127;
    if (e > 127) e = 127;
    for (int t = 0; t < n; ++t) code[t] = (uint8_t)e2m1_nearest_even(ldexp((double)p[t], -e));
    return (uint8_t)(e + 127);
}

static void pack_codes(const uint8_t* code, int n, uint8_t* packed /* 16 bytes */)
{
    memset(packed, 0, MXB / 2);
    for (int t = 0; t < n; ++t) packed[t >> 1] |= (uint8_t)((code[t] & 0xF) << ((t & 1) * 4));
}

/* ---------------------------------------------------------------------------------- */
/* Standalone stage: (x, B, tau, h) -> (Q_P, s_P)  (paper Sec. 4.3, kernel interface)   */
/* ---------------------------------------------------------------------------------- */

/* producer: 0 = EFQ, 1 = exp-then-quantize scale4, 2 = exp-then-quantize scale6, 3 = EFQ-LUT (tau, h unused).
 * scores [rows, ld] fp32 raw; row_max [rows] in scaled units; codes [rows, nblk*16]
 * packed low nibble first; scales [rows, nblk]; nblk = ceil(cols/32). */
void efq_oracle_probgen(const float* scores, int64_t ld, const float* row_max, int64_t rows, int64_t cols,
                        float sigma, float tau, float h, int producer, uint8_t* codes, uint8_t* scales)
{
    int64_t nblk = (cols + MXB - 1) / MXB;
    efq_consts K = consts_for(producer, sigma, tau, h);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < rows; ++i) {
        uint8_t c[MXB];
        for (int64_t b = 0; b < nblk; ++b) {
            int n = cols - b * MXB < MXB ? (int)(cols - b * MXB) : MXB;
            const float* r = scores + i * ld + b * MXB;
            uint8_t sb = is_efq(producer) ? efq_block(r, n, row_max[i], &K, c)
                                       : etq_block(r, n, row_max[i], sigma, producer - 1, c);
            scales[i * nblk + b] = sb;
            pack_codes(c, n, codes + (i * nblk + b) * (MXB / 2));
        }
    }
}

/* ---------------------------------------------------------------------------------- */
/* Online update over the key/value blocks of one query row (Algorithm 2)              */
/* ---------------------------------------------------------------------------------- */

/* r [n_keys] raw scores of one row (masked = -inf); vhat [n_keys, d] dequantised values.
 * Walks KV tiles of width Bc in ascending order with the running maximum, producing the
 * probability operand per 32-key block and accumulating numerator and denominator from
 * that same operand.  Optional dumps: codes [nblk*16], scales [nblk], m_s per tile. */
/* rescale_threshold T (scaled units, not in the paper; T = 0 is Algorithm 2 as printed): the maximum that shifts
 * the scores is kept from tile to tile while the true running maximum exceeds it by at most T, and replaced by
 * the true running maximum otherwise:
 *     cand = max(m, tile maximum);   m <- cand  if m = -inf or T <= 0 or fl(fl(sigma cand) - fl(sigma m)) > T,
 *                                    m unchanged otherwise.
 * Shifted scores may then be positive (up to T); the scale rule is shift-equivariant, so only the block exponents
 * move, and alpha = 1 for every tile that keeps m. */
static void online_row(const float* r, int64_t n_keys, const float* vhat, int d, int64_t Bc,
                       const efq_consts* K, int producer, float rescale_threshold, double* out /* [d] */,
                       uint8_t* codes_out, uint8_t* scales_out, float* ms_out)
{
    double* A = (double*)calloc((size_t)d, sizeof(double));
    double l = 0.0;
    float m_raw = -INFINITY;
    float m_s_old = -INFINITY;
    int64_t ntile = (n_keys + Bc - 1) / Bc;
    uint8_t c[MXB];
    for (int64_t j = 0; j < ntile; ++j) {
        int64_t t0 = j * Bc;
        int64_t t1 = t0 + Bc < n_keys ? t0 + Bc : n_keys;
        float cand = m_raw;
        for (int64_t t = t0; t < t1; ++t)
            if (r[t] > cand) cand = r[t]; /* Eq. rowmax-update */
        if (m_raw == -INFINITY || !(rescale_threshold > 0.0f)) {
            m_raw = cand;
        } else {
            float sc = K->sigma * cand;
            float su = K->sigma * m_raw;
            float diff = sc - su;
            if (diff > rescale_threshold) m_raw = cand;
        }
        float m_s = K->sigma * m_raw;
        if (ms_out) ms_out[j] = m_s;
        if (m_raw == -INFINITY) { /* nothing visible yet: operand is all zero */
            for (int64_t t = t0; t < t1; t += MXB) {
                if (scales_out) scales_out[t / MXB] = 0;
                if (codes_out) memset(codes_out + (t / MXB) * (MXB / 2), 0, MXB / 2);
            }
            continue;
        }
        double alpha = (m_s_old == -INFINITY) ? 0.0 : exp((double)m_s_old - (double)m_s); /* Eq. alpha */
        for (int ch = 0; ch < d; ++ch) A[ch] *= alpha;
        l *= alpha;
        for (int64_t t = t0; t < t1; t += MXB) {
            int n = t1 - t < MXB ? (int)(t1 - t) : MXB;
            uint8_t sb = is_efq(producer) ? efq_block(r + t, n, m_s, K, c)
                                       : etq_block(r + t, n, m_s, K->sigma, producer == 4 ? 0 : producer - 1, c);
            if (scales_out) scales_out[t / MXB] = sb;
            if (codes_out) pack_codes(c, n, codes_out + (t / MXB) * (MXB / 2));
            double s = ldexp(1.0, (int)sb - 127);
            for (int u = 0; u < n; ++u) {
                double p = s * C8[c[u]]; /* p~_t = s_b * C8[c_t] */
                if (producer == 4 && r[t + u] != -INFINITY) {   /* context variant: FP32 exponential in the denominator */
                    float x = K->sigma * r[t + u];
                    x = x - m_s;
                    l += (double)(float)exp((double)x);
                    if (p == 0.0) continue;
                } else {
                    if (p == 0.0) continue;
                    l += p;                                     /* Eq. denominator-basic */
                }
                const float* vr = vhat + (t + u) * d;
                for (int ch = 0; ch < d; ++ch) A[ch] += p * (double)vr[ch]; /* Eq. numerator-basic */
            }
        }
        m_s_old = m_s;
    }
    for (int ch = 0; ch < d; ++ch) out[ch] = l > 0.0 ? A[ch] / l : 0.0;
    free(A);
}

/* Standalone form of the online walk on caller-supplied raw scores (used to check a
 * kernel's codes bit-for-bit on the kernel's own FP32 scores).
 * scores [rows, ld]; codes [rows, nblk*16]; scales [rows, nblk]; ms [rows, ntile]. */
void efq_oracle_online_codes(const float* scores, int64_t ld, int64_t rows, int64_t n_keys, int64_t Bc,
                             float sigma, float tau, float h, int producer, float rescale_threshold,
                             uint8_t* codes, uint8_t* scales, float* ms)
{
    int64_t nblk = (n_keys + MXB - 1) / MXB;
    int64_t ntile = (n_keys + Bc - 1) / Bc;
    efq_consts K = consts_for(producer, sigma, tau, h);
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t i = 0; i < rows; ++i) {
        double dummy[1];
        float zero = 0.0f;
        /* d = 0: no value accumulation */
        online_row(scores + i * ld, n_keys, &zero, 0, Bc, &K, producer, rescale_threshold, dummy,
                   codes + i * nblk * (MXB / 2), scales + i * nblk, ms ? ms + i * ntile : NULL);
    }
}

/* ---------------------------------------------------------------------------------- */
/* Attention forward on sampled query rows                                             */
/* ---------------------------------------------------------------------------------- */

static int64_t visible_keys(int64_t i, int64_t Sq, int64_t Sk, int causal)
{
    if (!causal) return Sk;
    int64_t n = i + Sk - Sq + 1; /* bottom-right aligned */
    if (n < 0) n = 0;
    if (n > Sk) n = Sk;
    return n;
}

/* q [B,Hq,Sq,d], k, v [B,Hkv,Sk,d] as fp32 (exact widenings of the bf16 inputs).
 * rows [n_rows, 3] = (b, head, query index).  path: 0 = exact (double, unquantised),
 * 1 = EFQ, 2 = ETQ scale4, 3 = ETQ scale6, 4 = EFQ-LUT, 5 = ETQ scale4 with FP32 denominator.  out [n_rows, d] fp32.
 * Optional dumps (NULL to skip), each row-major over the sampled rows:
 *   raw [n_rows, Sk] (-inf where masked), codes [n_rows, nblk*16], scales [n_rows, nblk],
 *   ms [n_rows, ntile]. */
void efq_oracle_attention_rows(const float* q, const float* k, const float* v,
                               int B, int Hq, int Hkv, int64_t Sq, int64_t Sk, int d, int causal,
                               float sigma, float tau, float h, int64_t Bc, int path, float rescale_threshold,
                               const int64_t* rows, int64_t n_rows, float* out,
                               float* raw, uint8_t* codes, uint8_t* scales, float* ms)
{
    (void)B;
    int group = Hq / Hkv;
    int64_t nblk = (Sk + MXB - 1) / MXB;
    int64_t ntile = (Sk + Bc - 1) / Bc;
    efq_consts K = consts_for(path - 1, sigma, tau, h);

    /* which (b, kv head) pairs are needed */
    int n_kv = B * Hkv;
    char* need = (char*)calloc((size_t)n_kv, 1);
    for (int64_t n = 0; n < n_rows; ++n) need[rows[3 * n] * Hkv + rows[3 * n + 1] / group] = 1;

    for (int kv = 0; kv < n_kv; ++kv) {
        if (!need[kv]) continue;
        const float* kh = k + (int64_t)kv * Sk * d;
        const float* vh = v + (int64_t)kv * Sk * d;
        float* khat = NULL;
        float* vhat = NULL;
        if (path != 0) {
            khat = (float*)malloc(sizeof(float) * (size_t)(Sk * d));
            vhat = (float*)malloc(sizeof(float) * (size_t)(Sk * d));
            efq_oracle_mxfp4_rows(kh, Sk, d, khat, NULL, NULL);
            efq_oracle_mxfp4_cols(vh, Sk, d, vhat, NULL, NULL);
        }
#pragma omp parallel for schedule(dynamic, 1)
        for (int64_t n = 0; n < n_rows; ++n) {
            int64_t b = rows[3 * n], hq = rows[3 * n + 1], i = rows[3 * n + 2];
            if (b * Hkv + hq / group != kv) continue;
            const float* qrow = q + ((b * Hq + hq) * Sq + i) * d;
            int64_t nvis = visible_keys(i, Sq, Sk, causal);
            float* o = out + n * d;
            if (path == 0) {
                /* exact: stable softmax in double */
                double* s = (double*)malloc(sizeof(double) * (size_t)(nvis > 0 ? nvis : 1));
                double mx = -INFINITY;
                for (int64_t t = 0; t < nvis; ++t) {
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += (double)qrow[c] * (double)kh[t * d + c];
                    s[t] = acc * (double)sigma;
                    if (s[t] > mx) mx = s[t];
                }
                double* acc = (double*)calloc((size_t)d, sizeof(double));
                double l = 0.0;
                for (int64_t t = 0; t < nvis; ++t) {
                    double p = exp(s[t] - mx);
                    l += p;
                    for (int c = 0; c < d; ++c) acc[c] += p * (double)vh[t * d + c];
                }
                for (int c = 0; c < d; ++c) o[c] = l > 0.0 ? (float)(acc[c] / l) : 0.0f;
                free(acc);
                free(s);
                continue;
            }
            float qhat[1024];
            efq_oracle_mxfp4_rows(qrow, 1, d, qhat, NULL, NULL);
            float* r = (float*)malloc(sizeof(float) * (size_t)Sk);
            for (int64_t t = 0; t < Sk; ++t) {
                if (t >= nvis) {
                    r[t] = -INFINITY;
                    continue;
                }
                double acc = 0.0;
                for (int c = 0; c < d; ++c) acc += (double)qhat[c] * (double)khat[t * d + c];
                r[t] = (float)acc;
            }
            double* od = (double*)malloc(sizeof(double) * (size_t)d);
            online_row(r, Sk, vhat, d, Bc, &K, path - 1, rescale_threshold, od,
                       codes ? codes + n * nblk * (MXB / 2) : NULL,
                       scales ? scales + n * nblk : NULL, ms ? ms + n * ntile : NULL);
            for (int c = 0; c < d; ++c) o[c] = (float)od[c];
            if (raw) memcpy(raw + n * Sk, r, sizeof(float) * (size_t)Sk);
            free(od);
            free(r);
        }
        free(khat);
        free(vhat);
    }
    free(need);
}
