// Fused block-scaled FP4 attention forward with in-register probability generation
// (Algorithm 2 looped over KV tiles, Algorithm 1 per 32-key microscaling block), sm_100a.
//
// One CTA owns one 128-row query tile of one (batch, head) and walks the KV tiles of width 128:
//   warp 0      TMA producer: Q tile once, then K_j / V^T_j code tiles (SW64 layout) and their
//               512-byte scale tiles through 4-stage mbarrier rings
//   warps 1, 2  MMA issuers (one elected lane each): scale tiles smem -> TMEM (tcgen05.cp), then warp 1
//               S_j = Q^ K^_j^T  and warp 2  [dA | dl] = P~_j [V^_j | 1]  as kind::mxf4 block-scaled MMAs,
//               FP32 accumulators in TMEM; S runs up to two tiles ahead of P~V.  The 16 "ones" rows appended to V^T give the denominator
//               P~1 from the very operand that feeds the numerator.
//   warps 12-15 historical rescaling: when a row's maximum grew in tile j, its accumulator row and denominator in
//               TMEM are multiplied by alpha_j after P~V_{j-1} and before P~V_j, beside the code generation.
//   warps 4-11  probability generation, two groups of four warps: group 0 takes the even KV tiles,
//               group 1 the odd ones, so one group's latency-bound steps (TMEM load, hand-over of the
//               running maximum, accumulator rescaling) overlap the other group's code generation.
//               Thread = query row: the 128 scores of the row come from TMEM straight into registers;
//               block maxima, scale and codes are thread-local; codes go as 16-byte packed stores into
//               the swizzled shared-memory A operand, the four scale bytes as one word into the scale
//               tile.  No FP16/FP32 probability tile exists anywhere.  Per tile a warp publishes once (running
//               maximum, alpha, hand-back of the S buffer), asks each barrier one step before it needs the
//               answer, and sends for the scores of its next tile as soon as its registers are free.
// The online recurrence is unchanged: when a row's maximum grows, the accumulator rows in TMEM
// are rescaled by alpha = exp(m_old - m_new) before the next P~V MMA is released (warps 12-15).
//
// TMEM columns: S double buffer 2 x 128 | O 144 (128 channels + 16 denominator) | scale factors.
// Every wait is bounded; on expiry the CTA records EFQ_ERR_DEVICE_TIMEOUT in the workspace status
// word, all roles drain, TMEM is released and the kernel returns.
#include <cuda.h>
#include <cuda_runtime.h>

#include <mutex>

#include <vector>

#include "efq_common.cuh"
#include "efq_internal.cuh"
#include "efq_producers.cuh"
#include "sm100_ptx.cuh"

namespace efq {

namespace {

constexpr int kTile = 128;            // query rows per CTA and keys per KV tile (Bc)
constexpr int kStages = 4;            // K and V ring depth
constexpr int kThreads = 512;         // 16 warps = 4 warpgroups: {TMA, QK, PV, idle}, 2 x probability generation, rescaling
constexpr int kGroupWarps = 4;        // warps per probability group (one thread per query row)
constexpr int kTileBytes = kTile * 64;          // 128 rows x 64 B of packed E2M1
constexpr int kSfBytes = 512;
constexpr int kVStageBytes = kTileBytes + 1024; // + 16 ones rows
constexpr uint64_t kTimeoutCycles = 1500000000ull;

// TMEM column map
constexpr uint32_t kColS = 0;         // 2 x 128
constexpr uint32_t kColO = 256;       // 144
constexpr uint32_t kColSfQ = 400;     // 4
constexpr uint32_t kColSfK = 404;     // 2 x 4
constexpr uint32_t kColSfP = 412;     // 2 x 4
constexpr uint32_t kColSfV = 420;     // 2 x 8 (4 for V, 4 for the ones rows)
constexpr uint32_t kTmemCols = 512;

struct __align__(1024) Smem {
    uint8_t q[kTileBytes];
    uint8_t k[kStages][kTileBytes];
    uint8_t v[kStages][kVStageBytes];
    uint8_t p[2][kTileBytes];
    uint8_t sf_q[kSfBytes];
    uint8_t sf_k[kStages][kSfBytes];
    uint8_t sf_v[kStages][kSfBytes];
    uint8_t sf_p[2][kSfBytes];
    uint8_t sf_ones[kSfBytes];
    float lsum_x[2][kTile];   // FP32-denominator baseline only: each group's sum of exponentials ...
    float mref_x[2][kTile];   // ... and the scaled maximum it refers to
    float runmax[2][kTile];   // running row maximum after the group's latest tile, raw score units
    float alpha[4][kTile];    // [tile mod 4]: rescale factor of the tile, per row (1 where the maximum did not grow)
    uint64_t q_full;
    uint64_t k_full[kStages], k_empty[kStages];
    uint64_t v_full[kStages], v_empty[kStages];
    uint64_t s_full[2], s_empty[2];
    uint64_t p_full[2], p_empty[2];
    uint64_t x_bar[2][4];     // [group][lane quarter]: runmax of the group's latest tile is published
    uint64_t a_bar[4][4];     // [tile mod 4][lane quarter]: alpha of that tile is published
    uint64_t o_ready[2];      // accumulator rows rescaled (or found unchanged) for the tile of this parity
    uint64_t o_done;          // the last P~V of the work item has completed
    uint64_t l_bar;           // FP32-denominator baseline only: all eight probability warps have written lsum_x / mref_x
    uint32_t tmem_base;
    volatile uint32_t abort_flag;
};

struct FwdParams {
    int B, Hq, Hkv;
    int64_t Sq, Sk, Sq_pad, Sk_pad;
    int causal;
    ProducerConsts K;
    const uint8_t* sf_q;      // [B*Hq*Sq_pad/128][512]
    const uint8_t* sf_k;      // [B*Hkv*Sk_pad/128][512]
    const uint8_t* sf_v;
    float* o;
    int64_t o_head, o_row;    // strides of o in elements: row i of (batch b, head h) starts at o[(b * Hq + h) * o_head + i * o_row]
    uint32_t* status;
    efq_debug_t dbg;
    int has_dbg;
    int packed;               // dense batch with few query tokens: the query heads of a KV group share one query tile
    const SeqDesc* seqs;      // packed variable-length batch: sequence table and one item per CTA (device memory);
    const ItemDesc* items;    //   NULL for a [B, H, S, d] batch, whose items follow from the block index
    int64_t v_tiles_per_head; // packed batch: 128-key tiles per KV head in the V^T code matrix (all sequences)
    int inject_skip_loads;    // test hook: the TMA thread loads Q only, so the first wait on K/V runs out
    float rescale_threshold;  // 0: Algorithm 2; > 0: the shifting maximum is kept while the true one is at most this far above
};

// Bounded wait of one thread.  Returns false on timeout (recorded in the status word) or CTA-wide abort.
// The polling loop is kept to the barrier test itself; the abort flag and the clock are looked at every 64th
// round only, because every instruction a waiting warp issues is taken from the warps that compute.
__device__ __forceinline__ bool wait1(uint64_t* bar, uint32_t parity, Smem* sm, uint32_t* status)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t spins = 1;; ++spins) {
        if (ptx::mbar_try_wait_suspend(bar, parity, 20000u)) return true;
        if ((spins & 63u) == 0u) {
            if (sm->abort_flag) return false;
            if (static_cast<uint64_t>(clock64() - t0) > kTimeoutCycles) {
                sm->abort_flag = 1;
                atomicExch(status, static_cast<uint32_t>(EFQ_ERR_DEVICE_TIMEOUT));
                return false;
            }
        }
    }
}
// The same wait executed by all lanes of a warp.  All lanes poll the same barrier; only the rare timeout path
// can split a warp, so the verdict is made warp-uniform there and nowhere else.
__device__ __forceinline__ bool wait_all(uint64_t* bar, uint32_t parity, Smem* sm, uint32_t* status)
{
    if (ptx::mbar_try_wait(bar, parity)) return true;
    const bool ok = wait1(bar, parity, sm, status);
    return __all_sync(__activemask(), ok);
}

__device__ __forceinline__ uint32_t p_swizzled_offset(uint32_t row, uint32_t chunk)
{
    return (row >> 3) * 512u + (row & 7u) * 64u + ((chunk ^ ((row >> 1) & 3u)) << 4);
}

template <int PRODUCER, bool DEBUG, bool FIX8>
__global__ void __launch_bounds__(kThreads, 1)
attention_fwd_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_k,
                     const __grid_constant__ CUtensorMap map_v, const FwdParams P)
{
    extern __shared__ uint8_t smem_raw[];
    Smem* sm = reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // ---- work item.  [B, H, S, d] batch: heaviest query tiles first, the heads of a GQA group adjacent.  Packed
    // variable-length batch: the item and its sequence come from the tables.  Either way the item is one 128-row
    // query tile: rows q0 .. q0 + 127 of query head head0, or - "packed", when the sequence has so few query tokens
    // that the G query heads of a KV group fit into one tile - row r = token r % Sq of query head head0 + r / Sq.
    const int G = P.Hq / P.Hkv;
    int64_t Sq, Sk, o_base, q0;
    int b, head0, hkv, q_row, k_row0, v_x0, v_y0;
    int64_t sfv_tile0;
    bool packed;
    if (P.items != nullptr) {
        const ItemDesc it = P.items[blockIdx.x];
        const SeqDesc sd = P.seqs[it.seq];
        Sq = sd.Sq; Sk = sd.Sk; o_base = sd.o_off; b = it.seq;
        packed = sd.packed != 0;
        if (packed) { hkv = it.head; head0 = hkv * G; q0 = 0; q_row = sd.q_row0 + hkv * kTile; }
        else { head0 = it.head; hkv = head0 / G; q0 = static_cast<int64_t>(it.qt) * kTile; q_row = sd.q_row0 + head0 * sd.Sq_pad + it.qt * kTile; }
        k_row0 = sd.k_row0 + hkv * sd.Sk_pad;
        v_x0 = sd.k_col0 / 2;
        v_y0 = hkv * kTile;
        sfv_tile0 = static_cast<int64_t>(hkv) * P.v_tiles_per_head + sd.k_col0 / kTile;
    } else {
        Sq = P.Sq; Sk = P.Sk;
        packed = P.packed != 0;
        const int64_t n_qtiles = packed ? 1 : P.Sq_pad / kTile;
        const int64_t heads = packed ? P.Hkv : P.Hq;          // heads that own query tiles
        const int64_t bh_count = static_cast<int64_t>(P.B) * heads;
        const int64_t item = blockIdx.x;
        const int64_t qt = n_qtiles - 1 - item / bh_count;
        const int64_t bh = item % bh_count;
        b = static_cast<int>(bh / heads);
        const int hh = static_cast<int>(bh % heads);
        if (packed) { hkv = hh; head0 = hkv * G; q0 = 0; q_row = static_cast<int>(bh * kTile); }
        else { head0 = hh; hkv = hh / G; q0 = qt * kTile; q_row = static_cast<int>(bh * P.Sq_pad + q0); }
        const int64_t kvh = static_cast<int64_t>(b) * P.Hkv + hkv;
        k_row0 = static_cast<int>(kvh * P.Sk_pad);
        v_x0 = 0;
        v_y0 = static_cast<int>(kvh * kTile);
        sfv_tile0 = kvh * (P.Sk_pad / kTile);
        o_base = static_cast<int64_t>(b) * P.Hq * P.o_head;
    }
    const int64_t shift = Sk - Sq;                         // causal: query i sees keys <= i + shift
    int64_t n_tiles = (Sk + kTile - 1) / kTile;
    if (P.causal) {
        int64_t last_row = packed ? Sq - 1 : (q0 + kTile - 1 < Sq ? q0 + kTile - 1 : Sq - 1);
        int64_t last_key = last_row + shift;               // may be negative: nothing visible
        int64_t need = last_key < 0 ? 0 : last_key / kTile + 1;
        if (need < n_tiles) n_tiles = need;
    }

    // ---- setup
    if (threadIdx.x == 0) {
        ptx::mbar_init(&sm->q_full, 1);
        ptx::mbar_init(&sm->o_done, 1);
        ptx::mbar_init(&sm->l_bar, 2 * kGroupWarps);
        for (int s = 0; s < kStages; ++s) {
            ptx::mbar_init(&sm->k_full[s], 1);
            ptx::mbar_init(&sm->k_empty[s], 1);
            ptx::mbar_init(&sm->v_full[s], 1);
            ptx::mbar_init(&sm->v_empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            ptx::mbar_init(&sm->s_full[i], 1);
            ptx::mbar_init(&sm->s_empty[i], kGroupWarps);
            ptx::mbar_init(&sm->p_full[i], kGroupWarps);
            ptx::mbar_init(&sm->p_empty[i], 1);
            ptx::mbar_init(&sm->o_ready[i], 4);
            for (int qd = 0; qd < 4; ++qd) ptx::mbar_init(&sm->x_bar[i][qd], 1);
        }
        for (int i = 0; i < 4; ++i)
            for (int qd = 0; qd < 4; ++qd) ptx::mbar_init(&sm->a_bar[i][qd], 1);
        sm->abort_flag = (*reinterpret_cast<volatile uint32_t*>(P.status) != 0u) ? 1u : 0u;
        ptx::mbar_init_fence();
    }
    // constant parts of the B operand of P~V: 16 rows of E2M1 1.0 (0x22) after each V^T stage, unit scales
    for (int i = threadIdx.x; i < kStages * 256; i += kThreads)
        reinterpret_cast<uint32_t*>(sm->v[i / 256] + kTileBytes)[i % 256] = 0x22222222u;
    for (int i = threadIdx.x; i < kSfBytes / 4; i += kThreads)
        reinterpret_cast<uint32_t*>(sm->sf_ones)[i] = (i < 64 && (i & 3) == 0) ? 0x7f7f7f7fu : 0u;
    ptx::fence_proxy_async_smem();
    if (warp == 1) ptx::tmem_alloc(&sm->tmem_base, kTmemCols);
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = sm->tmem_base;
    const bool run = sm->abort_flag == 0 && n_tiles > 0;

    // Register budget: the probability warpgroups take what the other two give up.  setmaxnreg moves registers
    // inside the CTA's own allocation only (512 threads x 128 at launch = 16 x 128 per lane), so the budgets must
    // add up to no more than that: 4 x 56 + 8 x 200 + 4 x 56 = 2048.  A role that asks for more waits for good.
    if (warp < 4) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    if (run && warp == 0 && lane == 0) {
        // =============================== TMA producer (one thread) ===============================
        ptx::mbar_arrive_expect_tx(&sm->q_full, kTileBytes + kSfBytes);
        ptx::tma_load_2d(sm->q, &map_q, 0, q_row, &sm->q_full);
        ptx::bulk_load_1d(sm->sf_q, P.sf_q + static_cast<int64_t>(q_row / kTile) * kSfBytes, kSfBytes, &sm->q_full);
        const int64_t sfk_tile0 = k_row0 / kTile;
        int s = 0;
        uint32_t ph = 0;
        for (int64_t j = 0; j < (P.inject_skip_loads ? 0 : n_tiles); ++j) {
            // Stage barriers of their own: a waiter on a barrier that other roles may complete twice before it
            // looks (S runs ahead) could not tell which completion it sees by parity.
            if (!wait1(&sm->k_empty[s], ph ^ 1u, sm, P.status)) break;
            ptx::mbar_arrive_expect_tx(&sm->k_full[s], kTileBytes + kSfBytes);
            ptx::tma_load_2d(sm->k[s], &map_k, 0, k_row0 + static_cast<int>(j * kTile), &sm->k_full[s]);
            ptx::bulk_load_1d(sm->sf_k[s], P.sf_k + (sfk_tile0 + j) * kSfBytes, kSfBytes, &sm->k_full[s]);
            if (!wait1(&sm->v_empty[s], ph ^ 1u, sm, P.status)) break;
            ptx::mbar_arrive_expect_tx(&sm->v_full[s], kTileBytes + kSfBytes);
            ptx::tma_load_2d(sm->v[s], &map_v, v_x0 + static_cast<int>(j * 64), v_y0, &sm->v_full[s]);
            ptx::bulk_load_1d(sm->sf_v[s], P.sf_v + (sfv_tile0 + j) * kSfBytes, kSfBytes, &sm->v_full[s]);
            if (++s == kStages) { s = 0; ph ^= 1u; }
        }
    } else if (run && warp == 1) {
        // =============================== S = Q K^T issuer ===============================
        // The whole warp runs the loop with warp-uniform state; one elected lane issues the tcgen05
        // instructions.  Descriptors differ from tile to tile only in the start-address field (address >> 4).
        const uint64_t d_sw64 = ptx::smem_desc(0, 16, 512, ptx::kLayoutSw64);
        const uint64_t d_sf = ptx::smem_desc(0, 16, 128, ptx::kLayoutNone);
        const uint64_t dq0 = d_sw64 + (ptx::smem_u32(sm->q) >> 4);
        const uint32_t sfq = tmem + kColSfQ;
        bool ok = wait_all(&sm->q_full, 0, sm, P.status);
        ptx::tc_fence_after_sync();
        if (ok && ptx::elect_one()) ptx::tmem_cp_sf(sfq, d_sf + (ptx::smem_u32(sm->sf_q) >> 4));
        int ks = 0;
        uint32_t kph = 0;
        for (int64_t t = 0; ok && t < n_tiles; ++t) {
            const int sb = static_cast<int>(t & 1);
            if (!wait_all(&sm->k_full[ks], kph, sm, P.status)) break;
            if (!wait_all(&sm->s_empty[sb], static_cast<uint32_t>((t >> 1) & 1) ^ 1u, sm, P.status)) break;
            ptx::tc_fence_after_sync();
            if (ptx::elect_one()) {
                const uint32_t sfk = tmem + kColSfK + 4 * sb;
                ptx::tmem_cp_sf(sfk, d_sf + (ptx::smem_u32(sm->sf_k[ks]) >> 4));
                const uint64_t dk0 = d_sw64 + (ptx::smem_u32(sm->k[ks]) >> 4);
                const uint32_t d_s = tmem + kColS + 128 * sb;
                ptx::mma_mxf4(d_s, dq0, dk0, ptx::mxf4_idesc(128, 0), sfq, sfk, 0u);
                ptx::mma_mxf4(d_s, dq0 + 2, dk0 + 2, ptx::mxf4_idesc(128, 2), sfq | (2u << 30), sfk | (2u << 30), 1u);
                ptx::mma_commit(&sm->s_full[sb]);
                ptx::mma_commit(&sm->k_empty[ks]);
            }
            __syncwarp();
            if (++ks == kStages) { ks = 0; kph ^= 1u; }
        }
    } else if (run && warp == 2) {
        // =============================== [dA | dl] = P~ [V | 1] issuer ===============================
        const uint64_t d_sw64 = ptx::smem_desc(0, 16, 512, ptx::kLayoutSw64);
        const uint64_t d_sf = ptx::smem_desc(0, 16, 128, ptx::kLayoutNone);
        if (ptx::elect_one()) {
            const uint64_t d1 = d_sf + (ptx::smem_u32(sm->sf_ones) >> 4);
            ptx::tmem_cp_sf(tmem + kColSfV + 4, d1);
            ptx::tmem_cp_sf(tmem + kColSfV + 12, d1);
        }
        __syncwarp();
        int vs = 0;
        uint32_t vph = 0;
        for (int64_t j = 0; j < n_tiles; ++j) {
            const int pb = static_cast<int>(j & 1);
            if (!wait_all(&sm->v_full[vs], vph, sm, P.status)) break;
            if (!wait_all(&sm->p_full[pb], static_cast<uint32_t>((j >> 1) & 1), sm, P.status)) break;
            if (!wait_all(&sm->o_ready[pb], static_cast<uint32_t>((j >> 1) & 1), sm, P.status)) break;
            ptx::tc_fence_after_sync();
            if (ptx::elect_one()) {
                const uint32_t sfp = tmem + kColSfP + 4 * pb;
                const uint32_t sfv = tmem + kColSfV + 8 * pb;
                ptx::tmem_cp_sf(sfp, d_sf + (ptx::smem_u32(sm->sf_p[pb]) >> 4));
                ptx::tmem_cp_sf(sfv, d_sf + (ptx::smem_u32(sm->sf_v[vs]) >> 4));
                const uint64_t dp0 = d_sw64 + (ptx::smem_u32(sm->p[pb]) >> 4);
                const uint64_t dv0 = d_sw64 + (ptx::smem_u32(sm->v[vs]) >> 4);
                ptx::mma_mxf4(tmem + kColO, dp0, dv0, ptx::mxf4_idesc(144, 0), sfp, sfv, j > 0 ? 1u : 0u);
                ptx::mma_mxf4(tmem + kColO, dp0 + 2, dv0 + 2, ptx::mxf4_idesc(144, 2), sfp | (2u << 30), sfv | (2u << 30), 1u);
                ptx::mma_commit(&sm->p_empty[pb]);
                ptx::mma_commit(&sm->v_empty[vs]);
                if (j + 1 == n_tiles) ptx::mma_commit(&sm->o_done);
            }
            __syncwarp();
            if (++vs == kStages) { vs = 0; vph ^= 1u; }
        }
    }
    } else if (warp >= 12) {
    // =============================== historical rescaling (Eq. alpha) ===============================
    // One warp per TMEM lane quarter.  When a row's maximum grew in tile j, its accumulator row and its
    // denominator are multiplied by alpha_j after P~V_{j-1} has landed and before P~V_j is released; this runs
    // beside the code generation of tile j instead of inside it.
    asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
    const int quarter = warp & 3;
    const uint32_t row = quarter * 32 + lane;
    const uint32_t o_addr = tmem + (static_cast<uint32_t>(quarter * 32) << 16) + kColO;
    if (run) {
        for (int64_t j = 0; j < n_tiles; ++j) {
            const int sb = static_cast<int>(j & 1);
            // every tile, so that each phase of this barrier is seen in order
            if (!wait_all(&sm->a_bar[j & 3][quarter], static_cast<uint32_t>((j >> 2) & 1), sm, P.status)) break;
            if (j > 0) {
                const float alpha = sm->alpha[j & 3][row];
                const bool any = __any_sync(0xffffffffu, alpha != 1.0f);
                // every tile, so that each phase of this barrier is seen in order
                if (!wait_all(&sm->p_empty[sb ^ 1], static_cast<uint32_t>(((j - 1) >> 1) & 1), sm, P.status)) break;
                if (any) {
                    ptx::tc_fence_after_sync();
                    uint32_t o[32];
                    const uint64_t alpha2 = pack2(alpha, alpha);
                    uint32_t lcol = 0;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        ptx::tmem_ld32<0>(o_addr + 32 * c, o);
                        if (c == 0) lcol = ptx::tmem_ld1(o_addr + 128);     // the denominator travels with the first chunk
                        ptx::tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {
                            uint64_t v2;
                            asm("mov.b64 %0, {%1, %2};" : "=l"(v2) : "r"(o[i]), "r"(o[i + 1]));
                            asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(v2) : "l"(v2), "l"(alpha2));
                            asm("mov.b64 {%0, %1}, %2;" : "=r"(o[i]), "=r"(o[i + 1]) : "l"(v2));
                        }
                        ptx::tmem_st32<0>(o_addr + 32 * c, o);
                        if (c == 0) ptx::tmem_st1(o_addr + 128, __float_as_uint(__uint_as_float(lcol) * alpha));
                        ptx::tmem_wait_st();   // the store reads o[] asynchronously: not before this may o[] be reused
                    }
                    ptx::tc_fence_before_sync();
                }
            }
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&sm->o_ready[sb]);
        }
    }
    } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 200;");
    const int quarter = warp & 3;                       // TMEM lane quarter this warp may touch
    const int group = (warp - 4) >> 2;                  // group 0 takes the even KV tiles, group 1 the odd ones
    const uint32_t row = quarter * 32 + lane;           // row inside the query tile: one thread owns one row
    // this thread's query: token index inside the sequence, query head, and whether the row exists
    int64_t grow;
    int hq;
    bool row_valid;
    if (packed) {
        const int lq = static_cast<int>(Sq);
        const int gq = static_cast<int>(row) / lq;
        grow = static_cast<int>(row) - gq * lq;
        hq = head0 + gq;
        row_valid = gq < G;
    } else {
        grow = q0 + row;
        hq = head0;
        row_valid = grow < Sq;
    }
    const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
    if (run) {
        // =============================== probability generation ===============================
        const ProducerConsts K = P.K;
        int64_t limit = P.causal ? grow + shift : Sk - 1; // last visible key of this row
        if (limit > Sk - 1) limit = Sk - 1;
        const bool dbg_row = DEBUG && P.has_dbg && b == P.dbg.batch && hq == P.dbg.head && grow >= P.dbg.q_begin &&
                             grow < P.dbg.q_end && row_valid;
        const int64_t drow = grow - P.dbg.q_begin;
        const int64_t nblk_all = (Sk + 31) / 32;
        const int64_t ntile_all = (Sk + kTile - 1) / kTile;
        bool ok = true;
        bool in_flight = false;           // the scores of this tile were asked for at the end of the group's previous tile
        // FP32-denominator baseline (PRODUCER 6): this thread's sum of the row's FP32 exponentials over the group's
        // own tiles, relative to the scaled maximum m_ref of the latest of them
        float lsum = 0.0f, m_ref = -INFINITY;
        float r[128];
        const uint32_t s_addr = tmem + lane_base + kColS + 128 * group;

        for (int64_t j = group; j < n_tiles; j += 2) {
            const int sb = group;                                         // S, P and exchange buffers belong to the group
            const uint32_t ph2 = static_cast<uint32_t>((j >> 1) & 1);

            // ---- scores of tile j: TMEM -> registers (Algorithm 2, step 1 happened on the tensor core)
            if (!in_flight) {
                if (!wait_all(&sm->s_full[sb], ph2, sm, P.status)) { ok = false; break; }
                ptx::tc_fence_after_sync();
                ptx::tmem_ld32f<0>(s_addr, r);
                ptx::tmem_ld32f<32>(s_addr + 32, r);
                ptx::tmem_ld32f<64>(s_addr + 64, r);
                ptx::tmem_ld32f<96>(s_addr + 96, r);
            }
            float bmax[4];
            bool have_prev;
            {
                // polls whose answers are needed later travel while the scores do
                have_prev = j == 0 || ptx::mbar_try_wait(&sm->x_bar[sb ^ 1][quarter], static_cast<uint32_t>(((j - 1) >> 1) & 1));
                ptx::tmem_wait_ld();
                ptx::tc_fence_before_sync();          // the S buffer is handed back with the joint publication below
                const int64_t key0 = j * kTile;
                if (key0 + 127 > limit) {     // diagonal or ragged tile: keys past the row's limit are masked in place
#pragma unroll
                    for (int i = 0; i < 128; ++i)
                        if (key0 + i > limit) r[i] = -INFINITY;
                }
            }
#pragma unroll
            for (int g = 0; g < 4; ++g) bmax[g] = block_max32(&r[32 * g]);

            // ---- running row maximum (Eq. rowmax-update): handed over from the group that owns tile j-1
            float m_prev = -INFINITY;
            if (j > 0) {
                if (!have_prev && !wait_all(&sm->x_bar[sb ^ 1][quarter], static_cast<uint32_t>(((j - 1) >> 1) & 1), sm, P.status)) { ok = false; break; }
                m_prev = sm->runmax[sb ^ 1][row];
            }
            float m_new = fmaxf(fmaxf(m_prev, bmax[0]), max3(bmax[1], bmax[2], bmax[3]));
            if (P.rescale_threshold > 0.0f && m_prev != -INFINITY) {      // optional policy: keep the old maximum
                const float ahead = __fsub_rn(__fmul_rn(K.sigma, m_new), __fmul_rn(K.sigma, m_prev));
                if (!(ahead > P.rescale_threshold)) m_new = m_prev;
            }
            const float m_s_prev = __fmul_rn(K.sigma, m_prev);
            const float m_s = __fmul_rn(K.sigma, m_new);
            const bool grew = m_new > m_prev && m_prev != -INFINITY;      // history exists and must be rescaled
            const float alpha = grew ? ex2_approx(__fmul_rn(__fsub_rn(m_s_prev, m_s), K.LOG2E)) : 1.0f;
            // One publication for both readers: the running maximum for the other group, alpha for the rescaling
            // warps.  alpha sits in a ring of four tiles: slot j mod 4 was last read for tile j-4, before P~V_{j-4}
            // was released, and this group waited for the end of P~V_{j-4} before it stored the codes of tile j-2.
            sm->runmax[sb][row] = m_new;
            sm->alpha[j & 3][row] = alpha;
            __syncwarp();
            if (lane == 0) {
                ptx::mbar_arrive(&sm->x_bar[sb][quarter]);
                ptx::mbar_arrive(&sm->a_bar[j & 3][quarter]);
                ptx::mbar_arrive(&sm->s_empty[sb]);           // every lane's scores are in registers (wait::ld above)
            }
            // P~V of tile j-2 reads the group's P buffer: asked here, answered while block 0 is computed
            const bool have_p = ptx::mbar_try_wait(&sm->p_empty[sb], ph2 ^ 1u);

            if (PRODUCER == 6) {          // bring the sum to the new reference maximum (two tiles of alpha in one step)
                if (lsum != 0.0f) lsum *= ex2_approx(__fmul_rn(__fsub_rn(m_ref, m_s), K.LOG2E));
                m_ref = m_s;
            }
            // ---- probability operand (Algorithm 1 per block): codes and scales straight into the MMA operand
            uint32_t sfword = 0;
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint4 codes;
                uint32_t byte;
                produce32<PRODUCER, FIX8>(&r[g * 32], bmax[g], m_s, K, codes, byte, &lsum);
                if (g == 0 && !have_p) {      // P~V of tile j-2 must have finished: it reads the group's P buffer
                    if (!wait_all(&sm->p_empty[sb], ph2 ^ 1u, sm, P.status)) { ok = false; break; }
                }
                *reinterpret_cast<uint4*>(sm->p[sb] + p_swizzled_offset(row, g)) = codes;
                sfword |= byte << (8 * g);
                if (DEBUG && dbg_row) {
                    const int64_t blk = j * 4 + g;
                    if (blk < nblk_all) {
                        if (P.dbg.codes) *reinterpret_cast<uint4*>(P.dbg.codes + (drow * nblk_all + blk) * 16) = codes;
                        if (P.dbg.scales) P.dbg.scales[drow * nblk_all + blk] = static_cast<uint8_t>(byte);
                    }
                }
            }
            if (!ok) break;               // the bounded wait inside the block loop gave up
            *reinterpret_cast<uint32_t*>(sm->sf_p[sb] + (row & 31u) * 16u + (row >> 5) * 4u) = sfword;
            if (DEBUG && dbg_row) {
                if (P.dbg.raw_scores) {
                    for (int i = 0; i < 128; ++i)
                        if (j * kTile + i < Sk) P.dbg.raw_scores[drow * Sk + j * kTile + i] = r[i];
                }
                if (P.dbg.row_max) P.dbg.row_max[drow * ntile_all + j] = m_s;
            }

            // The registers are free: if S of the group's next tile is there already (it is as a rule, S runs ahead),
            // its scores set out now and travel while the operand is handed over and the loop turns.
            in_flight = j + 2 < n_tiles && ptx::mbar_try_wait(&sm->s_full[sb], ph2 ^ 1u);
            if (in_flight) {
                ptx::tc_fence_after_sync();
                ptx::tmem_ld32f<0>(s_addr, r);
                ptx::tmem_ld32f<32>(s_addr + 32, r);
                ptx::tmem_ld32f<64>(s_addr + 64, r);
                ptx::tmem_ld32f<96>(s_addr + 96, r);
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&sm->p_full[sb]);
        }
        ptx::tmem_wait_ld();              // nothing may be in flight when a bounded wait gave up inside the loop

        if (PRODUCER == 6) {              // both groups' partial denominators meet in shared memory
            sm->lsum_x[group][row] = lsum;
            sm->mref_x[group][row] = m_ref;
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&sm->l_bar);
        }
        // ---- final normalisation O = A / l: each group writes 64 of the 128 channels
        // (a barrier of its own: a group that skipped a phase of the other group's p_empty could not tell
        // an old completion from the last one by parity)
        if (ok) ok = wait_all(&sm->o_done, 0, sm, P.status);
        if (ok && PRODUCER == 6) ok = wait_all(&sm->l_bar, 0, sm, P.status);
        if (ok) {
            ptx::tc_fence_after_sync();
            uint32_t o[64];
            const uint32_t o_addr = tmem + lane_base + kColO + 64 * group;
            ptx::tmem_ld32<0>(o_addr, o);
            ptx::tmem_ld32<32>(o_addr + 32, o);
            const uint32_t lcol = ptx::tmem_ld1(tmem + lane_base + kColO + 128);
            ptx::tmem_wait_ld();
            if (row_valid) {
                float l = __uint_as_float(lcol);
                if (PRODUCER == 6) {
                    // the accumulator refers to the maximum of the last tile, the larger of the two groups' references
                    const float l0 = sm->lsum_x[0][row], l1 = sm->lsum_x[1][row];
                    const float m0 = sm->mref_x[0][row], m1 = sm->mref_x[1][row];
                    const float mf = fmaxf(m0, m1);
                    l = (l0 != 0.0f ? l0 * ex2_approx(__fmul_rn(__fsub_rn(m0, mf), K.LOG2E)) : 0.0f) +
                        (l1 != 0.0f ? l1 * ex2_approx(__fmul_rn(__fsub_rn(m1, mf), K.LOG2E)) : 0.0f);
                }
                const float inv = l > 0.0f ? 1.0f / l : 0.0f;
                float4* dst = reinterpret_cast<float4*>(P.o + (o_base + hq * P.o_head + grow * P.o_row + 64 * group));
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float4 v;
                    v.x = __uint_as_float(o[4 * i + 0]) * inv;
                    v.y = __uint_as_float(o[4 * i + 1]) * inv;
                    v.z = __uint_as_float(o[4 * i + 2]) * inv;
                    v.w = __uint_as_float(o[4 * i + 3]) * inv;
                    dst[i] = v;
                }
            }
        }
    } else if (sm->abort_flag == 0) {
        // no visible key for the whole tile: rows are zero
        if (row_valid) {
            float4* dst = reinterpret_cast<float4*>(P.o + (o_base + hq * P.o_head + grow * P.o_row + 64 * group));
            for (int i = 0; i < 16; ++i) dst[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    }

    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) ptx::tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kMaxDevices = 64;   // device ordinals the per-device tables of this file cover

EncodeTiledFn get_encode()
{
    static std::once_flag once;
    static EncodeTiledFn fn = nullptr;
    std::call_once(once, [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    });
    return fn;
}

// [rows, row_bytes] u8 matrix, box 64 B x 128 rows, 64-byte swizzle.  A descriptor depends on nothing but
// (base, row_bytes, rows), so the last few are kept: a serving loop that calls with the same workspace and shape
// (decode steps above all) does not pay for three driver calls per forward.
struct MapCacheEntry {
    const void* base;
    uint64_t row_bytes, rows;
    CUtensorMap map;
};
constexpr int kMapCacheSize = 24;
std::mutex g_map_mutex;
MapCacheEntry g_map_cache[kMapCacheSize] = {};
int g_map_next = 0;

bool encode_map(CUtensorMap* map, const void* base, uint64_t row_bytes, uint64_t rows)
{
    {
        std::lock_guard<std::mutex> lock(g_map_mutex);
        for (int i = 0; i < kMapCacheSize; ++i) {
            const MapCacheEntry& e = g_map_cache[i];
            if (e.base == base && e.row_bytes == row_bytes && e.rows == rows) {
                *map = e.map;
                return true;
            }
        }
    }
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[2] = {row_bytes, rows};
    cuuint64_t strides[1] = {row_bytes};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    if (enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    std::lock_guard<std::mutex> lock(g_map_mutex);
    g_map_cache[g_map_next] = MapCacheEntry{base, row_bytes, rows, *map};
    g_map_next = (g_map_next + 1) % kMapCacheSize;
    return true;
}

struct Workspace {
    size_t status, qc, qsf, kc, ksf, vt, vsf, total;
    int64_t Sq_pad, Sk_pad;
};

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

Workspace plan_workspace(int B, int Hq, int Hkv, int64_t Sq, int64_t Sk)
{
    Workspace w;
    w.Sq_pad = (Sq + kTile - 1) / kTile * kTile;
    w.Sk_pad = (Sk + kTile - 1) / kTile * kTile;
    size_t off = 0;
    w.status = off; off += 1024;
    w.qc = off;  off = align_up(off + static_cast<size_t>(B) * Hq * w.Sq_pad * 64, 1024);
    w.qsf = off; off = align_up(off + static_cast<size_t>(B) * Hq * (w.Sq_pad / kTile) * kSfBytes, 1024);
    w.kc = off;  off = align_up(off + static_cast<size_t>(B) * Hkv * w.Sk_pad * 64, 1024);
    w.ksf = off; off = align_up(off + static_cast<size_t>(B) * Hkv * (w.Sk_pad / kTile) * kSfBytes, 1024);
    w.vt = off;  off = align_up(off + static_cast<size_t>(B) * Hkv * 128 * (w.Sk_pad / 2), 1024);
    w.vsf = off; off = align_up(off + static_cast<size_t>(B) * Hkv * (w.Sk_pad / kTile) * kSfBytes, 1024);
    w.total = off;
    return w;
}

bool shape_ok(int B, int Hq, int Hkv, int64_t Sq, int64_t Sk, int d)
{
    return B > 0 && Hq > 0 && Hkv > 0 && Sq > 0 && Sk > 0 && d == 128 && Hq % Hkv == 0 &&
           static_cast<int64_t>(B) * Hq * ((Sq + kTile - 1) / kTile * kTile) < (1ll << 31) &&
           static_cast<int64_t>(B) * Hkv * ((Sk + kTile - 1) / kTile * kTile) < (1ll << 31);
}

template <int PRODUCER, bool DEBUG, bool FIX8>
cudaError_t launch_one(dim3 grid, size_t smem, cudaStream_t stream, const CUtensorMap& mq, const CUtensorMap& mk,
                       const CUtensorMap& mv, const FwdParams& P)
{
    // the shared-memory attribute belongs to (function, device): set once for each
    static std::mutex mu;
    static bool done[kMaxDevices] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!done[dev]) {
            cudaError_t e = cudaFuncSetAttribute(attention_fwd_kernel<PRODUCER, DEBUG, FIX8>,
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
            if (e != cudaSuccess) return e;
            done[dev] = true;
        }
    }
    attention_fwd_kernel<PRODUCER, DEBUG, FIX8><<<grid, kThreads, smem, stream>>>(mq, mk, mv, P);
    return cudaGetLastError();
}

template <int PRODUCER>
cudaError_t launch_main(bool debug, bool fix8, dim3 grid, size_t smem, cudaStream_t stream, const CUtensorMap& mq,
                        const CUtensorMap& mk, const CUtensorMap& mv, const FwdParams& P)
{
    if constexpr (PRODUCER != 0) {     // the 8 -> 7 fix belongs to the affine rule alone
        return debug ? launch_one<PRODUCER, true, false>(grid, smem, stream, mq, mk, mv, P)
                     : launch_one<PRODUCER, false, false>(grid, smem, stream, mq, mk, mv, P);
    } else {
        if (debug) return fix8 ? launch_one<PRODUCER, true, true>(grid, smem, stream, mq, mk, mv, P)
                               : launch_one<PRODUCER, true, false>(grid, smem, stream, mq, mk, mv, P);
        return fix8 ? launch_one<PRODUCER, false, true>(grid, smem, stream, mq, mk, mv, P)
                    : launch_one<PRODUCER, false, false>(grid, smem, stream, mq, mk, mv, P);
    }
}

// The query heads of a KV group share one 128-row query tile when they fit: a decode step (one query token) of a
// model with 4 query heads per KV head then fills 4 rows of one tile instead of 1 row of each of 4 tiles, and each
// K/V tile is loaded once per KV head.  Rows are independent of one another on the whole path, so the result is
// the unpacked one bit for bit.
bool use_packed_tile(int Hq, int Hkv, int64_t Sq) { return Hq / Hkv > 1 && static_cast<int64_t>(Hq / Hkv) * Sq <= kTile; }

cudaError_t launch_forward(int producer, bool debug, bool fix8, int64_t items, cudaStream_t stream, const CUtensorMap& mq,
                           const CUtensorMap& mk, const CUtensorMap& mv, const FwdParams& P)
{
    if (items <= 0 || items > 0x7fffffffll) return cudaErrorInvalidValue;
    dim3 grid(static_cast<unsigned>(items));
    // more than half of the SM's shared memory: one CTA per SM, since each CTA takes all 512 TMEM columns
    const size_t smem = sizeof(Smem) + 1024 > 120 * 1024 ? sizeof(Smem) + 1024 : 120 * 1024;
    switch (producer) {
        case 0: return launch_main<0>(debug, fix8, grid, smem, stream, mq, mk, mv, P);
        case 1: return launch_main<1>(debug, fix8, grid, smem, stream, mq, mk, mv, P);
        case 2: return launch_main<2>(debug, fix8, grid, smem, stream, mq, mk, mv, P);
        case 3: return launch_main<3>(debug, fix8, grid, smem, stream, mq, mk, mv, P);
        case 4: return launch_main<4>(debug, fix8, grid, smem, stream, mq, mk, mv, P);
        case 5: return launch_main<5>(debug, fix8, grid, smem, stream, mq, mk, mv, P);
        case 6: return launch_main<6>(debug, fix8, grid, smem, stream, mq, mk, mv, P);
        default: return cudaErrorInvalidValue;
    }
}

// fma(r, A, Bb) can reach 8 only if the residual of a block maximum, below ln 1.5, maps that high
bool needs_fix8(float tau, float h) { return (log(1.5) - static_cast<double>(tau)) * static_cast<double>(h) + 1.0 > 7.999; }

efq_status_t check_device()
{
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return EFQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return EFQ_ERR_CUDA;
    return major == 10 ? EFQ_OK : EFQ_ERR_ARCH;
}

efq_status_t attention_impl(const void* q, const void* k, const void* v, float* o, int B, int Hq, int Hkv, int64_t Sq,
                            int64_t Sk, int d, int causal, float softmax_scale, int producer, float tau, float h,
                            void* workspace, size_t workspace_bytes, const efq_debug_t* debug, cudaStream_t stream,
                            bool do_quantize, bool do_forward, bool inject_skip_loads = false, float rescale_threshold = 0.0f)
{
    // q [B, Hq, Sq, d], k, v [B, Hkv, Sk, d], o [B, Hq, Sq, d]
    if (!q || !k || !v || !o) return EFQ_ERR_INVALID_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || Hq % Hkv != 0) return EFQ_ERR_INVALID_ARG;
    if (d != 128) return EFQ_ERR_UNSUPPORTED;
    if (!shape_ok(B, Hq, Hkv, Sq, Sk, d)) return EFQ_ERR_UNSUPPORTED;
    if (producer < 0 || producer > 6) return EFQ_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.0f)) softmax_scale = static_cast<float>(1.0 / sqrt(static_cast<double>(d)));
    if (!isfinite(softmax_scale) || !isfinite(tau) || !isfinite(h) || !(h > 0.0f)) return EFQ_ERR_INVALID_ARG;
    auto mis = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; };
    if (mis(q, 16) || mis(k, 16) || mis(v, 16) || mis(o, 16)) return EFQ_ERR_ALIGNMENT;
    const Workspace w = plan_workspace(B, Hq, Hkv, Sq, Sk);
    if (!workspace || workspace_bytes < w.total) return EFQ_ERR_WORKSPACE;
    if (mis(workspace, 256)) return EFQ_ERR_ALIGNMENT;
    const efq_status_t dev_st = check_device();
    if (dev_st != EFQ_OK) return dev_st;

    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const bool packed = use_packed_tile(Hq, Hkv, Sq);
    const int G = Hq / Hkv;
    const int64_t q_rows = packed ? static_cast<int64_t>(B) * Hkv * kTile : static_cast<int64_t>(B) * Hq * w.Sq_pad;
    if (do_quantize) {
        QuantSeg sq{}, sk{}, sv{};
        sq.src = static_cast<const __nv_bfloat16*>(q);
        sq.heads = packed ? static_cast<int64_t>(B) * Hkv : static_cast<int64_t>(B) * Hq;
        sq.S = packed ? G * Sq : Sq;
        sq.S_pad = packed ? kTile : w.Sq_pad;
        sq.head_stride = Sq * 128; sq.row_stride = 128;
        sq.pack_lq = packed ? static_cast<int32_t>(Sq) : 0; sq.pack_G = packed ? G : 1;
        sq.codes = ws + w.qc; sq.sf = ws + w.qsf;
        sk.src = static_cast<const __nv_bfloat16*>(k);
        sk.heads = static_cast<int64_t>(B) * Hkv; sk.S = Sk; sk.S_pad = w.Sk_pad;
        sk.head_stride = Sk * 128; sk.row_stride = 128; sk.pack_G = 1;
        sk.codes = ws + w.kc; sk.sf = ws + w.ksf;
        sv = sk;
        sv.src = static_cast<const __nv_bfloat16*>(v);
        sv.codes = ws + w.vt; sv.sf = ws + w.vsf;
        sv.v_row_bytes = w.Sk_pad / 2; sv.v_x0 = 0; sv.v_sf_tiles_per_head = w.Sk_pad / kTile; sv.v_sf_tile0 = 0;
        // one launch for the three operands; it also clears the status words the forward starts from
        if (launch_quantize_qkv(sq, sk, sv, reinterpret_cast<uint32_t*>(ws + w.status), stream) != cudaSuccess) return EFQ_ERR_CUDA;
    }
    if (!do_forward) return EFQ_OK;

    CUtensorMap mq, mk, mv;
    if (!encode_map(&mq, ws + w.qc, 64, static_cast<uint64_t>(q_rows))) return EFQ_ERR_CUDA;
    if (!encode_map(&mk, ws + w.kc, 64, static_cast<uint64_t>(B) * Hkv * w.Sk_pad)) return EFQ_ERR_CUDA;
    if (!encode_map(&mv, ws + w.vt, static_cast<uint64_t>(w.Sk_pad / 2), static_cast<uint64_t>(B) * Hkv * 128)) return EFQ_ERR_CUDA;

    FwdParams P{};
    P.B = B; P.Hq = Hq; P.Hkv = Hkv; P.Sq = Sq; P.Sk = Sk; P.Sq_pad = w.Sq_pad; P.Sk_pad = w.Sk_pad;
    P.causal = causal ? 1 : 0;
    P.K = producer == 3 ? make_producer_consts_lut(softmax_scale) : make_producer_consts(softmax_scale, tau, h);
    P.sf_q = ws + w.qsf; P.sf_k = ws + w.ksf; P.sf_v = ws + w.vsf;
    P.o = o;
    P.o_head = Sq * 128;
    P.o_row = 128;
    P.status = reinterpret_cast<uint32_t*>(ws + w.status);
    P.packed = packed ? 1 : 0;
    P.seqs = nullptr; P.items = nullptr; P.v_tiles_per_head = 0;
    P.inject_skip_loads = inject_skip_loads ? 1 : 0;
    P.rescale_threshold = rescale_threshold;
    P.has_dbg = debug ? 1 : 0;
    if (debug) P.dbg = *debug; else P.dbg = efq_debug_t{};

    const int64_t items = packed ? static_cast<int64_t>(B) * Hkv : (w.Sq_pad / kTile) * B * Hq;
    return launch_forward(producer, debug != nullptr, needs_fix8(tau, h), items, stream, mq, mk, mv, P) == cudaSuccess ? EFQ_OK
                                                                                                                  : EFQ_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------
// Packed variable-length batch: every sequence quantised by itself, all of them in two launches
// ------------------------------------------------------------------------------------------------
// Workspace: status words | tables (sequence table, item table, quantiser jobs, their CTA prefix sums) |
// Q codes [rows of all sequences, 64 B] | Q scale tiles | K codes | K scale tiles |
// V^T codes [Hkv * 128, sum of Sk_pad / 2 B] (the sequences side by side along the keys) | V scale tiles.
struct VarlenPlan {
    int n_active;                    // sequences with query and key tokens
    int64_t q_rows, k_rows, k_cols;  // rows of the Q and K code matrices, keys along V^T (all padded to 128)
    int64_t items, quant_ctas;
    size_t tables, seqs_off, items_off, jobs_off, prefix_off, qc, qsf, kc, ksf, vt, vsf, total;
};

// checks the two prefix arrays and lays the workspace out; false with st set on bad input
bool plan_varlen(const int64_t* cu_q, const int64_t* cu_k, int n_seqs, int Hq, int Hkv, int d, VarlenPlan& p, efq_status_t& st)
{
    st = EFQ_OK;
    if (!cu_q || !cu_k || n_seqs < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0) { st = EFQ_ERR_INVALID_ARG; return false; }
    if (d != 128) { st = EFQ_ERR_UNSUPPORTED; return false; }
    if (n_seqs > 0 && (cu_q[0] != 0 || cu_k[0] != 0)) { st = EFQ_ERR_INVALID_ARG; return false; }
    p = VarlenPlan{};
    for (int s = 0; s < n_seqs; ++s) {
        const int64_t lq = cu_q[s + 1] - cu_q[s], lk = cu_k[s + 1] - cu_k[s];
        if (lq < 0 || lk < 0) { st = EFQ_ERR_INVALID_ARG; return false; }
        if (lq == 0 || lk == 0) continue;
        const bool packed = use_packed_tile(Hq, Hkv, lq);
        const int64_t lq_pad = packed ? kTile : (lq + kTile - 1) / kTile * kTile, lk_pad = (lk + kTile - 1) / kTile * kTile;
        ++p.n_active;
        p.q_rows += (packed ? Hkv : Hq) * lq_pad;
        p.k_rows += Hkv * lk_pad;
        p.k_cols += lk_pad;
        p.items += packed ? Hkv : (lq_pad / kTile) * Hq;
        p.quant_ctas += ((packed ? Hkv : Hq) * lq_pad * 4 + 255) / 256 + (Hkv * lk_pad * 4 + 255) / 256 + (Hkv * (lk_pad / 32) + 1) / 2;
    }
    // 32-bit tile coordinates and grid sizes
    if (p.q_rows >= (1ll << 31) || p.k_rows >= (1ll << 31) || p.k_cols >= (1ll << 31) || p.items >= (1ll << 31) ||
        p.quant_ctas >= (1ll << 31)) { st = EFQ_ERR_UNSUPPORTED; return false; }
    size_t off = 1024;
    p.seqs_off = off;   off = align_up(off + sizeof(SeqDesc) * p.n_active, 256);
    p.items_off = off;  off = align_up(off + sizeof(ItemDesc) * static_cast<size_t>(p.items), 256);
    p.jobs_off = off;   off = align_up(off + sizeof(QuantJob) * 3 * p.n_active, 256);
    p.prefix_off = off; off = align_up(off + sizeof(int32_t) * (3 * p.n_active + 1), 1024);
    p.tables = off - 1024;
    p.qc = off;  off = align_up(off + static_cast<size_t>(p.q_rows) * 64, 1024);
    p.qsf = off; off = align_up(off + static_cast<size_t>(p.q_rows / kTile) * kSfBytes, 1024);
    p.kc = off;  off = align_up(off + static_cast<size_t>(p.k_rows) * 64, 1024);
    p.ksf = off; off = align_up(off + static_cast<size_t>(p.k_rows / kTile) * kSfBytes, 1024);
    p.vt = off;  off = align_up(off + static_cast<size_t>(Hkv) * 128 * (p.k_cols / 2), 1024);
    p.vsf = off; off = align_up(off + static_cast<size_t>(Hkv) * (p.k_cols / kTile) * kSfBytes, 1024);
    p.total = off;
    return true;
}

}  // namespace
}  // namespace efq

extern "C" size_t efq_attention_workspace_bytes(int B, int Hq, int Hkv, int64_t Sq, int64_t Sk, int d)
{
    if (!efq::shape_ok(B, Hq, Hkv, Sq, Sk, d)) return 0;
    return efq::plan_workspace(B, Hq, Hkv, Sq, Sk).total;
}

// Producer ids inside the library: 0 = EFQ (affine rule), 1 / 2 = exp-then-quantize scale4 / scale6, 3 = EFQ-LUT,
// 4 = exp-then-quantize scale4 with the scale folded into the exponential, 5 = the same with 2 of 8 exponentials by polynomial,
// 6 = exp-then-quantize scale4 whose denominator is the sum of the FP32 exponentials (the ones columns are ignored).
static bool read_params(const efq_params_t* params, float& tau, float& h, bool& lut, float& threshold, efq_status_t& st)
{
    tau = -3.06f;
    h = 2.30f;
    lut = false;
    threshold = 0.0f;
    st = EFQ_OK;
    if (params) {
        if (params->variant != 0 && params->variant != 1) { st = EFQ_ERR_UNSUPPORTED; return false; }
        if (params->kv_tile != 0 && params->kv_tile != 128) { st = EFQ_ERR_UNSUPPORTED; return false; }
        if (!(params->rescale_threshold >= 0.0f)) { st = EFQ_ERR_INVALID_ARG; return false; }   // negative or NaN
        threshold = params->rescale_threshold;
        lut = params->variant == 1;
        if (!lut) {                 // the LUT variant has its own fixed (tau16, h16): tau and h are not read
            tau = params->tau;
            h = params->h;
        }
    }
    return true;
}

extern "C" efq_status_t efq_attention_fwd(const void* q, const void* k, const void* v, float* o, int B, int Hq, int Hkv,
                                          int64_t Sq, int64_t Sk, int d, int causal, float softmax_scale,
                                          const efq_params_t* params, void* workspace, size_t workspace_bytes,
                                          const efq_debug_t* debug, void* stream)
{
    float tau, h, threshold;
    bool lut;
    efq_status_t st;
    if (!read_params(params, tau, h, lut, threshold, st)) return st;
    return efq::attention_impl(q, k, v, o, B, Hq, Hkv, Sq, Sk, d, causal, softmax_scale, lut ? 3 : 0, tau, h, workspace,
                               workspace_bytes, debug, static_cast<cudaStream_t>(stream), true, true, false, threshold);
}

extern "C" efq_status_t exp_then_quantize_attention_fwd(const void* q, const void* k, const void* v, float* o, int B,
                                                        int Hq, int Hkv, int64_t Sq, int64_t Sk, int d, int causal,
                                                        float softmax_scale, int scale_mode, void* workspace,
                                                        size_t workspace_bytes, const efq_debug_t* debug, void* stream)
{
    if (scale_mode < 0 || scale_mode > 4) return EFQ_ERR_INVALID_ARG;
    return efq::attention_impl(q, k, v, o, B, Hq, Hkv, Sq, Sk, d, causal, softmax_scale, scale_mode >= 2 ? scale_mode + 2 : 1 + scale_mode, 0.0f, 1.0f,
                               workspace, workspace_bytes, debug, static_cast<cudaStream_t>(stream), true, true);
}

extern "C" efq_status_t efq_attention_fwd_inject_timeout(const void* q, const void* k, const void* v, float* o, int B,
                                                         int Hq, int Hkv, int64_t Sq, int64_t Sk, int d, void* workspace,
                                                         size_t workspace_bytes, void* stream)
{
    return efq::attention_impl(q, k, v, o, B, Hq, Hkv, Sq, Sk, d, 0, 0.0f, 0, -3.06f, 2.30f, workspace, workspace_bytes,
                               nullptr, static_cast<cudaStream_t>(stream), true, true, true);
}

extern "C" efq_status_t efq_quantize_qkv(const void* q, const void* k, const void* v, int B, int Hq, int Hkv, int64_t Sq,
                                         int64_t Sk, int d, void* workspace, size_t workspace_bytes, void* stream)
{
    const void* nz_o = reinterpret_cast<const void*>(16);   // no output is written by the preparation step
    return efq::attention_impl(q, k, v, static_cast<float*>(const_cast<void*>(nz_o)), B, Hq, Hkv, Sq, Sk, d, 0, 0.0f, 0,
                               -3.06f, 2.30f, workspace, workspace_bytes, nullptr, static_cast<cudaStream_t>(stream), true,
                               false);
}

extern "C" efq_status_t efq_attention_fwd_quantized(float* o, int B, int Hq, int Hkv, int64_t Sq, int64_t Sk, int d,
                                                    int causal, float softmax_scale, int producer,
                                                    const efq_params_t* params, void* workspace, size_t workspace_bytes,
                                                    const efq_debug_t* debug, void* stream)
{
    float tau, h, threshold;
    bool lut;
    efq_status_t st;
    if (!read_params(params, tau, h, lut, threshold, st)) return st;
    if (producer == 0 && lut) producer = 3;
    const void* nz = reinterpret_cast<const void*>(16);   // operands already live in the workspace
    return efq::attention_impl(nz, nz, nz, o, B, Hq, Hkv, Sq, Sk, d, causal, softmax_scale, producer, tau, h, workspace,
                               workspace_bytes, debug, static_cast<cudaStream_t>(stream), false, true, false, threshold);
}

extern "C" efq_status_t efq_attention_fwd_host(const void* q_host, const void* k_host, const void* v_host, float* o_host,
                                               void* q_dev, void* k_dev, void* v_dev, float* o_dev, int B, int Hq, int Hkv,
                                               int64_t Sq, int64_t Sk, int d, int causal, float softmax_scale, int producer,
                                               const efq_params_t* params, void* workspace, size_t workspace_bytes,
                                               void* stream)
{
    if (!q_host || !k_host || !v_host || !o_host || !q_dev || !k_dev || !v_dev || !o_dev) return EFQ_ERR_INVALID_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0) return EFQ_ERR_INVALID_ARG;
    float tau, h, threshold;
    bool lut;
    efq_status_t st;
    if (!read_params(params, tau, h, lut, threshold, st)) return st;
    if (producer == 0 && lut) producer = 3;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t qb = static_cast<size_t>(B) * Hq * Sq * d * 2, kb = static_cast<size_t>(B) * Hkv * Sk * d * 2;
    if (cudaMemcpyAsync(q_dev, q_host, qb, cudaMemcpyHostToDevice, s) != cudaSuccess) return EFQ_ERR_CUDA;
    if (cudaMemcpyAsync(k_dev, k_host, kb, cudaMemcpyHostToDevice, s) != cudaSuccess) return EFQ_ERR_CUDA;
    if (cudaMemcpyAsync(v_dev, v_host, kb, cudaMemcpyHostToDevice, s) != cudaSuccess) return EFQ_ERR_CUDA;
    st = efq::attention_impl(q_dev, k_dev, v_dev, o_dev, B, Hq, Hkv, Sq, Sk, d, causal, softmax_scale, producer, tau, h,
                             workspace, workspace_bytes, nullptr, s, true, true, false, threshold);
    if (st != EFQ_OK) return st;
    if (cudaMemcpyAsync(o_host, o_dev, static_cast<size_t>(B) * Hq * Sq * d * 4, cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return EFQ_ERR_CUDA;
    return EFQ_OK;
}

namespace efq {
namespace {
// dst takes src's status if src reports one (keeps the first problem seen across the chunks of a pipelined call)
__global__ void merge_status_kernel(uint32_t* dst, const uint32_t* src, int overwrite)
{
    const uint32_t v = *src;
    if (overwrite || v != 0u) *dst = v;
}
}  // namespace
}  // namespace efq

extern "C" efq_status_t efq_attention_fwd_host_pipelined(const void* q_host, const void* k_host, const void* v_host,
                                                         float* o_host, void* q_dev, void* k_dev, void* v_dev,
                                                         float* o_dev, int B, int Hq, int Hkv, int64_t Sq, int64_t Sk,
                                                         int d, int causal, float softmax_scale, int producer,
                                                         const efq_params_t* params, void* workspace,
                                                         size_t workspace_bytes, int n_chunks, void* stream_in,
                                                         void* stream_compute, void* stream_out)
{
    if (!q_host || !k_host || !v_host || !o_host || !q_dev || !k_dev || !v_dev || !o_dev) return EFQ_ERR_INVALID_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || Hq % Hkv != 0 || n_chunks <= 0) return EFQ_ERR_INVALID_ARG;
    if (!workspace) return EFQ_ERR_WORKSPACE;
    float tau, h, threshold;
    bool lut;
    efq_status_t st;
    if (!read_params(params, tau, h, lut, threshold, st)) return st;
    if (producer == 0 && lut) producer = 3;
    cudaStream_t s_in = static_cast<cudaStream_t>(stream_in), s_c = static_cast<cudaStream_t>(stream_compute),
                 s_out = static_cast<cudaStream_t>(stream_out);
    // chunks are runs of KV heads inside one batch entry: contiguous slices of q, k, v and o
    int per_batch = n_chunks / B;
    if (per_batch < 1) per_batch = 1;
    if (per_batch > Hkv) per_batch = Hkv;
    const int heads_per_chunk = (Hkv + per_batch - 1) / per_batch;
    const int group = Hq / Hkv;
    if (B == 1 && heads_per_chunk >= Hkv)        // nothing to overlap: the plain form on the compute stream
        return efq_attention_fwd_host(q_host, k_host, v_host, o_host, q_dev, k_dev, v_dev, o_dev, B, Hq, Hkv, Sq, Sk, d,
                                      causal, softmax_scale, producer == 3 ? 0 : producer, params, workspace,
                                      workspace_bytes, stream_compute);
    if (!efq::shape_ok(1, heads_per_chunk * group, heads_per_chunk, Sq, Sk, d)) return EFQ_ERR_UNSUPPORTED;
    const size_t slot = efq::plan_workspace(1, heads_per_chunk * group, heads_per_chunk, Sq, Sk).total;
    if (workspace_bytes < slot + 256) return EFQ_ERR_WORKSPACE;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    uint32_t* agg = reinterpret_cast<uint32_t*>(ws + slot);          // first problem seen by any chunk
    if (cudaMemsetAsync(agg, 0, 4, s_c) != cudaSuccess) return EFQ_ERR_CUDA;

    const size_t q_head = static_cast<size_t>(Sq) * d * 2, kv_head = static_cast<size_t>(Sk) * d * 2;
    const size_t o_head = static_cast<size_t>(Sq) * d * 4;
    cudaEvent_t ev = nullptr;
    auto fail = [&](efq_status_t code) { if (ev) cudaEventDestroy(ev); return code; };
    // The staging buffers are reused from call to call: this call's input copies must not overtake the forwards
    // of an earlier call that still read them, so stream_in first waits for what stream_compute holds now.
    if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return EFQ_ERR_CUDA;
    if (cudaEventRecord(ev, s_c) != cudaSuccess || cudaStreamWaitEvent(s_in, ev, 0) != cudaSuccess) return fail(EFQ_ERR_CUDA);
    cudaEventDestroy(ev);
    ev = nullptr;
    for (int b = 0; b < B; ++b) {
        for (int h0 = 0; h0 < Hkv; h0 += heads_per_chunk) {
            const int nh = h0 + heads_per_chunk <= Hkv ? heads_per_chunk : Hkv - h0;
            const size_t q_off = (static_cast<size_t>(b) * Hq + static_cast<size_t>(h0) * group) * q_head;
            const size_t kv_off = (static_cast<size_t>(b) * Hkv + h0) * kv_head;
            const size_t o_off = (static_cast<size_t>(b) * Hq + static_cast<size_t>(h0) * group) * o_head;
            const uint8_t* qh = static_cast<const uint8_t*>(q_host) + q_off;
            const uint8_t* kh = static_cast<const uint8_t*>(k_host) + kv_off;
            const uint8_t* vh = static_cast<const uint8_t*>(v_host) + kv_off;
            uint8_t* qd = static_cast<uint8_t*>(q_dev) + q_off;
            uint8_t* kd = static_cast<uint8_t*>(k_dev) + kv_off;
            uint8_t* vd = static_cast<uint8_t*>(v_dev) + kv_off;
            uint8_t* od = reinterpret_cast<uint8_t*>(o_dev) + o_off;
            // inputs of this chunk: stream_in
            if (cudaMemcpyAsync(qd, qh, q_head * nh * group, cudaMemcpyHostToDevice, s_in) != cudaSuccess) return fail(EFQ_ERR_CUDA);
            if (cudaMemcpyAsync(kd, kh, kv_head * nh, cudaMemcpyHostToDevice, s_in) != cudaSuccess) return fail(EFQ_ERR_CUDA);
            if (cudaMemcpyAsync(vd, vh, kv_head * nh, cudaMemcpyHostToDevice, s_in) != cudaSuccess) return fail(EFQ_ERR_CUDA);
            if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return EFQ_ERR_CUDA;
            if (cudaEventRecord(ev, s_in) != cudaSuccess || cudaStreamWaitEvent(s_c, ev, 0) != cudaSuccess) return fail(EFQ_ERR_CUDA);
            cudaEventDestroy(ev);     // released once the recorded work has completed
            ev = nullptr;
            // forward of this chunk: stream_compute (in order, so the one workspace slot is reused safely)
            st = efq::attention_impl(qd, kd, vd, reinterpret_cast<float*>(od), 1, nh * group, nh, Sq, Sk, d, causal,
                                     softmax_scale, producer, tau, h, ws, slot, nullptr, s_c, true, true, false, threshold);
            if (st != EFQ_OK) return st;
            efq::merge_status_kernel<<<1, 1, 0, s_c>>>(agg, reinterpret_cast<const uint32_t*>(ws), 0);
            if (cudaGetLastError() != cudaSuccess) return EFQ_ERR_CUDA;
            if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return EFQ_ERR_CUDA;
            if (cudaEventRecord(ev, s_c) != cudaSuccess || cudaStreamWaitEvent(s_out, ev, 0) != cudaSuccess) return fail(EFQ_ERR_CUDA);
            cudaEventDestroy(ev);
            ev = nullptr;
            // output of this chunk: stream_out
            if (cudaMemcpyAsync(static_cast<uint8_t*>(static_cast<void*>(o_host)) + o_off, od, o_head * nh * group,
                                cudaMemcpyDeviceToHost, s_out) != cudaSuccess)
                return EFQ_ERR_CUDA;
        }
    }
    // the status word efq_poll_status() reads takes the aggregate; stream_compute then waits for the last copies,
    // so that synchronising stream_compute alone completes the call
    efq::merge_status_kernel<<<1, 1, 0, s_c>>>(reinterpret_cast<uint32_t*>(ws), agg, 1);
    if (cudaGetLastError() != cudaSuccess) return EFQ_ERR_CUDA;
    if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess) return EFQ_ERR_CUDA;
    if (cudaEventRecord(ev, s_out) != cudaSuccess || cudaStreamWaitEvent(s_c, ev, 0) != cudaSuccess) return fail(EFQ_ERR_CUDA);
    cudaEventDestroy(ev);
    return EFQ_OK;
}

// ------------------------------------------------------------------------------------------------
// Packed variable-length batch: the sequences of the batch lie one after the other along the token axis
// ------------------------------------------------------------------------------------------------
extern "C" size_t efq_attention_varlen_workspace_bytes(const int64_t* cu_seqlens_q, const int64_t* cu_seqlens_k, int n_seqs,
                                                       int Hq, int Hkv, int d)
{
    efq_status_t st;
    efq::VarlenPlan p;
    if (!efq::plan_varlen(cu_seqlens_q, cu_seqlens_k, n_seqs, Hq, Hkv, d, p, st)) return 0;
    return p.total;
}

extern "C" efq_status_t efq_attention_fwd_varlen(const void* q, const void* k, const void* v, float* o,
                                                 const int64_t* cu_seqlens_q, const int64_t* cu_seqlens_k, int n_seqs,
                                                 int Hq, int Hkv, int d, int causal, float softmax_scale, int producer,
                                                 const efq_params_t* params, void* workspace, size_t workspace_bytes,
                                                 void* stream)
{
    using namespace efq;
    float tau, h, threshold;
    bool lut;
    efq_status_t st;
    if (!read_params(params, tau, h, lut, threshold, st)) return st;
    if (producer == 0 && lut) producer = 3;
    if (producer < 0 || producer > 6) return EFQ_ERR_INVALID_ARG;
    VarlenPlan p;
    if (!plan_varlen(cu_seqlens_q, cu_seqlens_k, n_seqs, Hq, Hkv, d, p, st)) return st;
    if (n_seqs == 0 || cu_seqlens_q[n_seqs] == 0) return EFQ_OK;     // no query token: nothing to write
    if (!q || !k || !v || !o) return EFQ_ERR_INVALID_ARG;
    if (!(softmax_scale > 0.0f)) softmax_scale = static_cast<float>(1.0 / sqrt(static_cast<double>(d)));
    if (!isfinite(softmax_scale) || !isfinite(tau) || !isfinite(h) || !(h > 0.0f)) return EFQ_ERR_INVALID_ARG;
    auto mis = [](const void* ptr, uintptr_t a) { return (reinterpret_cast<uintptr_t>(ptr) & (a - 1)) != 0; };
    if (mis(q, 16) || mis(k, 16) || mis(v, 16) || mis(o, 16)) return EFQ_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < p.total) return EFQ_ERR_WORKSPACE;
    if (mis(workspace, 256)) return EFQ_ERR_ALIGNMENT;
    const efq_status_t dev_st = check_device();
    if (dev_st != EFQ_OK) return dev_st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    const int G = Hq / Hkv;

    // host copies of the tables, in the layout of the workspace's table region
    std::vector<uint8_t> tables(p.tables, 0);
    SeqDesc* seqs = reinterpret_cast<SeqDesc*>(tables.data() + (p.seqs_off - 1024));
    ItemDesc* items = reinterpret_cast<ItemDesc*>(tables.data() + (p.items_off - 1024));
    QuantJob* jobs = reinterpret_cast<QuantJob*>(tables.data() + (p.jobs_off - 1024));
    int32_t* prefix = reinterpret_cast<int32_t*>(tables.data() + (p.prefix_off - 1024));
    const __nv_bfloat16* qb = static_cast<const __nv_bfloat16*>(q);
    const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k);
    const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(v);
    int64_t q_row = 0, k_row = 0, k_col = 0, n_items = 0, ctas = 0;
    int a = 0;
    for (int i = 0; i < n_seqs; ++i) {
        const int64_t q0 = cu_seqlens_q[i], k0 = cu_seqlens_k[i];
        const int64_t lq = cu_seqlens_q[i + 1] - q0, lk = cu_seqlens_k[i + 1] - k0;
        if (lq == 0) continue;
        if (lk == 0) {               // no key at all: the rows are zero, as for a causal row that sees nothing
            if (cudaMemsetAsync(o + q0 * Hq * 128, 0, static_cast<size_t>(lq) * Hq * 128 * sizeof(float), s) != cudaSuccess) return EFQ_ERR_CUDA;
            continue;
        }
        const bool packed = use_packed_tile(Hq, Hkv, lq);
        const int64_t lq_pad = packed ? kTile : (lq + kTile - 1) / kTile * kTile, lk_pad = (lk + kTile - 1) / kTile * kTile;
        SeqDesc& sd = seqs[a];
        sd.Sq = lq; sd.Sk = lk; sd.o_off = q0 * Hq * 128;
        sd.q_row0 = static_cast<int32_t>(q_row); sd.Sq_pad = static_cast<int32_t>(lq_pad);
        sd.k_row0 = static_cast<int32_t>(k_row); sd.Sk_pad = static_cast<int32_t>(lk_pad);
        sd.k_col0 = static_cast<int32_t>(k_col); sd.packed = packed ? 1 : 0;
        // work items: heaviest query tiles of a sequence first, the heads of a GQA group adjacent
        if (packed) {
            for (int hk = 0; hk < Hkv; ++hk) items[n_items++] = ItemDesc{a, 0, hk, 0};
        } else {
            for (int64_t qt = lq_pad / kTile - 1; qt >= 0; --qt)
                for (int hh = 0; hh < Hq; ++hh) items[n_items++] = ItemDesc{a, static_cast<int32_t>(qt), hh, 0};
        }
        // quantiser jobs: the sequence's own Q, K, V (token-major source: a head is 128 elements, a token H * 128)
        QuantJob& jq = jobs[3 * a];
        QuantJob& jk = jobs[3 * a + 1];
        QuantJob& jv = jobs[3 * a + 2];
        jq.kind = kQuantRows; jk.kind = kQuantRows; jv.kind = kQuantV;
        jq.seg.src = qb + q0 * Hq * 128;
        jq.seg.heads = packed ? Hkv : Hq; jq.seg.S = packed ? G * lq : lq; jq.seg.S_pad = lq_pad;
        jq.seg.head_stride = 128; jq.seg.row_stride = static_cast<int64_t>(Hq) * 128;
        jq.seg.pack_lq = packed ? static_cast<int32_t>(lq) : 0; jq.seg.pack_G = packed ? G : 1;
        jq.seg.codes = ws + p.qc + q_row * 64; jq.seg.sf = ws + p.qsf + (q_row / kTile) * kSfBytes;
        jk.seg.src = kb + k0 * Hkv * 128;
        jk.seg.heads = Hkv; jk.seg.S = lk; jk.seg.S_pad = lk_pad;
        jk.seg.head_stride = 128; jk.seg.row_stride = static_cast<int64_t>(Hkv) * 128; jk.seg.pack_G = 1;
        jk.seg.codes = ws + p.kc + k_row * 64; jk.seg.sf = ws + p.ksf + (k_row / kTile) * kSfBytes;
        jv.seg = jk.seg;
        jv.seg.src = vb + k0 * Hkv * 128;
        jv.seg.codes = ws + p.vt; jv.seg.sf = ws + p.vsf;
        jv.seg.v_row_bytes = p.k_cols / 2; jv.seg.v_x0 = k_col / 2;
        jv.seg.v_sf_tiles_per_head = p.k_cols / kTile; jv.seg.v_sf_tile0 = k_col / kTile;
        for (int t = 0; t < 3; ++t) {
            prefix[3 * a + t] = static_cast<int32_t>(ctas);
            ctas += quantize_job_ctas(jobs[3 * a + t]);
        }
        q_row += (packed ? Hkv : Hq) * lq_pad;
        k_row += Hkv * lk_pad;
        k_col += lk_pad;
        ++a;
    }
    if (p.n_active == 0)             // nothing to launch: the status word still has to read "no problem"
        return cudaMemsetAsync(ws, 0, 4, s) == cudaSuccess ? EFQ_OK : EFQ_ERR_CUDA;
    prefix[3 * p.n_active] = static_cast<int32_t>(ctas);

    // Pageable host memory: the call returns once the bytes sit in the driver's staging area, so the vector may go.
    if (cudaMemcpyAsync(ws + 1024, tables.data(), p.tables, cudaMemcpyHostToDevice, s) != cudaSuccess) return EFQ_ERR_CUDA;
    if (launch_quantize_jobs(reinterpret_cast<const QuantJob*>(ws + p.jobs_off), reinterpret_cast<const int32_t*>(ws + p.prefix_off),
                             3 * p.n_active, ctas, reinterpret_cast<uint32_t*>(ws), s) != cudaSuccess)
        return EFQ_ERR_CUDA;

    CUtensorMap mq, mk, mv;
    if (!encode_map(&mq, ws + p.qc, 64, static_cast<uint64_t>(p.q_rows))) return EFQ_ERR_CUDA;
    if (!encode_map(&mk, ws + p.kc, 64, static_cast<uint64_t>(p.k_rows))) return EFQ_ERR_CUDA;
    if (!encode_map(&mv, ws + p.vt, static_cast<uint64_t>(p.k_cols / 2), static_cast<uint64_t>(Hkv) * 128)) return EFQ_ERR_CUDA;

    FwdParams P{};
    P.B = p.n_active; P.Hq = Hq; P.Hkv = Hkv; P.Sq = 0; P.Sk = 0; P.Sq_pad = 0; P.Sk_pad = 0;
    P.causal = causal ? 1 : 0;
    P.K = producer == 3 ? make_producer_consts_lut(softmax_scale) : make_producer_consts(softmax_scale, tau, h);
    P.sf_q = ws + p.qsf; P.sf_k = ws + p.ksf; P.sf_v = ws + p.vsf;
    P.o = o;
    P.o_head = 128;                                   // token-major: a head is 128 elements, a token Hq * 128
    P.o_row = static_cast<int64_t>(Hq) * 128;
    P.status = reinterpret_cast<uint32_t*>(ws);
    P.packed = 0;
    P.seqs = reinterpret_cast<const SeqDesc*>(ws + p.seqs_off);
    P.items = reinterpret_cast<const ItemDesc*>(ws + p.items_off);
    P.v_tiles_per_head = p.k_cols / kTile;
    P.inject_skip_loads = 0;
    P.rescale_threshold = threshold;
    P.has_dbg = 0;
    P.dbg = efq_debug_t{};
    return launch_forward(producer, false, needs_fix8(tau, h), n_items, s, mq, mk, mv, P) == cudaSuccess ? EFQ_OK : EFQ_ERR_CUDA;
}

extern "C" efq_status_t efq_poll_status(void* workspace, void* stream)
{
    if (!workspace) return EFQ_ERR_INVALID_ARG;
    uint32_t word = 0;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, workspace, 4, cudaMemcpyDeviceToHost, s) != cudaSuccess) return EFQ_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return EFQ_ERR_CUDA;
    return word == 0 ? EFQ_OK : (word == EFQ_ERR_DEVICE_TIMEOUT ? EFQ_ERR_DEVICE_TIMEOUT : EFQ_ERR_CUDA);
}

// ------------------------------------------------------------------------------------------------
// Forward without a caller-supplied workspace
// ------------------------------------------------------------------------------------------------
// Scratch for efq_attention_fwd_static: lives in the library image, one copy per device that loads it.
static __device__ __align__(256) uint8_t g_static_scratch[EFQ_STATIC_SCRATCH_BYTES];

namespace {

constexpr int kMaxDevices = 64;   // device ordinals this table covers
std::mutex g_static_mutex;
void* g_static_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device ordinal

// The array's name is only a host-side handle; kernels need its device address, which differs per device.
// Looked up once per device with that device current.
efq_status_t static_scratch_for_current_device(void** out)
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return EFQ_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return EFQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return EFQ_ERR_CUDA;
        g_static_ptr[dev] = p;
    }
    *out = g_static_ptr[dev];
    return EFQ_OK;
}

}  // namespace

extern "C" efq_status_t efq_attention_fwd_static(const void* q, const void* k, const void* v, float* o, int B, int Hq,
                                                 int Hkv, int64_t Sq, int64_t Sk, int d, int causal,
                                                 float softmax_scale, const efq_params_t* params, void* stream)
{
    float tau, h, threshold;
    bool lut;
    efq_status_t st;
    if (!read_params(params, tau, h, lut, threshold, st)) return st;
    // the argument rules of efq_attention_fwd, in its order, before the size of the problem is looked at
    if (!q || !k || !v || !o) return EFQ_ERR_INVALID_ARG;
    if (B <= 0 || Hq <= 0 || Hkv <= 0 || Sq <= 0 || Sk <= 0 || Hq % Hkv != 0) return EFQ_ERR_INVALID_ARG;
    if (d != 128) return EFQ_ERR_UNSUPPORTED;
    const size_t need = efq_attention_workspace_bytes(B, Hq, Hkv, Sq, Sk, d);
    if (need == 0) return EFQ_ERR_UNSUPPORTED;
    if (need > EFQ_STATIC_SCRATCH_BYTES) return EFQ_ERR_STATIC_LIMIT;
    void* scratch = nullptr;
    st = static_scratch_for_current_device(&scratch);
    if (st != EFQ_OK) return st;
    return efq::attention_impl(q, k, v, o, B, Hq, Hkv, Sq, Sk, d, causal, softmax_scale, lut ? 3 : 0, tau, h, scratch,
                               EFQ_STATIC_SCRATCH_BYTES, nullptr, static_cast<cudaStream_t>(stream), true, true, false, threshold);
}
