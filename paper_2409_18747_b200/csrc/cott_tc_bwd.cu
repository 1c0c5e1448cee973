// Fused causal backward for d = 64 (bf16 I/O, fp32 accumulation and states): one walk over the
// sequence produces dQ, dK and dV (the three formulas printed after Eq. 7 plus the chain rule
// through the row normalisation and the stabilisation factor of Eq. 4) and the dm sum.
//
// One CTA walks one sequence group forward in time in chunks of 128 tokens.  Per chunk, with
// q^, k^ the rows normalised in shared memory (Eq. 2/3) and M the lower-triangular mask that
// keeps the diagonal (Eq. 6):
//     G   = dO V^T . M                      (128 x 128, scores of the dQ^ and dK^ streams)
//     P   = K^ Q^^T . M^T                   (128 x 128, scores of the dV' stream)
//     dQ^ = G K^   + dO Sq                  Sq = sum over earlier chunks of V^T K^  (d_v x d_k)
//     dK^ = G^T Q^ + V  R^T                 R  = sum over later chunks of Q^^T dO  (d_k x d_v)
//     dV' = P dO   + K^ R
// The paper notes that dK and dV share one cumulative sum that runs backward in time while
// dQ's runs forward.  Here both live in one walk: Sq is accumulated chunk by chunk, and R is
// obtained by taking the sum over the group and everything after it (computed by a
// partial-state pass beforehand) and removing each chunk as the walk passes it.  The two
// updates are one tensor-core product: the 128 x 128 fp32 accumulator [V | Q^]^T [K^ | dO]
// holds Sq in its upper-left block and the accumulated Q^^T dO in its lower-right block, which
// starts at minus the suffix sum, so that block always equals -R (the two other blocks are
// never read).  G is formed once: masked and rounded to bf16 it sits in shared memory, where
// it is the K-major A operand of G K^ and the MN-major A operand of G^T Q^.
//
// Every tensor is read once (q, k, v, dO) and written once (dq, dk, dv): the normalised rows
// and their reciprocal norms, which the chain rule needs, are the tiles the products use.
#include <stdlib.h>
#include "cott_internal.h"
#include "cott_sm100.cuh"
#include "cott_tc_common.cuh"

namespace cott {

using namespace sm100;
using namespace tc;

namespace {

constexpr int kC = 128;                 // tokens per chunk
constexpr int kD = 64;                  // per-head dimension this kernel serves
constexpr int kTile = kC * kD * 2;      // one 128 x 64 bf16 tile
constexpr int kWorkerWarps = 16;        // four worker groups of four warps (one warp per TMEM lane quadrant)
constexpr int kGroupThreads = 128;
constexpr int kThreads = (kWorkerWarps + 4) * 32;   // + score, output, state-update and copy threads

// Shared-memory plan.  A stage holds the four tiles of one chunk; [V | Q] and [K | dO] are
// adjacent pairs, so each pair is one 128-wide MN-major operand of the state update.
struct L {
    static constexpr int kOffV = 0, kOffQ = kTile, kOffK = 2 * kTile, kOffDO = 3 * kTile;
    static constexpr int kStage = 4 * kTile;
    static constexpr int kStages = 2;
    static constexpr int kOffG = kStages * kStage;          // masked scores G, bf16, 128 x 128 (two half tiles)
    static constexpr int kStateTile = kD * kD * 2;           // bf16 copy of one 64 x 64 state
    // bf16 copies of the two states.  R is needed by the chunk whose update has just been applied
    // (the "early" copy: two buffers, chunk parity), Sq by the next chunk (the "late" copy: one
    // buffer).
    static constexpr int kOffLb = kOffG + 2 * kTile;
    static constexpr int kOffEb = kOffLb + kStateTile;
    static constexpr int kOffStQ = kOffEb + 2 * kStateTile;  // staging of the dq rows of a chunk
    static constexpr int kOffStK = kOffStQ + kTile;          // staging of the dk rows
    static constexpr int kOffCtl = kOffStK + kTile;
    // control block: mbarriers (first 512 bytes), tensor-memory slot, abort flag and wait
    // limit, reciprocal row norms of the two stages, dm scratch
    static constexpr int kOffTmemSlot = kCtlTmemSlot, kOffAbort = kCtlAbort;
    static constexpr int kOffRq = 1024;                      // float2 [2][128]: 1 / max(||q||, eps), 1 if not clamped
    static constexpr int kOffRk = kOffRq + 2 * kC * 8;
    static constexpr int kOffDmRed = kOffRk + 2 * kC * 8;    // float [32]
    static constexpr int kCtlBytes = kOffDmRed + 128;
    static constexpr int kDynBytes = kOffCtl + kCtlBytes + 1024;   // + alignment slack
};

struct BwdParams {
    const float* sq_part;    // [BH, n_groups, 64 * 64] partial states V^T K^ of every group but the last, or NULL
    const float* r_part;     // [BH, n_groups, 64 * 64] partial states Q^^T dO of every group
    float* dm_partial;       // [BH, n_groups]
    float* dm_out;           // dm[H]
    int* status;             // workspace status words
    const float* m; const float* seq_len; float seq_len_scalar;
    int H; int N; int group; int n_groups;
    int wait_limit_kcycles;
    int head_first_mask;     // bit i: in tensor map i (q, k, v, dO, dq, dk, dv) the head index comes before the token index
    int no_state;            // the whole sequence is one chunk: both states are zero wherever they are read, no update
    const float* sq_fwd;     // the forward call's partial states K^^T V ([BH, n_groups * split, 64 * 64]) or NULL
    int sq_fwd_split;
    // Packed variable-length batch (VARLEN instances): rows of all sequences back to back, sequence
    // b = rows cu_seqlens[b] .. cu_seqlens[b + 1] - 1, cut into groups from its first row on; the rows
    // of a ragged last chunk leave as plain stores: dq, dk, dv as global memory with their
    // token and head strides in elements.
    const int* cu_seqlens;
    void* out_rows[3]; long long out_sn[3], out_sh[3]; int out_w[3];
    // A segment of a longer causal sequence (all three NULL otherwise), fp32 [BH, 64, 64] in the
    // [key][value] layout of a caller's state: what earlier tokens left in the running state of
    // Eq. 8 (it contains c), the gradient that later tokens send into the state this segment hands
    // on, and where the gradient of state_in goes.  The dm sum is then taken over the value rows,
    // <dV'_j, v_j>, which sees d_state_out and does not see state_in.
    const float* state_in; const float* d_state_out; float* d_state_in;
    int dm_by_v;
};


#ifdef COTT_TIMING
// Debug build only: SM-clock stamps of CTA 0, chunks kStampC0 .. + 3, eight slots for each of
// eight roles (0: worker group A; 1, 2: the two halves of worker group B; 4-7: score, output,
// state, copy threads), each by its first thread.
#ifndef COTT_STAMP_C0
#define COTT_STAMP_C0 4
#endif
__device__ long long g_bwd_stamps[8 * 4 * 8];
__device__ long long g_bwd_cta[256 * 4];   // per CTA: global-timer ns at entry, after the prologue, after the walk, at exit
__device__ __forceinline__ long long gtime_ns() { long long t; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t)); return t; }
#define CSTAMP(slot) do { if (threadIdx.x == 0 && blockIdx.x < 256) g_bwd_cta[blockIdx.x * 4 + (slot)] = gtime_ns(); } while (0)
__device__ long long g_state_stamps[3 * 16 * 4];   // state kernel, CTA 0: role (worker, mma, copy) x chunk x slot
#define SSTAMP(role, cc, slot)                                                                     \
    do {                                                                                           \
        if (blockIdx.x == 0 && (cc) < 16 && ((role) == 0 ? threadIdx.x == 0 : true))              \
            g_state_stamps[((role) * 16 + (cc)) * 4 + (slot)] = clock64();                        \
    } while (0)
#define BSTAMP(role, cc, slot)                                                                     \
    do {                                                                                           \
        if (blockIdx.x == 0 && (cc) >= COTT_STAMP_C0 && (cc) < COTT_STAMP_C0 + 4 &&               \
            ((role) < 3 ? (threadIdx.x == ((role) == 0 ? 0 : ((role) + 1) * 128)) : true))                                   \
            g_bwd_stamps[((role) * 4 + ((cc) - COTT_STAMP_C0)) * 8 + (slot)] = clock64();         \
    } while (0)
#else
#define BSTAMP(role, cc, slot) do {} while (0)
#define CSTAMP(slot) do {} while (0)
#define SSTAMP(role, cc, slot) do {} while (0)
#endif

// K-major operand of 64 columns: K step kk (16 elements) advances the address by 32 bytes.
// K-major operand of 128 columns (two half tiles 16 KB apart): steps 4..7 are in the second half.
// MN-major operand: rows are the contraction index, a K step is 16 rows = 2048 bytes; the
// leading byte offset is the distance between 64-wide blocks of the M / N index.
__device__ __forceinline__ uint32_t kstep128(int kk) { return ((kk >> 2) * 16384u + (kk & 3) * 32u) >> 4; }

// P[128 x 128] = X[128 x 64] A[128 x 64]^T, both K-major.
__device__ __forceinline__ void issue_scores(uint32_t tP, uint32_t x, uint32_t a) {
    constexpr uint32_t idesc = instr_desc_bf16(128, 128, false, false);
    const uint32_t xl = smem_desc_lo(x, 16), al = smem_desc_lo(a, 16);
#pragma unroll
    for (int kk = 0; kk < kD / 16; ++kk) mma_ss_w(tP, xl + kk * 2u, kDescHi, al + kk * 2u, kDescHi, idesc, kk > 0);
}
// Out[128 x 64] = G[128 x 128] B[128 x 64]: G K-major from shared memory, B MN-major.
__device__ __forceinline__ void issue_g_b(uint32_t tO, uint32_t g, uint32_t bt) {
    constexpr uint32_t idesc = instr_desc_bf16(128, kD, false, true);
    const uint32_t gl = smem_desc_lo(g, 16), bl = smem_desc_lo(bt, 16384);
#pragma unroll
    for (int kk = 0; kk < kC / 16; ++kk) mma_ss_w(tO, gl + kstep128(kk), kDescHi, bl + kk * 128u, kDescHi, idesc, kk > 0);
}
// Out[128 x 64] = G^T[128 x 128] B[128 x 64]: G read MN-major (its columns are the M index), B MN-major.
__device__ __forceinline__ void issue_gt_b(uint32_t tO, uint32_t g, uint32_t bt) {
    constexpr uint32_t idesc = instr_desc_bf16(128, kD, true, true);
    const uint32_t gl = smem_desc_lo(g, 16384), bl = smem_desc_lo(bt, 16384);
#pragma unroll
    for (int kk = 0; kk < kC / 16; ++kk) mma_ss_w(tO, gl + kk * 128u, kDescHi, bl + kk * 128u, kDescHi, idesc, kk > 0);
}
// Out[128 x 64] = P~[128 x 128] B[128 x 64]: P~ (bf16, two per column) in tensor memory, B MN-major.
__device__ __forceinline__ void issue_pt_b(uint32_t tO, uint32_t tPt, uint32_t bt) {
    constexpr uint32_t idesc = instr_desc_bf16(128, kD, false, true);
    const uint32_t bl = smem_desc_lo(bt, 16384);
#pragma unroll
    for (int kk = 0; kk < kC / 16; ++kk) mma_ts_w(tO, tPt + kk * 8u, bl + kk * 128u, kDescHi, idesc, kk > 0);
}
// Out[128 x 64] += X[128 x 64] St[64 x 64], St read MN-major (its rows are the contraction index).
__device__ __forceinline__ void issue_x_state(uint32_t tO, uint32_t x, uint32_t st, bool acc_first = true) {
    constexpr uint32_t idesc = instr_desc_bf16(128, kD, false, true);
    const uint32_t xl = smem_desc_lo(x, 16), sl = smem_desc_lo(st, kD * 128u);
#pragma unroll
    for (int kk = 0; kk < kD / 16; ++kk)
        mma_ss_w(tO, xl + kk * 2u, kDescHi, sl + kk * 128u, kDescHi, idesc, (acc_first || kk > 0) ? 1u : 0u);
}
// Out[128 x 64] += X[128 x 64] St^T, St read K-major (its columns are the contraction index).
__device__ __forceinline__ void issue_x_state_t(uint32_t tO, uint32_t x, uint32_t st, bool acc_first = true) {
    constexpr uint32_t idesc = instr_desc_bf16(128, kD, false, false);
    const uint32_t xl = smem_desc_lo(x, 16), sl = smem_desc_lo(st, 16);
#pragma unroll
    for (int kk = 0; kk < kD / 16; ++kk)
        mma_ss_w(tO, xl + kk * 2u, kDescHi, sl + kk * 2u, kDescHi, idesc, (acc_first || kk > 0) ? 1u : 0u);
}
// State[128 x 128] += [V | Q^]^T [K^ | dO]: both operands MN-major, 128 wide (two tiles 16 KB apart).
__device__ __forceinline__ void issue_update(uint32_t tS, uint32_t vq, uint32_t kdo) {
    constexpr uint32_t idesc = instr_desc_bf16(128, 128, true, true);
    const uint32_t al = smem_desc_lo(vq, 16384), bl = smem_desc_lo(kdo, 16384);
#pragma unroll
    for (int kk = 0; kk < kC / 16; ++kk) mma_ss_w(tS, al + kk * 128u, kDescHi, bl + kk * 128u, kDescHi, idesc, 1u);
}

// Thread roles.  Warps 0-15 are row workers (warp w owns TMEM lanes / tile rows
// 32 (w % 4) .. + 31, one row per thread) in two groups of eight, see below.
// Lane 0 of warp 16 issues the score products, of warp 17 the six output products, of warp 18
// the state update, of warp 19 every TMA load and store.  The roles meet only through
// mbarriers, every wait bounded.  Every per-chunk barrier is a pair indexed by chunk parity:
// the two-stage ring keeps all roles within one chunk of each other (the tiles of chunk c + 2
// are requested only after every epilogue of chunk c), so a phase parity names one chunk.
// BIDIR: the bidirectional backward (all-ones mask).  Both states are then totals over the whole
// sequence -- S^T = V^T K^ and R = Q^^T dO, summed in the prologue from the partial states of ALL
// groups -- and every chunk's rows are plain products with them,
//     dQ^ = dO S^T ,   dK^ = V R^T ,   dV' = K^ R ,
// so the score products, the masks, the state update and the per-chunk state copies fall away;
// loads, row norms, epilogues, stores and the dm sum are those of the causal walk.
// SEG: a segment of a longer causal sequence (cott_bwd_stateful): the running states start from
// the caller's, and dm is summed over the value rows.  An instance of its own, so that the plain
// causal walk carries none of it.
template <bool BIDIR, bool VARLEN, bool SEG = false>
__global__ void __launch_bounds__(kThreads, 1)
tc_bwd_fused_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmDO,
                    const __grid_constant__ CUtensorMap tmDQ, const __grid_constant__ CUtensorMap tmDK,
                    const __grid_constant__ CUtensorMap tmDV, BwdParams p) {
    // Tensor-memory columns: State 128 | P1[2] 128 each (G scores; then dQ^ in its columns 0-63
    // and dK^ in 64-127) | P2 128 (P scores; then P~ packed in columns 0-63, dV' in 64-127).
    constexpr uint32_t colS = 0, colP1 = 128, colP2 = 384;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + L::kOffCtl;
    enum { B_FULL = 0, B_NREADY = 16, B_P1FULL = 32, B_P2FULL = 48, B_GREADY = 64, B_PTREADY = 80,
           B_UFULL = 96, B_CEREADY = 112, B_OQFULL = 128, B_OKFULL = 144, B_OVFULL = 160,
           B_EQDONE = 176, B_EKDONE = 192, B_EVDONE = 208, B_OVFREE = 224, B_CLREADY = 240,
           B_STQFREE = 256 /* dq rows read */, B_STKFREE = 264, B_B1READ = 272 /* [4 quadrants][2] */,
           B_STVFREE = 336 /* dv rows read (same tile as dq) */, B_END = 344 };
    auto bar = [&](int which, int c) { return bars + which + 8 * (c & 1); };
    auto par = [&](int c) { return (uint32_t)((c >> 1) & 1); };
    const uint32_t tmem_slot = bars + L::kOffTmemSlot;
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + L::kOffCtl + L::kOffTmemSlot);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kOffCtl + L::kOffAbort);
    float2* rq_buf = reinterpret_cast<float2*>(gbase + L::kOffCtl + L::kOffRq);   // [2][128]
    float2* rk_buf = reinterpret_cast<float2*>(gbase + L::kOffCtl + L::kOffRk);
    float* dm_red = reinterpret_cast<float*>(gbase + L::kOffCtl + L::kOffDmRed);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    CSTAMP(0);
    const int g = blockIdx.x % p.n_groups, bh = blockIdx.x / p.n_groups;
    const int bseq = bh / p.H, h = bh % p.H;
    const int b = VARLEN ? 0 : bseq;                   // batch coordinate of the tensor maps
    // (packed batch: group g of a sequence starts g groups behind its first row and may lie wholly
    // behind its last one -- a CTA with nothing to do)
    const int seq0 = VARLEN ? p.cu_seqlens[bseq] : 0, seq1 = VARLEN ? p.cu_seqlens[bseq + 1] : p.N;
    const int tok0 = seq0 + g * p.group;
    const int tok1 = min(seq1, tok0 + p.group);
    const int n_chunks = tok1 > tok0 ? (tok1 - tok0 + kC - 1) / kC : 0;
    // (a packed batch: the last chunk of a sequence may hold rows of the next one -- they are made
    // inert by normalising them to zero, and that chunk's output rows are stored one by one)
    const bool ragged_last = VARLEN && ((tok1 - tok0) % kC) != 0;
    auto chunk_row = [&](int c) { return tok0 + c * kC; };
    const bool is_score = warp == kWorkerWarps, is_out = warp == kWorkerWarps + 1;
    const bool is_upd = warp == kWorkerWarps + 2, is_copy = warp == kWorkerWarps + 3;

    if (is_score) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(bars + B_FULL + 8 * i, 1);
            mbar_init(bars + B_NREADY + 8 * i, 2 * kGroupThreads);
            mbar_init(bars + B_P1FULL + 8 * i, 1);
            mbar_init(bars + B_P2FULL + 8 * i, 1);
            mbar_init(bars + B_GREADY + 8 * i, 2 * kGroupThreads);
            mbar_init(bars + B_PTREADY + 8 * i, 2 * kGroupThreads);
            mbar_init(bars + B_UFULL + 8 * i, 1);
            mbar_init(bars + B_CEREADY + 8 * i, kGroupThreads);
            mbar_init(bars + B_CLREADY + 8 * i, kGroupThreads);
            mbar_init(bars + B_OQFULL + 8 * i, 1);
            mbar_init(bars + B_OKFULL + 8 * i, 1);
            mbar_init(bars + B_OVFULL + 8 * i, 1);
            mbar_init(bars + B_EQDONE + 8 * i, kGroupThreads);
            mbar_init(bars + B_EKDONE + 8 * i, kGroupThreads);
            mbar_init(bars + B_EVDONE + 8 * i, 2 * kGroupThreads);
            mbar_init(bars + B_OVFREE + 8 * i, 2 * kGroupThreads);
            for (int qq = 0; qq < 4; ++qq) mbar_init(bars + B_B1READ + 16 * qq + 8 * i, 32);
        }
        mbar_init(bars + B_STQFREE, 1);
        mbar_init(bars + B_STKFREE, 1);
        mbar_init(bars + B_STVFREE, 1);
        *abort_flag = 0;
        abort_flag[3] = p.wait_limit_kcycles;
        mbar_fence_init();
        fence_proxy_async();
    }
    if (is_copy && lane == 0) {
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmDO);
        tma_prefetch_desc(&tmDQ); tma_prefetch_desc(&tmDK); tma_prefetch_desc(&tmDV);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_g;
    auto stage = [&](int c) { return base + (uint32_t)(c & 1) * L::kStage; };
    auto stage_g = [&](int c) { return gbase + (c & 1) * L::kStage; };

    // One 128 x 64 tile of tensor map `which` at token row `row` (4-D map: column, then head and
    // token ordered by stride, then batch).
    auto coords = [&](int which, int row, int& c1, int& c2) {
        const bool hf = (p.head_first_mask >> which) & 1;
        c1 = hf ? h : row; c2 = hf ? row : h;
    };
    auto issue_loads = [&](int c) {
        const uint32_t fb = bar(B_FULL, c), st = stage(c);
        const int row = chunk_row(c);
        int c1, c2;
        mbar_expect_tx(fb, 4 * kTile);
        coords(3, row, c1, c2); tma_load_4d(st + L::kOffDO, &tmDO, fb, 0, c1, c2, b);
        coords(2, row, c1, c2); tma_load_4d(st + L::kOffV, &tmV, fb, 0, c1, c2, b);
        coords(0, row, c1, c2); tma_load_4d(st + L::kOffQ, &tmQ, fb, 0, c1, c2, b);
        coords(1, row, c1, c2); tma_load_4d(st + L::kOffK, &tmK, fb, 0, c1, c2, b);
    };
    // The kernels before this one in the stream (the partial-state passes of the same call)
    // write none of q, k, v, dO: the first tiles are requested before the wait for them.
    if (is_copy && lane == 0)
        for (int c = 0; c < 2 && c < n_chunks; ++c) issue_loads(c);
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const float s_b = p.seq_len ? p.seq_len[bseq]
                                : (p.seq_len_scalar > 0.f ? p.seq_len_scalar : (float)(VARLEN ? max(seq1 - seq0, 1) : p.N));
    const float cfac = stab_factor(p.m[h], s_b);

    const int wg = warp >> 2, q4 = warp & 3;
    const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
    const int row = q4 * 32 + lane;               // tile row / TMEM lane of a worker thread

    if (warp < kWorkerWarps) {
        // Initial state: worker group wg fills columns 32 wg .. + 31 of the 128 x 128 accumulator.
        // Rows 0-63, columns 0-63 hold Sq: the sum of the partial states of the groups before
        // this one.  Rows 64-127, columns 64-127 hold minus R: minus the sum over this group
        // and all later ones (the update adds every chunk, so the block is then minus what is
        // left).  The two other blocks are never read and start at zero.
        uint32_t r[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) r[i] = 0u;
        const bool upper = row < 64;
        if (upper == (wg < 2)) {
            float acc[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) acc[i] = 0.f;
            const float* src = upper ? p.sq_part : p.r_part;
            const int g_lo = BIDIR ? 0 : (upper ? 0 : g), g_hi = BIDIR ? p.n_groups : (upper ? g : p.n_groups);
            const size_t off = (size_t)(row & 63) * kD + (size_t)(wg & 1) * 32;
            if (!BIDIR && upper && p.sq_fwd != nullptr) {
                // V^T K^ of the groups before this one is the transpose of what the forward call
                // left: element (row, col) of Sq is element (col, row) of K^^T V.
                const int parts = g * p.sq_fwd_split;
                const float* sf = p.sq_fwd + (size_t)bh * p.n_groups * p.sq_fwd_split * kD * kD + (size_t)(wg & 1) * 32 * kD + (row & 63);
                for (int pp = 0; pp < parts; ++pp) {
                    const float* sg = sf + (size_t)pp * kD * kD;
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc[i] += __ldg(sg + (size_t)i * kD);
                }
            } else if (src != nullptr) {
                for (int gg = g_lo; gg < g_hi; ++gg) {
                    const float* sg = src + ((size_t)bh * p.n_groups + gg) * kD * kD + off;
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        const float4 v = *reinterpret_cast<const float4*>(sg + i);
                        acc[i] += v.x; acc[i + 1] += v.y; acc[i + 2] += v.z; acc[i + 3] += v.w;
                    }
                }
            }
            if constexpr (SEG) {
                // Segment of a longer sequence: Sq starts from the caller's state (its transpose,
                // without the factor c the state carries), R from the gradient of the outgoing state.
                const float* extra = upper ? p.state_in : p.d_state_out;
                if (extra != nullptr) {
                    const float* eb = extra + (size_t)bh * kD * kD;
                    const float f = upper ? 1.0f / cfac : 1.0f;
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        const int col = (wg & 1) * 32 + i;
                        // upper: Sq[row = value index][col = key index] = state_in[col][row] / c;
                        // lower: R[row = key index][col = value index] = d_state_out[row][col]
                        acc[i] += f * (upper ? __ldg(eb + (size_t)col * kD + (row & 63)) : __ldg(eb + (size_t)(row & 63) * kD + col));
                    }
                }
                // the first group's R is the sum over the whole segment plus d_state_out: d_state_in
                if (!upper && g == 0 && p.d_state_in != nullptr) {
                    float* db = p.d_state_in + (size_t)bh * kD * kD + (size_t)(row & 63) * kD + (wg & 1) * 32;
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        *reinterpret_cast<float4*>(db + i) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
                }
            }
            if (BIDIR && g == 0) {
                // dm of the bidirectional case needs no row sums at all: sum_i <q^_i, dO_i S^T> is
                // the element-wise product of the two totals, <S, R>, formed here in fp32 from the
                // partial states -- none of the bf16 roundings of the walk enters it.  The upper
                // threads hold S^T (row b, 32 columns a), the lower ones R (row a, 32 columns b):
                // S^T crosses over through the output staging tiles (unused until the first
                // epilogue), rows padded to 65 words so that neither side has bank conflicts.
                float* sT = reinterpret_cast<float*>(gbase + L::kOffStQ);
                if (upper) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) sT[row * 65 + (wg & 1) * 32 + i] = acc[i];
                }
                asm volatile("bar.sync 1, 256;" ::: "memory");
                if (!upper) {
                    float t = 0.f;
                    const int a_ = row & 63, b0 = (wg & 1) * 32;
#pragma unroll
                    for (int i = 0; i < 32; ++i) t = fmaf(acc[i], sT[(b0 + i) * 65 + a_], t);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
                    if (lane == 0) dm_red[4 + (wg & 1) * 2 + (q4 & 1)] = t;
                }
            } else if (BIDIR && !upper && lane == 0) {
                dm_red[4 + (wg & 1) * 2 + (q4 & 1)] = 0.f;
            }
            if (upper || BIDIR) {
                // Sq is what the first chunk reads before any update: its bf16 copy goes to the
                // late-copy buffer.  (Bidirectional: both totals are copied here, once: S^T to
                // the late-copy buffer, R to the first early-copy buffer.)
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(acc[i]);
                uint8_t* dst = gbase + (upper ? L::kOffLb : L::kOffEb);
#pragma unroll
                for (int i = 0; i < 32; i += 8)
                    *reinterpret_cast<uint4*>(dst + swz(row & 63, (uint32_t)((wg & 1) * 4 + (i >> 3)))) = pack8(&r[i]);
            } else {
#pragma unroll
                for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(-acc[i]);
            }
        }
        if (!BIDIR) {
            tmem_st32(tmem + lane_base + colS + wg * 32, r);
            tmem_wait_st();
        }
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    float dm_acc = 0.f;
    CSTAMP(1);

    if (is_copy) {
        // ------------------------------------------------------------------ copy thread
        // Stores each output tile as soon as its epilogue has staged it, and refills the stage as
        // soon as it has been read: v and dO when the chunk's last products have completed, q
        // and k when their epilogues (which read the normalised rows) are done as well.  The dq
        // staging tile takes the dv rows of the same chunk once the dq store has read it, so the
        // stage itself never waits for a store.
        if (lane == 0 && n_chunks > 0) {
            for (int c = 0; c < n_chunks; ++c) {
                const uint32_t st = stage(c);
                const int trow = chunk_row(c);
                const bool more = c + 2 < n_chunks;
                const uint32_t fb = bar(B_FULL, c);      // (same barrier for chunk c + 2)
                const int nrow = chunk_row(c + 2);
                int c1, c2;
                if (!wait_or_abort(bar(B_EQDONE, c), par(c), abort_flag)) break;
                BSTAMP(7, c, 0);
                const bool by_rows = ragged_last && c == n_chunks - 1;      // the workers stored this chunk's rows themselves
                if (!by_rows) { coords(4, trow, c1, c2); tma_store_4d(&tmDQ, base + L::kOffStQ, 0, c1, c2, b); }
                tma_store_commit();
                tma_store_wait_read0();
                mbar_arrive(bars + B_STQFREE);           // the tile may take the dv rows of the chunk
                if (more) {
                    if (!wait_or_abort(bar(B_OVFULL, c), par(c), abort_flag)) break;
                    if (!BIDIR && !wait_or_abort(bar(B_UFULL, c), par(c), abort_flag)) break;
                    mbar_expect_tx(fb, 4 * kTile);
                    coords(3, nrow, c1, c2); tma_load_4d(st + L::kOffDO, &tmDO, fb, 0, c1, c2, b);
                    // (dm over the value rows: the dV epilogue still reads the v tile)
                    if (!SEG) { coords(2, nrow, c1, c2); tma_load_4d(st + L::kOffV, &tmV, fb, 0, c1, c2, b); }
                    coords(0, nrow, c1, c2); tma_load_4d(st + L::kOffQ, &tmQ, fb, 0, c1, c2, b);
                    BSTAMP(7, c, 1);
                }
                if (!wait_or_abort(bar(B_EKDONE, c), par(c), abort_flag)) break;
                if (!by_rows) { coords(5, trow, c1, c2); tma_store_4d(&tmDK, base + L::kOffStK, 0, c1, c2, b); }
                tma_store_commit();
                if (more) { coords(1, nrow, c1, c2); tma_load_4d(st + L::kOffK, &tmK, fb, 0, c1, c2, b); }
                BSTAMP(7, c, 2);
                if (!wait_or_abort(bar(B_EVDONE, c), par(c), abort_flag)) break;
                if (more && SEG) { coords(2, nrow, c1, c2); tma_load_4d(st + L::kOffV, &tmV, fb, 0, c1, c2, b); }
                if (!by_rows) { coords(6, trow, c1, c2); tma_store_4d(&tmDV, base + L::kOffStQ, 0, c1, c2, b); }
                tma_store_commit();
                tma_store_wait_read1();
                mbar_arrive(bars + B_STKFREE);
                tma_store_wait_read0();
                mbar_arrive(bars + B_STVFREE);           // the tile may take the dq rows of the next chunk
                BSTAMP(7, c, 3);
            }
            tma_store_wait_all0();
        }
    } else if (is_score) {
        // ------------------------------------------------------------------ score thread
        if (lane == 0 && !BIDIR) {
            for (int c = 0; c < n_chunks; ++c) {
                const uint32_t st = stage(c);
                if (!wait_or_abort(bar(B_FULL, c), par(c), abort_flag)) break;
                BSTAMP(4, c, 0);
                // (the score columns of this parity were drained by the epilogues of chunk
                // c - 2, which the request for this chunk's tiles waited for)
                tc_fence_after();
                issue_scores(tmem + colP1 + (c & 1) * 128, st + L::kOffDO, st + L::kOffV);
                tc_commit(bar(B_P1FULL, c));
                BSTAMP(4, c, 1);
                if (!wait_or_abort(bar(B_NREADY, c), par(c), abort_flag)) break;
                BSTAMP(4, c, 2);
                if (c >= 1 && !wait_or_abort(bar(B_OVFREE, c - 1), par(c - 1), abort_flag)) break;
                BSTAMP(4, c, 3);
                tc_fence_after();
                issue_scores(tmem + colP2, st + L::kOffK, st + L::kOffQ);
                tc_commit(bar(B_P2FULL, c));
                BSTAMP(4, c, 4);
            }
        }
    } else if (is_upd) {
        // ------------------------------------------------------------------ state-update thread
        if (lane == 0 && !BIDIR) {
            for (int c = 0; c < n_chunks; ++c) {
                const uint32_t st = stage(c);
                if (!wait_or_abort(bar(B_NREADY, c), par(c), abort_flag)) break;
                // the workers have copied the state the previous update left
                BSTAMP(6, c, 0);
                if (c >= 1 && !wait_or_abort(bar(B_CEREADY, c - 1), par(c - 1), abort_flag)) break;
                if (c >= 1 && !wait_or_abort(bar(B_CLREADY, c - 1), par(c - 1), abort_flag)) break;
                BSTAMP(6, c, 1);
                tc_fence_after();
                if (!p.no_state) issue_update(tmem + colS, st + L::kOffV, st + L::kOffK);
                tc_commit(bar(B_UFULL, c));
                BSTAMP(6, c, 2);
            }
        }
    } else if (is_out) {
        // ------------------------------------------------------------------ output-product thread
        if (lane == 0 && BIDIR) {
            // every chunk: three products of its rows with the two totals
            const uint32_t st_t = base + L::kOffLb, rt = base + L::kOffEb;
            for (int c = 0; c < n_chunks; ++c) {
                const uint32_t st = stage(c);
                const uint32_t tP1 = tmem + colP1 + (c & 1) * 128;
                if (!wait_or_abort(bar(B_NREADY, c), par(c), abort_flag)) break;
                // (the accumulators of this parity were drained by the epilogues of chunk c - 2,
                // which the request for this chunk's tiles waited for)
                tc_fence_after();
                issue_x_state(tP1, st + L::kOffDO, st_t, false);          // dQ^ = dO S^T
                tc_commit(bar(B_OQFULL, c));
                issue_x_state_t(tP1 + 64, st + L::kOffV, rt, false);      // dK^ = V R^T
                tc_commit(bar(B_OKFULL, c));
                // the one dV' accumulator: drained by the epilogue of the chunk before
                if (c >= 1 && !wait_or_abort(bar(B_OVFREE, c - 1), par(c - 1), abort_flag)) break;
                tc_fence_after();
                issue_x_state(tmem + colP2 + 64, st + L::kOffK, rt, false);   // dV' = K^ R
                tc_commit(bar(B_OVFULL, c));
            }
        }
        if (lane == 0 && !BIDIR) {
            const uint32_t gt = base + L::kOffG;
            for (int c = 0; c < n_chunks; ++c) {
                const uint32_t st = stage(c);
                const uint32_t tP1 = tmem + colP1 + (c & 1) * 128;
                BSTAMP(5, c, 0);
                if (!wait_or_abort(bar(B_GREADY, c), par(c), abort_flag)) break;
                BSTAMP(5, c, 1);
                if (!wait_or_abort(bar(B_NREADY, c), par(c), abort_flag)) break;
                // dQ^ reads the copy of Sq made after the previous chunk's update (chunk 0: the
                // prologue's); dK^ and dV' need R after this chunk's own update.
                const uint32_t late = base + L::kOffLb, early = base + L::kOffEb + (c & 1) * L::kStateTile;
                if (c >= 1 && !wait_or_abort(bar(B_CLREADY, c - 1), par(c - 1), abort_flag)) break;
                tc_fence_after();
                issue_g_b(tP1, gt, st + L::kOffK);
                issue_x_state(tP1, st + L::kOffDO, late);
                tc_commit(bar(B_OQFULL, c));
                BSTAMP(5, c, 2);
                if (!wait_or_abort(bar(B_CEREADY, c), par(c), abort_flag)) break;
                BSTAMP(5, c, 3);
                tc_fence_after();
                issue_gt_b(tP1 + 64, gt, st + L::kOffQ);
                issue_x_state_t(tP1 + 64, st + L::kOffV, early);
                tc_commit(bar(B_OKFULL, c));
                BSTAMP(5, c, 4);
                if (!wait_or_abort(bar(B_PTREADY, c), par(c), abort_flag)) break;
                BSTAMP(5, c, 5);
                tc_fence_after();
                issue_pt_b(tmem + colP2 + 64, tmem + colP2, st + L::kOffDO);
                issue_x_state(tmem + colP2 + 64, st + L::kOffK, early);
                tc_commit(bar(B_OVFULL, c));
                BSTAMP(5, c, 6);
            }
        }
    } else {
        // ------------------------------------------------------------------ row workers
        // Two groups of eight warps, each running ONE sequence of jobs per chunk (few distinct
        // instruction streams on the SM at a time: the roles share its instruction caches).  A
        // warp has a TMEM lane quadrant q4 and a half hw: lanes / rows 32 q4 .. + 31, and one
        // half of whatever the job splits in two.
        //   group A (warps 0-7):  mask of G, bf16 state copies, mask of P, row norms of the next
        //                         chunk (hw 0: the q tile, hw 1: the k tile);
        //   group B (warps 8-15): projection epilogue (hw 0: dQ, hw 1: dK), then half of the
        //                         dV epilogue each.
        bool alive = n_chunks > 0;
        auto wait = [&](uint32_t bar_, uint32_t parity) {
            if (alive && !wait_or_abort(bar_, parity, abort_flag)) alive = false;
            return alive;
        };
        const int w8 = warp & 7, hw = w8 >> 2;
        if (warp < 8) {
            // -------------------------------------------------------------- group A
            // x^ = x / max(||x||, eps) on this thread's row of its tile, in place; leaves
            // (1 / max(||x||, eps), 1 if not clamped) for the projection epilogue.
            auto normalise = [&](int c) {
                if (tid == 0) BSTAMP(3, c, 0);
                if (!wait(bar(B_FULL, c), par(c))) return;
                if (tid == 0) BSTAMP(3, c, 1);
                uint8_t* tile = stage_g(c) + (hw == 0 ? L::kOffQ : L::kOffK);
                uint4 w[8];
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                for (int j = 0; j < 8; ++j) w[j] = *reinterpret_cast<const uint4*>(tile + swz(row, j));
#pragma unroll
                for (int j = 0; j < 8; j += 2) {
                    const __nv_bfloat162* e0 = reinterpret_cast<const __nv_bfloat162*>(&w[j]);
                    const __nv_bfloat162* e1 = reinterpret_cast<const __nv_bfloat162*>(&w[j + 1]);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 f0 = __bfloat1622float2(e0[i]), f1 = __bfloat1622float2(e1[i]);
                        a0 = fmaf(f0.x, f0.x, a0); a1 = fmaf(f0.y, f0.y, a1);
                        a2 = fmaf(f1.x, f1.x, a2); a3 = fmaf(f1.y, f1.y, a3);
                    }
                }
                const float nrm = sqrtf((a0 + a1) + (a2 + a3));
                float rn = 1.0f / fmaxf(nrm, kEps);
                if (VARLEN && chunk_row(c) + row >= tok1) rn = 0.f;      // a row of the next sequence
                // x * rn in packed bf16 arithmetic with the scale split in two bf16 terms
                // (rn = hi + lo to 2^-17): round(x hi + round(x lo)) is x rn rounded once, up to a
                // second rounding of the small term -- two instructions per pair of elements
                // instead of unpacking, two multiplies and a conversion.
                const __nv_bfloat16 hi = __float2bfloat16_rn(rn);
                const __nv_bfloat16 lo = __float2bfloat16_rn(rn - __bfloat162float(hi));
                const __nv_bfloat162 hi2 = __halves2bfloat162(hi, hi), lo2 = __halves2bfloat162(lo, lo);
                // Bidirectional: what the rounding of x^ to bf16 drops, x rn - x^, goes to the
                // (unused) score buffer as 7-bit fixed point, for the first-order correction of dm in
                // the projection epilogue: units of 2^-15 (|x rn - x^| <= 2^-9 since |x^| <= 1),
                // formed in packed bf16 arithmetic as well (x hi - x^ is a difference of close
                // values, exact before its one rounding).  In bf16, r + 192 = 128 + (r + 64) for
                // |r| <= 63, so the low byte of the sum is r + 64.
                uint8_t* res = gbase + L::kOffG + (c & 1) * 16384 + hw * 8192 + row * 64;
                const __nv_bfloat16 sc15 = __float2bfloat16_rn(32768.f);
                const __nv_bfloat162 hi2s = __hmul2(hi2, __halves2bfloat162(sc15, sc15)), lo2s = __hmul2(lo2, __halves2bfloat162(sc15, sc15));
                const __nv_bfloat162 nsc = __halves2bfloat162(__float2bfloat16_rn(-32768.f), __float2bfloat16_rn(-32768.f));
                const __nv_bfloat162 c63 = __halves2bfloat162(__float2bfloat16_rn(63.f), __float2bfloat16_rn(63.f));
                const __nv_bfloat162 c192 = __halves2bfloat162(__float2bfloat16_rn(192.f), __float2bfloat16_rn(192.f));
                uint32_t rb[4];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    __nv_bfloat162* e = reinterpret_cast<__nv_bfloat162*>(&w[j]);
                    uint32_t t[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const __nv_bfloat162 x = e[i];
                        e[i] = __hfma2(x, hi2, __hmul2(x, lo2));
                        if (BIDIR) {
                            __nv_bfloat162 r = __hfma2(x, lo2s, __hfma2(x, hi2s, __hmul2(e[i], nsc)));
                            r = __hadd2(__hmin2(__hmax2(r, __hneg2(c63)), c63), c192);
                            t[i] = *reinterpret_cast<const uint32_t*>(&r);
                        }
                    }
                    *reinterpret_cast<uint4*>(tile + swz(row, j)) = w[j];
                    if (BIDIR) {
                        rb[(j & 1) * 2] = __byte_perm(t[0], t[1], 0x6420);
                        rb[(j & 1) * 2 + 1] = __byte_perm(t[2], t[3], 0x6420);
                        if (j & 1)
                            *reinterpret_cast<uint4*>(res + ((((j >> 1) ^ (row >> 1)) & 3) << 4)) = make_uint4(rb[0], rb[1], rb[2], rb[3]);
                    }
                }
                (hw == 0 ? rq_buf : rk_buf)[(c & 1) * kC + row] = make_float2(rn, nrm > kEps ? 1.f : 0.f);
                fence_proxy_async();
                mbar_arrive(bar(B_NREADY, c));
                if (tid == 0) BSTAMP(3, c, 2);
            };
            normalise(0);
            if (BIDIR) {
                for (int c = 1; c < n_chunks && alive; ++c) normalise(c);
            }
            for (int c = 0; !BIDIR && c < n_chunks && alive; ++c) {
                // ---- G[i][j] = dO_i . v_j, kept for j <= i (diagonal kept, Eq. 6), rounded to bf16,
                // into shared memory; this warp's half: column blocks 2 hw and 2 hw + 1.  Per
                // 32 x 32 block (row block q4, column block cb) the mask is all-keep, all-zero or
                // a triangle; the first two are warp-uniform branches (a per-lane condition around
                // every element would diverge).  G is free once the products of the previous chunk
                // that read it have completed.
                if (c >= 1 && !(wait(bar(B_OQFULL, c - 1), par(c - 1)) && wait(bar(B_OKFULL, c - 1), par(c - 1)))) break;
                BSTAMP(0, c, 0);
                if (!wait(bar(B_P1FULL, c), par(c))) break;
                BSTAMP(0, c, 1);
                tc_fence_after();
#pragma unroll
                for (int hb = 0; hb < 2; ++hb) {
                    const int cb = 2 * hw + hb;
                    uint8_t* gdst = gbase + L::kOffG + hw * 16384;
                    if (cb <= q4) {                      // warp-uniform
                        uint32_t r[32];
                        tmem_ld32(tmem + lane_base + colP1 + (c & 1) * 128 + cb * 32, r);
                        tmem_wait_ld();
                        if (cb == q4) {                  // the diagonal block: a triangle
#pragma unroll
                            for (int j = 0; j < 32; ++j) r[j] = (j <= lane) ? r[j] : 0u;
                        }
#pragma unroll
                        for (int i = 0; i < 32; i += 8)
                            *reinterpret_cast<uint4*>(gdst + swz(row, hb * 4 + (i >> 3))) = pack8(&r[i]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 4; ++i)
                            *reinterpret_cast<uint4*>(gdst + swz(row, hb * 4 + i)) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
                fence_proxy_async();
                tc_fence_before();
                mbar_arrive(bar(B_GREADY, c));
                BSTAMP(0, c, 2);
                // ---- bf16 copy of R after this chunk's update (rows 64-127 hold minus it), which
                // this chunk's V R^T and K^ R need; this warp's half: 32 columns.
                if (!wait(bar(B_UFULL, c), par(c))) break;
                BSTAMP(0, c, 3);
                if (row >= 64) {
                    tc_fence_after();
                    uint32_t s2[32];
                    tmem_ld32(tmem + lane_base + colS + 64 + hw * 32, s2);
                    tmem_wait_ld();
                    uint8_t* dst = gbase + L::kOffEb + (c & 1) * L::kStateTile;
#pragma unroll
                    for (int i = 0; i < 32; ++i) s2[i] ^= 0x80000000u;
#pragma unroll
                    for (int i = 0; i < 32; i += 8)
                        *reinterpret_cast<uint4*>(dst + swz(row & 63, hw * 4 + (i >> 3))) = pack8(&s2[i]);
                    fence_proxy_async();
                    tc_fence_before();
                    mbar_arrive(bar(B_CEREADY, c));
                }
                BSTAMP(0, c, 4);
                // ---- P[j][i] = k^_j . q^_i, kept for i >= j, rounded to bf16 and packed two per
                // column over the start of the score columns themselves: packed block cb lands
                // in columns 16 cb .. + 15, i.e. blocks 0, 1 inside fp32 block 0 and blocks 2, 3
                // inside fp32 block 1.  The hw = 0 warp reads fp32 blocks 0 and 1 before it
                // writes; the hw = 1 warp (fp32 blocks 2, 3) writes into block 1 and therefore
                // waits until its sibling has read it.
                if (!wait(bar(B_P2FULL, c), par(c))) break;
                BSTAMP(0, c, 5);
                tc_fence_after();
                {
                    const uint32_t sib = bars + B_B1READ + 16 * q4 + 8 * (c & 1);
                    if (hw == 1 && !wait(sib, par(c))) break;
                    uint32_t pk[2][16];
#pragma unroll
                    for (int hb = 0; hb < 2; ++hb) {
                        const int cb = 2 * hw + hb;
                        if (cb >= q4) {                  // warp-uniform
                            uint32_t r[32];
                            tmem_ld32(tmem + lane_base + colP2 + cb * 32, r);
                            tmem_wait_ld();
                            if (cb == q4) {
#pragma unroll
                                for (int j = 0; j < 32; ++j) r[j] = (j >= lane) ? r[j] : 0u;
                            }
#pragma unroll
                            for (int j = 0; j < 16; ++j) pk[hb][j] = pack_bf16(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
                        } else {
#pragma unroll
                            for (int j = 0; j < 16; ++j) pk[hb][j] = 0u;
                        }
                    }
                    // (both fp32 blocks of this warp have been read -- or need not be: now the
                    // sibling may write into block 1, and this warp into blocks 0 / 1)
                    if (hw == 0) { tc_fence_before(); mbar_arrive(sib); }
                    tmem_st16(tmem + lane_base + colP2 + hw * 32, pk[0]);
                    tmem_st16(tmem + lane_base + colP2 + hw * 32 + 16, pk[1]);
                    tmem_wait_st();
                }
                tc_fence_before();
                mbar_arrive(bar(B_PTREADY, c));
                BSTAMP(0, c, 6);
                // ---- row norms of the next chunk
                if (c + 1 < n_chunks) normalise(c + 1);
                BSTAMP(0, c, 7);
                // ---- bf16 copy of Sq (rows 0-63) for the next chunk's dO Sq.  One buffer: the
                // product of this chunk that reads the previous copy must have completed.
                if (row < 64 && alive) {
                    if (!wait(bar(B_OQFULL, c), par(c))) break;
                    tc_fence_after();
                    uint32_t s2[32];
                    tmem_ld32(tmem + lane_base + colS + hw * 32, s2);
                    tmem_wait_ld();
                    uint8_t* dst = gbase + L::kOffLb;
#pragma unroll
                    for (int i = 0; i < 32; i += 8)
                        *reinterpret_cast<uint4*>(dst + swz(row & 63, hw * 4 + (i >> 3))) = pack8(&s2[i]);
                    fence_proxy_async();
                    tc_fence_before();
                    mbar_arrive(bar(B_CLREADY, c));
                }
            }
        } else {
            // -------------------------------------------------------------- group B
            const bool isq = hw == 0;
            const int off_tile = isq ? L::kOffQ : L::kOffK;
            const float2* rn_buf = isq ? rq_buf : rk_buf;
            uint8_t* out_tile = gbase + (isq ? L::kOffStQ : L::kOffStK);
            const uint32_t free_bar = bars + (isq ? B_STVFREE : B_STKFREE);
            for (int c = 0; c < n_chunks && alive; ++c) {
                // ---- projection epilogue (chain rule through x^ = x / max(||x||, eps)): with a
                // the fp32 accumulator row, x^ the normalised row and rn = (1 / max(||x||, eps),
                // 1 if not clamped):   out = c rn.x (a - x^ <x^, a> rn.y),  bf16, into the
                // output's staging tile (free once the store of the previous chunk has read it).
                BSTAMP(1 + hw, c, 0);
                if (!wait(bar(isq ? B_OQFULL : B_OKFULL, c), par(c))) break;
                // (the dq tile also takes the dv rows of every chunk: the store of dv of chunk
                // c - 1 must have read it)
                if (c >= 1 && !wait(free_bar, (uint32_t)((c - 1) & 1))) break;
                BSTAMP(1 + hw, c, 1);
                tc_fence_after();
                {
                    // Two sweeps over the accumulator row: holding all of it next to the tile
                    // chunks does not fit the register budget (and a single spilled value in this
                    // loop costs more than the second round trip to tensor memory).
                    const uint32_t tacc = tmem + lane_base + colP1 + (c & 1) * 128 + (isq ? 0 : 64);
                    const uint8_t* tile = stage_g(c) + off_tile;
                    const float2 rn = rn_buf[(c & 1) * kC + row];
                    const uint8_t* res = gbase + L::kOffG + (c & 1) * 16384 + hw * 8192 + row * 64;
                    float d0 = 0.f, d1 = 0.f;
                    __nv_bfloat162 ec[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) ec[i] = __halves2bfloat162(__float2bfloat16_rn(0.f), __float2bfloat16_rn(0.f));
#pragma unroll 1
                    for (int hf = 0; hf < 2; ++hf) {
                        uint32_t a[32];
                        tmem_ld32(tacc + hf * 32, a);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint4 w = *reinterpret_cast<const uint4*>(tile + swz(row, hf * 4 + j));
                            const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 f = __bfloat1622float2(e[i]);
                                d0 = fmaf(f.x, __uint_as_float(a[8 * j + 2 * i]), d0);
                                d1 = fmaf(f.y, __uint_as_float(a[8 * j + 2 * i + 1]), d1);
                            }
                            if (BIDIR) {
                                // <x rn - x^, a>: the part of <x^, a> that the bf16 rounding of x^ lost,
                                // in packed bf16 arithmetic (a correction: one percent of it is plenty).
                                // Byte m of the residuals next to 0x43 is the bf16 number 128 + m.
                                const uint2 rw = *reinterpret_cast<const uint2*>(res + ((((hf * 2 + (j >> 1)) ^ (row >> 1)) & 3) << 4) + (j & 1) * 8);
                                const __nv_bfloat162 c192 = __halves2bfloat162(__float2bfloat16_rn(192.f), __float2bfloat16_rn(192.f));
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const uint32_t word = i < 2 ? rw.x : rw.y;
                                    const uint32_t pr = __byte_perm(word, 0x43434343u, (i & 1) ? 0x4342 : 0x4140);
                                    const __nv_bfloat162 r = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&pr), c192);
                                    const __nv_bfloat162 ab = __floats2bfloat162_rn(__uint_as_float(a[8 * j + 2 * i]), __uint_as_float(a[8 * j + 2 * i + 1]));
                                    ec[i] = __hfma2(r, ab, ec[i]);
                                }
                            }
                        }
                    }
                    float dot = d0 + d1;
                    if (BIDIR) {
                        // dm = <S, R> (formed in the prologue) + sum_i <dq^_i, dQ^_i> + sum_j <dk^_j, dK^_j>,
                        // dx^ the rounding residuals: exact to second order in the bf16 roundings.
                        const float2 s01 = __bfloat1622float2(__hadd2(ec[0], ec[1])), s23 = __bfloat1622float2(__hadd2(ec[2], ec[3]));
                        const float corr = ((s01.x + s01.y) + (s23.x + s23.y)) * (1.f / 32768.f);
                        dm_acc += corr;
                        dot += corr;
                    } else if (isq && !SEG) {
                        dm_acc += dot;    // <q^_i, dQ^_i> of the unscaled accumulator (rows past N are zero)
                    }
                    // out = sc (a - coef x^), rounded to bf16 once
                    const float sc = cfac * rn.x, mc = -(dot * rn.y) * sc;
#pragma unroll 1
                    for (int hf = 0; hf < 2; ++hf) {
                        uint32_t a[32];
                        tmem_ld32(tacc + hf * 32, a);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint4 w = *reinterpret_cast<const uint4*>(tile + swz(row, hf * 4 + j));
                            const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w);
                            uint4 o;
                            uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 f = __bfloat1622float2(e[i]);
                                ow[i] = pack_bf16(fmaf(f.x, mc, __uint_as_float(a[8 * j + 2 * i]) * sc),
                                                  fmaf(f.y, mc, __uint_as_float(a[8 * j + 2 * i + 1]) * sc));
                            }
                            if (VARLEN && ragged_last && c == n_chunks - 1) {
                                const long long grow = (long long)chunk_row(c) + row;
                                if (grow < tok1 && (hf * 4 + j) * 8 < p.out_w[hw])
                                    *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out_rows[hw]) + grow * p.out_sn[hw] +
                                                              (long long)h * p.out_sh[hw] + (hf * 4 + j) * 8) = o;
                            } else {
                                *reinterpret_cast<uint4*>(out_tile + swz(row, hf * 4 + j)) = o;
                            }
                        }
                    }
                }
                fence_proxy_async();
                tc_fence_before();
                mbar_arrive(bar(isq ? B_EQDONE : B_EKDONE, c));
                BSTAMP(1 + hw, c, 2);
                // ---- dV epilogue, this warp's half of the columns: c dV', bf16, into the dq staging
                // tile once the store of this chunk's dq rows has read it.
                if (!wait(bar(B_OVFULL, c), par(c))) break;
                BSTAMP(1 + hw, c, 3);
                if (!wait(bars + B_STQFREE, (uint32_t)(c & 1))) break;
                tc_fence_after();
                {
                    uint32_t a[32];
                    tmem_ld32(tmem + lane_base + colP2 + 64 + hw * 32, a);
                    tmem_wait_ld();
                    tc_fence_before();
                    mbar_arrive(bar(B_OVFREE, c));     // the P columns may take the next chunk's scores
                    uint8_t* tile = gbase + L::kOffStQ;
                    if (SEG && (long long)chunk_row(c) + row < tok1) {
                        // dm of a segment: <dV'_j, v_j> of the unscaled accumulator with the raw v row
                        // (the copy thread keeps the v tile until this epilogue is done)
                        const uint8_t* vt = stage_g(c) + L::kOffV;
                        float t0 = 0.f, t1 = 0.f;
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint4 w = *reinterpret_cast<const uint4*>(vt + swz(row, hw * 4 + j));
                            const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float2 f = __bfloat1622float2(e[i]);
                                t0 = fmaf(f.x, __uint_as_float(a[8 * j + 2 * i]), t0);
                                t1 = fmaf(f.y, __uint_as_float(a[8 * j + 2 * i + 1]), t1);
                            }
                        }
                        dm_acc += t0 + t1;
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(a[8 * j]) * cfac, __uint_as_float(a[8 * j + 1]) * cfac);
                        o.y = pack_bf16(__uint_as_float(a[8 * j + 2]) * cfac, __uint_as_float(a[8 * j + 3]) * cfac);
                        o.z = pack_bf16(__uint_as_float(a[8 * j + 4]) * cfac, __uint_as_float(a[8 * j + 5]) * cfac);
                        o.w = pack_bf16(__uint_as_float(a[8 * j + 6]) * cfac, __uint_as_float(a[8 * j + 7]) * cfac);
                        if (VARLEN && ragged_last && c == n_chunks - 1) {
                            const long long grow = (long long)chunk_row(c) + row;
                            if (grow < tok1 && (hw * 4 + j) * 8 < p.out_w[2])
                                *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out_rows[2]) + grow * p.out_sn[2] +
                                                          (long long)h * p.out_sh[2] + (hw * 4 + j) * 8) = o;
                        } else {
                            *reinterpret_cast<uint4*>(tile + swz(row, hw * 4 + j)) = o;
                        }
                    }
                }
                fence_proxy_async();
                mbar_arrive(bar(B_EVDONE, c));
                BSTAMP(1 + hw, c, 4);
            }
            if (isq || BIDIR || SEG) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) dm_acc += __shfl_xor_sync(0xffffffffu, dm_acc, o);
                if (lane == 0) dm_red[(isq ? 0 : 12) + q4] = dm_acc;
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    CSTAMP(2);
    {
        int* last_flag = reinterpret_cast<int*>(&dm_red[8]);
        if (tid == 0) {
            // Fixed-order reduction of the CTA's dm term.
            if (!*abort_flag)
                p.dm_partial[(size_t)bh * p.n_groups + g] = BIDIR ? ((dm_red[4] + dm_red[5]) + (dm_red[6] + dm_red[7])) +
                                                                          (((dm_red[0] + dm_red[1]) + (dm_red[2] + dm_red[3])) +
                                                                           ((dm_red[12] + dm_red[13]) + (dm_red[14] + dm_red[15])))
                                                                  : ((dm_red[0] + dm_red[1]) + (dm_red[2] + dm_red[3])) +
                                                                        (SEG ? (dm_red[12] + dm_red[13]) + (dm_red[14] + dm_red[15]) : 0.f);
            __threadfence();
            *last_flag = atomicAdd(&p.status[4], 1) == (int)gridDim.x - 1;
        }
        __syncthreads();
        if (*last_flag) {
            // Every CTA's partial sum is visible: dm_h = sum_b dc/dm(b,h) * sum_g T_{b,h,g}, T the
            // sum over rows of <q^, dQ^>, dc/dm = -ln(s_b) sigma(m_h) (1 - sigma(m_h)) c_{b,h};
            // fixed order, so deterministic.  One warp per head.
            __threadfence();
            const int n_b = (int)gridDim.x / (p.n_groups * p.H);
            const int per = n_b * p.n_groups;
            for (int hh = warp; hh < p.H; hh += kThreads / 32) {
                const float sg = 1.0f / (1.0f + expf(-p.m[hh]));
                float part = 0.f;
                for (int i = lane; i < per; i += 32) {
                    const int bb = i / p.n_groups, gg = i - bb * p.n_groups;
                    const float sb2 = p.seq_len ? p.seq_len[bb]
                                                : (p.seq_len_scalar > 0.f ? p.seq_len_scalar
                                                   : (float)(VARLEN ? max(p.cu_seqlens[bb + 1] - p.cu_seqlens[bb], 1) : p.N));
                    const float ls = logf(sb2);
                    part += __ldcg(&p.dm_partial[((size_t)bb * p.H + hh) * p.n_groups + gg]) *
                            (-ls * sg * (1.0f - sg) * expf(-sg * ls));
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                if (lane == 0) p.dm_out[hh] = part;
            }
            if (tid == 0) p.status[4] = 0;
        }
    }
    if (*abort_flag) {
        // A wait gave up.  Give the copies and products still in flight time to land (they need
        // microseconds; nothing here waits without a limit), then report: status word 0 = 1,
        // word 1 = where the first wait gave up, word 2 = the CTA.
        for (int i = 0; i < 100; ++i) __nanosleep(1000);
        __syncthreads();
        if (tid == 0 && atomicCAS(p.status, 0, 1) == 0) {
            p.status[1] = *abort_flag;
            p.status[2] = (int)blockIdx.x | (3 << 24);
        }
    }
    CSTAMP(3);
    if (is_score) tmem_dealloc(tmem, 512);
}


// ---------------------------------------------------------------------------------------------
// Partial states of every group for the walk above, both at once: per chunk one product
// [V | Q^]^T [K^ | dO] accumulates V^T K^ (rows 0-63, columns 0-63) and Q^^T dO (rows 64-127,
// columns 64-127) of the group; the two other blocks are not used.  One CTA per (b, h, group):
// 8 warps normalise the q and k rows of a chunk in shared memory, one thread issues the
// products, one the TMA loads (a ring of three 64 KB stages).  The chunks of a group are visited
// last to first, so that the tiles still in L2 afterwards are the ones the walk asks for first.
constexpr int kStThreads = 10 * 32;
constexpr int kStStages = 3;
constexpr int kStStagesR = 6;       // when only Q^^T dO is needed: stages of two tiles, twice as many

struct StateParams {
    float* sq_out;           // [BH, n_groups, 64 * 64]
    float* r_out;            // [BH, n_groups, 64 * 64]
    int* status;
    int H; int N; int group; int n_groups;
    int clear_status;
    int wait_limit_kcycles;
    int head_first_mask;     // bit i: in tensor map i (q, k, v, dO) the head index comes before the token index
    int all_sq;              // bidirectional backward: V^T K^ of the last group is read too
    int no_sq;               // V^T K^ comes from the forward call's workspace: no group loads k and v
    int grid_groups;         // groups 0 .. grid_groups - 1 of every (b, h) are computed (a causal forward never reads the last one's)
    const int* cu_seqlens;   // VARLEN instances: packed batch
};

// RONLY: no group needs V^T K^ (the forward call's partial states serve): a stage holds q and dO
// only, the product is the 64 x 64 Q^^T dO (rows 16 i .. 16 i + 15 of the result sit in lanes
// 32 i .. 32 i + 15 of the accumulator), and the ring is twice as deep.
template <bool RONLY, bool VARLEN>
__global__ void __launch_bounds__(kStThreads, 1)
tc_bwd_state_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmDO, StateParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + L::kOffCtl;
    constexpr int NS = RONLY ? kStStagesR : kStStages;
    constexpr uint32_t kSt = RONLY ? 2u * kTile : (uint32_t)L::kStage;     // bytes of a stage
    constexpr uint32_t oQ = RONLY ? 0u : (uint32_t)L::kOffQ, oDO = RONLY ? (uint32_t)kTile : (uint32_t)L::kOffDO;
    enum { S_FULL = 0, S_NREADY = 64, S_UFULL = 128 };         // rings of NS, indexed by chunk % NS
    auto bar = [&](int which, int c) { return bars + which + 8 * (c % NS); };
    auto par = [&](int c) { return (uint32_t)((c / NS) & 1); };
    const uint32_t tmem_slot = bars + L::kOffTmemSlot;
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + L::kOffCtl + L::kOffTmemSlot);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kOffCtl + L::kOffAbort);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = blockIdx.x % p.grid_groups, bh = blockIdx.x / p.grid_groups;
    const int bseq = bh / p.H, h = bh % p.H;
    const int b = VARLEN ? 0 : bseq;                   // batch coordinate of the tensor maps
    const int tok0 = (VARLEN ? p.cu_seqlens[bseq] : 0) + g * p.group;
    const int tok1 = min(VARLEN ? p.cu_seqlens[bseq + 1] : p.N, tok0 + p.group);
    const int n_chunks = tok1 > tok0 ? (tok1 - tok0 + kC - 1) / kC : 0;
    const bool is_mma = warp == 8, is_copy = warp == 9;
    // Nobody reads V^T K^ of the last group: its CTA leaves the v and k slots at zero (the product
    // then adds nothing to that block) and loads q and dO only.
    const bool need_sq = !RONLY && !p.no_sq && (p.all_sq || g + 1 < p.n_groups);

    if (is_mma) {
        tmem_alloc(tmem_slot, 128);
        tmem_relinquish();
    }
    if (tid == 0) {
        for (int i = 0; i < NS; ++i) {
            mbar_init(bars + S_FULL + 8 * i, 1);
            mbar_init(bars + S_NREADY + 8 * i, 256);
            mbar_init(bars + S_UFULL + 8 * i, 1);
        }
        *abort_flag = 0;
        abort_flag[3] = p.wait_limit_kcycles;
        mbar_fence_init();
        fence_proxy_async();
    }
    if (is_copy && lane == 0) {
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmDO);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_g;
    auto stage = [&](int c) { return base + (uint32_t)(c % NS) * kSt; };
    auto issue_loads = [&](int c) {
        const uint32_t fb = bar(S_FULL, c), st = stage(c);
        const int row = tok0 + (n_chunks - 1 - c) * kC;
        mbar_expect_tx(fb, (need_sq ? 4 : 2) * kTile);
        auto load = [&](uint32_t dst, const CUtensorMap* tm, int which) {
            const bool hf = (p.head_first_mask >> which) & 1;
            tma_load_4d(dst, tm, fb, 0, hf ? h : row, hf ? row : h, b);
        };
        load(st + oQ, &tmQ, 0);
        load(st + oDO, &tmDO, 3);
        if (need_sq) { load(st + L::kOffK, &tmK, 1); load(st + L::kOffV, &tmV, 2); }
    };
    if (!RONLY && !need_sq) {
        for (int i = tid; i < kStStages * 2 * (kTile / 16); i += kStThreads) {
            const int s3 = i / (2 * (kTile / 16)), r2 = i % (2 * (kTile / 16));
            const int off = s3 * L::kStage + (r2 < kTile / 16 ? L::kOffV : L::kOffK) + (r2 % (kTile / 16)) * 16;
            *reinterpret_cast<uint4*>(gbase + off) = make_uint4(0u, 0u, 0u, 0u);
        }
        fence_proxy_async();
    }
    // The first kernel of a library call may follow a kernel that produced its inputs: nothing
    // is read before the wait.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.clear_status && blockIdx.x == 0 && tid < 8) p.status[tid] = 0;   // status words and the dm counter

    if (is_copy) {
        if (lane == 0) {
            for (int c = 0; c < NS && c < n_chunks; ++c) { issue_loads(c); SSTAMP(2, c, 0); }
            for (int c = 0; c + NS < n_chunks; ++c) {
                if (!wait_or_abort(bar(S_UFULL, c), par(c), abort_flag)) break;
                issue_loads(c + NS);
                SSTAMP(2, c + NS, 0);
            }
        }
    } else if (is_mma) {
        if (lane == 0) {
            for (int c = 0; c < n_chunks; ++c) {
                const uint32_t st = stage(c);
                if (!wait_or_abort(bar(S_NREADY, c), par(c), abort_flag)) break;
                SSTAMP(1, c, 0);
                tc_fence_after();
                constexpr uint32_t idesc = RONLY ? instr_desc_bf16(64, 64, true, true) : instr_desc_bf16(128, 128, true, true);
                const uint32_t al = smem_desc_lo(st + (RONLY ? oQ : (uint32_t)L::kOffV), 16384);
                const uint32_t bl = smem_desc_lo(st + (RONLY ? oDO : (uint32_t)L::kOffK), 16384);
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)
                    mma_ss_w(tmem, al + kk * 128u, kDescHi, bl + kk * 128u, kDescHi, idesc, (c > 0 || kk > 0) ? 1u : 0u);
                tc_commit(bar(S_UFULL, c));
            }
        }
    } else {
        // row workers: warps 0-3 normalise the q rows of a chunk, warps 4-7 the k rows
        bool alive = n_chunks > 0;
        const int q4 = warp & 3, hw = warp >> 2, row = q4 * 32 + lane;
        for (int c = 0; c < n_chunks && alive; ++c) {
            SSTAMP(0, c, 0);
            if (!wait_or_abort(bar(S_FULL, c), par(c), abort_flag)) { alive = false; break; }
            SSTAMP(0, c, 1);
            if (hw == 1 && !need_sq) { mbar_arrive(bar(S_NREADY, c)); continue; }
            uint8_t* tile = gbase + (c % NS) * kSt + (hw == 0 ? oQ : (uint32_t)L::kOffK);
            uint4 w[8];
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = *reinterpret_cast<const uint4*>(tile + swz(row, j));
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                const __nv_bfloat162* e0 = reinterpret_cast<const __nv_bfloat162*>(&w[j]);
                const __nv_bfloat162* e1 = reinterpret_cast<const __nv_bfloat162*>(&w[j + 1]);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 f0 = __bfloat1622float2(e0[i]), f1 = __bfloat1622float2(e1[i]);
                    a0 = fmaf(f0.x, f0.x, a0); a1 = fmaf(f0.y, f0.y, a1);
                    a2 = fmaf(f1.x, f1.x, a2); a3 = fmaf(f1.y, f1.y, a3);
                }
            }
            float rn = 1.0f / fmaxf(sqrtf((a0 + a1) + (a2 + a3)), kEps);
            // (a packed batch: rows of the next sequence in a ragged chunk count for nothing)
            if (VARLEN && tok0 + (n_chunks - 1 - c) * kC + row >= tok1) rn = 0.f;
            // (the same two-term packed scaling as in the walk: its q^, k^ must be the same bits)
            const __nv_bfloat16 hi = __float2bfloat16_rn(rn);
            const __nv_bfloat16 lo = __float2bfloat16_rn(rn - __bfloat162float(hi));
            const __nv_bfloat162 hi2 = __halves2bfloat162(hi, hi), lo2 = __halves2bfloat162(lo, lo);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                __nv_bfloat162* e = reinterpret_cast<__nv_bfloat162*>(&w[j]);
#pragma unroll
                for (int i = 0; i < 4; ++i) e[i] = __hfma2(e[i], hi2, __hmul2(e[i], lo2));
                *reinterpret_cast<uint4*>(tile + swz(row, j)) = w[j];
            }
            fence_proxy_async();
            mbar_arrive(bar(S_NREADY, c));
            SSTAMP(0, c, 2);
        }
        if (VARLEN && n_chunks == 0) {
            // A group behind the end of its sequence (packed batch): its partial states are zero.
            const size_t slot = ((size_t)bh * p.n_groups + g) * kD * kD;
            for (int i = tid; i < kD * kD / 4; i += 256) {
                reinterpret_cast<float4*>(p.r_out + slot)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (!RONLY && p.sq_out != nullptr) reinterpret_cast<float4*>(p.sq_out + slot)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        }
        if (alive && wait_or_abort(bar(S_UFULL, n_chunks - 1), par(n_chunks - 1), abort_flag)) {
            // the group's partial states, fp32: rows 0-63 -> Sq, rows 64-127 -> R (32 columns per thread)
            tc_fence_after();
            const bool upper = row < 64;
            uint32_t r[32];
            tmem_ld32(tmem + ((uint32_t)(q4 * 32) << 16) + (RONLY ? 0 : (upper ? 0 : 64)) + hw * 32, r);
            tmem_wait_ld();
            // (the 64-row accumulator: lanes 0-15 of every quadrant hold rows 16 q4 .. 16 q4 + 15)
            const int orow = RONLY ? q4 * 16 + (lane & 15) : (row & 63);
            float* dst = ((upper && !RONLY) ? p.sq_out : p.r_out) + ((size_t)bh * p.n_groups + g) * kD * kD + (size_t)orow * kD + hw * 32;
            if (!RONLY || lane < 16) {
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                    *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(r[i]), __uint_as_float(r[i + 1]),
                                                                       __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 100; ++i) __nanosleep(1000);
        __syncthreads();
        if (tid == 0 && atomicCAS(p.status, 0, 1) == 0) {
            p.status[1] = *abort_flag;
            p.status[2] = (int)blockIdx.x | (4 << 24);
        }
    }
    if (is_mma) tmem_dealloc(tmem, 128);
}

}  // namespace

cudaError_t launch_tc_bwd_fused(const TcBwdFusedArgs& a, int B, int H, int N, cudaStream_t st) {
    const void* ptrs[7] = {a.q, a.k, a.v, a.d_o, a.dq, a.dk, a.dv};
    const RowLayout lays[7] = {a.l_qkv, a.l_qkv, a.l_v, a.l_do, a.l_dqkv, a.l_dqkv, a.l_dv};
    // real column counts (<= 64): tiles are zero-filled beyond them and stores clipped
    const int wk = a.w_k > 0 ? a.w_k : kD, wv = a.w_v > 0 ? a.w_v : kD;
    const int dims[7] = {wk, wk, wv, wv, wk, wk, wv};
    if (wk > kD || wv > kD) return cudaErrorInvalidValue;
    CUtensorMap tm[7];
    BwdParams p;
    p.head_first_mask = 0;
    // A packed batch is one tensor of total_tokens rows per head (batch extent 1).
    const int map_B = a.cu_seqlens ? 1 : B, map_N = a.cu_seqlens ? a.total_tokens : N;
    for (int i = 0; i < 7; ++i) {
        bool hf = false;
        if (!make_tile_map(&tm[i], ptrs[i], map_B, H, map_N, dims[i], lays[i], &hf)) return cudaErrorInvalidValue;
        p.head_first_mask |= (hf ? 1 : 0) << i;
    }
    p.cu_seqlens = a.cu_seqlens;
    for (int i = 0; i < 3; ++i) {
        const RowLayout lo = resolve_layout(lays[4 + i], H, map_N, dims[4 + i]);
        p.out_rows[i] = const_cast<void*>(ptrs[4 + i]); p.out_sn[i] = lo.sn; p.out_sh[i] = lo.sh; p.out_w[i] = dims[4 + i];
    }
    p.sq_part = a.sq_part; p.r_part = a.r_part; p.dm_partial = a.dm_partial; p.dm_out = a.dm_out;
    const bool segment = !a.bidir && (a.state_in || a.d_state_out || a.d_state_in);
    p.state_in = a.bidir ? nullptr : a.state_in; p.d_state_out = a.bidir ? nullptr : a.d_state_out;
    p.d_state_in = a.bidir ? nullptr : a.d_state_in; p.dm_by_v = segment ? 1 : 0;
    p.status = a.status; p.m = a.m; p.seq_len = a.seq_len; p.seq_len_scalar = a.seq_len_scalar;
    p.H = H; p.N = N; p.group = a.group; p.n_groups = a.n_groups;
    p.wait_limit_kcycles = wait_limit_kcycles();
    p.sq_fwd = a.bidir ? nullptr : a.sq_fwd; p.sq_fwd_split = a.sq_fwd_split > 0 ? a.sq_fwd_split : 1;
    // One chunk per (b, h): nothing precedes it (Sq = 0) and nothing follows it (R = 0 once its own
    // update is taken out again), so the states stay zero and no partial-state pass is needed.
    p.no_state = (!a.bidir && !segment && a.n_groups == 1 && N <= kC && !a.sq_part && !a.r_part) ? 1 : 0;
    if (!p.no_state && !a.r_part) return cudaErrorInvalidValue;
    if (segment && a.cu_seqlens) return cudaErrorInvalidValue;
    auto kern = segment ? tc_bwd_fused_kernel<false, false, true>
                        : a.cu_seqlens ? (a.bidir ? tc_bwd_fused_kernel<true, true> : tc_bwd_fused_kernel<false, true>)
                                       : (a.bidir ? tc_bwd_fused_kernel<true, false> : tc_bwd_fused_kernel<false, false>);
    if (cudaError_t e = configure_smem_once(reinterpret_cast<const void*>(kern), L::kDynBytes); e != cudaSuccess)
        return e;
    const int prof = profile_begin_launch(3, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(B * H * a.n_groups));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = L::kDynBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.plain_launch ? 0 : 1;
    cudaError_t le = cudaLaunchKernelEx(&cfg, kern, tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], tm[6], p);
    profile_end_launch(prof, st);
    note_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

cudaError_t launch_tc_bwd_states(const TcBwdFusedArgs& a, float* sq_out, float* r_out, int clear_status, int B, int H,
                                 int N, cudaStream_t st) {
    const void* ptrs[4] = {a.q, a.k, a.v, a.d_o};
    const RowLayout lays[4] = {a.l_qkv, a.l_qkv, a.l_v, a.l_do};
    const int wk = a.w_k > 0 ? a.w_k : kD, wv = a.w_v > 0 ? a.w_v : kD;
    const int dims[4] = {wk, wk, wv, wv};
    if (wk > kD || wv > kD) return cudaErrorInvalidValue;
    CUtensorMap tm[4];
    StateParams p;
    p.head_first_mask = 0;
    const int map_B = a.cu_seqlens ? 1 : B, map_N = a.cu_seqlens ? a.total_tokens : N;
    for (int i = 0; i < 4; ++i) {
        bool hf = false;
        if (!make_tile_map(&tm[i], ptrs[i], map_B, H, map_N, dims[i], lays[i], &hf)) return cudaErrorInvalidValue;
        p.head_first_mask |= (hf ? 1 : 0) << i;
    }
    p.cu_seqlens = a.cu_seqlens;
    p.sq_out = sq_out; p.r_out = r_out; p.status = a.status;
    p.H = H; p.N = N; p.group = a.group; p.n_groups = a.n_groups;
    p.clear_status = clear_status;
    p.all_sq = a.bidir;
    p.no_sq = (!a.bidir && a.sq_fwd != nullptr) ? 1 : 0;
    p.grid_groups = a.n_groups;
    p.wait_limit_kcycles = wait_limit_kcycles();
    static_assert(kStStages * L::kStage <= L::kOffCtl && kStStagesR * 2 * kTile <= L::kOffCtl, "the stage ring overlaps the control block");
    auto kern = a.cu_seqlens ? tc_bwd_state_kernel<false, true> : (p.no_sq ? tc_bwd_state_kernel<true, false> : tc_bwd_state_kernel<false, false>);
    if (a.cu_seqlens) p.no_sq = 0;
    if (cudaError_t e = configure_smem_once(reinterpret_cast<const void*>(kern), L::kOffCtl + L::kCtlBytes + 1024); e != cudaSuccess)
        return e;
    const int prof = profile_begin_launch(0, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(B * H * a.n_groups));
    cfg.blockDim = dim3(kStThreads);
    cfg.dynamicSmemBytes = L::kOffCtl + L::kCtlBytes + 1024;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.plain_launch ? 0 : 1;
    cudaError_t le = cudaLaunchKernelEx(&cfg, kern, tm[0], tm[1], tm[2], tm[3], p);
    profile_end_launch(prof, st);
    note_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

// Partial states A^^T B of groups 0 .. grid_groups - 1 of every (b, h), A's rows normalised
// (the forward's K^^T V): the q / dO-only instance of the kernel above on another pair of tensors.
cudaError_t launch_tc_pair_states(const void* a_rows, const void* b_rows, const RowLayout& l_a, const RowLayout& l_b,
                                  int w_a, int w_b, float* out, int* status, int clear_status, int B, int H, int N,
                                  int group, int n_groups, int grid_groups, int plain_launch, cudaStream_t st) {
    if (w_a > kD || w_b > kD || grid_groups < 1 || grid_groups > n_groups) return cudaErrorInvalidValue;
    const void* ptrs[4] = {a_rows, a_rows, b_rows, b_rows};            // (the k and v maps are not used)
    const RowLayout lays[4] = {l_a, l_a, l_b, l_b};
    const int dims[4] = {w_a, w_a, w_b, w_b};
    CUtensorMap tm[4];
    StateParams p;
    p.head_first_mask = 0;
    for (int i = 0; i < 4; ++i) {
        bool hf = false;
        if (!make_tile_map(&tm[i], ptrs[i], B, H, N, dims[i], lays[i], &hf)) return cudaErrorInvalidValue;
        p.head_first_mask |= (hf ? 1 : 0) << i;
    }
    p.sq_out = nullptr; p.r_out = out; p.status = status;
    p.H = H; p.N = N; p.group = group; p.n_groups = n_groups; p.grid_groups = grid_groups;
    p.clear_status = clear_status; p.all_sq = 0; p.no_sq = 1; p.cu_seqlens = nullptr;
    p.wait_limit_kcycles = wait_limit_kcycles();
    auto kern = tc_bwd_state_kernel<true, false>;
    if (cudaError_t e = configure_smem_once(reinterpret_cast<const void*>(kern), L::kOffCtl + L::kCtlBytes + 1024); e != cudaSuccess)
        return e;
    const int prof = profile_begin_launch(0, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(B * H * grid_groups));
    cfg.blockDim = dim3(kStThreads);
    cfg.dynamicSmemBytes = L::kOffCtl + L::kCtlBytes + 1024;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = plain_launch ? 0 : 1;
    cudaError_t le = cudaLaunchKernelEx(&cfg, kern, tm[0], tm[1], tm[2], tm[3], p);
    profile_end_launch(prof, st);
    note_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace cott

#ifdef COTT_TIMING
// Debug build only: copies the 256 stamps (8 roles x 4 chunks x 8 slots) to the host.
extern "C" int cott_debug_bwd_stamps(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, cott::g_bwd_stamps, sizeof(long long) * 256);
}
extern "C" int cott_debug_state_stamps(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, cott::g_state_stamps, sizeof(long long) * 192);
}
extern "C" int cott_debug_bwd_cta(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, cott::g_bwd_cta, sizeof(long long) * 1024);
}
#endif
