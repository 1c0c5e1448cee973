// Tensor-core running-sum walk (bf16 I/O, fp32 accumulation and state) for d in {64,128}.
//
// One CTA walks one sequence group in chunks of 128 tokens.  With operand roles (X, A, Bv),
// per chunk (Eq. 6 restricted to the chunk plus the running state of Eq. 7/8):
//     P      = X A^T                      (128 x 128, tcgen05, fp32 in TMEM)
//     Out    = (P . M) Bv  +  X State     (two MMAs into one TMEM accumulator)
//     State += A^T Bv                     (d x d fp32, resident in TMEM)
// Forward pass: (X,A,Bv) = (Q, K^, V).  The three gradient streams are the same walk with
// other roles, two of them backward in time (the formulas printed after Eq. 7):
//     dQ^: (dO, V, K^)        dK^: (V, dO, Q^) reversed        dV': (K, Q^, dO) reversed
// Tiles arrive by TMA with the 128-byte swizzle.  The operand whose row scale sits on a
// contraction index (K^ or Q^) is normalised in shared memory; every other scale (the X row
// norm, the stabilisation factor c of Eq. 4) multiplies fp32 accumulator rows in the
// epilogue.  States are kept without c.
//
// Modes:  MODE_STATE   only accumulates the group's partial state and writes it (phase A);
//         MODE_CAUSAL  the chunk walk starting from the group's prefix / suffix state;
//         MODE_READOUT Out = X State for a fixed state (bidirectional form, Eq. 5).
#include <stdlib.h>
#include "cott_internal.h"
#include "cott_sm100.cuh"

namespace cott {

using namespace sm100;

namespace {

constexpr int kChunk = 128;
constexpr int kTcThreads = 608;   // 16 row-worker warps + control warp + store warp + state-update warp
constexpr int kWaitLimitMsDefault = 2000;   // bound of every device-side wait: far above any legitimate one

struct TcWalkParams {
    const float* init;      // [BH, n_groups, d*d] unscaled group states, or NULL
    int init_transposed;    // 1: init holds the transposes of the states this walk needs
    int state_rev;          // state-only pass: visit the chunks of a group last to first
    int init_split;         // init_sum: entries of `init` per group (a finer state-pass partition)
    int init_sum;           // 0: init holds this group's start state; 1: it holds raw partial
                            // states, to be summed here over the groups before (after, when
                            // time runs backward; all, for the read-out) this one
    float* state_out;       // MODE_STATE: [BH, n_groups, d*d] partial states (unscaled)
    float* dm_partial;      // a stream that carries a part of the dm sum: [BH, n_groups]
    const float* dm_extra;  // the finalising stream: the other stream's [BH, n_groups] part, or NULL
    float* dm_out;          // that stream: dm[H], written by the CTA that finishes last (or NULL)
    int init_has_scale;     // init is a caller's state (contains c): divide by c on the way in
    float* state_final;     // causal walk, one group: [BH, d*d] state after the last token, times c (or NULL)
    int* status;            // workspace status word
    const float* m; const float* seq_len; float seq_len_scalar;
    int H; int N; int group; int n_groups;
    int first_group; int grid_groups;   // groups this launch covers: one CTA per (b, h, group)
    int plain_launch;                   // host side only: launch without programmatic serialization
    int clear_status;                   // first kernel of a call: CTA 0 zeroes the status words
    int wait_limit_kcycles;             // bound of every wait, in units of 1024 SM cycles
    // Packed variable-length batch: rows of all sequences back to back in one [T, H, d]
    // tensor, sequence b = rows cu_seqlens[b] .. cu_seqlens[b+1]-1, cut into groups from its first row on.
    const int* cu_seqlens;              // NULL: every (b, h) has N rows of its own
    void* out_rows; long long out_sn, out_sh;   // Out as plain global memory (rows of a ragged last chunk)
    int head_first_mask;                // bit i: in tensor map i (X, A, Bv, raw rows, Out) the head index
                                        // comes before the token index (its stride is the smaller one)
    int d_out;                          // columns Out really has (<= d): boxes wholly beyond are not stored
};

enum { MODE_STATE = 0, MODE_CAUSAL = 1, MODE_READOUT = 2 };

// Output stream a kernel instance serves.  The operand roles, the direction of time and the
// epilogue are compile-time properties, so that every instance carries only its own code (the
// walk is sensitive to instruction-cache misses: ncu showed 'no instruction' as the top stall
// of the d = 128 causal walk when all variants shared one body).
//   S_FWD: X rows normalised in the epilogue, A normalised in shared memory, plain store
//   S_DQ : Bv normalised, projection epilogue, also sums <q^, dQ^> for dm
//   S_DK : as S_DQ, time reversed
//   S_DV : as S_FWD, time reversed
enum { S_FWD = 0, S_DQ = 1, S_DK = 2, S_DV = 3 };

constexpr int kWorkerWarps = 16;                      // row-worker warps (4 per TMEM lane quadrant)
constexpr int kWorkers = kWorkerWarps * 32;
constexpr int kGroupThreads = kWorkers / 2;           // the workers act as two groups of eight warps

#ifdef COTT_TIMING
// Debug build only: SM-clock timestamps of one CTA of the causal walk of one output stream,
// chunks kStampC0 .. kStampC0 + 3, eight slots per chunk for each of five roles (0 = thread 0
// of group P, 1 = thread 256 of group O, 2 = control, 3 = state update, 4 = store thread),
// written straight to a device array that cott_debug_stamps copies out.  Slots 5-7 of role 0 in
// the first stamped chunk hold: kernel entry, the return of the wait for the previous kernel,
// the end of the prologue.
#ifndef COTT_STAMP_STREAM
#define COTT_STAMP_STREAM 0   // which output stream's walk is stamped (0 forward, 1 dQ, 2 dK, 3 dV)
#endif
#ifndef COTT_STAMP_CTA
#define COTT_STAMP_CTA 0
#endif
#ifndef COTT_STAMP_D
#define COTT_STAMP_D 64
#endif
#ifndef COTT_STAMP_C0
#define COTT_STAMP_C0 4
#endif
constexpr int kStampC0 = COTT_STAMP_C0;
__device__ long long g_cott_stamps[5 * 4 * 8];
#define COTT_STAMP_AT(role, cc, slot)                                                          \
    do {                                                                                       \
        if (D == COTT_STAMP_D && MODE == MODE_CAUSAL && STREAM == COTT_STAMP_STREAM &&         \
            blockIdx.x == COTT_STAMP_CTA && (cc) >= kStampC0 && (cc) < kStampC0 + 4 &&         \
            ((role) == 0 ? threadIdx.x == 0 : (role) == 1 ? threadIdx.x == 256 : true))        \
            g_cott_stamps[((role) * 4 + ((cc) - kStampC0)) * 8 + (slot)] = clock64();          \
    } while (0)
#else
#define COTT_STAMP_AT(role, cc, slot) do {} while (0)
#endif
constexpr int kStampBytes = 0;

// Shared-memory plan.  A stage holds the tiles one chunk needs from TMA: (A, Bv) for the
// state-only pass, (X, A, Bv) for the causal walk, (X) for the read-out.
template <int D, int MODE> struct Smem {
    static constexpr int kTile = kChunk * D * 2;          // one 128 x D bf16 tile
    static constexpr bool kHasX = MODE != MODE_STATE;
    static constexpr bool kHasAB = MODE != MODE_READOUT;
    static constexpr int kTilesPerStage = (kHasX ? 1 : 0) + (kHasAB ? 2 : 0);
    static constexpr int kStages = MODE == MODE_CAUSAL ? (D == 128 ? 2 : 3)
                                 : MODE == MODE_STATE ? (D == 128 ? 3 : 4) : 4;
    static constexpr int kStage = kTilesPerStage * kTile;
    static constexpr int kOffX = 0;
    static constexpr int kOffA = kHasX ? kTile : 0;
    static constexpr int kOffB = kOffA + kTile;
    static constexpr int kOffOut = kHasAB ? kOffB : kOffX;             // output staging slot
    // bf16 copy of the state for the X State product.  The d = 64 causal walk keeps two copies
    // (chunk parity), so that the copy of chunk c can be written while X State of chunk c
    // still reads the previous one; at d = 128 there is room for one.
    static constexpr int kSbBufs = (MODE == MODE_CAUSAL && D == 64) ? 2 : 1;
    static constexpr int kSb = (MODE == MODE_STATE) ? 0 : D * D * 2 * kSbBufs;
    static constexpr int kOffSb = kStages * kStage;
    // Output staging.  The d = 64 causal walk has room for two buffers of its own (chunk
    // parity): the whole stage of chunk c can then be refilled as soon as the chunk's last MMA
    // has read it, instead of after its epilogue and output store -- with a ring of three
    // stages the refill latency, not the arithmetic, sets the pace of the walk.  Every other
    // case stages the output in a slot of the chunk's stage that is dead by then.
    static constexpr int kOutBufs = (MODE == MODE_CAUSAL && D == 64) ? 2 : 0;
    static constexpr int kOffOutBuf = kOffSb + kSb;
    static constexpr int kOffBar = kOffOutBuf + kOutBufs * kTile;   // mbarriers, TMEM slot, abort flag
    // Row scales of X wait in rx[kRx][128] from the norm phase of a chunk to its output
    // epilogue; three buffers are needed because X and A of chunk c+2 can land (and be
    // normalised) before every worker has finished the epilogue of chunk c.
    // (Four in the d = 64 causal walk, where group P may compute the scale of chunk c + 1
    // while group O has not yet begun the epilogue of chunk c - 2.)
    static constexpr int kRx = (MODE == MODE_CAUSAL && D == 64) ? 4 : (kStages < 3 ? 3 : kStages);
    static constexpr int kBarBytes = 384;                 // mbarriers, TMEM slot, abort flag
    static constexpr int kOffRx = kOffBar + kBarBytes;    // rx[kRx][128] floats, dm scratch
    static constexpr int kCtlBytes = kBarBytes + kRx * 512 + 64 + (D == 64 ? kStampBytes : 0);
    // Gradient epilogues need a fourth tile (raw q, k or v rows) and a 4 KB exchange area
    // for per-row partial sums.  The causal walk at d = 128 has no room for either: it puts
    // the tile in the A slot and the exchange area in the X slot, both dead by then.  Every
    // other case has a buffer behind the control block, allocated only when needed.
    static constexpr bool kProjInA = (MODE == MODE_CAUSAL && D == 128);
    // Causal walk at d = 128 (two-stage ring): Bv, loaded last and needed last, has a barrier
    // of its own so that the scores of a chunk do not wait for it.  Measured: helps the
    // two-stage ring, costs a little with the three stages of d = 64.
    static constexpr bool kSplitB = (MODE == MODE_CAUSAL && D == 128);
    static constexpr int kOffProj = (kOffBar + kCtlBytes + 1023) / 1024 * 1024;
    static constexpr int kXch = 2048;
    static constexpr int dyn_bytes(bool with_proj) {
        return ((with_proj && !kProjInA) ? kOffProj + kTile + kXch : kOffBar + kCtlBytes) + 1024;  // + align slack
    }
};

// tcgen05.mma chains (one thread).  All tiles are 128-byte-swizzled rows of 128 bytes; a
// 128-column (256-byte) row is split into two half tiles 16 KB apart.
template <int D>
__device__ __forceinline__ void issue_p(uint32_t tP, uint32_t x, uint32_t a) {
    constexpr uint32_t idesc = instr_desc_bf16(128, 128, false, false);
    constexpr uint32_t hi = smem_desc_hi(1024);
    const uint32_t xl = smem_desc_lo(x, 16), al = smem_desc_lo(a, 16);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = ((kk >> 2) * 16384u + (kk & 3) * 32u) >> 4;
        mma_ss_w(tP, xl + off, hi, al + off, hi, idesc, kk > 0);
    }
}
template <int D>
__device__ __forceinline__ void issue_xs(uint32_t tO, uint32_t x, uint32_t sb) {
    constexpr uint32_t idesc = instr_desc_bf16(128, D, false, true);
    constexpr uint32_t hi = smem_desc_hi(1024);
    const uint32_t xl = smem_desc_lo(x, 16), sl = smem_desc_lo(sb, D * 128u);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = ((kk >> 2) * 16384u + (kk & 3) * 32u) >> 4;
        mma_ss_w(tO, xl + off, hi, sl + kk * 128u, hi, idesc, kk > 0);
    }
}
template <int D>
__device__ __forceinline__ void issue_pb(uint32_t tO, uint32_t tPt, uint32_t bv, bool acc_first) {
    // P~ (bf16, packed two per column) is the A operand in tensor memory: 8 columns per K = 16.
    constexpr uint32_t idesc = instr_desc_bf16(128, D, false, true);
    constexpr uint32_t hi = smem_desc_hi(1024);
    const uint32_t bl = smem_desc_lo(bv, 16384);
    mma_ts_w(tO, tPt, bl, hi, idesc, acc_first);
#pragma unroll
    for (int kk = 1; kk < kChunk / 16; ++kk)
        mma_ts_w(tO, tPt + kk * 8u, bl + kk * 128u, hi, idesc, 1u);
}
template <int D>
__device__ __forceinline__ void issue_atb(uint32_t tS, uint32_t a, uint32_t bv, bool acc_first) {
    constexpr uint32_t idesc = instr_desc_bf16(D, D, true, true);
    constexpr uint32_t hi = smem_desc_hi(1024);
    const uint32_t al = smem_desc_lo(a, 16384), bl = smem_desc_lo(bv, 16384);
    mma_ss_w(tS, al, hi, bl, hi, idesc, acc_first);
#pragma unroll
    for (int kk = 1; kk < kChunk / 16; ++kk)
        mma_ss_w(tS, al + kk * 128u, hi, bl + kk * 128u, hi, idesc, 1u);
}

// Bounded wait that also gives up as soon as any thread of the CTA has given up.
// The thread that gives up first leaves a record of where: bit 31 set, warp index in bits
// 16-20, byte offset of the barrier inside the barrier block in bits 4-13, parity in bit 0.
// (The abort flag sits 236 bytes into the barrier block.)
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();   // SM cycle counter: far cheaper to read than the global timer
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 15u) == 1) {
            if (*abort_flag) return false;
            // the limit (in units of 1024 SM cycles) sits three words behind the abort flag
            if (clock64() - t0 > ((long long)abort_flag[3] << 10)) {
                const uint32_t bars = (uint32_t)__cvta_generic_to_shared((const void*)abort_flag) - 236u;
                const uint32_t where = 0x80000000u | ((threadIdx.x >> 5) << 16) | (((bar - bars) & 0x3FFu) << 4) | (parity & 1u);
                atomicCAS(const_cast<int*>(abort_flag), 0, (int)where);
                return false;
            }
        }
    }
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Sum of squares of eight bf16 values, on two independent accumulators.
__device__ __forceinline__ void sumsq8(const uint4& w, float& a0, float& a1) {
    const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float2 f = __bfloat1622float2(e[i]);
        a0 = fmaf(f.x, f.x, a0);
        a1 = fmaf(f.y, f.y, a1);
    }
}

__device__ __forceinline__ uint4 pack8(const uint32_t* r) {
    uint4 w;
    w.x = pack_bf16(__uint_as_float(r[0]), __uint_as_float(r[1]));
    w.y = pack_bf16(__uint_as_float(r[2]), __uint_as_float(r[3]));
    w.z = pack_bf16(__uint_as_float(r[4]), __uint_as_float(r[5]));
    w.w = pack_bf16(__uint_as_float(r[6]), __uint_as_float(r[7]));
    return w;
}

// QW (16 or 32) consecutive accumulator columns of this thread's TMEM lane.
template <int QW> __device__ __forceinline__ void tmem_ldq(uint32_t taddr, uint32_t (&r)[QW]);
template <> __device__ __forceinline__ void tmem_ldq<32>(uint32_t taddr, uint32_t (&r)[32]) { tmem_ld32(taddr, r); }
template <> __device__ __forceinline__ void tmem_ldq<16>(uint32_t taddr, uint32_t (&r)[16]) { tmem_ld16(taddr, r); }
template <int QW> __device__ __forceinline__ void tmem_stq(uint32_t taddr, const uint32_t (&r)[QW]);
template <> __device__ __forceinline__ void tmem_stq<32>(uint32_t taddr, const uint32_t (&r)[32]) { tmem_st32(taddr, r); }
template <> __device__ __forceinline__ void tmem_stq<16>(uint32_t taddr, const uint32_t (&r)[16]) { tmem_st16(taddr, r); }


// Thread roles: warps 0-15 are the row workers, in two groups of eight that work on different
// chunks at once (score masking + state copy / row norms + output epilogue).  Lane 0 of
// warp 16 is the control thread (scores, P~ Bv and X State MMAs), of warp 17 the store thread
// (output stores, stage refills, epilogue-tile loads), of warp 18 the state-update thread
// (State += A^T Bv in the causal walk).  The roles meet only through mbarriers, every wait
// bounded.
// VARLEN (packed variable-length batch) is a compile-time property as well: the walk is
// sensitive to its instruction footprint and register count, and the dense instances were
// measurably slower (C5 N=131072: 577 us against 515 us) with the packed-batch code in them.
template <int D, int MODE, int STREAM, bool VARLEN>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_walk_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmA,
               const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmP,
               const __grid_constant__ CUtensorMap tmO, TcWalkParams p) {
    using L = Smem<D, MODE>;
    constexpr int NST = L::kStages;
    constexpr int NH = D / 64;                       // 64-column half tiles per row
    constexpr uint32_t kTmemCols = 512;
    // Columns: State d | P 128 (fp32 scores) | P~ 64 (bf16 masked scores, packed) | Out | P~.
    // d = 64 double-buffers Out.  P~ has two buffers (chunk parity; the second one takes the
    // last 64 columns): the scores of chunk c + 1 may be issued ahead of P~ Bv of chunk c, so
    // the mask of chunk c + 1 can finish while that product still reads P~ of chunk c.
    constexpr uint32_t colS = 0, colP = D, colPt0 = D + 128, colPt1 = 448, colO0 = D + 192;
    static_assert(D + 192 + (D == 64 ? 2 : 1) * D <= 448, "tensor-memory columns overlap");
    auto colPt = [&](int c) { return (c & 1) ? colPt1 : colPt0; };
    constexpr int kOBufs = (D == 64) ? 2 : 1;
    constexpr int QW = D / 4;                        // accumulator columns per worker thread
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + L::kOffBar;
    // Barriers that a fast role could otherwise lap are arrays indexed by stage or by chunk
    // parity, so a phase parity always names one chunk; no waiter ever skips a phase.
    const uint32_t bar_full = bars;            // [NST] (<= 4) TMA landed: X and A (causal walk), all tiles otherwise
    const uint32_t bar_a_ready = bars + 32;    // [NST] X scale known, A normalised (all workers)
    const uint32_t bar_p_full = bars + 64;     //       scores done (commit)
    const uint32_t bar_s_full = bars + 256;    // [4]   state update done (commit)
    const uint32_t bar_pt_ready = bars + 88;   //       masked scores in tensor memory (all workers)
    const uint32_t bar_sb_ready = bars + 96;   // [2]   bf16 state copy written (all workers); the second one sits at bars + 240
    const uint32_t bar_o_full = bars + 288;    // [4]   output accumulator complete (commit)
    const uint32_t bar_o_free = bars + 120;    // [2]   output accumulator drained (all workers)
    const uint32_t bar_proj = bars + 136;      // [2]   epilogue tile landed (second one only with two tile buffers)
    const uint32_t bar_e_done = bars + 320;    // [4]   output rows of the chunk staged (all workers)
    const uint32_t bar_xch = bars + 160;       //       per-row partial sums exchanged (all workers)
    const uint32_t bar_full_b = bars + 168;    // [NST] causal walk: Bv landed (it is loaded last and needed last)
    const uint32_t bar_b_ready = bars + 200;   // [NST] causal walk: Bv normalised, when it is the one (all workers)
    const uint32_t bar_out_free = bars + 352;  // [2]   own output buffers: the store of the chunk has read its buffer
    const uint32_t tmem_slot = bars + 232;
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + L::kOffBar + 232);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kOffBar + 236);
    // Barriers with waiters that only the data flow holds back (the store thread, the
    // state-update thread, a worker group behind the other) are rings of four indexed by
    // chunk: the stage ring (at most four deep) keeps every role within three chunks of the
    // others, so a phase parity always names one chunk.
    auto sfull_bar = [&](int c) { return bar_s_full + 8 * (c & 3); };
    auto sfull_par = [&](int c) { return (uint32_t)((c >> 2) & 1); };
    auto ofull_bar = [&](int c) { return bar_o_full + 8 * (c & 3); };
    auto ofull_par = [&](int c) { return (uint32_t)((c >> 2) & 1); };
    auto edone_bar = [&](int c) { return bar_e_done + 8 * (c & 3); };
    auto edone_par = [&](int c) { return (uint32_t)((c >> 2) & 1); };
    auto sb_bar = [&](int c) { return (c & 1) ? bars + 240 : bar_sb_ready; };
    auto sb_par = [&](int c) { return (uint32_t)((c >> 1) & 1); };
    // Byte offset of the state copy X State of chunk c reads (written after chunk c - 1, or by
    // the prologue for c = 0).
    auto sb_off = [&](int c) { return (uint32_t)(L::kSbBufs == 2 ? ((c + 1) & 1) * (D * D * 2) : 0); };
    constexpr int NRX = L::kRx;
    float* rx_buf = reinterpret_cast<float*>(gbase + L::kOffRx);                 // [NRX][128]
    float* dm_red = reinterpret_cast<float*>(gbase + L::kOffRx + NRX * 512);     // [16]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    COTT_STAMP_AT(0, kStampC0, 5);
    const int g = p.first_group + blockIdx.x % p.grid_groups, bh = blockIdx.x / p.grid_groups;
    const int b = bh / p.H, h = bh % p.H;
    constexpr bool varlen = VARLEN;
    // (packed batch: group g of sequence b starts g groups behind the sequence's first row and may
    // lie wholly behind its last one -- a CTA with nothing to do)
    const int seq0 = varlen ? p.cu_seqlens[b] : 0, seq1 = varlen ? p.cu_seqlens[b + 1] : p.N;
    const int tok0 = seq0 + g * p.group;
    const int tok1 = min(seq1, tok0 + p.group);
    const int n_chunks = tok1 > tok0 ? (tok1 - tok0 + kChunk - 1) / kChunk : 0;
    // Packed batch: the chunks of a sequence start at its first row, so only its last chunk can
    // hold rows of the next sequence.  Those rows take no part: the operand that is normalised
    // in shared memory gets zeros there (it is one of the two operands of the state update and
    // either the key side of the scores or the value side of P~ Bv), their outputs are not
    // stored, and they add nothing to dm.
    const int bcoord = varlen ? 0 : b;                 // batch coordinate of the tensor maps
    const bool ragged_last = varlen && ((tok1 - tok0) % kChunk) != 0;
    constexpr bool kNormBv = STREAM == S_DQ || STREAM == S_DK;
    constexpr bool kXNorm = STREAM == S_FWD || STREAM == S_DV;
    constexpr bool kReverse = STREAM == S_DK || STREAM == S_DV;
    // The dV' stream has a plain epilogue: the sum over rows of <dV'_j, v_j> that dm needs
    // equals the sum over rows of <q^_i, dQ^_i> (both are the sum over the attended pairs (i, j)
    // of (q^_i . k^_j)(dO_i . v_j)), and the dQ^ stream's projection epilogue already forms
    // <q_i, dQ^_i> for every row, so that stream accumulates it and the dV' stream needs neither
    // the raw v rows nor the per-row exchange.
    constexpr int kEpi = (STREAM == S_FWD || STREAM == S_DV) ? EPI_PLAIN : EPI_PROJ;
    constexpr bool with_proj = (MODE != MODE_STATE) && (kEpi != EPI_PLAIN);
    const bool is_ctrl = warp == kWorkerWarps;
    const bool is_store = warp == kWorkerWarps + 1;
    const bool is_upd = warp == kWorkerWarps + 2;

    if (is_ctrl) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    if (tid == 0) {
        for (int i = 0; i < NST; ++i) {
            mbar_init(bar_full + 8 * i, L::kSplitB ? 1 : 2); mbar_init(bar_a_ready + 8 * i, kGroupThreads);
            mbar_init(bar_full_b + 8 * i, 1); mbar_init(bar_b_ready + 8 * i, kGroupThreads);
        }
        mbar_init(bar_p_full, 1);
        for (int i = 0; i < 4; ++i) { mbar_init(bar_s_full + 8 * i, 1); mbar_init(bar_o_full + 8 * i, 1); mbar_init(bar_e_done + 8 * i, kGroupThreads); }
        mbar_init(bar_pt_ready, kGroupThreads); mbar_init(bar_sb_ready, kGroupThreads);
        mbar_init(bars + 240, kGroupThreads);
        mbar_init(bar_o_free, kGroupThreads); mbar_init(bar_o_free + 8, kGroupThreads);
        mbar_init(bar_proj, 1); mbar_init(bar_proj + 8, 1);
        mbar_init(bar_xch, kGroupThreads);
        mbar_init(bar_out_free, 1); mbar_init(bar_out_free + 8, 1);
        *abort_flag = 0;
        abort_flag[3] = p.wait_limit_kcycles;
        mbar_fence_init();
        fence_proxy_async();
    }
    if (is_ctrl && lane == 0) {
        tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmA); tma_prefetch_desc(&tmB);
        tma_prefetch_desc(&tmP); tma_prefetch_desc(&tmO);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_g;
    auto stage_x = [&](int s) { return base + s * L::kStage + L::kOffX; };
    auto stage_a = [&](int s) { return base + s * L::kStage + L::kOffA; };
    auto stage_b = [&](int s) { return base + s * L::kStage + L::kOffB; };
    // Chunk visited at step c.  The state-only pass may take either order (its result does not
    // depend on it): it takes the opposite of the walk that follows, so that the tiles it
    // read last -- still in L2 -- are the ones the walk needs first.
    const bool backward = (MODE == MODE_STATE) ? (p.state_rev != 0) : kReverse;
    auto chunk_row = [&](int c) { return tok0 + (backward ? (n_chunks - 1 - c) : c) * kChunk; };
    // Step at which the sequence's last chunk (the only one that can be ragged) is visited.
    const int last_visit_of_ragged = backward ? 0 : n_chunks - 1;

    // TMA loads (issued by single threads of the control and the store warp).
    // The tensor maps are 4-D (column, then head and token ordered by stride, then batch), so
    // that [B,H,N,d], [B,N,H,d] and rows inside a fused projection output are read in place.
    auto load_tile = [&](uint32_t dst, const CUtensorMap* tm, uint32_t bar, int row, int which) {
        const bool hf = (p.head_first_mask >> which) & 1;   // head index before the token index
        const int c1 = hf ? h : row, c2 = hf ? row : h;
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) tma_load_4d(dst + hh * 16384, tm, bar, hh * 64, c1, c2, bcoord);
    };
    // Loads of chunk c: part 1 = X and A, part 2 = Bv (X alone in the read-out pass).
    auto issue_loads = [&](int c, bool part1, bool part2) {
        const int s = c % NST;
        const uint32_t bar = bar_full + 8 * s;
        const int row = chunk_row(c);
        if (L::kSplitB) {
            if (part1) {
                mbar_expect_tx(bar, 2 * L::kTile);
                load_tile(stage_x(s), &tmX, bar, row, 0);
                load_tile(stage_a(s), &tmA, bar, row, 1);
            }
            if (part2) {
                mbar_expect_tx(bar_full_b + 8 * s, L::kTile);
                load_tile(stage_b(s), &tmB, bar_full_b + 8 * s, row, 2);
            }
        } else {
            // One barrier for the stage, two arrivals: each part arms its own byte count
            // before its copies (the parts may come from different threads).
            constexpr int kPart1Tiles = L::kHasAB ? (L::kHasX ? 2 : 1) : 0;
            if (part1) {
                mbar_expect_tx(bar, kPart1Tiles * L::kTile);
                if (L::kHasAB) {
                    if (L::kHasX) load_tile(stage_x(s), &tmX, bar, row, 0);
                    load_tile(stage_a(s), &tmA, bar, row, 1);
                }
            }
            if (part2) {
                mbar_expect_tx(bar, L::kTile);
                if (L::kHasAB) load_tile(stage_b(s), &tmB, bar, row, 2);
                else load_tile(stage_x(s), &tmX, bar, row, 0);
            }
        }
    };
    // Raw q, k or v rows of chunk c for the gradient epilogues: into the A slot of the chunk's
    // stage once the state update has read it (d = 128 causal walk, control thread), else into
    // a buffer of its own once the previous chunk's epilogue is done (store thread).
    auto load_proj = [&](int c) {
        constexpr bool two = L::kOutBufs > 0 && !L::kProjInA;   // two tile buffers (see below)
        const uint32_t proj_u = L::kProjInA ? stage_a(c % NST)
                                            : base + ((two && (c & 1)) ? L::kOffOutBuf + L::kTile : L::kOffProj);
        // One barrier per chunk parity wherever the tile of chunk c + 1 can be requested before
        // the epilogue of chunk c has seen its own: arming a barrier whose phase still waits for
        // bytes would be a second arrival on a count of one.  (In the A slot the request follows
        // the state update of c + 1, which only follows the epilogue of c - 1.)
        const uint32_t pbar = (two || L::kProjInA) ? bar_proj + 8 * (c & 1) : bar_proj;
        mbar_expect_tx(pbar, L::kTile);
        load_tile(proj_u, &tmP, pbar, chunk_row(c), 3);
    };
    // Every kernel but the first of a library call follows a kernel of the same call, which
    // writes none of the tensors loaded here: its first tiles are requested before the wait
    // for that kernel, so their HBM latency overlaps its tail.
    const bool early_loads = p.clear_status == 0 && n_chunks > 0;
    if (early_loads && is_ctrl && lane == 0)
        for (int c = 0; c < NST && c < n_chunks; ++c) issue_loads(c, true, true);
    // Everything above touched only this CTA's own resources.  From here on global memory
    // written by the previous kernel of the stream is read (and its inputs overwritten).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    COTT_STAMP_AT(0, kStampC0, 6);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.clear_status && blockIdx.x == 0 && tid < 8) p.status[tid] = 0;   // status words and the dm counter
    // The first kernel of a call may follow a kernel that produced its inputs: its first tiles
    // are requested here, right behind the wait.
    if (!early_loads && is_ctrl && lane == 0)
        for (int c = 0; c < NST && c < n_chunks; ++c) issue_loads(c, true, true);

    const float s_b = p.seq_len ? p.seq_len[b]
                                : (p.seq_len_scalar > 0.f ? p.seq_len_scalar
                                                          : (float)(varlen ? max(seq1 - seq0, 1) : p.N));
    const float cfac = stab_factor(p.m[h], s_b);

    // Accumulator mapping of a worker thread: TMEM lane quadrant q, column quarter cq, row.
    const int q = warp & 3, cq = (warp >> 2) & 3;
    const uint32_t lane_base = (uint32_t)(q * 32) << 16;
    const int arow = q * 32 + lane;                   // row of P / Out held by this thread
    // State rows: M = 128 maps row r to lane r; M = 64 maps row r to lane (r%16) + 32*(r/16).
    const bool owns_srow = (D == 128) || (lane < 16);
    const int srow = (D == 128) ? arow : q * 16 + (lane & 15);
    const uint32_t sb = base + L::kOffSb;

    // bf16 copy of QW state columns of this thread's row into the MN-major state tile.
    auto write_sb = [&](const uint32_t (&r)[QW], int c0) {
#pragma unroll
        for (int i = 0; i < QW; i += 8) {
            const int col = c0 + i;
            const uint32_t off = (col >> 6) * (D * 128u) + swz(srow, (col & 63) >> 3);
            *reinterpret_cast<uint4*>(gbase + L::kOffSb + sb_off(0) + off) = pack8(&r[i]);
        }
    };

    const bool init_state = p.init != nullptr;
    if (init_state && warp < kWorkerWarps) {
        // Initial state of the group: fp32 into TMEM, bf16 copy into shared memory.  With
        // init_sum the exclusive prefix (suffix / total) over the groups' partial states is
        // formed here, in group order, instead of by a separate scan launch.
        // Element (srow, cq*QW + i) of group gg's state; a transposed source (the state of a
        // sibling gradient stream, which is this stream's state transposed) is read by columns.
        const int n_init = p.n_groups * p.init_split;     // entries of `init` per (b, h)
        const float* src = p.init + (size_t)bh * n_init * D * D;
        auto load4 = [&](int gg, int i) -> float4 {
            const float* sg = src + (size_t)gg * D * D;
            if (!p.init_transposed) return *reinterpret_cast<const float4*>(sg + (size_t)srow * D + cq * QW + i);
            const float* col = sg + (size_t)(cq * QW + i) * D + srow;
            return make_float4(col[0], col[D], col[2 * D], col[3 * D]);
        };
        uint32_t r[QW];
        if (!p.init_sum) {
#pragma unroll
            for (int i = 0; i < QW; i += 4) {
                float4 v = owns_srow ? load4(g, i) : make_float4(0.f, 0.f, 0.f, 0.f);
                if (p.init_has_scale) { const float ic = 1.0f / cfac; v.x *= ic; v.y *= ic; v.z *= ic; v.w *= ic; }
                r[i] = __float_as_uint(v.x); r[i + 1] = __float_as_uint(v.y);
                r[i + 2] = __float_as_uint(v.z); r[i + 3] = __float_as_uint(v.w);
            }
        } else {
            float acc[QW];
#pragma unroll
            for (int i = 0; i < QW; ++i) acc[i] = 0.f;
            const int g_lo = (MODE == MODE_READOUT) ? 0 : (kReverse ? (g + 1) * p.init_split : 0);
            const int g_hi = (MODE == MODE_READOUT) ? n_init : (kReverse ? n_init : g * p.init_split);
            if (owns_srow) {
                for (int gg = g_lo; gg < g_hi; ++gg) {
#pragma unroll
                    for (int i = 0; i < QW; i += 4) {
                        const float4 v = load4(gg, i);
                        acc[i] += v.x; acc[i + 1] += v.y; acc[i + 2] += v.z; acc[i + 3] += v.w;
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < QW; ++i) r[i] = __float_as_uint(acc[i]);
        }
        if (MODE == MODE_CAUSAL) { tmem_stq<QW>(tmem + lane_base + colS + cq * QW, r); tmem_wait_st(); }
        if (MODE != MODE_STATE && owns_srow) write_sb(r, cq * QW);
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    float dm_acc = 0.f;
    COTT_STAMP_AT(0, kStampC0, 7);

    // The stage of chunk c is refilled with chunk c + NST by the store thread, in two steps
    // when possible: X and A as soon as the last MMAs that read the stage have completed, Bv
    // -- the output staging slot -- after the chunk's output store has drained.
    constexpr bool split_refill = MODE == MODE_CAUSAL && !(with_proj && L::kProjInA);
    constexpr bool own_out = L::kOutBufs > 0;     // output staged outside the stage ring
    // Gradient epilogues of that walk: one output buffer, and the other 16 KB hold a second
    // buffer for the raw rows, so that the rows of chunk c + 2 are requested when the epilogue
    // of chunk c is done and their latency is not part of any epilogue.
    constexpr bool proj2 = own_out && with_proj && !L::kProjInA;
    constexpr bool out_pair = own_out && !proj2;  // two output buffers (chunk parity)
    // Which worker group normalises the contraction-side tile / computes the X row scales in
    // the d = 64 causal walk.  Group O is the busy one (it has the epilogue), so: the forward
    // walk gives the X scales to group P; the gradient walks, whose epilogues are longer and
    // whose scores leave group P idle most of the time, give it the tile.
    constexpr bool kTileNormInP = own_out && kEpi != EPI_PLAIN;
    constexpr bool kXScaleInP = own_out && kEpi == EPI_PLAIN;
    // Where the normalised operand is Bv (dQ^ and dK^ streams) the scores need only the raw X
    // and A tiles: they are issued as soon as the tiles have landed, and the normalisation is
    // waited for before P~ Bv and the state update.
    constexpr bool kScoresOnFull = own_out && kNormBv;
    constexpr bool proj_bar2 = proj2 || (with_proj && L::kProjInA);     // barrier per chunk parity (see load_proj)
    auto proj_bar = [&](int c) { return proj_bar2 ? bar_proj + 8 * (c & 1) : bar_proj; };
    auto proj_par = [&](int c) { return (uint32_t)((proj_bar2 ? (c >> 1) : c) & 1); };
    auto proj_off = [&](int c) { return (proj2 && (c & 1)) ? L::kOffOutBuf + L::kTile : L::kOffProj; };
    auto out_off = [&](int c) { return L::kOffOutBuf + (out_pair ? (c & 1) * L::kTile : 0); };

    if (is_ctrl) {
        // ------------------------------------------------------------------ control thread
        if (lane == 0 && n_chunks > 0) {
            bool alive = true;
            auto wait = [&](uint32_t bar, uint32_t parity) {
                if (alive && !wait_or_abort(bar, parity, abort_flag)) alive = false;
                return alive;
            };
            // First MMA batch of chunk c: scores, X State (needs the previous chunk's state
            // copy and a drained output buffer), state update.
            auto scores = [&](int c) {
                const int s = c % NST;
                tc_fence_after();
                issue_p<D>(tmem + colP, stage_x(s), stage_a(s));
                tc_commit(bar_p_full);
            };
            auto batch1 = [&](int c, bool scores_issued) {
                const int s = c % NST;
                if (!wait((kScoresOnFull ? bar_full : bar_a_ready) + 8 * s, (c / NST) & 1)) return;
                COTT_STAMP_AT(2, c - 1, 4);
                const bool acc = init_state || c > 0;
                // Scores first: they need neither the state copy nor the output buffer.
                if (MODE == MODE_CAUSAL && !scores_issued) scores(c);
                if (MODE != MODE_STATE) {
                    if (MODE == MODE_CAUSAL && c >= 1 && !wait(sb_bar(c - 1), sb_par(c - 1))) return;
                    COTT_STAMP_AT(2, c - 1, 5);
                    // The output accumulator this chunk writes must have been drained: by chunk
                    // c - 2 with two buffers, by chunk c - 1 with one.
                    if (kOBufs == 2) { if (c >= 2 && !wait(bar_o_free + 8 * (c & 1), ((c >> 1) & 1) ^ 1)) return; }
                    else if (c >= 1 && !wait(bar_o_free + 8 * ((c - 1) & 1), ((c - 1) >> 1) & 1)) return;
                }
                tc_fence_after();
                COTT_STAMP_AT(2, c - 1, 6);
                const uint32_t tO = tmem + colO0 + (c % kOBufs) * D;
                if (MODE == MODE_CAUSAL) {
                    // (The state update of the chunk is issued by the state-update thread.)
                    if (acc) issue_xs<D>(tO, stage_x(s), sb + sb_off(c));
                    COTT_STAMP_AT(2, c - 1, 7);
                } else if (MODE == MODE_STATE) {
                    issue_atb<D>(tmem + colS, stage_a(s), stage_b(s), acc);
                    tc_commit(sfull_bar(c));
                } else {
                    issue_xs<D>(tO, stage_x(s), sb);
                    tc_commit(ofull_bar(c));
                }
            };
            batch1(0, false);
            for (int c = 0; c < n_chunks && alive; ++c) {
                const int s = c % NST;
                bool next_scores = false;
                COTT_STAMP_AT(2, c, 0);
                if (MODE == MODE_CAUSAL) {
                    if (!wait(bar_pt_ready, c & 1)) break;
                    COTT_STAMP_AT(2, c, 1);
                    // The masked scores of chunk c have left the score columns.  If the next
                    // chunk's tiles are ready its scores go in ahead of P~ Bv of this one: the
                    // mask of the next chunk, not the epilogue of this one, waits on the tensor
                    // core here.
                    if (c + 1 < n_chunks &&
                        mbar_try_wait((kScoresOnFull ? bar_full : bar_a_ready) + 8 * ((c + 1) % NST),
                                      ((c + 1) / NST) & 1)) {
                        scores(c + 1);
                        next_scores = true;
                    }
                    COTT_STAMP_AT(2, c, 2);
                    // Bv is needed from here on: landed, and normalised if it is the operand
                    // whose row scale sits on the contraction index.
                    if (L::kSplitB) {
                        if (!wait(bar_full_b + 8 * s, (c / NST) & 1)) break;
                        if (kNormBv && !wait(bar_b_ready + 8 * s, (c / NST) & 1)) break;
                    }
                    if (kScoresOnFull && !wait(bar_a_ready + 8 * s, (c / NST) & 1)) break;
                    tc_fence_after();
                    const bool acc = init_state || c > 0;
                    issue_pb<D>(tmem + colO0 + (c % kOBufs) * D, tmem + colPt(c), stage_b(s), acc);
                    tc_commit(ofull_bar(c));
                    COTT_STAMP_AT(2, c, 3);
                    if (with_proj && L::kProjInA) {
                        // The A slot is free once the state update has read it.
                        if (!wait(sfull_bar(c), sfull_par(c))) break;
                        load_proj(c);
                    }
                }
                if (c + 1 < n_chunks) { batch1(c + 1, next_scores); if (!alive) break; }
            }
        }
    } else if (is_upd) {
        // ------------------------------------------------------------------ state-update thread
        // Causal walk: State += A^T Bv of chunk c depends on the chunk's tiles and on the
        // workers having copied the previous state, not on the scores; issued from a thread of
        // its own it neither waits behind the masked scores nor holds up their MMAs.
        if (lane == 0 && MODE == MODE_CAUSAL) {
            for (int c = 0; c < n_chunks; ++c) {
                const int s = c % NST;
                COTT_STAMP_AT(3, c, 0);
                if (!wait_or_abort(bar_a_ready + 8 * s, (c / NST) & 1, abort_flag)) break;
                COTT_STAMP_AT(3, c, 1);
                if (L::kSplitB) {
                    if (!wait_or_abort(bar_full_b + 8 * s, (c / NST) & 1, abort_flag)) break;
                    if (kNormBv && !wait_or_abort(bar_b_ready + 8 * s, (c / NST) & 1, abort_flag)) break;
                }
                // the workers have read the fp32 state of the previous chunk
                if (c >= 1 && !wait_or_abort(sb_bar(c - 1), sb_par(c - 1), abort_flag)) break;
                COTT_STAMP_AT(3, c, 2);
                // Nothing else ties this thread to group O: stay within two chunks of its
                // epilogue, so that the ring of state-update barriers cannot lap it.
                if (c >= 2 && !wait_or_abort(edone_bar(c - 2), edone_par(c - 2), abort_flag)) break;
                COTT_STAMP_AT(3, c, 3);
                tc_fence_after();
                issue_atb<D>(tmem + colS, stage_a(s), stage_b(s), init_state || c > 0);
                tc_commit(sfull_bar(c));
                COTT_STAMP_AT(3, c, 4);
            }
        }
    } else if (is_store) {
        // ------------------------------------------------------------------ store thread
        // Refills the stages and stores the output rows the workers staged.  Kept off the
        // control thread: issuing a TMA copy costs it about as much as several MMAs, and the
        // wait for a store's shared-memory read would stall the MMA issue.
        if (lane == 0) {
            bool alive = n_chunks > 0;
            if (alive && with_proj && !L::kProjInA) {
                load_proj(0);
                if (proj2 && n_chunks > 1) load_proj(1);
            }
            for (int c = 0; c < n_chunks && alive; ++c) {
                const int s = c % NST;
                const bool more = c + NST < n_chunks;
                COTT_STAMP_AT(4, c, 0);
                // X and A (everything in the state-only pass) as soon as the chunk's last MMA,
                // the state update, has completed.
                if ((MODE == MODE_STATE || split_refill) && more) {
                    if (!wait_or_abort(sfull_bar(c), sfull_par(c), abort_flag)) { alive = false; break; }
                    // (causal walk: the other MMAs of the chunk come from another thread)
                    if (MODE == MODE_CAUSAL &&
                        !wait_or_abort(ofull_bar(c), ofull_par(c), abort_flag)) { alive = false; break; }
                    COTT_STAMP_AT(4, c, 1);
                    issue_loads(c + NST, true, MODE == MODE_STATE || own_out);
                    COTT_STAMP_AT(4, c, 2);
                }
                if (MODE == MODE_STATE) continue;
                if (!wait_or_abort(edone_bar(c), edone_par(c), abort_flag)) { alive = false; break; }
                COTT_STAMP_AT(4, c, 3);
                if (with_proj && !L::kProjInA) {                // the tile buffer of chunk c is free now
                    if (proj2) { if (c + 2 < n_chunks) load_proj(c + 2); }
                    else if (c + 1 < n_chunks) load_proj(c + 1);
                }
                const uint32_t src = own_out ? base + out_off(c) : base + s * L::kStage + L::kOffOut;
#pragma unroll
                // (the rows of a ragged last chunk of a packed batch were written by the workers)
                for (int hh = 0; hh < ((ragged_last && c == last_visit_of_ragged) ? 0 : NH); ++hh) {
                    if (hh * 64 >= p.d_out) break;
                    const bool hfo = (p.head_first_mask >> 4) & 1;
                    const int row = chunk_row(c);
                    tma_store_4d(&tmO, src + hh * 16384, hh * 64, hfo ? h : row, hfo ? row : h, bcoord);
                }
                tma_store_commit();
                COTT_STAMP_AT(4, c, 4);
                if (out_pair) {
                    // The previous chunk's store has read its buffer: the epilogue of the
                    // chunk after this one may fill it again.
                    if (c >= 1) { tma_store_wait_read1(); mbar_arrive(bar_out_free + 8 * ((c - 1) & 1)); }
                } else if (own_out) {
                    tma_store_wait_read0();                      // one buffer: the next epilogue waits for this
                    mbar_arrive(bar_out_free);
                } else if (more) {
                    tma_store_wait_read0();
                    issue_loads(c + NST, !split_refill, true);
                }
                COTT_STAMP_AT(4, c, 5);
            }
            // (the stream that carries the dm sum drains its stores after the dm tail instead,
            // so that the tail runs while the last store is still on its way)
            if (MODE != MODE_STATE && p.dm_partial == nullptr) tma_store_wait_all0();
        }
    } else {
        // ------------------------------------------------------------------ row workers
        // Two groups of eight warps work on different chunks at the same time, so that the
        // long-latency steps of one (TMEM loads, shared-memory round trips) hide behind the
        // other:  group P (warps 0-7)  masks the scores and refreshes the bf16 state copy;
        //         group O (warps 8-15) computes the row norms of the next chunk and runs the
        //         output epilogue of the current one.
        // Each group covers all four TMEM lane quadrants with two warps (column halves).  In
        // the state-only pass both groups normalise, on alternate chunks.
        bool alive = n_chunks > 0;
        auto wait = [&](uint32_t bar, uint32_t parity) {
            if (alive && !wait_or_abort(bar, parity, abort_flag)) alive = false;
            return alive;
        };
        const int grp = warp >> 3, w8 = warp & 7, hf = w8 >> 2;
        constexpr int HW = D / 2;                     // accumulator columns per thread in the chunk loops
        constexpr int NPIECE = HW / 32;               // 32-column pieces of that range
        // Norm mapping inside a group: lanes l and l^16 share a row (two column halves).
        const int nrow = w8 * 16 + (lane & 15), nhalf = lane >> 4;
        constexpr int NC = D / 16;                    // 16-byte chunks in half a row
        auto tile_h_ptr = [&](uint8_t* tile, int j) {
            const int ch = nhalf * NC + j;            // chunk index within the row
            return tile + (ch >> 3) * 16384 + swz(nrow, ch & 7);
        };
        auto pair_sum = [&](float v) { return v + __shfl_xor_sync(0xffffffffu, v, 16); };
        // x^ = x / max(||x||, eps) on this thread's half row, in place, rounded to bf16.
        auto normalise_half_row = [&](uint8_t* nt, int c) {
            uint4 wn[NC];
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
            for (int j = 0; j < NC; ++j) wn[j] = *reinterpret_cast<const uint4*>(tile_h_ptr(nt, j));
#pragma unroll
            for (int j = 0; j < NC; j += 2) { sumsq8(wn[j], a0, a1); sumsq8(wn[j + 1], a2, a3); }
            float r = 1.0f / fmaxf(sqrtf(pair_sum((a0 + a1) + (a2 + a3))), kEps);
            if (varlen && chunk_row(c) + nrow >= tok1) r = 0.f;     // a row of the next sequence
#pragma unroll
            for (int j = 0; j < NC; ++j) {
                const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&wn[j]);
                uint4 o;
                uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float2 f = __bfloat1622float2(e[i]);
                    ow[i] = pack_bf16(f.x * r, f.y * r);
                }
                *reinterpret_cast<uint4*>(tile_h_ptr(nt, j)) = o;
            }
            fence_proxy_async();
        };
        // Row norms of chunk c, in two parts that either worker group can run: the
        // contraction-side operand is normalised in place (the scores wait for this part); the
        // X row scale (times c) is left in rx_buf[c % NRX] for the output epilogue.
        auto norm_tile = [&](int c) {
            const int s = c % NST;
            if (!wait(bar_full + 8 * s, (c / NST) & 1)) return;
            COTT_STAMP_AT(1, c - 1, 7);
            // In the split causal walk Bv arrives on its own barrier and is normalised later.
            if (L::kHasAB && !(L::kSplitB && kNormBv))
                normalise_half_row(gbase + s * L::kStage + (kNormBv ? L::kOffB : L::kOffA), c);
            mbar_arrive(bar_a_ready + 8 * s);
        };
        // Only streams whose X rows are normalised keep a scale per row; the others use c itself.
        // Ordering of these shared-memory writes before the epilogue that reads them (other
        // threads, other row mapping): when group P computes the scales, through its arrival on
        // the masked-scores barrier of the same chunk.  When group O does: with a single output
        // accumulator (d = 128) the scales of chunk c + 1 are written during iteration c, before
        // the thread's arrival on `o_free` of chunk c, which X State of chunk c + 1 and hence
        // its epilogue wait for -- so they may follow the tile's normalisation, off the path to
        // the chunk's scores; chunk 0 has no such arrival and gets a barrier of the group
        // instead.  With two accumulators `o_free` of chunk c does not gate chunk c + 1: there
        // the scales come BEFORE the normalisation, whose arrival on `a_ready` the chunk's MMAs
        // and hence its epilogue follow.
        auto x_scale = [&](int c) {
            if (!L::kHasX || !kXNorm) return;
            const int s = c % NST;
            float rx = cfac;
            {
                if (!wait(bar_full + 8 * s, (c / NST) & 1)) return;
                const uint8_t* xt = gbase + s * L::kStage + L::kOffX;
                float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
                for (int j = 0; j < NC; j += 2) {
                    sumsq8(*reinterpret_cast<const uint4*>(tile_h_ptr(const_cast<uint8_t*>(xt), j)), a0, a1);
                    sumsq8(*reinterpret_cast<const uint4*>(tile_h_ptr(const_cast<uint8_t*>(xt), j + 1)), a2, a3);
                }
                rx = cfac / fmaxf(sqrtf(pair_sum((a0 + a1) + (a2 + a3))), kEps);
            }
            if (nhalf == 0) rx_buf[(c % NRX) * 128 + nrow] = rx;
        };
        auto norm_phase = [&](int c) { x_scale(c); if (alive) norm_tile(c); };
        // Split causal walk, Bv is the normalised operand (dQ^ and dK^ streams).
        auto norm_b = [&](int c) {
            const int s = c % NST;
            if (!wait(bar_full_b + 8 * s, (c / NST) & 1)) return;
            normalise_half_row(gbase + s * L::kStage + L::kOffB, c);
            mbar_arrive(bar_b_ready + 8 * s);
        };
        // bf16 copy of 32 state columns of this thread's row into the MN-major state tile.
        auto write_sb32 = [&](const uint32_t (&r)[32], int c0, uint32_t buf) {
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
                const int col = c0 + i;
                const uint32_t off = (col >> 6) * (D * 128u) + swz(srow, (col & 63) >> 3);
                *reinterpret_cast<uint4*>(gbase + L::kOffSb + buf + off) = pack8(&r[i]);
            }
        };

        if (MODE == MODE_STATE) {
            // Both groups normalise, on alternate chunks, and follow every state update (a
            // parity names one chunk only if no phase is skipped).
            for (int c = 0; c < n_chunks && alive; ++c) {
                if ((c & 1) == grp) norm_phase(c);
                if (c >= 1 && !wait(sfull_bar(c - 1), sfull_par(c - 1))) break;
            }
            if (alive) wait(sfull_bar(n_chunks - 1), sfull_par(n_chunks - 1));
        } else if (grp == 0) {
            // -------------------------------------------------------------- group P
            if (kTileNormInP) norm_tile(0);
            if (kXScaleInP) x_scale(0);
            for (int c = 0; MODE == MODE_CAUSAL && c < n_chunks && alive; ++c) {
                // Masked scores -> bf16 operand P~ in tensor memory.  Forward: row i keeps
                // columns j <= i (diagonal kept, Eq. 6); backward in time: j >= i.  Per
                // 32 x 32 block (row block q, column block cb) the mask is all-keep, all-zero
                // or, on the diagonal, a triangle; the first two cases are warp-uniform.
                COTT_STAMP_AT(0, c, 0);
                if (!wait(bar_p_full, c & 1)) break;
                tc_fence_after();
                COTT_STAMP_AT(0, c, 1);
#pragma unroll 1
                for (int sbk = 0; sbk < 2; ++sbk) {
                    const int cb = 2 * hf + sbk;
                    const bool keep_all = kReverse ? (cb > q) : (cb < q);
                    const bool diag = cb == q;
                    uint32_t r[32];
                    if (keep_all || diag) {
                        tmem_ld32(tmem + lane_base + colP + cb * 32, r);
                        tmem_wait_ld();
                        if (diag) {
#pragma unroll
                            for (int j = 0; j < 32; ++j) {
                                const bool keep = kReverse ? (j >= lane) : (j <= lane);
                                r[j] = keep ? r[j] : 0u;
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = 0u;
                    }
                    // bf16, two scores per column (even column index in the low half): this
                    // block's 32 k-values are 16 columns of the A-operand region.
                    uint32_t pk[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        pk[j] = pack_bf16(__uint_as_float(r[2 * j]), __uint_as_float(r[2 * j + 1]));
                    tmem_st16(tmem + lane_base + colPt(c) + cb * 16, pk);
                }
                tmem_wait_st();
                COTT_STAMP_AT(0, c, 2);
                tc_fence_before();
                mbar_arrive(bar_pt_ready);
                // The next chunk's scores wait for its normalised tile: before the state copy.
                if (kTileNormInP && c + 1 < n_chunks) { norm_tile(c + 1); if (!alive) break; }
                // bf16 copy of the updated state for the next chunk's X State product.
                if (c + 1 < n_chunks) {
                    if (!wait(sfull_bar(c), sfull_par(c))) break;
                    // A single copy is still being read by this chunk's X State product.
                    if (L::kSbBufs == 1 && !wait(ofull_bar(c), ofull_par(c))) break;
                    tc_fence_after();
                    COTT_STAMP_AT(0, c, 3);
#pragma unroll 1
                    for (int pc = 0; pc < NPIECE; ++pc) {
                        uint32_t r[32];
                        tmem_ld32(tmem + lane_base + colS + hf * HW + pc * 32, r);
                        tmem_wait_ld();
                        if (owns_srow) write_sb32(r, hf * HW + pc * 32, sb_off(c + 1));
                    }
                    fence_proxy_async();
                    tc_fence_before();
                    mbar_arrive(sb_bar(c));
                    COTT_STAMP_AT(0, c, 4);
                }
                if (kXScaleInP && c + 1 < n_chunks) { x_scale(c + 1); if (!alive) break; }
            }
        } else {
            // -------------------------------------------------------------- group O
            if (kOBufs == 1) {
                if (!kTileNormInP) norm_tile(0);
                if (!kXScaleInP && alive) x_scale(0);
                // Chunk 0 has no earlier arrival of this group between these writes and the
                // epilogue that reads them: the group meets once here.  Every thread of the
                // group gets here exactly once (the waits above are bounded and return).
                if (kXNorm && !kXScaleInP) asm volatile("bar.sync 1, %0;" ::"n"(kGroupThreads) : "memory");
            } else {
                if (!kXScaleInP) x_scale(0);
                if (!kTileNormInP && alive) norm_tile(0);
            }
            if (L::kSplitB && kNormBv && alive) norm_b(0);
            for (int c = 0; c < n_chunks && alive; ++c) {
                const int s = c % NST;
                uint8_t* st = gbase + s * L::kStage;
                COTT_STAMP_AT(1, c, 0);
                if (c + 1 < n_chunks) {
                    if (kOBufs == 1) {
                        if (!kTileNormInP) norm_tile(c + 1);
                        if (!kXScaleInP && alive) x_scale(c + 1);
                    } else {
                        if (!kXScaleInP) x_scale(c + 1);
                        if (!kTileNormInP && alive) norm_tile(c + 1);
                    }
                    if (!alive) break;
                }
                COTT_STAMP_AT(1, c, 1);
                // ---- output epilogue of chunk c: accumulator -> bf16 rows in the staging slot
                if (!wait(ofull_bar(c), ofull_par(c))) break;
                tc_fence_after();
                COTT_STAMP_AT(1, c, 2);
                const uint32_t tO = tmem + lane_base + colO0 + (c % kOBufs) * D + hf * HW;
                const float rx = kXNorm ? rx_buf[(c % NRX) * 128 + arow] : cfac;
                uint32_t r[HW];
#pragma unroll
                for (int pc = 0; pc < NPIECE; ++pc)
                    tmem_ld32(tO + pc * 32, *reinterpret_cast<uint32_t(*)[32]>(&r[pc * 32]));
                tmem_wait_ld();
                tc_fence_before();
                mbar_arrive(bar_o_free + 8 * (c & 1));
                float coef = 0.f, rp = 1.f;
                const uint8_t* proj = L::kProjInA ? (st + L::kOffA) : (gbase + proj_off(c));
                auto proj_chunk = [&](int i) {       // 8 raw values next to accumulator columns hf*HW + i ..
                    const int col = hf * HW + i;
                    return *reinterpret_cast<const uint4*>(proj + (col >> 6) * 16384 + swz(arow, (col & 63) >> 3));
                };
                if (with_proj) {
                    if (!wait(proj_bar(c), proj_par(c))) break;
                    // Per-row <p, acc> and ||p||^2: each of the two column-half threads sums its
                    // part; the parts meet in shared memory.
                    float2* xch = reinterpret_cast<float2*>(L::kProjInA ? (st + L::kOffX)
                                                                        : (gbase + L::kOffProj + L::kTile));
                    float ss0 = 0.f, ss1 = 0.f, dp0 = 0.f, dp1 = 0.f;
#pragma unroll
                    for (int i = 0; i < HW; i += 8) {
                        const uint4 w = proj_chunk(i);
                        const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float2 f = __bfloat1622float2(e[j]);
                            ss0 = fmaf(f.x, f.x, ss0); ss1 = fmaf(f.y, f.y, ss1);
                            dp0 = fmaf(f.x, __uint_as_float(r[i + 2 * j]), dp0);
                            dp1 = fmaf(f.y, __uint_as_float(r[i + 2 * j + 1]), dp1);
                        }
                    }
                    xch[hf * 128 + arow] = make_float2(ss0 + ss1, dp0 + dp1);
                    mbar_arrive(bar_xch);
                    if (!wait(bar_xch, c & 1)) break;
                    const float2 e0 = xch[arow], e1 = xch[128 + arow];
                    const float ss = e0.x + e1.x, dp = e0.y + e1.y;
                    if (kEpi == EPI_PROJ) {
                        // g = rx * acc;  out = (g - p^ <p^, g>) / max(||p||, eps); clamped branch: g / eps
                        const float nrm = sqrtf(ss);
                        rp = 1.0f / fmaxf(nrm, kEps);
                        coef = nrm > kEps ? dp * rx * rp * rp : 0.f;
                        // <q^_i, dQ^_i> of the unscaled accumulator, once per row (see kEpi)
                        if (STREAM == S_DQ && hf == 0 && !(varlen && chunk_row(c) + arow >= tok1))
                            dm_acc += dp * rp;
                        // The dQ^ stream's sum uses k^ rounded to bf16 (its Bv operand).  To first
                        // order the sum with the exact k^ is larger by sum_j <k^_j - bf16(k^_j), dK^_j>,
                        // and this stream has both factors: the raw k rows and the dK^ accumulator.
                        // dm is a heavily cancelling sum, so this rounding is its largest error.
                        if (STREAM == S_DK && p.dm_partial != nullptr && !(varlen && chunk_row(c) + arow >= tok1)) {
                            const float rpe = nrm > kEps ? rp : 0.f;     // (a clamped row has no such term worth keeping)
                            float c0 = 0.f, c1 = 0.f;
#pragma unroll
                            for (int i = 0; i < HW; i += 8) {
                                const uint4 w = proj_chunk(i);
                                const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
                                for (int j = 0; j < 4; ++j) {
                                    const float2 f = __bfloat1622float2(e[j]);
                                    const float kx = f.x * rpe, ky = f.y * rpe;
                                    c0 = fmaf(kx - __bfloat162float(__float2bfloat16_rn(kx)), __uint_as_float(r[i + 2 * j]), c0);
                                    c1 = fmaf(ky - __bfloat162float(__float2bfloat16_rn(ky)), __uint_as_float(r[i + 2 * j + 1]), c1);
                                }
                            }
                            dm_acc += c0 + c1;
                        }
                    }
                }
                // Scale, (project,) round to bf16, stage for the TMA store.  The staging slot is
                // the Bv slot, which the state update (issued behind P~ Bv) still reads: wait for it.
                COTT_STAMP_AT(1, c, 3);
                if (own_out) {
                    // Nothing else waits for the last state update: it must not be in flight
                    // when the CTA gives back its tensor memory.
                    if (c + 1 == n_chunks && !wait(sfull_bar(c), sfull_par(c))) break;
                }
                if (out_pair) {
                    // own buffer of this chunk parity: the store of chunk c - 2 has read it
                    if (c >= 2 && !wait(bar_out_free + 8 * (c & 1), ((c >> 1) & 1) ^ 1)) break;
                } else if (own_out) {
                    if (c >= 1 && !wait(bar_out_free, (c - 1) & 1)) break;   // the one buffer: store of chunk c - 1
                } else if (MODE == MODE_CAUSAL && !wait(sfull_bar(c), sfull_par(c))) break;
                COTT_STAMP_AT(1, c, 4);
                uint8_t* so = own_out ? gbase + out_off(c) : st + L::kOffOut;
#pragma unroll
                for (int i = 0; i < HW; i += 8) {
                    const int col = hf * HW + i;
                    float v[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(r[i + j]) * rx;
                    if (with_proj && kEpi == EPI_PROJ) {
                        const uint4 w = proj_chunk(i);
                        const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float2 f = __bfloat1622float2(e[j]);
                            v[2 * j] = (v[2 * j] - f.x * coef) * rp;
                            v[2 * j + 1] = (v[2 * j + 1] - f.y * coef) * rp;
                        }
                    }
                    uint4 w;
                    w.x = pack_bf16(v[0], v[1]); w.y = pack_bf16(v[2], v[3]);
                    w.z = pack_bf16(v[4], v[5]); w.w = pack_bf16(v[6], v[7]);
                    if (ragged_last && c == last_visit_of_ragged) {
                        // Packed batch, last chunk of the sequence: a tile store would overwrite
                        // rows of the next sequence; the rows that exist go out one by one.
                        const long long grow = (long long)chunk_row(c) + arow;
                        if (grow < tok1 && col < p.d_out)
                            *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out_rows) +
                                                      grow * p.out_sn + (long long)h * p.out_sh + col) = w;
                    } else {
                        *reinterpret_cast<uint4*>(so + (col >> 6) * 16384 + swz(arow, (col & 63) >> 3)) = w;
                    }
                }
                fence_proxy_async();
                mbar_arrive(edone_bar(c));
                COTT_STAMP_AT(1, c, 5);
                // Bv of the next chunk lands last; normalise it (when it is the one) after this
                // chunk's epilogue, before the tensor core needs it.
                if (L::kSplitB && kNormBv && c + 1 < n_chunks) { norm_b(c + 1); if (!alive) break; }
            }
        }

        if (MODE == MODE_STATE && varlen && n_chunks == 0 && p.state_out != nullptr) {
            // A group behind the end of its sequence: its partial state is zero.
            float4* dst = reinterpret_cast<float4*>(p.state_out + ((size_t)bh * p.n_groups + g) * D * D);
            for (int i = tid; i < D * D / 4; i += 16 * 32) dst[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (MODE == MODE_STATE && alive && p.state_out != nullptr) {
            // Partial state of this group, fp32, unscaled (every state update was waited for).
            tc_fence_after();
            float* dst = p.state_out + ((size_t)bh * p.n_groups + g) * D * D + (size_t)srow * D + cq * QW;
            uint32_t r[QW];
            tmem_ldq<QW>(tmem + lane_base + colS + cq * QW, r);
            tmem_wait_ld();
            if (owns_srow) {
#pragma unroll
                for (int i = 0; i < QW; i += 4)
                    *reinterpret_cast<float4*>(dst + i) =
                        make_float4(__uint_as_float(r[i]), __uint_as_float(r[i + 1]),
                                    __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
            }
        }
        if (MODE == MODE_CAUSAL && p.state_final != nullptr && alive) {
            // State after the last token of the (single) group, times c: the caller's Eq. 8 state.
            if (wait(sfull_bar(n_chunks - 1), sfull_par(n_chunks - 1))) {
                tc_fence_after();
                float* dst = p.state_final + (size_t)bh * D * D + (size_t)srow * D + cq * QW;
                uint32_t r[QW];
                tmem_ldq<QW>(tmem + lane_base + colS + cq * QW, r);
                tmem_wait_ld();
                if (owns_srow) {
#pragma unroll
                    for (int i = 0; i < QW; i += 4)
                        *reinterpret_cast<float4*>(dst + i) =
                            make_float4(__uint_as_float(r[i]) * cfac, __uint_as_float(r[i + 1]) * cfac,
                                        __uint_as_float(r[i + 2]) * cfac, __uint_as_float(r[i + 3]) * cfac);
                }
            }
        }
        if (MODE != MODE_STATE && p.dm_partial != nullptr) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) dm_acc += __shfl_xor_sync(0xffffffffu, dm_acc, o);
            if (lane == 0) dm_red[warp] = dm_acc;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (MODE != MODE_STATE && p.dm_partial != nullptr) {
        int* last_flag = reinterpret_cast<int*>(&dm_red[0]);
        if (tid == 0) {
            // Fixed-order reduction of the CTA's dm term (the warps of group O hold sums; in the
            // dQ^ stream only its first half).
            if (!*abort_flag)
                p.dm_partial[(size_t)bh * p.n_groups + g] = ((dm_red[8] + dm_red[9]) + (dm_red[10] + dm_red[11])) +
                                                             ((dm_red[12] + dm_red[13]) + (dm_red[14] + dm_red[15]));
            *last_flag = 0;
            if (p.dm_out != nullptr) {
                __threadfence();
                *last_flag = atomicAdd(&p.status[4], 1) == (int)gridDim.x - 1;
            }
        }
        __syncthreads();
        if (*last_flag) {
            // Every CTA's partial sum is visible: dm_h = sum_b dc/dm(b,h) * sum_g T_{b,h,g}, T the
            // sum over rows of <dV', V> (equally of <q^, dQ^>), dc/dm = -ln(s_b) sigma(m_h)
            // (1 - sigma(m_h)) c_{b,h}; fixed order, so deterministic.
            __threadfence();
            // One warp per head; lane l takes the (b, g) pairs l, l + 32, ... and the lanes meet
            // in a butterfly: the loads of a head go out together instead of one after the
            // other (this tail is the end of the last kernel of a backward call).
            const int n_b = (int)gridDim.x / (p.n_groups * p.H);
            const int per = n_b * p.n_groups;
            for (int hh = warp; hh < p.H; hh += kTcThreads / 32) {
                const float sg = 1.0f / (1.0f + expf(-p.m[hh]));
                float part = 0.f;
                for (int i = lane; i < per; i += 32) {
                    const int bb = i / p.n_groups, gg = i - bb * p.n_groups;
                    const float sb2 = p.seq_len ? p.seq_len[bb]
                                                : (p.seq_len_scalar > 0.f ? p.seq_len_scalar
                                                   : (float)(varlen ? max(p.cu_seqlens[bb + 1] - p.cu_seqlens[bb], 1) : p.N));
                    const float ls = logf(sb2);
                    const size_t idx = ((size_t)bb * p.H + hh) * p.n_groups + gg;
                    const float t_bh = __ldcg(&p.dm_partial[idx]) + (p.dm_extra ? __ldcg(&p.dm_extra[idx]) : 0.f);
                    part += t_bh * (-ls * sg * (1.0f - sg) * expf(-sg * ls));
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                if (lane == 0) p.dm_out[hh] = part;
            }
            if (tid == 0) p.status[4] = 0;
        }
    }
    if (MODE != MODE_STATE && p.dm_partial != nullptr && is_store && lane == 0) tma_store_wait_all0();
    if (*abort_flag) {
        // A wait gave up.  Before the CTA's shared memory and tensor memory go away, give the
        // copies and MMAs still in flight time to land (they need microseconds; nothing here
        // waits without a limit), then report: status word 0 = 1, word 1 = where the first
        // wait gave up, word 2 = the CTA.
        for (int i = 0; i < 100; ++i) __nanosleep(1000);
        __syncthreads();
        if (tid == 0 && atomicCAS(p.status, 0, 1) == 0) {
            p.status[1] = *abort_flag;
            p.status[2] = (int)blockIdx.x | (MODE << 24) | (STREAM << 28);
        }
    }
    if (is_ctrl) tmem_dealloc(tmem, kTmemCols);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    // (initialised once, thread-safe: a function-local static)
    static const EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) ==
                cudaSuccess && qres == cudaDriverEntryPointSuccess)
            return reinterpret_cast<EncodeTiledFn>(ptr);
        return nullptr;
    }();
    return fn;
}

}  // namespace

// Tensor map over a bf16 tensor of logical shape [B,H,N,d] with element strides (sb, sh, sn)
// and contiguous rows: 4-D, the head and token dimensions ordered by stride (dense [B,H,N,d]:
// token first; [B,N,H,d] or rows inside a fused projection output: head first); box = 128
// tokens x 64 columns of one (b,h), 128-byte swizzle; rows past N read as zero and are not
// written.  *head_first tells the kernel the order of the two middle coordinates.
bool make_tile_map(CUtensorMap* map, const void* ptr, int B, int H, int N, int d, const RowLayout& lay,
                   bool* head_first, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    const RowLayout l = resolve_layout(lay, H, N, d);
    if (l.sn < d || l.sh < d || l.sb < d || (l.sn & 7) || (l.sh & 7) || (l.sb & 7)) return false;
    const bool hf = l.sh < l.sn;
    *head_first = hf;
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)(hf ? H : N), (cuuint64_t)(hf ? N : H), (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)(hf ? l.sh : l.sn) * 2, (cuuint64_t)(hf ? l.sn : l.sh) * 2,
                             (cuuint64_t)l.sb * 2};
    cuuint32_t box[4] = {64, hf ? 1u : (cuuint32_t)box_rows, hf ? (cuuint32_t)box_rows : 1u, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// Tensor map over `rows` contiguous rows of d bf16 values (a dense [B,H,N,d] tensor seen as one
// list of rows): box = box_rows rows x 64 columns, 128-byte swizzle, coordinates (column, row, 0, 0).
bool make_rows_map(CUtensorMap* map, const void* ptr, long long rows, int d, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc || rows < 1 || d < 8 || (d & 7) || box_rows < 1 || box_rows > 256) return false;
    cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)rows, 1, 1};
    cuuint64_t strides[3] = {(cuuint64_t)d * 2, (cuuint64_t)rows * d * 2, (cuuint64_t)rows * d * 2};
    cuuint32_t box[4] = {64, (cuuint32_t)box_rows, 1, 1};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

namespace {

template <int D, int MODE, int STREAM, bool VARLEN>
cudaError_t launch_mode_v(const CUtensorMap* tm, const TcWalkParams& p, int BH, cudaStream_t st) {
    auto kern = tc_walk_kernel<D, MODE, STREAM, VARLEN>;
    // (the dV' stream has a plain epilogue, like the forward pass)
    constexpr bool with_proj = (MODE != MODE_STATE) && (STREAM == S_DQ || STREAM == S_DK);
    {   // (per kernel and device: the attribute belongs to a function on one device)
        cudaError_t e = configure_smem_once(reinterpret_cast<const void*>(kern), Smem<D, MODE>::dyn_bytes(with_proj));
        if (e != cudaSuccess) return e;
    }
    const int prof = profile_begin_launch(MODE, st);
    // Programmatic dependent launch: this kernel may start (allocate TMEM, set up barriers,
    // prefetch tensor maps) while the previous kernel of the stream drains; it waits for that
    // kernel's memory with griddepcontrol.wait before touching any global data.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(BH * p.grid_groups));
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = Smem<D, MODE>::dyn_bytes(with_proj);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.plain_launch ? 0 : 1;
    cudaError_t le = cudaLaunchKernelEx(&cfg, kern, tm[0], tm[1], tm[2], tm[3], tm[4], p);
    profile_end_launch(prof, st);
    note_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

template <int D, int MODE, int STREAM>
cudaError_t launch_mode(const CUtensorMap* tm, const TcWalkParams& p, int BH, cudaStream_t st) {
    return p.cu_seqlens ? launch_mode_v<D, MODE, STREAM, true>(tm, p, BH, st)
                        : launch_mode_v<D, MODE, STREAM, false>(tm, p, BH, st);
}

template <int D>
cudaError_t launch_d(int mode, int stream_kind, const CUtensorMap* tm, const TcWalkParams& p, int BH,
                     cudaStream_t st) {
    if (mode == MODE_STATE)   // only the operand that is normalised distinguishes the instances
        return (stream_kind == S_DQ || stream_kind == S_DK) ? launch_mode<D, MODE_STATE, S_DQ>(tm, p, BH, st)
                                                            : launch_mode<D, MODE_STATE, S_FWD>(tm, p, BH, st);
    if (mode == MODE_CAUSAL) {
        switch (stream_kind) {
            case S_FWD: return launch_mode<D, MODE_CAUSAL, S_FWD>(tm, p, BH, st);
            case S_DQ: return launch_mode<D, MODE_CAUSAL, S_DQ>(tm, p, BH, st);
            case S_DK: return launch_mode<D, MODE_CAUSAL, S_DK>(tm, p, BH, st);
            default: return launch_mode<D, MODE_CAUSAL, S_DV>(tm, p, BH, st);
        }
    }
    switch (stream_kind) {
        case S_FWD: return launch_mode<D, MODE_READOUT, S_FWD>(tm, p, BH, st);
        case S_DQ: return launch_mode<D, MODE_READOUT, S_DQ>(tm, p, BH, st);
        case S_DK: return launch_mode<D, MODE_READOUT, S_DK>(tm, p, BH, st);
        default: return launch_mode<D, MODE_READOUT, S_DV>(tm, p, BH, st);
    }
}

}  // namespace

cudaError_t launch_tc_walk(const TcWalkArgs& a, int B, int H, int N, int d, cudaStream_t st) {
    const int BH = B * H;
    // Unused operands still need a valid map: point them at a tensor that exists.
    const void* any = a.x ? a.x : a.a;
    const RowLayout any_l = a.x ? a.lx : a.la;
    const void* ptrs[5] = {a.x ? a.x : any, a.a ? a.a : any, a.bv ? a.bv : any,
                           a.proj ? a.proj : any, a.out ? a.out : any};
    const RowLayout lays[5] = {a.x ? a.lx : any_l, a.a ? a.la : any_l, a.bv ? a.lbv : any_l,
                               a.proj ? a.lproj : any_l, a.out ? a.lout : any_l};
    CUtensorMap tm[5];
    int head_first_mask = 0;
    // A packed batch is one tensor of total_tokens rows per head (batch extent 1).
    const int map_B = a.cu_seqlens ? 1 : B, map_N = a.cu_seqlens ? a.total_tokens : N;
    const int d_xa = a.d_xa > 0 ? a.d_xa : d, d_bo = a.d_bo > 0 ? a.d_bo : d;
    if (d_xa > d || d_bo > d) return cudaErrorInvalidValue;
    // (an unused operand's map points at x or a)
    const int dims[5] = {d_xa, d_xa, a.bv ? d_bo : d_xa, a.proj ? d_bo : d_xa, a.out ? d_bo : d_xa};
    for (int i = 0; i < 5; ++i) {
        bool hf = false;
        if (!make_tile_map(&tm[i], ptrs[i], map_B, H, map_N, dims[i], lays[i], &hf)) return cudaErrorInvalidValue;
        head_first_mask |= (hf ? 1 : 0) << i;
    }
    TcWalkParams p;
    p.head_first_mask = head_first_mask;
    p.cu_seqlens = a.cu_seqlens;
    p.d_out = d_bo;
    {
        const RowLayout lo = resolve_layout(a.lout, H, map_N, d_bo);
        p.out_rows = a.out; p.out_sn = lo.sn; p.out_sh = lo.sh;
    }
    p.init = a.init; p.state_out = a.state_out; p.dm_partial = a.dm_partial; p.dm_extra = a.dm_extra; p.dm_out = a.dm_out; p.status = a.status;
    p.init_has_scale = a.init_has_scale; p.state_final = a.state_final;
    p.m = a.m; p.seq_len = a.seq_len; p.seq_len_scalar = a.seq_len_scalar;
    p.H = H; p.N = N; p.group = a.group; p.n_groups = a.n_groups;
    p.init_sum = a.init_sum; p.init_transposed = a.init_transposed;
    p.init_split = (a.init_sum && a.init_split > 1) ? a.init_split : 1;
    p.state_rev = (a.mode == MODE_STATE) ? a.reverse : 0;
    const bool subset = a.mode == MODE_STATE && a.grid_groups > 0;
    p.first_group = subset ? a.first_group : 0;
    p.grid_groups = subset ? a.grid_groups : a.n_groups;
    // (a packed batch reads cu_seqlens before anything else: no early start behind a kernel
    // that may have produced it)
    p.plain_launch = a.plain_launch || a.cu_seqlens != nullptr;
    p.clear_status = a.clear_status;
    p.wait_limit_kcycles = wait_limit_kcycles();
    if (p.first_group < 0 || p.first_group + p.grid_groups > a.n_groups) return cudaErrorInvalidValue;
    // The four combinations of roles the library uses, as compile-time kernel variants.
    int kind;
    if (a.epilogue == EPI_PLAIN && !a.norm_bv && a.x_norm && !a.reverse) kind = S_FWD;
    else if (a.epilogue == EPI_PROJ && a.norm_bv && !a.x_norm && !a.reverse) kind = S_DQ;
    else if (a.epilogue == EPI_PROJ && a.norm_bv && !a.x_norm && a.reverse) kind = S_DK;
    else if (a.epilogue == EPI_DV && !a.norm_bv && a.x_norm && a.reverse) kind = S_DV;
    else if (a.mode == MODE_STATE) kind = a.norm_bv ? S_DQ : S_FWD;
    else return cudaErrorInvalidValue;
    if (d == 128) return launch_d<128>(a.mode, kind, tm, p, BH, st);
    if (d == 64) return launch_d<64>(a.mode, kind, tm, p, BH, st);
    return cudaErrorInvalidValue;
}

}  // namespace cott

#ifdef COTT_TIMING
// Debug build only: copies the 160 timestamps (5 roles x 4 chunks x 8 slots) to the host.
extern "C" int cott_debug_stamps(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, cott::g_cott_stamps, sizeof(long long) * 160);
}
#endif
