// Bidirectional backward in one launch for d <= 64 (bf16 I/O, fp32 accumulation), one CTA per
// (b, h) or per (sequence, head) of a packed batch.
//
// With an all-ones mask the gradients of O = c Q^ (K^^T V) (the right-hand side of Eq. 5) are
// plain products with two d x d totals over the whole sequence,
//     S = K^^T V ,  R = Q^^T dO :     dQ^ = dO S^T ,   dK^ = V R^T ,   dV' = K^ R ,
// followed by the chain rule through the row normalisation (Eq. 2/3) and the factor c (Eq. 4).
//
// Phase 1 streams the (k, v) and (q, dO) tile pairs of the sequence once: the k and q rows are
// normalised in shared memory and S, R accumulate in tensor memory (M = 64 products).  Between
// the phases the two totals are rounded to bf16 operands in shared memory, and their fp32
// element-wise product gives the dm sum, sum_i <q^_i, dQ^_i> = <S, R>.  Phase 2 streams the pairs
// (dO, q) and (v, k) again (they come from L2): one product per output tile -- none of them needs
// a normalised operand, since K^ R = diag(1 / ||k||) (K R) -- and one thread per row applies the
// row scale, the projection and c, with x^ = x / ||x|| formed in fp32 from the raw row; the
// gradient rows are staged in the tiles they were computed from and stored from there.  The bf16
// rounding of q^ and k^ before the state products is the only rounding that enters dm; its
// first-order terms, sum_i <q^_i - bf16(q^_i), dQ^_i> + sum_j <k^_j - bf16(k^_j), dK^_j>, are added
// by the same threads.
// Two CTAs share an SM (113 KB of shared memory, 256 tensor-memory columns each): three tile pairs
// are in flight per CTA.
#include "cott_internal.h"
#include "cott_sm100.cuh"
#include "cott_tc_common.cuh"

namespace cott {

using namespace sm100;
using namespace tc;

namespace {

constexpr int kC = 128;                 // tokens per chunk
constexpr int kD = 64;
constexpr int kTile = kC * kD * 2;      // one 128 x 64 bf16 tile
constexpr int kWorkerWarps = 8;
constexpr int kThreads = (kWorkerWarps + 3) * 32;   // + product thread, load thread, store thread

// Three stages of two tiles: a ring that the tile pairs of both phases go through in turn.
struct L {
    static constexpr int kStages = 3;
    static constexpr int kOffSb = kStages * 2 * kTile;      // bf16 copy of S (64 x 64)
    static constexpr int kOffRb = kOffSb + kD * kD * 2;     // bf16 copy of R
    static constexpr int kOffCtl = kOffRb + kD * kD * 2;
    static constexpr int kOffDmRed = 640;                   // float [16] + a flag, inside the control block
    static constexpr int kCtlBytes = 1024;
    static constexpr int kDynBytes = kOffCtl + kCtlBytes;   // (no slack: the base must be aligned, see the kernel)
};

struct BidirBwdParams {
    float* dm_partial; float* dm_out; int* status;
    const float* m; const float* seq_len; float seq_len_scalar;
    int H; int N;
    int wait_limit_kcycles;
    int head_first_mask;     // bit i: in tensor map i (q, k, v, dO, dq, dk, dv) the head index comes before the token index
    // Packed variable-length batch (NULL: dense): every tensor is [1, H, total_tokens, d], sequence
    // b = rows cu_seqlens[b] .. cu_seqlens[b + 1] - 1; the rows of a ragged last chunk leave as
    // plain stores: dq, dk, dv as global memory with their token and head strides in elements.
    const int* cu_seqlens;
    void* out_rows[3]; long long out_sn[3], out_sh[3]; int out_w[3];
};

// Out[128 x 64] = X[128 x 64] St, St read MN-major (its rows are the contraction index).
__device__ __forceinline__ void issue_x_state(uint32_t tO, uint32_t x, uint32_t st) {
    constexpr uint32_t idesc = instr_desc_bf16(128, kD, false, true);
    const uint32_t xl = smem_desc_lo(x, 16), sl = smem_desc_lo(st, kD * 128u);
#pragma unroll
    for (int kk = 0; kk < kD / 16; ++kk) mma_ss_w(tO, xl + kk * 2u, kDescHi, sl + kk * 128u, kDescHi, idesc, kk > 0 ? 1u : 0u);
}
// Out[128 x 64] = X[128 x 64] St^T, St read K-major (its columns are the contraction index).
__device__ __forceinline__ void issue_x_state_t(uint32_t tO, uint32_t x, uint32_t st) {
    constexpr uint32_t idesc = instr_desc_bf16(128, kD, false, false);
    const uint32_t xl = smem_desc_lo(x, 16), sl = smem_desc_lo(st, 16);
#pragma unroll
    for (int kk = 0; kk < kD / 16; ++kk) mma_ss_w(tO, xl + kk * 2u, kDescHi, sl + kk * 2u, kDescHi, idesc, kk > 0 ? 1u : 0u);
}

#ifdef COTT_TIMING
// Debug build only: SM-clock stamps of CTA 0 for the first 32 items: role (0, 1: first thread of the
// two worker halves; 2: product, 3: load, 4: store thread) x item x slot.
__device__ long long g_bb_stamps[5 * 32 * 4];
#define BBSTAMP(role, g, slot) do { if (blockIdx.x == 0 && (g) < 32) g_bb_stamps[((role) * 32 + (g)) * 4 + (slot)] = clock64(); } while (0)
#else
#define BBSTAMP(role, g, slot) do { } while (0)
#endif

template <bool VARLEN>
__global__ void __launch_bounds__(kThreads, 2)
tc_bidir_bwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmDO,
                    const __grid_constant__ CUtensorMap tmDQ, const __grid_constant__ CUtensorMap tmDK,
                    const __grid_constant__ CUtensorMap tmDV, BidirBwdParams p) {
    // Tensor-memory columns.  Phase 1: S 64 | R 64.  Phase 2: dQ^ [2] 64 each (chunk parity, over
    // S and R, which have been copied by then) | dK^ 64 | dV' 64.
    constexpr uint32_t colS = 0, colR = 64, colQ = 0, colK = 128, colV = 192;
    // Six tiles, two state copies and the control block are all of the 113 KB a CTA can have when
    // two share an SM: there is no room to round the base up, so it must come aligned to the
    // 1024 bytes of the swizzle pattern (checked below, reported as an error otherwise).
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    uint8_t* gbase = smem_raw;
    const uint32_t bars = base + L::kOffCtl;
    // The tile pairs of both phases are one sequence of items: g = 0 .. 2 n - 1 are the (k, v)
    // (even g) and (q, dO) (odd g) pairs of phase 1, g = 2 n .. 4 n - 1 the (dO, q) (even g - 2 n)
    // and (v, k) (odd) pairs of phase 2; item g uses stage g % 3.
    // By stage: FULL (tiles landed; both phases, so its phase parity is (g / 3) & 1), READY (rows
    // normalised) and UFULL (product done, stage free) in phase 1, EDONE (gradient rows staged) in
    // phase 2.  PH1DONE, SBREADY once; the dQ^ accumulators QFULL / QDRAIN by chunk parity; KFULL /
    // KDRAIN for the dK^, dV' pair.
    // A wait asks whether the barrier's current phase differs in parity from the one named: it is
    // only meaningful while the barrier is less than two phases away from that one.  Hence every
    // waiter follows every phase of a barrier it uses -- the row workers wait for the tiles of
    // every item, also those the other half handles.
    enum { B_FULL = 0, B_READY = 24, B_UFULL = 48, B_EDONE = 72, B_PH1DONE = 96, B_SBREADY = 104, B_QFULL = 112,
           B_QDRAIN = 128, B_KFULL = 144, B_KDRAIN = 152, B_SFREE = 160 /* by stage: the stores have read the tiles */ };
    const uint32_t tmem_slot = bars + kCtlTmemSlot;
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + L::kOffCtl + kCtlTmemSlot);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kOffCtl + kCtlAbort);
    float* dm_red = reinterpret_cast<float*>(gbase + L::kOffCtl + L::kOffDmRed);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (base & 1023u) {
        if (tid == 0 && atomicCAS(p.status, 0, 1) == 0) {
            p.status[1] = (int)0x80007FF0u;
            p.status[2] = (int)blockIdx.x | (7 << 24);
        }
        return;
    }
    const int bh = blockIdx.x, bseq = bh / p.H, h = bh % p.H;
    const int b = VARLEN ? 0 : bseq;                   // batch coordinate of the tensor maps
    const int tok0 = VARLEN ? p.cu_seqlens[bseq] : 0;
    const int tok1 = VARLEN ? p.cu_seqlens[bseq + 1] : p.N;
    const int n_chunks = (tok1 - tok0 + kC - 1) / kC;
    const int n1 = 2 * n_chunks, n_items = 4 * n_chunks;
    // (a packed batch: the last chunk of a sequence may hold rows of the next one -- they are
    // normalised to zero in phase 1, and that chunk's gradient rows are stored one by one)
    const bool ragged_last = VARLEN && ((tok1 - tok0) % kC) != 0;
    const bool is_mma = warp == kWorkerWarps, is_copy = warp == kWorkerWarps + 1, is_store = warp == kWorkerWarps + 2;

    if (is_mma) {
        tmem_alloc(tmem_slot, 256);
        tmem_relinquish();
    }
    if (tid == 0) {
        for (int i = 0; i < L::kStages; ++i) {
            mbar_init(bars + B_FULL + 8 * i, 1);
            mbar_init(bars + B_READY + 8 * i, 128);
            mbar_init(bars + B_UFULL + 8 * i, 1);
            mbar_init(bars + B_EDONE + 8 * i, 128);
            mbar_init(bars + B_SFREE + 8 * i, 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bars + B_QFULL + 8 * i, 1);
            mbar_init(bars + B_QDRAIN + 8 * i, 128);
        }
        mbar_init(bars + B_PH1DONE, 1);
        mbar_init(bars + B_SBREADY, 256);
        mbar_init(bars + B_KFULL, 1);
        mbar_init(bars + B_KDRAIN, 128);
        *abort_flag = 0;
        abort_flag[3] = p.wait_limit_kcycles;
        mbar_fence_init();
        fence_proxy_async();
    }
    if (tid < 16) dm_red[tid] = 0.f;
    if (is_copy && lane == 0) {
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmDO);
    }
    if (is_store && lane == 0) {
        tma_prefetch_desc(&tmDQ); tma_prefetch_desc(&tmDK); tma_prefetch_desc(&tmDV);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_g;
    auto coords = [&](int which, int row, int& c1, int& c2) {
        const bool hf = (p.head_first_mask >> which) & 1;
        c1 = hf ? h : row; c2 = hf ? row : h;
    };
    auto load = [&](uint32_t dst, const CUtensorMap* tm, int which, uint32_t fb, int row) {
        int c1, c2;
        coords(which, row, c1, c2);
        tma_load_4d(dst, tm, fb, 0, c1, c2, b);
    };
    // (a packed batch reads cu_seqlens above: its launch is a plain one)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const float s_b = p.seq_len ? p.seq_len[bseq]
                                : (p.seq_len_scalar > 0.f ? p.seq_len_scalar : (float)(VARLEN ? max(tok1 - tok0, 1) : p.N));
    const float cfac = stab_factor(p.m[h], s_b);
    auto par = [&](int c) { return (uint32_t)(c & 1); };
    auto chunk_row = [&](int c) { return tok0 + c * kC; };
    // item g: its stage, the parity of its phase on the stage's FULL / READY / UFULL barriers, and
    // (phase 2) on the stage's EDONE barrier, whose first use is the first item >= 2 n on the stage
    auto stage_of = [&](int g) { return g % L::kStages; };
    auto fpar = [&](int g) { return (uint32_t)((g / L::kStages) & 1); };
    auto epar = [&](int g) {
        const int st = g % L::kStages, first = n1 + ((st - n1 % L::kStages) + L::kStages) % L::kStages;
        return (uint32_t)(((g - first) / L::kStages) & 1);
    };
    auto stage_base = [&](int g) { return (uint32_t)(stage_of(g) * 2) * (uint32_t)kTile; };

    if (is_copy) {
        // ------------------------------------------------------------------ load thread
        if (lane == 0 && n_chunks > 0) {
            for (int g = 0; g < n_items; ++g) {
                const int st = stage_of(g);
                // the stage's previous item: its product (phase 1) or its stores (phase 2) must be done with the tiles
                if (g >= L::kStages) {
                    const int prev = g - L::kStages;
                    if (!wait_or_abort(bars + (prev < n1 ? B_UFULL : B_SFREE) + 8 * st, prev < n1 ? fpar(prev) : epar(prev), abort_flag)) break;
                }
                const uint32_t fb = bars + B_FULL + 8 * st, dst = base + stage_base(g);
                BBSTAMP(3, g, 0);
                mbar_expect_tx(fb, 2 * kTile);
                if (g < n1) {
                    const int c = g >> 1, s = g & 1;       // (k, v) or (q, dO): the rows to normalise first
                    load(dst, s == 0 ? &tmK : &tmQ, s == 0 ? 1 : 0, fb, chunk_row(c));
                    load(dst + kTile, s == 0 ? &tmV : &tmDO, s == 0 ? 2 : 3, fb, chunk_row(c));
                } else {
                    const int j = g - n1, c = j >> 1, s = j & 1;   // (dO, q) or (v, k): the product's operand first
                    load(dst, s == 0 ? &tmDO : &tmV, s == 0 ? 3 : 2, fb, chunk_row(c));
                    load(dst + kTile, s == 0 ? &tmQ : &tmK, s == 0 ? 0 : 1, fb, chunk_row(c));
                }
            }
        }
    } else if (is_store) {
        // ------------------------------------------------------------------ store thread
        // The gradient rows of a phase-2 item are staged in its own tiles (dq over q; dk over k, dv
        // over v); the stage is free for the next load once the stores have read them.  (A thread of
        // its own: waiting for that read must not hold up the loads of the other stages.)
        if (lane == 0 && n_chunks > 0) {
            for (int g = n1; g < n_items; ++g) {
                const int st = stage_of(g);
                if (!wait_or_abort(bars + B_EDONE + 8 * st, epar(g), abort_flag)) break;
                BBSTAMP(4, g, 0);
                const int j = g - n1, c = j >> 1, trow = chunk_row(c);
                const uint32_t sb = base + stage_base(g);
                int c1, c2;
                if (!(ragged_last && c == n_chunks - 1)) {      // (else the workers stored the rows themselves)
                    if ((j & 1) == 0) {
                        coords(4, trow, c1, c2); tma_store_4d(&tmDQ, sb + kTile, 0, c1, c2, b);
                    } else {
                        coords(5, trow, c1, c2); tma_store_4d(&tmDK, sb + kTile, 0, c1, c2, b);
                        coords(6, trow, c1, c2); tma_store_4d(&tmDV, sb, 0, c1, c2, b);
                    }
                }
                tma_store_commit();
                tma_store_wait_read0();
                BBSTAMP(4, g, 1);
                mbar_arrive(bars + B_SFREE + 8 * st);
            }
            tma_store_wait_all0();
        }
    } else if (is_mma) {
        // ------------------------------------------------------------------ product thread
        if (lane == 0 && n_chunks > 0) {
            bool ok = true;
            for (int g = 0; g < n1; ++g) {
                // S (+)= K^^T V, R (+)= Q^^T dO: both operands MN-major (rows = tokens = contraction index)
                const int c = g >> 1, s = g & 1, st = stage_of(g);
                if (!wait_or_abort(bars + B_READY + 8 * st, fpar(g), abort_flag)) { ok = false; break; }
                BBSTAMP(2, g, 0);
                tc_fence_after();
                constexpr uint32_t idesc = instr_desc_bf16(kD, kD, true, true);
                const uint32_t at = base + stage_base(g);
                const uint32_t al = smem_desc_lo(at, 16384), bl = smem_desc_lo(at + kTile, 16384);
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)
                    mma_ss_w(tmem + (s == 0 ? colS : colR), al + kk * 128u, kDescHi, bl + kk * 128u, kDescHi, idesc, (c > 0 || kk > 0) ? 1u : 0u);
                tc_commit(bars + B_UFULL + 8 * st);
                BBSTAMP(2, g, 1);
                if (g + 1 == n1) tc_commit(bars + B_PH1DONE);
            }
            if (ok && wait_or_abort(bars + B_SBREADY, 0u, abort_flag)) {
                for (int g = n1; g < n_items; ++g) {
                    const int j = g - n1, c = j >> 1, s = j & 1;
                    if (!wait_or_abort(bars + B_FULL + 8 * stage_of(g), fpar(g), abort_flag)) break;
                    BBSTAMP(2, g, 0);
                    const uint32_t sb = base + stage_base(g);
                    if (s == 0) {
                        // dQ^ = dO S^T into the accumulator of the chunk's parity (drained by chunk c - 2)
                        const int a = c & 1;
                        if (c >= 2 && !wait_or_abort(bars + B_QDRAIN + 8 * a, (uint32_t)(((c >> 1) - 1) & 1), abort_flag)) break;
                        tc_fence_after();
                        issue_x_state_t(tmem + colQ + a * 64, sb, base + L::kOffSb);
                        tc_commit(bars + B_QFULL + 8 * a);
                        BBSTAMP(2, g, 1);
                    } else {
                        // dK^ = V R^T, dV' = K R (raw k rows: their scale is applied to the product's rows)
                        if (c >= 1 && !wait_or_abort(bars + B_KDRAIN, par(c - 1), abort_flag)) break;
                        tc_fence_after();
                        issue_x_state_t(tmem + colK, sb, base + L::kOffRb);
                        issue_x_state(tmem + colV, sb + kTile, base + L::kOffRb);
                        tc_commit(bars + B_KFULL);
                        BBSTAMP(2, g, 1);
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ row workers
        // Eight warps: TMEM lane quadrant q4 = warp & 3, half hw = warp >> 2.  Half 0 serves the even
        // items of both phases (k rows, then the dq rows), half 1 the odd ones (q rows, then dk and dv).
        bool alive = n_chunks > 0;
        auto wait = [&](uint32_t bar_, uint32_t parity) {
            if (alive && !wait_or_abort(bar_, parity, abort_flag)) alive = false;
            return alive;
        };
        const int q4 = warp & 3, hw = warp >> 2, row = q4 * 32 + lane;
        const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
        // phase 1: a thread normalises one row of the first tile of its items
        for (int g = 0; g < n1 && alive; ++g) {
            if (!wait(bars + B_FULL + 8 * stage_of(g), fpar(g))) break;
            if ((g & 1) != hw) continue;
            if ((tid & 127) == 0) BBSTAMP(hw, g, 0);
            const int c = g >> 1;
            uint8_t* tile = gbase + stage_base(g);
            uint4 w[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) w[j] = *reinterpret_cast<const uint4*>(tile + swz(row, j));
            float rn;
            normalise_row64(w, kEps, &rn);
            if (VARLEN && chunk_row(c) + row >= tok1) {          // a row of the next sequence
#pragma unroll
                for (int j = 0; j < 8; ++j) w[j] = make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) *reinterpret_cast<uint4*>(tile + swz(row, j)) = w[j];
            fence_proxy_async();
            mbar_arrive(bars + B_READY + 8 * stage_of(g));
            if ((tid & 127) == 0) BBSTAMP(hw, g, 2);
        }
        // the totals: fp32 in tensor memory (M = 64: row r sits in lane 32 (r / 16) + r % 16), bf16
        // copies into shared memory, and <S, R> for dm
        if (alive && wait(bars + B_PH1DONE, 0u)) {
            tc_fence_after();
            uint32_t sv[32], rv[32];
            tmem_ld32(tmem + lane_base + colS + hw * 32, sv);
            tmem_ld32(tmem + lane_base + colR + hw * 32, rv);
            tmem_wait_ld();
            float t = 0.f;
            if (lane < 16) {
                const int srow = q4 * 16 + lane;
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    *reinterpret_cast<uint4*>(gbase + L::kOffSb + swz(srow, hw * 4 + (i >> 3))) = pack8(&sv[i]);
                    *reinterpret_cast<uint4*>(gbase + L::kOffRb + swz(srow, hw * 4 + (i >> 3))) = pack8(&rv[i]);
                }
#pragma unroll
                for (int i = 0; i < 32; ++i) t = fmaf(__uint_as_float(sv[i]), __uint_as_float(rv[i]), t);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if (lane == 0) dm_red[warp] = t;
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bars + B_SBREADY);
        } else {
            alive = false;
        }
        // phase 2: every thread owns row `row` of its stage's chunks.
        // Projection (chain rule through x^ = x / max(||x||, eps)) of an accumulator row a, with
        // x^ = x rn in fp32 from the raw row: out = c rn (a - x^ <x^, a> [not clamped]), bf16, written
        // over the raw row.  Returns <x^ - bf16(x^), a>, bf16(x^) the operand phase 1 used.
        float dm_acc = 0.f;
        auto project = [&](uint32_t tacc, uint8_t* tile, float rn, bool clamped, int c, int which) {
            const __nv_bfloat16 hi = __float2bfloat16_rn(rn);
            const __nv_bfloat16 lo = __float2bfloat16_rn(rn - __bfloat162float(hi));
            const __nv_bfloat162 hi2 = __halves2bfloat162(hi, hi), lo2 = __halves2bfloat162(lo, lo);
            float d0 = 0.f, d1 = 0.f, e0 = 0.f, e1 = 0.f;
            // (two sweeps over the accumulator row, the raw row read from the tile chunk by chunk:
            // holding either next to the other does not fit the register budget)
#pragma unroll 1
            for (int hf = 0; hf < 2; ++hf) {
                uint32_t a[32];
                tmem_ld32(tacc + hf * 32, a);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint4 wj = *reinterpret_cast<const uint4*>(tile + swz(row, hf * 4 + j));
                    const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&wj);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        // <x, a> with the raw row (times rn afterwards) and <bf16(x^), a>
                        const float2 x = __bfloat1622float2(e[i]);
                        const float2 xh = __bfloat1622float2(__hfma2(e[i], hi2, __hmul2(e[i], lo2)));
                        const float a0 = __uint_as_float(a[8 * j + 2 * i]), a1 = __uint_as_float(a[8 * j + 2 * i + 1]);
                        d0 = fmaf(x.x, a0, d0); d1 = fmaf(x.y, a1, d1);
                        e0 = fmaf(xh.x, a0, e0); e1 = fmaf(xh.y, a1, e1);
                    }
                }
            }
            const float dot = (d0 + d1) * rn;                       // <x^, a>
            const float sc = cfac * rn, mc = (clamped ? 0.f : -dot * sc) * rn;   // (times rn: applied to the raw row)
#pragma unroll 1
            for (int hf = 0; hf < 2; ++hf) {
                uint32_t a[32];
                tmem_ld32(tacc + hf * 32, a);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint4 wj = *reinterpret_cast<const uint4*>(tile + swz(row, hf * 4 + j));
                    const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&wj);
                    uint4 o;
                    uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const float2 x = __bfloat1622float2(e[i]);
                        ow[i] = pack_bf16(fmaf(x.x, mc, __uint_as_float(a[8 * j + 2 * i]) * sc),
                                          fmaf(x.y, mc, __uint_as_float(a[8 * j + 2 * i + 1]) * sc));
                    }
                    if (VARLEN && ragged_last && c == n_chunks - 1) {
                        const long long grow = (long long)chunk_row(c) + row;
                        if (grow < tok1 && (hf * 4 + j) * 8 < p.out_w[which])
                            *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out_rows[which]) + grow * p.out_sn[which] +
                                                      (long long)h * p.out_sh[which] + (hf * 4 + j) * 8) = o;
                    } else {
                        *reinterpret_cast<uint4*>(tile + swz(row, hf * 4 + j)) = o;
                    }
                }
            }
            return dot - (e0 + e1);                                 // <x^ - bf16(x^), a>
        };
        for (int g = n1; g < n_items && alive; ++g) {
            if (!wait(bars + B_FULL + 8 * stage_of(g), fpar(g))) break;
            if (((g - n1) & 1) != hw) continue;
            if ((tid & 127) == 0) BBSTAMP(hw, g, 0);
            const int c = (g - n1) >> 1;
            // the raw q (half 0) or k (half 1) row, its norm
            uint8_t* xt = gbase + stage_base(g) + kTile;
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                const uint4 w0 = *reinterpret_cast<const uint4*>(xt + swz(row, j));
                const uint4 w1 = *reinterpret_cast<const uint4*>(xt + swz(row, j + 1));
                const __nv_bfloat162* e0 = reinterpret_cast<const __nv_bfloat162*>(&w0);
                const __nv_bfloat162* e1 = reinterpret_cast<const __nv_bfloat162*>(&w1);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 f0 = __bfloat1622float2(e0[i]), f1 = __bfloat1622float2(e1[i]);
                    a0 = fmaf(f0.x, f0.x, a0); a1 = fmaf(f0.y, f0.y, a1);
                    a2 = fmaf(f1.x, f1.x, a2); a3 = fmaf(f1.y, f1.y, a3);
                }
            }
            const float nrm = sqrtf((a0 + a1) + (a2 + a3));
            float rn = 1.0f / fmaxf(nrm, kEps);
            const bool clamped = !(nrm > kEps);
            if (VARLEN && chunk_row(c) + row >= tok1) rn = 0.f;      // a row of the next sequence: nothing to dm, never stored
            if (hw == 0) {
                const int a = c & 1;
                if (!wait(bars + B_QFULL + 8 * a, (uint32_t)((c >> 1) & 1))) break;
                if ((tid & 127) == 0) BBSTAMP(hw, g, 1);
                tc_fence_after();
                dm_acc += project(tmem + lane_base + colQ + a * 64, xt, rn, clamped, c, 0);
                tc_fence_before();
                mbar_arrive(bars + B_QDRAIN + 8 * a);
            } else {
                if (!wait(bars + B_KFULL, par(c))) break;
                if ((tid & 127) == 0) BBSTAMP(hw, g, 1);
                tc_fence_after();
                dm_acc += project(tmem + lane_base + colK, xt, rn, clamped, c, 1);
                // dv = c K^ R: the rows of K R times c / max(||k||, eps), over the v rows (both
                // products that read them are done)
                uint8_t* vt = gbase + stage_base(g);
                const float sc = cfac * rn;
#pragma unroll 1
                for (int hf = 0; hf < 2; ++hf) {
                    uint32_t a[32];
                    tmem_ld32(tmem + lane_base + colV + hf * 32, a);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(a[8 * j]) * sc, __uint_as_float(a[8 * j + 1]) * sc);
                        o.y = pack_bf16(__uint_as_float(a[8 * j + 2]) * sc, __uint_as_float(a[8 * j + 3]) * sc);
                        o.z = pack_bf16(__uint_as_float(a[8 * j + 4]) * sc, __uint_as_float(a[8 * j + 5]) * sc);
                        o.w = pack_bf16(__uint_as_float(a[8 * j + 6]) * sc, __uint_as_float(a[8 * j + 7]) * sc);
                        if (VARLEN && ragged_last && c == n_chunks - 1) {
                            const long long grow = (long long)chunk_row(c) + row;
                            if (grow < tok1 && (hf * 4 + j) * 8 < p.out_w[2])
                                *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out_rows[2]) + grow * p.out_sn[2] +
                                                          (long long)h * p.out_sh[2] + (hf * 4 + j) * 8) = o;
                        } else {
                            *reinterpret_cast<uint4*>(vt + swz(row, hf * 4 + j)) = o;
                        }
                    }
                }
                tc_fence_before();
                mbar_arrive(bars + B_KDRAIN);
            }
            fence_proxy_async();
            mbar_arrive(bars + B_EDONE + 8 * stage_of(g));
            if ((tid & 127) == 0) BBSTAMP(hw, g, 2);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dm_acc += __shfl_xor_sync(0xffffffffu, dm_acc, o);
        if (lane == 0) dm_red[8 + warp] = dm_acc;
    }
    tc_fence_before();
    __syncthreads();
    {
        int* last_flag = reinterpret_cast<int*>(&dm_red[16]);
        if (tid == 0) {
            // Fixed-order reduction of the CTA's dm term: <S, R> and the first-order terms.
            float t = 0.f;
            for (int i = 0; i < 16; ++i) t += dm_red[i];
            if (!*abort_flag) p.dm_partial[bh] = t;
            __threadfence();
            *last_flag = atomicAdd(&p.status[4], 1) == (int)gridDim.x - 1;
        }
        __syncthreads();
        if (*last_flag) {
            // Every CTA's sum is visible: dm_h = sum_b dc/dm(b,h) T_{b,h}, dc/dm = -ln(s_b) sigma(m_h)
            // (1 - sigma(m_h)) c_{b,h}; fixed order, so deterministic.  One warp per head.
            __threadfence();
            const int n_b = (int)gridDim.x / p.H;
            for (int hh = warp; hh < p.H; hh += kThreads / 32) {
                const float sg = 1.0f / (1.0f + expf(-p.m[hh]));
                float part = 0.f;
                for (int bb = lane; bb < n_b; bb += 32) {
                    const float sb2 = p.seq_len ? p.seq_len[bb]
                                                : (p.seq_len_scalar > 0.f ? p.seq_len_scalar
                                                   : (float)(VARLEN ? max(p.cu_seqlens[bb + 1] - p.cu_seqlens[bb], 1) : p.N));
                    const float ls = logf(sb2);
                    part += __ldcg(&p.dm_partial[(size_t)bb * p.H + hh]) * (-ls * sg * (1.0f - sg) * expf(-sg * ls));
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                if (lane == 0) p.dm_out[hh] = part;
            }
            if (tid == 0) p.status[4] = 0;
        }
    }
    if (*abort_flag) {
        // A wait gave up: let the copies and products in flight land, then report where.
        for (int i = 0; i < 100; ++i) __nanosleep(1000);
        __syncthreads();
        if (tid == 0 && atomicCAS(p.status, 0, 1) == 0) {
            p.status[1] = *abort_flag;
            p.status[2] = (int)blockIdx.x | (7 << 24);
        }
    }
    if (is_mma) tmem_dealloc(tmem, 256);
}

}  // namespace

cudaError_t launch_tc_bidir_bwd(const TcBwdFusedArgs& a, int B, int H, int N, cudaStream_t st) {
    const void* ptrs[7] = {a.q, a.k, a.v, a.d_o, a.dq, a.dk, a.dv};
    const RowLayout lays[7] = {a.l_qkv, a.l_qkv, a.l_v, a.l_do, a.l_dqkv, a.l_dqkv, a.l_dv};
    // real column counts (<= 64): tiles are zero-filled beyond them and stores clipped
    const int wk = a.w_k > 0 ? a.w_k : kD, wv = a.w_v > 0 ? a.w_v : kD;
    const int dims[7] = {wk, wk, wv, wv, wk, wk, wv};
    if (wk > kD || wv > kD) return cudaErrorInvalidValue;
    CUtensorMap tm[7];
    BidirBwdParams p;
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
    p.dm_partial = a.dm_partial; p.dm_out = a.dm_out; p.status = a.status;
    p.m = a.m; p.seq_len = a.seq_len; p.seq_len_scalar = a.seq_len_scalar;
    p.H = H; p.N = N;
    p.wait_limit_kcycles = wait_limit_kcycles();
    auto kern = a.cu_seqlens ? tc_bidir_bwd_kernel<true> : tc_bidir_bwd_kernel<false>;
    if (cudaError_t e = configure_smem_once(reinterpret_cast<const void*>(kern), L::kDynBytes); e != cudaSuccess)
        return e;
    // Two CTAs of 113 KB fill an SM's shared memory: ask for the largest carve-out.
    if (cudaError_t e = cudaFuncSetAttribute(reinterpret_cast<const void*>(kern), cudaFuncAttributePreferredSharedMemoryCarveout,
                                             (int)cudaSharedmemCarveoutMaxShared); e != cudaSuccess)
        return e;
    const int prof = profile_begin_launch(7, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(B * H));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = L::kDynBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = a.cu_seqlens ? 0 : 1;
    cudaError_t le = cudaLaunchKernelEx(&cfg, kern, tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], tm[6], p);
    profile_end_launch(prof, st);
    note_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace cott

#ifdef COTT_TIMING
// Debug build only: copies the stamps (5 roles x 32 items x 4 slots) to the host.
extern "C" int cott_debug_bidir_bwd_stamps(long long* out) {
    return (int)cudaMemcpyFromSymbol(out, cott::g_bb_stamps, sizeof(long long) * 640);
}
#endif
