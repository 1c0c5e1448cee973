// Bidirectional forward in one launch for d = 64 (bf16 I/O, fp32 accumulation): the right-hand
// side of Eq. 5, O = c Q^ (K^^T V), one CTA per (b, h).
//
// Phase 1 streams the k and v tiles of the sequence once: the k rows are normalised in shared
// memory (Eq. 2/3) and S += K^^T V accumulates the d x d state in tensor memory.  Phase 2 turns
// S into a bf16 operand and streams the q tiles: per chunk of 128 tokens one product Q S, whose
// fp32 rows are multiplied by c / max(||q||, eps) (the stabilisation factor of Eq. 4 and the
// query's row norm), rounded to bf16 and stored.  Every tensor is read or written exactly once,
// and nothing but the optional state export goes through global memory in between.
// Three CTAs share an SM (74 KB of shared memory and 128 tensor-memory columns each), so that a
// batch of a few hundred (b, h) pairs is resident all at once and one CTA's load latency hides
// behind the others' work; the output rows are staged in the q tile they were computed from.
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
constexpr int kThreads = (kWorkerWarps + 2) * 32;   // + product thread, copy thread

struct L {
    static constexpr int kSlots = 4;                        // ring of tile slots: (k, v) pairs in phase 1, q tiles in phase 2
    static constexpr int kOffSb = kSlots * kTile;           // bf16 copy of the state (64 x 64)
    static constexpr int kOffCtl = kOffSb + kD * kD * 2;
    static constexpr int kCtlBytes = 1024;                  // mbarriers, tensor-memory slot, abort flag and wait limit
    static constexpr int kDynBytes = kOffCtl + kCtlBytes + 1024;
};

struct BidirParams {
    float* state_out;        // NULL, or [BH, 64 * 64]: c K^^T V
    int* status;
    const float* m; const float* seq_len; float seq_len_scalar;
    int H; int N;
    int clear_status;
    int wait_limit_kcycles;
    int head_first_mask;     // bit i: in tensor map i (q, k, v, o) the head index comes before the token index
    // Packed variable-length batch (NULL: dense): every tensor is [1, H, total_tokens, d], sequence
    // b = rows cu_seqlens[b] .. cu_seqlens[b + 1] - 1, one CTA per (sequence, head).  The k rows of
    // the next sequence in a ragged last chunk are normalised to zero (they then add nothing to
    // the state), and that chunk's output rows leave as plain stores: o as global memory with its
    // token and head strides in elements.
    const int* cu_seqlens;
    void* out_rows; long long out_sn, out_sh; int out_w;
};

template <bool VARLEN>
__global__ void __launch_bounds__(kThreads, 3)
tc_bidir_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO, BidirParams p) {
    // Tensor-memory columns: S 64 | O 64.
    constexpr uint32_t colS = 0, colO = 64;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + L::kOffCtl;
    // Phase 1 (per chunk, pairs indexed by chunk parity): KV_FULL, K_READY, U_FULL.
    // Phase 2 (per chunk): Q_FULL[4], Q_READ[4] and E_DONE[4] by tile slot, O_FULL[2] and O_DRAIN[2] by chunk parity.
    // A waiter may only ask for the phase that follows the last one it saw complete on the same
    // barrier: asking for one further ahead passes at once (a fresh barrier counts as having
    // completed an odd phase), and asking for one the barrier has left two or more behind
    // blocks until the next phase of that parity.  Hence PH1_DONE for "the whole state is
    // there": the row workers take alternate chunks and do not follow every U_FULL phase.
    enum { B_KVFULL = 0, B_KREADY = 16, B_UFULL = 32, B_SBREADY = 48, B_PH1DONE = 56, B_QFULL = 64, B_OFULL = 96, B_ODRAIN = 112,
           B_EDONE = 128, B_QREAD = 160 };
    const uint32_t tmem_slot = bars + kCtlTmemSlot;
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + L::kOffCtl + kCtlTmemSlot);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kOffCtl + kCtlAbort);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x, bseq = bh / p.H, h = bh % p.H;
    const int b = VARLEN ? 0 : bseq;                   // batch coordinate of the tensor maps
    const int tok0 = VARLEN ? p.cu_seqlens[bseq] : 0;
    const int tok1 = VARLEN ? p.cu_seqlens[bseq + 1] : p.N;
    const int n_chunks = (tok1 - tok0 + kC - 1) / kC;
    const bool ragged_last = VARLEN && ((tok1 - tok0) % kC) != 0;
    auto chunk_row = [&](int c) { return tok0 + c * kC; };
    const bool is_mma = warp == kWorkerWarps, is_copy = warp == kWorkerWarps + 1;

    if (is_mma) {
        tmem_alloc(tmem_slot, 128);
        tmem_relinquish();
    }
    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(bars + B_KVFULL + 8 * i, 1);
            mbar_init(bars + B_KREADY + 8 * i, 128);
            mbar_init(bars + B_UFULL + 8 * i, 1);
            mbar_init(bars + B_OFULL + 8 * i, 1);
            mbar_init(bars + B_ODRAIN + 8 * i, 256);
        }
        mbar_init(bars + B_SBREADY, 256);
        mbar_init(bars + B_PH1DONE, 1);
        for (int i = 0; i < 4; ++i) {
            mbar_init(bars + B_QFULL + 8 * i, 1); mbar_init(bars + B_EDONE + 8 * i, 256); mbar_init(bars + B_QREAD + 8 * i, 256);
        }
        *abort_flag = 0;
        abort_flag[3] = p.wait_limit_kcycles;
        mbar_fence_init();
        fence_proxy_async();
    }
    if (is_copy && lane == 0) {
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmO);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_g;
    auto load = [&](uint32_t dst, const CUtensorMap* tm, int which, uint32_t fb, int row) {
        const bool hf = (p.head_first_mask >> which) & 1;
        tma_load_4d(dst, tm, fb, 0, hf ? h : row, hf ? row : h, b);
    };
    // The first kernel of a library call may follow a kernel that produced its inputs: nothing
    // is read before the wait.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.clear_status && blockIdx.x == 0 && tid < 8) p.status[tid] = 0;

    const float s_b = p.seq_len ? p.seq_len[bseq]
                                : (p.seq_len_scalar > 0.f ? p.seq_len_scalar : (float)(VARLEN ? max(tok1 - tok0, 1) : p.N));
    const float cfac = stab_factor(p.m[h], s_b);
    auto par2 = [&](int c) { return (uint32_t)((c >> 1) & 1); };
    auto par4 = [&](int c) { return (uint32_t)((c >> 2) & 1); };

    if (is_copy) {
        // ------------------------------------------------------------------ copy thread
        if (lane == 0 && n_chunks > 0) {
            bool ok = true;
            // phase 1: (k, v) of chunk c into slots 2 (c & 1), 2 (c & 1) + 1
            for (int c = 0; c < n_chunks && ok; ++c) {
                if (c >= 2 && !wait_or_abort(bars + B_UFULL + 8 * (c & 1), par2(c - 2), abort_flag)) { ok = false; break; }
                const uint32_t fb = bars + B_KVFULL + 8 * (c & 1), dst = base + (uint32_t)(2 * (c & 1)) * kTile;
                mbar_expect_tx(fb, 2 * kTile);
                load(dst, &tmK, 1, fb, chunk_row(c));
                load(dst + kTile, &tmV, 2, fb, chunk_row(c));
            }
            // phase 2: q of chunk c into slot c & 3, once the slot's last reader is done: a (k, v)
            // pair of phase 1 (the state update of the last chunk with that parity), then the
            // store of the output rows of chunk c - 4, which were staged in the slot
            auto store = [&](int e) {
                const bool hfo = (p.head_first_mask >> 3) & 1;
                // (the rows of a ragged last chunk of a packed batch were stored by the workers)
                if (!(ragged_last && e == n_chunks - 1))
                    tma_store_4d(&tmO, base + (uint32_t)(e & 3) * kTile, 0, hfo ? h : chunk_row(e), hfo ? chunk_row(e) : h, b);
                tma_store_commit();
            };
            for (int c = 0; c < n_chunks && ok; ++c) {
                if (c < 4) {
                    const int par = (c & 3) >> 1;                         // stage of phase 1 that used the slot
                    const int last = ((n_chunks - 1) & 1) == par ? n_chunks - 1 : n_chunks - 2;
                    if (last >= 0 && !wait_or_abort(bars + B_UFULL + 8 * par, par2(last), abort_flag)) { ok = false; break; }
                } else {
                    // stores issued so far: chunks 0 .. c - 3; all but the last must have read their tile
                    tma_store_wait_read1();
                }
                const uint32_t fb = bars + B_QFULL + 8 * (c & 3);
                mbar_expect_tx(fb, kTile);
                load(base + (uint32_t)(c & 3) * kTile, &tmQ, 0, fb, chunk_row(c));
                // the output rows of chunk c - 2, if staged meanwhile, go out between the loads
                if (c >= 2) {
                    const int e = c - 2;
                    if (!wait_or_abort(bars + B_EDONE + 8 * (e & 3), par4(e), abort_flag)) { ok = false; break; }
                    store(e);
                }
            }
            for (int e = (n_chunks >= 2 ? n_chunks - 2 : 0); e < n_chunks && ok; ++e) {
                if (!wait_or_abort(bars + B_EDONE + 8 * (e & 3), par4(e), abort_flag)) break;
                store(e);
            }
            tma_store_wait_all0();
        }
    } else if (is_mma) {
        // ------------------------------------------------------------------ product thread
        if (lane == 0 && n_chunks > 0) {
            bool ok = true;
            for (int c = 0; c < n_chunks; ++c) {
                // S (+)= K^^T V: both operands MN-major (rows = tokens = contraction index)
                if (!wait_or_abort(bars + B_KREADY + 8 * (c & 1), par2(c), abort_flag)) { ok = false; break; }
                tc_fence_after();
                constexpr uint32_t idesc = instr_desc_bf16(kD, kD, true, true);
                const uint32_t kt = base + (uint32_t)(2 * (c & 1)) * kTile;
                const uint32_t al = smem_desc_lo(kt, 16384), bl = smem_desc_lo(kt + kTile, 16384);
#pragma unroll
                for (int kk = 0; kk < kC / 16; ++kk)
                    mma_ss_w(tmem + colS, al + kk * 128u, kDescHi, bl + kk * 128u, kDescHi, idesc, (c > 0 || kk > 0) ? 1u : 0u);
                tc_commit(bars + B_UFULL + 8 * (c & 1));
                if (c + 1 == n_chunks) tc_commit(bars + B_PH1DONE);
            }
            if (ok && wait_or_abort(bars + B_SBREADY, 0u, abort_flag)) {
                for (int c = 0; c < n_chunks; ++c) {
                    // O = Q S: Q K-major, the bf16 state MN-major (its rows are the contraction index)
                    if (!wait_or_abort(bars + B_QFULL + 8 * (c & 3), par4(c), abort_flag)) break;
                    // (the one accumulator was drained by the epilogue of the chunk before)
                    if (c >= 1 && !wait_or_abort(bars + B_ODRAIN + 8 * ((c - 1) & 1), par2(c - 1), abort_flag)) break;
                    tc_fence_after();
                    constexpr uint32_t idesc = instr_desc_bf16(128, kD, false, true);
                    const uint32_t xl = smem_desc_lo(base + (uint32_t)(c & 3) * kTile, 16), sl = smem_desc_lo(base + L::kOffSb, kD * 128u);
#pragma unroll
                    for (int kk = 0; kk < kD / 16; ++kk)
                        mma_ss_w(tmem + colO, xl + kk * 2u, kDescHi, sl + kk * 128u, kDescHi, idesc, kk > 0);
                    tc_commit(bars + B_OFULL + 8 * (c & 1));
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ row workers
        // Eight warps: TMEM lane quadrant q4 = warp & 3, half hw = warp >> 2.
        bool alive = n_chunks > 0;
        auto wait = [&](uint32_t bar_, uint32_t parity) {
            if (alive && !wait_or_abort(bar_, parity, abort_flag)) alive = false;
            return alive;
        };
        const int q4 = warp & 3, hw = warp >> 2, row = q4 * 32 + lane;
        const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
        // phase 1: the two halves take alternate chunks; a thread normalises one k row
        for (int c = hw; c < n_chunks && alive; c += 2) {
            if (!wait(bars + B_KVFULL + 8 * (c & 1), par2(c))) break;
            uint8_t* tile = gbase + (2 * (c & 1)) * kTile;
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
            mbar_arrive(bars + B_KREADY + 8 * (c & 1));
        }
        // the state: fp32 in tensor memory (M = 64: row r sits in lane 32 (r / 16) + r % 16), bf16
        // copy into shared memory, optional export times c
        if (alive && wait(bars + B_PH1DONE, 0u)) {
            tc_fence_after();
            uint32_t r[32];
            tmem_ld32(tmem + lane_base + colS + hw * 32, r);
            tmem_wait_ld();
            if (lane < 16) {
                const int srow = q4 * 16 + lane;
#pragma unroll
                for (int i = 0; i < 32; i += 8)
                    *reinterpret_cast<uint4*>(gbase + L::kOffSb + swz(srow, hw * 4 + (i >> 3))) = pack8(&r[i]);
                if (p.state_out != nullptr) {
                    float* dst = p.state_out + (size_t)bh * kD * kD + (size_t)srow * kD + hw * 32;
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        *reinterpret_cast<float4*>(dst + i) = make_float4(__uint_as_float(r[i]) * cfac, __uint_as_float(r[i + 1]) * cfac,
                                                                           __uint_as_float(r[i + 2]) * cfac, __uint_as_float(r[i + 3]) * cfac);
                }
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bars + B_SBREADY);
        } else {
            alive = false;
        }
        // phase 2: every thread owns row `row` and the 32 accumulator columns of its half
        for (int c = 0; c < n_chunks && alive; ++c) {
            if (!wait(bars + B_QFULL + 8 * (c & 3), par4(c))) break;
            // c / max(||q||, eps): each of the two threads of a row sums the whole row (cheaper
            // than meeting through shared memory)
            const uint8_t* qt = gbase + (c & 3) * kTile;
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
            for (int j = 0; j < 8; j += 2) {
                const uint4 w0 = *reinterpret_cast<const uint4*>(qt + swz(row, j));
                const uint4 w1 = *reinterpret_cast<const uint4*>(qt + swz(row, j + 1));
                const __nv_bfloat162* e0 = reinterpret_cast<const __nv_bfloat162*>(&w0);
                const __nv_bfloat162* e1 = reinterpret_cast<const __nv_bfloat162*>(&w1);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 f0 = __bfloat1622float2(e0[i]), f1 = __bfloat1622float2(e1[i]);
                    a0 = fmaf(f0.x, f0.x, a0); a1 = fmaf(f0.y, f0.y, a1);
                    a2 = fmaf(f1.x, f1.x, a2); a3 = fmaf(f1.y, f1.y, a3);
                }
            }
            const float rx = cfac / fmaxf(sqrtf((a0 + a1) + (a2 + a3)), kEps);
            mbar_arrive(bars + B_QREAD + 8 * (c & 3));
            // the product has read the q tile and filled the accumulator: drain it, then stage
            // the rows where q was
            if (!wait(bars + B_OFULL + 8 * (c & 1), par2(c))) break;
            tc_fence_after();
            uint32_t a[32];
            tmem_ld32(tmem + lane_base + colO + hw * 32, a);
            tmem_wait_ld();
            tc_fence_before();
            mbar_arrive(bars + B_ODRAIN + 8 * (c & 1));
            // (both threads of a row sum the whole q row: the other one must be done with it)
            if (!wait(bars + B_QREAD + 8 * (c & 3), par4(c))) break;
            uint8_t* out = gbase + (c & 3) * kTile;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint4 o;
                o.x = pack_bf16(__uint_as_float(a[8 * j]) * rx, __uint_as_float(a[8 * j + 1]) * rx);
                o.y = pack_bf16(__uint_as_float(a[8 * j + 2]) * rx, __uint_as_float(a[8 * j + 3]) * rx);
                o.z = pack_bf16(__uint_as_float(a[8 * j + 4]) * rx, __uint_as_float(a[8 * j + 5]) * rx);
                o.w = pack_bf16(__uint_as_float(a[8 * j + 6]) * rx, __uint_as_float(a[8 * j + 7]) * rx);
                if (VARLEN && ragged_last && c == n_chunks - 1) {
                    const long long grow = (long long)chunk_row(c) + row;
                    if (grow < tok1 && (hw * 4 + j) * 8 < p.out_w)
                        *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(p.out_rows) + grow * p.out_sn + (long long)h * p.out_sh +
                                                  (hw * 4 + j) * 8) = o;
                } else {
                    *reinterpret_cast<uint4*>(out + swz(row, hw * 4 + j)) = o;
                }
            }
            fence_proxy_async();
            mbar_arrive(bars + B_EDONE + 8 * (c & 3));
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // A wait gave up: let the copies and products in flight land, then report where.
        for (int i = 0; i < 100; ++i) __nanosleep(1000);
        __syncthreads();
        if (tid == 0 && atomicCAS(p.status, 0, 1) == 0) {
            p.status[1] = *abort_flag;
            p.status[2] = (int)blockIdx.x | (5 << 24);
        }
    }
    if (is_mma) tmem_dealloc(tmem, 128);
}

}  // namespace

cudaError_t launch_tc_bidir_fwd(const void* q, const void* k, const void* v, void* o, const RowLayout& l_qkv,
                                const RowLayout& l_v, const RowLayout& l_o, float* state_out, int* status, const float* m, const float* seq_len,
                                float seq_len_scalar, int B, int H, int N, cudaStream_t st, int dk, int dv,
                                const int* cu_seqlens, int total_tokens) {
    const void* ptrs[4] = {q, k, v, o};
    const RowLayout lays[4] = {l_qkv, l_qkv, l_v, l_o};
    // real column counts (<= 64): tiles are zero-filled beyond them and stores clipped
    const int dims[4] = {dk > 0 ? dk : kD, dk > 0 ? dk : kD, dv > 0 ? dv : kD, dv > 0 ? dv : kD};
    CUtensorMap tm[4];
    BidirParams p;
    p.head_first_mask = 0;
    // A packed batch is one tensor of total_tokens rows per head (batch extent 1).
    const int map_B = cu_seqlens ? 1 : B, map_N = cu_seqlens ? total_tokens : N;
    for (int i = 0; i < 4; ++i) {
        bool hf = false;
        if (dims[i] > kD || !make_tile_map(&tm[i], ptrs[i], map_B, H, map_N, dims[i], lays[i], &hf)) return cudaErrorInvalidValue;
        p.head_first_mask |= (hf ? 1 : 0) << i;
    }
    p.cu_seqlens = cu_seqlens;
    {
        const RowLayout lo = resolve_layout(l_o, H, map_N, dims[3]);
        p.out_rows = o; p.out_sn = lo.sn; p.out_sh = lo.sh; p.out_w = dims[3];
    }
    if (cu_seqlens && state_out) return cudaErrorInvalidValue;
    p.state_out = state_out; p.status = status; p.m = m; p.seq_len = seq_len; p.seq_len_scalar = seq_len_scalar;
    p.H = H; p.N = N; p.clear_status = 1;
    p.wait_limit_kcycles = wait_limit_kcycles();
    auto kern = cu_seqlens ? tc_bidir_fwd_kernel<true> : tc_bidir_fwd_kernel<false>;
    if (cudaError_t e = configure_smem_once(reinterpret_cast<const void*>(kern), L::kDynBytes); e != cudaSuccess)
        return e;
    const int prof = profile_begin_launch(4, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(B * H));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = L::kDynBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = cu_seqlens ? 0 : 1;      // (a packed batch reads cu_seqlens before anything else: a plain launch)
    cudaError_t le = cudaLaunchKernelEx(&cfg, kern, tm[0], tm[1], tm[2], tm[3], p);
    profile_end_launch(prof, st);
    note_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace cott
