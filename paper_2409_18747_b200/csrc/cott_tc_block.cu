// A block of at most 64 tokens per (b, h) on a caller-held state (bf16 I/O, fp32 state): the
// recurrence of Eq. 8 taken a block at a time,
//     o_t   = c ( q^_t S_in / c  +  sum_{j <= t in the block} (q^_t . k^_j) v_j ),
//     S_out = S_in + c K^^T V ,
// i.e. multi-token decode steps and short segments of a chunked prefill.  The state (d x d fp32,
// 64 KB at d = 128) is read and written once per block whatever the number of tokens, and it is
// almost all the traffic: the kernel is built so that several CTAs share an SM (two at d = 128:
// 90 KB of shared memory and 256 tensor-memory columns; more at d = 64) and one CTA's state
// transfer hides behind the others' work -- the generic walk, one CTA per SM with a 128-row
// tile, spent most of such a call waiting on its own state.
// One CTA per (b, h): tiles of 64 rows, products with M = 64.
#include "cott_internal.h"
#include "cott_sm100.cuh"
#include "cott_tc_common.cuh"

namespace cott {

using namespace sm100;
using namespace tc;

namespace {

constexpr int kT = 64;                        // rows of a tile (tokens of a block)
constexpr int kBox = kT * 128;                // one box: 64 rows x 64 bf16 columns
constexpr int kWorkerWarps = 8;
constexpr int kThreads = (kWorkerWarps + 1) * 32;

template <int D>
struct BL {
    static constexpr int NH = D / 64;
    static constexpr int kTile = NH * kBox;                    // q, k or v: 64 rows x D columns
    static constexpr int kOffQ = 0, kOffK = kTile, kOffV = 2 * kTile;
    static constexpr int kOffSb = 3 * kTile;                    // bf16 copy of the incoming state, D x D
    static constexpr int kOffPt = kOffSb + D * D * 2;           // masked scores, bf16, 64 x 64
    static constexpr int kOffCtl = kOffPt + kBox;
    static constexpr int kOffRx = 1024;                         // float [64]: c / max(||q||, eps)
    static constexpr int kCtlBytes = kOffRx + 256;
    static constexpr int kDynBytes = kOffCtl + kCtlBytes + 1024;
};

struct BlockParams {
    const float* state_in;   // NULL (zero state) or [BH, D * D], contains c
    float* state_out;        // NULL or [BH, D * D]
    int* status;
    const float* m; const float* seq_len; float seq_len_scalar;
    int H; int N;            // N <= 64 tokens
    int d_out;               // columns o really has
    int wait_limit_kcycles;
    int head_first_mask;     // bit i: in tensor map i (q, k, v, o) the head index comes before the token index
};

// K step kk (16 elements) of a K-major operand of D columns stored as 64-column boxes of 64 rows.
__device__ __forceinline__ uint32_t kstep(int kk) { return ((kk >> 2) * (uint32_t)kBox + (kk & 3) * 32u) >> 4; }

template <int D>
__global__ void __launch_bounds__(kThreads, D == 128 ? 2 : 4)
tc_block_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO, BlockParams p) {
    using L = BL<D>;
    constexpr int NH = L::NH;
    constexpr bool kBig = D == 128;
    // Tensor-memory columns: state D | scores 64, then the output accumulator D (in their place).
    constexpr uint32_t colS = 0, colP = D;
    constexpr uint32_t kCols = 2 * D;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + L::kOffCtl;
    enum { B_FULL = 0, B_READY = 8, B_PFULL = 16, B_PTREADY = 24, B_OFULL = 32, B_UFULL = 40, B_EDONE = 48 };
    const uint32_t tmem_slot = bars + kCtlTmemSlot;
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + L::kOffCtl + kCtlTmemSlot);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kOffCtl + kCtlAbort);
    float* rx_buf = reinterpret_cast<float*>(gbase + L::kOffCtl + L::kOffRx);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool is_ctrl = warp == kWorkerWarps;
    const int bh = blockIdx.x, b = bh / p.H, h = bh % p.H;

    if (is_ctrl) {
        tmem_alloc(tmem_slot, kCols);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(bars + B_FULL, 1);
        mbar_init(bars + B_READY, 256);
        mbar_init(bars + B_PFULL, 1);
        mbar_init(bars + B_PTREADY, 256);
        mbar_init(bars + B_OFULL, 1);
        mbar_init(bars + B_UFULL, 1);
        mbar_init(bars + B_EDONE, 256);
        *abort_flag = 0;
        abort_flag[3] = p.wait_limit_kcycles;
        mbar_fence_init();
        fence_proxy_async();
    }
    if (is_ctrl && lane == 0) {
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV); tma_prefetch_desc(&tmO);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_g;
    // The only kernel of its call; the state and the rows may come from the kernel before it.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (blockIdx.x == 0 && tid < 8) p.status[tid] = 0;

    const float s_b = p.seq_len ? p.seq_len[b] : (p.seq_len_scalar > 0.f ? p.seq_len_scalar : (float)p.N);
    const float cfac = stab_factor(p.m[h], s_b);

    if (is_ctrl) {
        if (lane == 0) {
            const uint32_t fb = bars + B_FULL;
            mbar_expect_tx(fb, 3u * L::kTile);
            auto load = [&](uint32_t dst, const CUtensorMap* tm, int which) {
                const bool hf = (p.head_first_mask >> which) & 1;
#pragma unroll
                for (int hh = 0; hh < NH; ++hh) tma_load_4d(dst + hh * kBox, tm, fb, hh * 64, hf ? h : 0, hf ? 0 : h, b);
            };
            load(base + L::kOffQ, &tmQ, 0);
            load(base + L::kOffK, &tmK, 1);
            load(base + L::kOffV, &tmV, 2);
            bool ok = wait_or_abort(bars + B_READY, 0u, abort_flag);
            if (ok) {
                tc_fence_after();
                {   // scores P = Q K^^T (64 x 64), both operands K-major
                    constexpr uint32_t idesc = instr_desc_bf16(64, 64, false, false);
                    const uint32_t xl = smem_desc_lo(base + L::kOffQ, 16), al = smem_desc_lo(base + L::kOffK, 16);
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk)
                        mma_ss_w(tmem + colP, xl + kstep(kk), kDescHi, al + kstep(kk), kDescHi, idesc, kk > 0);
                    tc_commit(bars + B_PFULL);
                }
                {   // state update S += K^^T V: both MN-major (rows = tokens = contraction index)
                    constexpr uint32_t idesc = instr_desc_bf16(D, D, true, true);
                    const uint32_t al = smem_desc_lo(base + L::kOffK, kBox), bl = smem_desc_lo(base + L::kOffV, kBox);
#pragma unroll
                    for (int kk = 0; kk < kT / 16; ++kk)
                        mma_ss_w(tmem + colS, al + kk * 128u, kDescHi, bl + kk * 128u, kDescHi, idesc, 1u);
                    tc_commit(bars + B_UFULL);
                }
                ok = wait_or_abort(bars + B_PTREADY, 0u, abort_flag);
            }
            if (ok) {
                // O = Q S_in + P~ V in the columns the scores had (every worker has read them)
                tc_fence_after();
                constexpr uint32_t idesc = instr_desc_bf16(64, D, false, true);
                const uint32_t xl = smem_desc_lo(base + L::kOffQ, 16), sl = smem_desc_lo(base + L::kOffSb, D * 128u);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk)
                    mma_ss_w(tmem + colP, xl + kstep(kk), kDescHi, sl + kk * 128u, kDescHi, idesc, kk > 0);
                const uint32_t pl = smem_desc_lo(base + L::kOffPt, 16), vl = smem_desc_lo(base + L::kOffV, kBox);
#pragma unroll
                for (int kk = 0; kk < kT / 16; ++kk)
                    mma_ss_w(tmem + colP, pl + kk * 2u, kDescHi, vl + kk * 128u, kDescHi, idesc, 1u);
                tc_commit(bars + B_OFULL);
                ok = wait_or_abort(bars + B_EDONE, 0u, abort_flag);
            }
            if (ok) {
                const bool hfo = (p.head_first_mask >> 3) & 1;
#pragma unroll
                for (int hh = 0; hh < NH; ++hh)
                    if (hh * 64 < p.d_out) tma_store_4d(&tmO, base + L::kOffQ + hh * kBox, hh * 64, hfo ? h : 0, hfo ? 0 : h, b);
                tma_store_commit();
                tma_store_wait_all0();
            }
        }
    } else {
        // ------------------------------------------------------------------ row workers
        bool alive = true;
        auto wait = [&](uint32_t bar_, uint32_t parity) {
            if (alive && !wait_or_abort(bar_, parity, abort_flag)) alive = false;
            return alive;
        };
        const int q4 = warp & 3, hw = warp >> 2;
        const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
        // Rows of a 64-row accumulator sit in lanes 0-15 of every quadrant; a 128-row one uses all lanes.
        const int row64 = q4 * 16 + (lane & 15);
        const bool has64 = lane < 16;
        const int srow = kBig ? q4 * 32 + lane : row64;          // state row of this thread
        const bool has_s = kBig || has64;
        constexpr int SW = D / 2;                                 // state / output columns per thread
        // ---- incoming state: fp32 into tensor memory (divided by c: the kernels keep states
        // without it), bf16 copy into shared memory for Q S_in
        {
            const float ic = 1.0f / cfac;
            const float* src = p.state_in ? p.state_in + (size_t)bh * D * D + (size_t)srow * D + hw * SW : nullptr;
#pragma unroll 1
            for (int pc = 0; pc < SW / 32; ++pc) {
                uint32_t r[32];
#pragma unroll
                for (int i = 0; i < 32; i += 4) {
                    float4 v = (src && has_s) ? __ldg(reinterpret_cast<const float4*>(src + pc * 32 + i)) : make_float4(0.f, 0.f, 0.f, 0.f);
                    r[i] = __float_as_uint(v.x * ic); r[i + 1] = __float_as_uint(v.y * ic);
                    r[i + 2] = __float_as_uint(v.z * ic); r[i + 3] = __float_as_uint(v.w * ic);
                }
                tmem_st32(tmem + lane_base + colS + hw * SW + pc * 32, r);
                if (has_s) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        const int col = hw * SW + pc * 32 + i;
                        *reinterpret_cast<uint4*>(gbase + L::kOffSb + (col >> 6) * (D * 128u) + swz(srow, (col & 63) >> 3)) = pack8(&r[i]);
                    }
                }
            }
            tmem_wait_st();
        }
        // ---- row norms: four threads per row (a quarter of the columns each)
        if (wait(bars + B_FULL, 0u)) {
            const int nrow = tid >> 2, part = tid & 3;            // 64 rows x 4 parts
            constexpr int CH = D / 32;                            // 16-byte chunks per part
            float sq = 0.f, sk = 0.f;
            uint4 wk[CH];
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                const int ch = part * CH + j;
                const uint32_t off = (ch >> 3) * (uint32_t)kBox + swz(nrow, ch & 7);
                const uint4 wq = *reinterpret_cast<const uint4*>(gbase + L::kOffQ + off);
                wk[j] = *reinterpret_cast<const uint4*>(gbase + L::kOffK + off);
                const __nv_bfloat162* eq = reinterpret_cast<const __nv_bfloat162*>(&wq);
                const __nv_bfloat162* ek = reinterpret_cast<const __nv_bfloat162*>(&wk[j]);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 fq = __bfloat1622float2(eq[i]), fk = __bfloat1622float2(ek[i]);
                    sq = fmaf(fq.x, fq.x, sq); sq = fmaf(fq.y, fq.y, sq);
                    sk = fmaf(fk.x, fk.x, sk); sk = fmaf(fk.y, fk.y, sk);
                }
            }
            sq += __shfl_xor_sync(0xffffffffu, sq, 1); sk += __shfl_xor_sync(0xffffffffu, sk, 1);
            sq += __shfl_xor_sync(0xffffffffu, sq, 2); sk += __shfl_xor_sync(0xffffffffu, sk, 2);
            const float rk = 1.0f / fmaxf(sqrtf(sk), kEps);
            if (part == 0) rx_buf[nrow] = cfac / fmaxf(sqrtf(sq), kEps);
#pragma unroll
            for (int j = 0; j < CH; ++j) {
                const int ch = part * CH + j;
                __nv_bfloat162* e = reinterpret_cast<__nv_bfloat162*>(&wk[j]);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 f = __bfloat1622float2(e[i]);
                    e[i] = __floats2bfloat162_rn(f.x * rk, f.y * rk);
                }
                *reinterpret_cast<uint4*>(gbase + L::kOffK + (ch >> 3) * (uint32_t)kBox + swz(nrow, ch & 7)) = wk[j];
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bars + B_READY);
        }
        // ---- causal mask on the 64 x 64 scores (diagonal kept, Eq. 6), bf16 into shared memory
        if (wait(bars + B_PFULL, 0u)) {
            tc_fence_after();
            uint32_t r[32];
            tmem_ld32(tmem + lane_base + colP + hw * 32, r);
            tmem_wait_ld();
            if (has64) {
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = (hw * 32 + j <= row64) ? r[j] : 0u;
#pragma unroll
                for (int i = 0; i < 32; i += 8)
                    *reinterpret_cast<uint4*>(gbase + L::kOffPt + swz(row64, hw * 4 + (i >> 3))) = pack8(&r[i]);
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bars + B_PTREADY);
        }
        // ---- output rows: scale by c / max(||q||, eps), round, stage where q was
        if (wait(bars + B_OFULL, 0u)) {
            tc_fence_after();
            const float rx = rx_buf[row64];
#pragma unroll 1
            for (int pc = 0; pc < SW / 32; ++pc) {
                const int c0 = hw * SW + pc * 32;
                uint32_t a[32];
                tmem_ld32(tmem + lane_base + colP + c0, a);
                tmem_wait_ld();
                if (has64) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(a[8 * j]) * rx, __uint_as_float(a[8 * j + 1]) * rx);
                        o.y = pack_bf16(__uint_as_float(a[8 * j + 2]) * rx, __uint_as_float(a[8 * j + 3]) * rx);
                        o.z = pack_bf16(__uint_as_float(a[8 * j + 4]) * rx, __uint_as_float(a[8 * j + 5]) * rx);
                        o.w = pack_bf16(__uint_as_float(a[8 * j + 6]) * rx, __uint_as_float(a[8 * j + 7]) * rx);
                        const int ch = (c0 >> 3) + j;
                        *reinterpret_cast<uint4*>(gbase + L::kOffQ + (ch >> 3) * (uint32_t)kBox + swz(row64, ch & 7)) = o;
                    }
                }
            }
            fence_proxy_async();
            mbar_arrive(bars + B_EDONE);
        }
        // ---- outgoing state, times c
        if (p.state_out != nullptr && wait(bars + B_UFULL, 0u)) {
            tc_fence_after();
            float* dst = p.state_out + (size_t)bh * D * D + (size_t)srow * D + hw * SW;
#pragma unroll 1
            for (int pc = 0; pc < SW / 32; ++pc) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + colS + hw * SW + pc * 32, r);
                tmem_wait_ld();
                if (has_s) {
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        *reinterpret_cast<float4*>(dst + pc * 32 + i) =
                            make_float4(__uint_as_float(r[i]) * cfac, __uint_as_float(r[i + 1]) * cfac,
                                        __uint_as_float(r[i + 2]) * cfac, __uint_as_float(r[i + 3]) * cfac);
                }
            }
        } else if (alive) {
            wait(bars + B_UFULL, 0u);       // no product may be in flight when the tensor memory is given back
        }
    }
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 100; ++i) __nanosleep(1000);
        __syncthreads();
        if (tid == 0 && atomicCAS(p.status, 0, 1) == 0) {
            p.status[1] = *abort_flag;
            p.status[2] = (int)blockIdx.x | (7 << 24);
        }
    }
    if (is_ctrl) tmem_dealloc(tmem, kCols);
}

template <int D>
cudaError_t launch_d(const CUtensorMap* tm, const BlockParams& p, int BH, cudaStream_t st) {
    auto kern = tc_block_fwd_kernel<D>;
    if (cudaError_t e = configure_smem_once(reinterpret_cast<const void*>(kern), BL<D>::kDynBytes); e != cudaSuccess)
        return e;
    const int prof = profile_begin_launch(6, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)BH);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = BL<D>::kDynBytes;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t le = cudaLaunchKernelEx(&cfg, kern, tm[0], tm[1], tm[2], tm[3], p);
    profile_end_launch(prof, st);
    note_launch();
    return le != cudaSuccess ? le : cudaGetLastError();
}

}  // namespace

cudaError_t launch_tc_block_fwd(const void* q, const void* k, const void* v, void* o, const RowLayout& l_qk,
                                const RowLayout& l_v, const RowLayout& l_o, const float* state_in, float* state_out,
                                int* status, const float* m, const float* seq_len, float seq_len_scalar, int B, int H,
                                int N, int d, int dk, int dv, cudaStream_t st) {
    if (N < 1 || N > kT || (d != 64 && d != 128) || dk > d || dv > d) return cudaErrorInvalidValue;
    BlockParams p;
    p.state_in = state_in; p.state_out = state_out; p.status = status;
    p.m = m; p.seq_len = seq_len; p.seq_len_scalar = seq_len_scalar;
    p.H = H; p.N = N; p.d_out = dv;
    p.wait_limit_kcycles = wait_limit_kcycles();
    const void* ptrs[4] = {q, k, v, o};
    const RowLayout lays[4] = {l_qk, l_qk, l_v, l_o};
    const int widths[4] = {dk, dk, dv, dv};
    CUtensorMap tm[4];
    p.head_first_mask = 0;
    for (int i = 0; i < 4; ++i) {
        bool hf = false;
        if (!make_tile_map(&tm[i], ptrs[i], B, H, N, widths[i], lays[i], &hf, kT)) return cudaErrorInvalidValue;
        p.head_first_mask |= (hf ? 1 : 0) << i;
    }
    return d == 64 ? launch_d<64>(tm, p, B * H, st) : launch_d<128>(tm, p, B * H, st);
}

}  // namespace cott
