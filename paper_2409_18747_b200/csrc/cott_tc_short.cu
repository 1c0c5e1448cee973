// Short sequences (N <= 128 tokens, bf16 I/O, fp32 accumulation): the left-hand, quadratic side
// of Eq. 5 / the masked product of Eq. 6 with no running state at all.  The paper notes that
// this side is the cheaper one when the sequence is shorter than the head size; here the
// threshold is the 128-token tile of the tensor core.
//
// The rows of all (b, h) pairs of a dense [B,H,N,d] tensor are one long list of B H N rows, so a
// tile of 128 rows holds k = floor(128 / N) whole sequences of consecutive pairs.  One CTA per
// tile: a single score product P = Q K^^T (128 x 128), a block-diagonal mask -- a row keeps the
// columns of its own sequence, up to and including its own position when causal --, a single
// product O = P~ V, rows scaled by c / max(||q||, eps) (Eq. 2-4) and stored.  No state update,
// no state copy, no second launch; B H / k CTAs instead of B H, two per SM.
#include "cott_internal.h"
#include "cott_sm100.cuh"
#include "cott_tc_common.cuh"

namespace cott {

using namespace sm100;
using namespace tc;

namespace {

constexpr int kRows = 128;                    // rows of a tile
constexpr int kWorkerWarps = 8;
constexpr int kThreads = (kWorkerWarps + 1) * 32;     // + control warp (copies and products)

template <int D>
struct SL {
    static constexpr int kTile = kRows * D * 2;       // D / 64 boxes of 128 rows x 64 columns
    static constexpr int kOffQ = 0, kOffK = kTile, kOffV = 2 * kTile;
    static constexpr int kOffCtl = 3 * kTile;
    static constexpr int kDynBytes = kOffCtl + 1024 + 1024;
};

struct ShortParams {
    int* status;
    const float* m; const float* seq_len; float seq_len_scalar;
    int H; int N; int BH;
    int seqs_per_tile;       // k
    int causal;
    int d_out;               // columns o really has
    int wait_limit_kcycles;
};

template <int D>
__global__ void __launch_bounds__(kThreads, 2)
tc_short_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO, ShortParams p) {
    using L = SL<D>;
    constexpr int NH = D / 64;
    // Tensor-memory columns: scores, later the output accumulator 0..127 | masked bf16 scores 128..191.
    constexpr uint32_t colP = 0, colPt = 128;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bars = base + L::kOffCtl;
    enum { B_FULL = 0, B_KREADY = 8, B_PFULL = 16, B_PTREADY = 24, B_OFULL = 32, B_EDONE = 40 };
    const uint32_t tmem_slot = bars + kCtlTmemSlot;
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + L::kOffCtl + kCtlTmemSlot);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(gbase + L::kOffCtl + kCtlAbort);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool is_ctrl = warp == kWorkerWarps;
    const int rows_used = p.seqs_per_tile * p.N;              // rows of this tile that hold sequences
    const int row0 = (int)blockIdx.x * rows_used;             // first row of the tile in the list of B H N rows

    if (is_ctrl) {
        tmem_alloc(tmem_slot, 256);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(bars + B_FULL, 1);
        mbar_init(bars + B_KREADY, 256);
        mbar_init(bars + B_PFULL, 1);
        mbar_init(bars + B_PTREADY, 256);
        mbar_init(bars + B_OFULL, 1);
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
    // The only kernel of its call: it may follow a kernel that produced its inputs.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (blockIdx.x == 0 && tid < 8) p.status[tid] = 0;

    if (is_ctrl) {
        if (lane == 0) {
            // The copies bring rows_used rows per box; the rows below them are zeroed by the workers.
            const uint32_t fb = bars + B_FULL;
            mbar_expect_tx(fb, 3u * NH * (uint32_t)rows_used * 128u);
#pragma unroll
            for (int hh = 0; hh < NH; ++hh) {
                tma_load_4d(base + L::kOffQ + hh * 16384, &tmQ, fb, hh * 64, row0, 0, 0);
                tma_load_4d(base + L::kOffK + hh * 16384, &tmK, fb, hh * 64, row0, 0, 0);
                tma_load_4d(base + L::kOffV + hh * 16384, &tmV, fb, hh * 64, row0, 0, 0);
            }
            bool ok = wait_or_abort(bars + B_KREADY, 0u, abort_flag);
            if (ok) {
                // P = Q K^^T: both operands K-major
                tc_fence_after();
                constexpr uint32_t idesc = instr_desc_bf16(128, 128, false, false);
                const uint32_t xl = smem_desc_lo(base + L::kOffQ, 16), al = smem_desc_lo(base + L::kOffK, 16);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = ((kk >> 2) * 16384u + (kk & 3) * 32u) >> 4;
                    mma_ss_w(tmem + colP, xl + off, kDescHi, al + off, kDescHi, idesc, kk > 0);
                }
                tc_commit(bars + B_PFULL);
                ok = wait_or_abort(bars + B_PTREADY, 0u, abort_flag);
            }
            if (ok) {
                // O = P~ V: P~ from tensor memory (8 columns per K = 16), V MN-major; the
                // accumulator takes the place of the scores, which every worker has read
                tc_fence_after();
                constexpr uint32_t idesc = instr_desc_bf16(128, D, false, true);
                const uint32_t bl = smem_desc_lo(base + L::kOffV, 16384);
#pragma unroll
                for (int kk = 0; kk < kRows / 16; ++kk)
                    mma_ts_w(tmem + colP, tmem + colPt + kk * 8u, bl + kk * 128u, kDescHi, idesc, kk > 0);
                tc_commit(bars + B_OFULL);
                ok = wait_or_abort(bars + B_EDONE, 0u, abort_flag);
            }
            if (ok) {
#pragma unroll
                for (int hh = 0; hh < NH; ++hh)
                    if (hh * 64 < p.d_out) tma_store_4d(&tmO, base + L::kOffQ + hh * 16384, hh * 64, row0, 0, 0);
                tma_store_commit();
                tma_store_wait_all0();
            }
        }
    } else {
        // ------------------------------------------------------------------ row workers
        // TMEM lane quadrant q4 = warp & 3, column half hf = warp >> 2: two threads per row.
        bool alive = true;
        auto wait = [&](uint32_t bar_, uint32_t parity) {
            if (alive && !wait_or_abort(bar_, parity, abort_flag)) alive = false;
            return alive;
        };
        const int q4 = warp & 3, hf = warp >> 2, row = q4 * 32 + lane;
        const uint32_t lane_base = (uint32_t)(q4 * 32) << 16;
        const bool valid = row < rows_used;
        // rows the copies do not write: zero (a zero v row times a zero score must not be NaN)
        if (!valid) {
#pragma unroll
            for (int j = 0; j < 4 * NH; ++j) {
                const int ch = hf * 4 * NH + j;                       // 16-byte chunk of the row
                const uint32_t off = (ch >> 3) * 16384u + swz(row, ch & 7);
                *reinterpret_cast<uint4*>(gbase + L::kOffQ + off) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(gbase + L::kOffK + off) = make_uint4(0, 0, 0, 0);
                *reinterpret_cast<uint4*>(gbase + L::kOffV + off) = make_uint4(0, 0, 0, 0);
            }
        }
        // the row's sequence: pair index, scaling factor, first row of the sequence in the tile
        const int seq = row / p.N;
        const int pair = (int)blockIdx.x * p.seqs_per_tile + seq;
        const bool live = valid && pair < p.BH;
        float cfac = 0.f;
        if (live) {
            const int b = pair / p.H, h = pair % p.H;
            const float s_b = p.seq_len ? p.seq_len[b] : (p.seq_len_scalar > 0.f ? p.seq_len_scalar : (float)p.N);
            cfac = stab_factor(p.m[h], s_b);
        }
        const int lo = seq * p.N, hi = live ? (p.causal ? row : lo + p.N - 1) : -1;
        float rx = 0.f;
        if (wait(bars + B_FULL, 0u)) {
            // ||q|| and ||k|| over the whole row (each of the row's two threads sums all of it);
            // k is normalised in place, each thread its half of the columns
            float sq = 0.f, sk = 0.f;
#pragma unroll
            for (int ch = 0; ch < 8 * NH; ++ch) {
                const uint32_t off = (ch >> 3) * 16384u + swz(row, ch & 7);
                const uint4 wq = *reinterpret_cast<const uint4*>(gbase + L::kOffQ + off);
                const uint4 wk = *reinterpret_cast<const uint4*>(gbase + L::kOffK + off);
                const __nv_bfloat162* eq = reinterpret_cast<const __nv_bfloat162*>(&wq);
                const __nv_bfloat162* ek = reinterpret_cast<const __nv_bfloat162*>(&wk);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 fq = __bfloat1622float2(eq[i]), fk = __bfloat1622float2(ek[i]);
                    sq = fmaf(fq.x, fq.x, sq); sq = fmaf(fq.y, fq.y, sq);
                    sk = fmaf(fk.x, fk.x, sk); sk = fmaf(fk.y, fk.y, sk);
                }
            }
            rx = cfac / fmaxf(sqrtf(sq), kEps);
            const float rk = 1.0f / fmaxf(sqrtf(sk), kEps);
#pragma unroll
            for (int j = 0; j < 4 * NH; ++j) {
                const int ch = hf * 4 * NH + j;
                uint4* pk = reinterpret_cast<uint4*>(gbase + L::kOffK + (ch >> 3) * 16384u + swz(row, ch & 7));
                uint4 w = *pk;
                __nv_bfloat162* e = reinterpret_cast<__nv_bfloat162*>(&w);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float2 f = __bfloat1622float2(e[i]);
                    e[i] = __floats2bfloat162_rn(f.x * rk, f.y * rk);
                }
                *pk = w;
            }
            fence_proxy_async();
            mbar_arrive(bars + B_KREADY);
        }
        if (wait(bars + B_PFULL, 0u)) {
            // block-diagonal (causal) mask on this thread's 64 columns, packed to bf16 pairs
            tc_fence_after();
#pragma unroll 1
            for (int pc = 0; pc < 2; ++pc) {
                const int c0 = hf * 64 + pc * 32;
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + colP + c0, r);
                tmem_wait_ld();
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int ja = c0 + 2 * j, jb = ja + 1;
                    const float a = (ja >= lo && ja <= hi) ? __uint_as_float(r[2 * j]) : 0.f;
                    const float b2 = (jb >= lo && jb <= hi) ? __uint_as_float(r[2 * j + 1]) : 0.f;
                    pk[j] = pack_bf16(a, b2);
                }
                tmem_st16(tmem + lane_base + colPt + (c0 >> 1), pk);
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(bars + B_PTREADY);
        }
        if (wait(bars + B_OFULL, 0u)) {
            // this thread's D / 2 accumulator columns: scale, round, stage where q was
            tc_fence_after();
#pragma unroll 1
            for (int pc = 0; pc < D / 64; ++pc) {
                const int c0 = hf * (D / 2) + pc * 32;
                uint32_t a[32];
                tmem_ld32(tmem + lane_base + colP + c0, a);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint4 o;
                    o.x = pack_bf16(__uint_as_float(a[8 * j]) * rx, __uint_as_float(a[8 * j + 1]) * rx);
                    o.y = pack_bf16(__uint_as_float(a[8 * j + 2]) * rx, __uint_as_float(a[8 * j + 3]) * rx);
                    o.z = pack_bf16(__uint_as_float(a[8 * j + 4]) * rx, __uint_as_float(a[8 * j + 5]) * rx);
                    o.w = pack_bf16(__uint_as_float(a[8 * j + 6]) * rx, __uint_as_float(a[8 * j + 7]) * rx);
                    const int ch = (c0 >> 3) + j;
                    *reinterpret_cast<uint4*>(gbase + L::kOffQ + (ch >> 3) * 16384u + swz(row, ch & 7)) = o;
                }
            }
            fence_proxy_async();
            tc_fence_before();
            mbar_arrive(bars + B_EDONE);
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
            p.status[2] = (int)blockIdx.x | (6 << 24);
        }
    }
    if (is_ctrl) tmem_dealloc(tmem, 256);
}

template <int D>
cudaError_t launch_d(const CUtensorMap* tm, const ShortParams& p, int tiles, cudaStream_t st) {
    auto kern = tc_short_fwd_kernel<D>;
    if (cudaError_t e = configure_smem_once(reinterpret_cast<const void*>(kern), SL<D>::kDynBytes); e != cudaSuccess)
        return e;
    const int prof = profile_begin_launch(5, st);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)tiles);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = SL<D>::kDynBytes;
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

cudaError_t launch_tc_short_fwd(const void* q, const void* k, const void* v, void* o, int* status, const float* m,
                                const float* seq_len, float seq_len_scalar, int B, int H, int N, int d, int dk, int dv,
                                int causal, cudaStream_t st) {
    if (N < 1 || N > kRows || (d != 64 && d != 128) || dk > d || dv > d) return cudaErrorInvalidValue;
    ShortParams p;
    p.status = status; p.m = m; p.seq_len = seq_len; p.seq_len_scalar = seq_len_scalar;
    p.H = H; p.N = N; p.BH = B * H;
    p.seqs_per_tile = kRows / N;
    p.causal = causal; p.d_out = dv;
    p.wait_limit_kcycles = wait_limit_kcycles();
    const int rows_used = p.seqs_per_tile * N;
    const long long rows = (long long)B * H * N;
    const void* ptrs[4] = {q, k, v, o};
    const int widths[4] = {dk, dk, dv, dv};
    CUtensorMap tm[4];
    for (int i = 0; i < 4; ++i)
        if (!make_rows_map(&tm[i], ptrs[i], rows, widths[i], rows_used)) return cudaErrorInvalidValue;
    const int tiles = (p.BH + p.seqs_per_tile - 1) / p.seqs_per_tile;
    return d == 64 ? launch_d<64>(tm, p, tiles, st) : launch_d<128>(tm, p, tiles, st);
}

}  // namespace cott
