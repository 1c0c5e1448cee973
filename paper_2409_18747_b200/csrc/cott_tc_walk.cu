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
#include "cott_internal.h"
#include "cott_sm100.cuh"

namespace cott {

using namespace sm100;

namespace {

constexpr int kChunk = 128;
constexpr int kTcThreads = 128;
constexpr uint64_t kWaitTimeoutNs = 2000000000ull;  // 2 s: far above any legitimate wait

struct TcWalkParams {
    const float* init;      // [BH, n_groups, d*d] unscaled prefix / suffix / total states, or NULL
    float* state_out;       // MODE_STATE: [BH, n_groups, d*d] partial states (unscaled)
    float* dm_partial;      // EPI_DV: [BH, n_groups]
    int* status;            // workspace status word
    const float* m; const float* seq_len; float seq_len_scalar;
    int H; int N; int group; int n_groups;
    int norm_bv;            // 1: Bv is normalised in shared memory, 0: A is
    int x_norm;             // 1: rows of X are normalised (scale applied in the epilogue)
    int epilogue;           // Epilogue enum
    int reverse;            // 1: walk backward in time, mask keeps columns >= row
};

template <int D> struct Smem {
    static constexpr int kTile = kChunk * D * 2;          // one 128 x D bf16 tile
    static constexpr int kStage = 3 * kTile;              // X, A, Bv
    static constexpr int kSb = D * D * 2;                 // bf16 copy of the state
    static constexpr int kOffSb = 2 * kStage;
    static constexpr int kOffBar = kOffSb + kSb;          // full[2], mma, proj, tmem slot, dm scratch
    // d = 64 only, and only for launches whose epilogue needs a fourth tile: a dedicated
    // buffer behind everything else (d = 128 reuses the A slot instead).
    static constexpr int kOffProj = (kOffBar + 128 + 1023) / 1024 * 1024;
    static constexpr int dyn_bytes(bool with_proj) {
        return ((with_proj && D == 64) ? kOffProj + kTile : kOffBar + 128) + 1024;  // + align slack
    }
};

// tcgen05.mma chains (one thread).  All tiles are 128-byte-swizzled rows of 128 bytes; a
// 128-column (256-byte) row is split into two half tiles 16 KB apart.
template <int D>
__device__ __forceinline__ void issue_p(uint32_t tP, uint32_t x, uint32_t a) {
    constexpr uint32_t idesc = instr_desc_bf16(128, 128, false, false);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = (kk >> 2) * 16384u + (kk & 3) * 32u;
        mma_ss(tP, smem_desc(x + off, 16, 1024), smem_desc(a + off, 16, 1024), idesc, kk > 0);
    }
}
template <int D>
__device__ __forceinline__ void issue_xs(uint32_t tO, uint32_t x, uint32_t sb) {
    constexpr uint32_t idesc = instr_desc_bf16(128, D, false, true);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = (kk >> 2) * 16384u + (kk & 3) * 32u;
        mma_ss(tO, smem_desc(x + off, 16, 1024), smem_desc(sb + kk * 2048u, D * 128u, 1024), idesc,
               kk > 0);
    }
}
template <int D>
__device__ __forceinline__ void issue_pb(uint32_t tO, uint32_t p, uint32_t bv, bool acc_first) {
    constexpr uint32_t idesc = instr_desc_bf16(128, D, false, true);
#pragma unroll
    for (int kk = 0; kk < kChunk / 16; ++kk) {
        const uint32_t off = (kk >> 2) * 16384u + (kk & 3) * 32u;
        mma_ss(tO, smem_desc(p + off, 16, 1024), smem_desc(bv + kk * 2048u, 16384, 1024), idesc,
               (kk > 0) || acc_first);
    }
}
template <int D>
__device__ __forceinline__ void issue_atb(uint32_t tS, uint32_t a, uint32_t bv, bool acc_first) {
    constexpr uint32_t idesc = instr_desc_bf16(D, D, true, true);
#pragma unroll
    for (int kk = 0; kk < kChunk / 16; ++kk)
        mma_ss(tS, smem_desc(a + kk * 2048u, 16384, 1024), smem_desc(bv + kk * 2048u, 16384, 1024),
               idesc, (kk > 0) || acc_first);
}

// Sum of squares of a 128-byte-swizzled tile row held by this thread.
template <int D>
__device__ __forceinline__ float row_sumsq(const uint8_t* tile, int row) {
    float ss = 0.f;
#pragma unroll
    for (int ch = 0; ch < D / 8; ++ch) {
        uint4 w = *reinterpret_cast<const uint4*>(tile + (ch >> 3) * 16384 + swz(row, ch & 7));
        const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f = __bfloat1622float2(e[i]);
            ss += f.x * f.x + f.y * f.y;
        }
    }
    return ss;
}

// x^ = x / max(||x||, eps) on this thread's row, in place, rounded to bf16.
template <int D>
__device__ __forceinline__ void normalise_row_inplace(uint8_t* tile, int row) {
    uint4 w[D / 8];
    float ss = 0.f;
#pragma unroll
    for (int ch = 0; ch < D / 8; ++ch) {
        w[ch] = *reinterpret_cast<const uint4*>(tile + (ch >> 3) * 16384 + swz(row, ch & 7));
        const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w[ch]);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f = __bfloat1622float2(e[i]);
            ss += f.x * f.x + f.y * f.y;
        }
    }
    const float r = 1.0f / fmaxf(sqrtf(ss), kEps);
#pragma unroll
    for (int ch = 0; ch < D / 8; ++ch) {
        const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w[ch]);
        uint4 o;
        uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float2 f = __bfloat1622float2(e[i]);
            ow[i] = pack_bf16(f.x * r, f.y * r);
        }
        *reinterpret_cast<uint4*>(tile + (ch >> 3) * 16384 + swz(row, ch & 7)) = o;
    }
}

enum { MODE_STATE = 0, MODE_CAUSAL = 1, MODE_READOUT = 2 };

template <int D, int MODE>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_walk_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmA,
               const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmP,
               const __grid_constant__ CUtensorMap tmO, TcWalkParams p) {
    using L = Smem<D>;
    constexpr int NH = D / 64;                       // 64-column half tiles per row
    constexpr uint32_t kTmemCols = (D == 128) ? 512 : 256;
    constexpr uint32_t colS = 0, colO = D, colP = 2 * D;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_full0 = base + L::kOffBar, bar_full1 = bar_full0 + 8, bar_mma = bar_full0 + 16;
    const uint32_t bar_proj = bar_full0 + 24, tmem_slot = bar_full0 + 32;
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + L::kOffBar + 32);
    float* dm_red = reinterpret_cast<float*>(gbase + L::kOffBar + 64);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = blockIdx.x % p.n_groups, bh = blockIdx.x / p.n_groups;
    const int b = bh / p.H, h = bh % p.H;
    const int tok0 = g * p.group;
    const int tok1 = min(p.N, tok0 + p.group);
    const int n_chunks = (tok1 - tok0 + kChunk - 1) / kChunk;
    const bool with_proj = (MODE != MODE_STATE) && (p.epilogue != EPI_PLAIN);

    if (warp == 0) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(bar_full0, 1); mbar_init(bar_full1, 1); mbar_init(bar_mma, 1);
        mbar_init(bar_proj, 1);
        mbar_fence_init();
        fence_proxy_async();
        tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmA); tma_prefetch_desc(&tmB);
        tma_prefetch_desc(&tmP); tma_prefetch_desc(&tmO);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot_g;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;

    const float s_b = p.seq_len ? p.seq_len[b] : (p.seq_len_scalar > 0.f ? p.seq_len_scalar : (float)p.N);
    const float cfac = stab_factor(p.m[h], s_b);

    // State row held by this thread: with M = 128 accumulator rows map to lanes one to one;
    // with M = 64 row r sits in lane (r % 16) + 32 * (r / 16).
    const bool owns_row = (D == 128) || (lane < 16);
    const int srow = (D == 128) ? tid : warp * 16 + (lane & 15);
    const uint32_t sb = base + L::kOffSb;

    bool has_state = false;
    if (p.init != nullptr) {
        // Load the group's initial state into TMEM (fp32) and its bf16 copy into shared memory.
        const float* src = p.init + ((size_t)bh * p.n_groups + g) * D * D + (size_t)srow * D;
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 32) {
            uint32_t r[32];
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
                float4 v = owns_row ? *reinterpret_cast<const float4*>(src + c0 + i)
                                    : make_float4(0.f, 0.f, 0.f, 0.f);
                r[i] = __float_as_uint(v.x); r[i + 1] = __float_as_uint(v.y);
                r[i + 2] = __float_as_uint(v.z); r[i + 3] = __float_as_uint(v.w);
            }
            if (MODE == MODE_CAUSAL) tmem_st32(tmem + lane_base + colS + c0, r);
            if (owns_row) {
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    uint4 w;
                    w.x = pack_bf16(__uint_as_float(r[i]), __uint_as_float(r[i + 1]));
                    w.y = pack_bf16(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                    w.z = pack_bf16(__uint_as_float(r[i + 4]), __uint_as_float(r[i + 5]));
                    w.w = pack_bf16(__uint_as_float(r[i + 6]), __uint_as_float(r[i + 7]));
                    const int col = c0 + i;  // first of 8 columns
                    const uint32_t off = (col >> 6) * (D * 128u) + swz(srow, (col & 63) >> 3);
                    *reinterpret_cast<uint4*>(gbase + L::kOffSb + off) = w;
                }
            }
        }
        if (MODE == MODE_CAUSAL) tmem_wait_st();
        fence_proxy_async();
        has_state = true;
    }

    bool failed = false;
    uint32_t mma_phase = 0;
    float dm_acc = 0.f;
    auto stage_x = [&](int s) { return base + s * L::kStage; };
    auto stage_a = [&](int s) { return base + s * L::kStage + L::kTile; };
    auto stage_b = [&](int s) { return base + s * L::kStage + 2 * L::kTile; };
    // Chunk visited at step c (time runs backward when p.reverse).
    auto chunk_row = [&](int c) { return tok0 + (p.reverse ? (n_chunks - 1 - c) : c) * kChunk; };

    auto issue_loads = [&](int c) {
        const int s = c & 1;
        const uint32_t bar = s ? bar_full1 : bar_full0;
        const int row = chunk_row(c);
        constexpr uint32_t n_tiles = (MODE == MODE_STATE) ? 2 : (MODE == MODE_CAUSAL ? 3 : 1);
        mbar_expect_tx(bar, n_tiles * L::kTile);
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) {
            if (MODE != MODE_STATE) tma_load_3d(stage_x(s) + hh * 16384, &tmX, bar, hh * 64, row, bh);
            if (MODE != MODE_READOUT) {
                tma_load_3d(stage_a(s) + hh * 16384, &tmA, bar, hh * 64, row, bh);
                tma_load_3d(stage_b(s) + hh * 16384, &tmB, bar, hh * 64, row, bh);
            }
        }
    };

    if (tid == 0 && n_chunks > 0) issue_loads(0);

    for (int c = 0; c < n_chunks; ++c) {
        const int s = c & 1;
        if (tid == 0 && c + 1 < n_chunks) {
            tma_store_wait_read0();  // the store that read a slot of stage s^1 has drained
            issue_loads(c + 1);
        }
        bool ok = mbar_wait(s ? bar_full1 : bar_full0, (uint32_t)((c >> 1) & 1), kWaitTimeoutNs);
        if (__syncthreads_or(!ok)) { failed = true; break; }

        uint8_t* xs = gbase + s * L::kStage;
        uint8_t* as = xs + L::kTile;
        uint8_t* bs = xs + 2 * L::kTile;
        // Row scale of X (thread t owns token row t of the chunk), applied in the epilogue.
        float rx = cfac;
        if (MODE != MODE_STATE && p.x_norm) rx = cfac / fmaxf(sqrtf(row_sumsq<D>(xs, tid)), kEps);
        if (MODE != MODE_READOUT) {
            normalise_row_inplace<D>(p.norm_bv ? bs : as, tid);
            fence_proxy_async();
        }
        tc_fence_before();
        __syncthreads();

        if (tid == 0) {
            tc_fence_after();
            if (MODE == MODE_CAUSAL) {
                issue_p<D>(tmem + colP, stage_x(s), stage_a(s));
                if (has_state) issue_xs<D>(tmem + colO, stage_x(s), sb);
                issue_atb<D>(tmem + colS, stage_a(s), stage_b(s), has_state);
            } else if (MODE == MODE_STATE) {
                issue_atb<D>(tmem + colS, stage_a(s), stage_b(s), has_state);
            } else {
                issue_xs<D>(tmem + colO, stage_x(s), sb);
            }
            tc_commit(bar_mma);
        }
        ok = mbar_wait(bar_mma, mma_phase, kWaitTimeoutNs);
        mma_phase ^= 1;
        if (__syncthreads_or(!ok)) { failed = true; break; }
        tc_fence_after();

        // The tile the epilogue needs besides the accumulator (raw q, k or v rows): fetched
        // now so that it lands while the scores are processed.  d = 128 reuses the A slot
        // (both MMAs that read A have completed); d = 64 has a dedicated buffer.
        uint8_t* proj = (D == 128) ? as : gbase + L::kOffProj;
        const uint32_t proj_u = (D == 128) ? stage_a(s) : base + L::kOffProj;
        if (with_proj && tid == 0) {
            if (D == 64) tma_store_wait_read0();  // previous chunk's store out of this buffer
            mbar_expect_tx(bar_proj, L::kTile);
#pragma unroll
            for (int hh = 0; hh < NH; ++hh)
                tma_load_3d(proj_u + hh * 16384, &tmP, bar_proj, hh * 64, chunk_row(c), bh);
        }

        if (MODE == MODE_CAUSAL) {
            // Masked scores -> bf16 operand in the X slot (X is dead: both MMAs that read it
            // have completed).  Forward: row i keeps columns j <= i (the diagonal stays,
            // Eq. 6); backward in time: columns j >= i.
#pragma unroll
            for (int c0 = 0; c0 < kChunk; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + colP + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    uint4 w;
                    uint32_t* ww = reinterpret_cast<uint32_t*>(&w);
#pragma unroll
                    for (int j = 0; j < 8; j += 2) {
                        const int col = c0 + i + j;
                        const bool k0 = p.reverse ? (col >= tid) : (col <= tid);
                        const bool k1 = p.reverse ? (col + 1 >= tid) : (col + 1 <= tid);
                        ww[j >> 1] = pack_bf16(k0 ? __uint_as_float(r[i + j]) : 0.f,
                                               k1 ? __uint_as_float(r[i + j + 1]) : 0.f);
                    }
                    const int col = c0 + i;
                    *reinterpret_cast<uint4*>(xs + (col >> 6) * 16384 + swz(tid, (col & 63) >> 3)) = w;
                }
            }
            // bf16 copy of the updated state for the next chunk's X State product.
            if (c + 1 < n_chunks) {
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld32(tmem + lane_base + colS + c0, r);
                    tmem_wait_ld();
                    if (owns_row) {
#pragma unroll
                        for (int i = 0; i < 32; i += 8) {
                            uint4 w;
                            w.x = pack_bf16(__uint_as_float(r[i]), __uint_as_float(r[i + 1]));
                            w.y = pack_bf16(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                            w.z = pack_bf16(__uint_as_float(r[i + 4]), __uint_as_float(r[i + 5]));
                            w.w = pack_bf16(__uint_as_float(r[i + 6]), __uint_as_float(r[i + 7]));
                            const int col = c0 + i;
                            const uint32_t off = (col >> 6) * (D * 128u) + swz(srow, (col & 63) >> 3);
                            *reinterpret_cast<uint4*>(gbase + L::kOffSb + off) = w;
                        }
                    }
                }
            }
            fence_proxy_async();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
                issue_pb<D>(tmem + colO, stage_x(s), stage_b(s), has_state);
                tc_commit(bar_mma);
            }
            ok = mbar_wait(bar_mma, mma_phase, kWaitTimeoutNs);
            mma_phase ^= 1;
            if (__syncthreads_or(!ok)) { failed = true; break; }
            tc_fence_after();
        }
        has_state = true;

        if (MODE != MODE_STATE) {
            uint8_t* stage_out = bs;
            uint32_t stage_out_u = stage_b(s);
            float coef = 0.f, rp = 1.f;
            if (with_proj) {
                ok = mbar_wait(bar_proj, (uint32_t)(c & 1), kWaitTimeoutNs);
                if (__syncthreads_or(!ok)) { failed = true; break; }
                stage_out = proj; stage_out_u = proj_u;
                // First pass over the accumulator row: <p, g> and ||p||^2.
                float ss = 0.f, dp = 0.f;
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 32) {
                    uint32_t r[32];
                    tmem_ld32(tmem + lane_base + colO + c0, r);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        const int col = c0 + i;
                        uint4 w = *reinterpret_cast<const uint4*>(proj + (col >> 6) * 16384 +
                                                                  swz(tid, (col & 63) >> 3));
                        const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            float2 f = __bfloat1622float2(e[j]);
                            ss += f.x * f.x + f.y * f.y;
                            dp += f.x * __uint_as_float(r[i + 2 * j]) + f.y * __uint_as_float(r[i + 2 * j + 1]);
                        }
                    }
                }
                if (p.epilogue == EPI_PROJ) {
                    // g = rx * acc;  out = (g - p^ <p^, g>) / max(||p||, eps), clamped branch: g / eps
                    const float nrm = sqrtf(ss);
                    rp = 1.0f / fmaxf(nrm, kEps);
                    coef = nrm > kEps ? dp * rx * rp * rp : 0.f;
                } else {
                    dm_acc += dp * rx / cfac;  // <dV', v> with dV' = (rx / c) * acc
                }
            }
            // Output rows: scale, (project,) round to bf16, stage, TMA store.
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + colO + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    const int col = c0 + i;
                    uint8_t* dst = stage_out + (col >> 6) * 16384 + swz(tid, (col & 63) >> 3);
                    float v[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = __uint_as_float(r[i + j]) * rx;
                    if (with_proj && p.epilogue == EPI_PROJ) {
                        uint4 w = *reinterpret_cast<const uint4*>(dst);
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
                    *reinterpret_cast<uint4*>(dst) = w;
                }
            }
            fence_proxy_async();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
#pragma unroll
                for (int hh = 0; hh < NH; ++hh)
                    tma_store_3d(&tmO, stage_out_u + hh * 16384, hh * 64, chunk_row(c), bh);
                tma_store_commit();
            }
        }
    }

    if (MODE == MODE_STATE && !failed && p.state_out != nullptr) {
        // Partial state of this group, fp32, unscaled.
        float* dst = p.state_out + ((size_t)bh * p.n_groups + g) * D * D + (size_t)srow * D;
#pragma unroll
        for (int c0 = 0; c0 < D; c0 += 32) {
            uint32_t r[32];
            tmem_ld32(tmem + lane_base + colS + c0, r);
            tmem_wait_ld();
            if (owns_row) {
#pragma unroll
                for (int i = 0; i < 32; i += 4)
                    *reinterpret_cast<float4*>(dst + c0 + i) =
                        make_float4(__uint_as_float(r[i]), __uint_as_float(r[i + 1]),
                                    __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
            }
        }
    }
    if (MODE != MODE_STATE && p.dm_partial != nullptr && !failed) {
        // Fixed-order reduction of <dV', V> over the CTA.
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) dm_acc += __shfl_xor_sync(0xffffffffu, dm_acc, o);
        if (lane == 0) dm_red[warp] = dm_acc;
        __syncthreads();
        if (tid == 0)
            p.dm_partial[(size_t)bh * p.n_groups + g] = (dm_red[0] + dm_red[1]) + (dm_red[2] + dm_red[3]);
    }

    if (failed) {
        if (tid == 0) {
            atomicExch(p.status, 1);
            // Give outstanding loads a bounded chance to land before shared memory is released.
            mbar_wait(bar_full0, 0, 1000000ull);
            mbar_wait(bar_full1, 0, 1000000ull);
        }
    }
    if (tid == 0) tma_store_wait_all0();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) ==
                cudaSuccess && qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// Tensor map over a contiguous [BH, N, d] bf16 tensor: box = 128 rows x 64 columns of one
// (b,h) slice, 128-byte swizzle; rows past N read as zero and are not written.
bool make_tile_map(CUtensorMap* map, const void* ptr, int BH, int N, int d) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)BH};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)N * d * 2};
    cuuint32_t box[3] = {64, (cuuint32_t)kChunk, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides,
                     box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

template <int D, int MODE>
cudaError_t launch_mode(const CUtensorMap* tm, const TcWalkParams& p, int BH, cudaStream_t st) {
    auto kern = tc_walk_kernel<D, MODE>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Smem<D>::dyn_bytes(true));
        if (e != cudaSuccess) return e;
        configured = true;
    }
    const bool with_proj = (MODE != MODE_STATE) && (p.epilogue != EPI_PLAIN);
    kern<<<dim3((unsigned)(BH * p.n_groups)), kTcThreads, Smem<D>::dyn_bytes(with_proj), st>>>(
        tm[0], tm[1], tm[2], tm[3], tm[4], p);
    note_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_tc_walk(const TcWalkArgs& a, int B, int H, int N, int d, cudaStream_t st) {
    const int BH = B * H;
    // Unused operands still need a valid map: point them at a tensor that exists.
    const void* any = a.x ? a.x : a.a;
    const void* ptrs[5] = {a.x ? a.x : any, a.a ? a.a : any, a.bv ? a.bv : any,
                           a.proj ? a.proj : any, a.out ? a.out : any};
    CUtensorMap tm[5];
    for (int i = 0; i < 5; ++i)
        if (!make_tile_map(&tm[i], ptrs[i], BH, N, d)) return cudaErrorInvalidValue;
    TcWalkParams p;
    p.init = a.init; p.state_out = a.state_out; p.dm_partial = a.dm_partial; p.status = a.status;
    p.m = a.m; p.seq_len = a.seq_len; p.seq_len_scalar = a.seq_len_scalar;
    p.H = H; p.N = N; p.group = a.group; p.n_groups = a.n_groups;
    p.norm_bv = a.norm_bv; p.x_norm = a.x_norm; p.epilogue = a.epilogue; p.reverse = a.reverse;
    if (d == 128) {
        if (a.mode == MODE_STATE) return launch_mode<128, MODE_STATE>(tm, p, BH, st);
        if (a.mode == MODE_CAUSAL) return launch_mode<128, MODE_CAUSAL>(tm, p, BH, st);
        return launch_mode<128, MODE_READOUT>(tm, p, BH, st);
    }
    if (d == 64) {
        if (a.mode == MODE_STATE) return launch_mode<64, MODE_STATE>(tm, p, BH, st);
        if (a.mode == MODE_CAUSAL) return launch_mode<64, MODE_CAUSAL>(tm, p, BH, st);
        return launch_mode<64, MODE_READOUT>(tm, p, BH, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace cott
