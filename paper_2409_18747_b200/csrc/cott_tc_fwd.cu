// Tensor-core forward kernels (bf16 I/O, fp32 accumulation and state) for d in {64,128}.
//
// One CTA walks one sequence group in chunks of 128 tokens.  Per chunk (Eq. 6 restricted to
// the chunk plus the running state of Eq. 7/8):
//     P   = Q K^^T                      (128 x 128, tcgen05, fp32 in TMEM)
//     O   = (P . M) V  +  Q S_prev      (two MMAs into one TMEM accumulator)
//     S  += K^^T V                      (d x d fp32 state, resident in TMEM)
// Q, K, V tiles arrive by TMA with the 128-byte swizzle.  K is normalised in shared memory
// (k^ = k / max(||k||, eps)); the Q normalisation and the stabilisation factor c of Eq. 4
// are applied to the fp32 accumulator rows in the epilogue, so Q and V feed the MMAs as
// loaded.  The state S is kept unscaled; c multiplies outputs and exported states.
//
// Modes:  MODE_STATE  only accumulates the group's partial state and writes it (phase A);
//         MODE_CAUSAL the full chunk walk starting from the group's prefix state;
//         MODE_READOUT O = Q S for a fixed state (bidirectional form, Eq. 5 right side).
#include "cott_internal.h"
#include "cott_sm100.cuh"

namespace cott {

using namespace sm100;

namespace {

constexpr int kChunk = 128;
constexpr int kTcThreads = 128;
constexpr uint64_t kWaitTimeoutNs = 2000000000ull;  // 2 s: far above any legitimate wait

struct TcFwdParams {
    const float* init;      // [BH, n_groups, d*d] unscaled prefix / total states, or NULL
    float* state_out;       // MODE_STATE: [BH, n_groups, d*d] partial states (unscaled)
    int* status;            // workspace status word
    const float* m; const float* seq_len; float seq_len_scalar;
    int H; int N; int group; int n_groups;
};

template <int D> struct Smem {
    static constexpr int kTile = kChunk * D * 2;          // one 128 x D bf16 tile
    static constexpr int kStage = 3 * kTile;              // Q, K, V
    static constexpr int kSb = D * D * 2;                 // bf16 copy of the state
    static constexpr int kOffSb = 2 * kStage;
    static constexpr int kOffBar = kOffSb + kSb;          // full[2], mma, tmem slot, flag
    static constexpr int kTotal = kOffBar + 64;
    static constexpr int kDyn = kTotal + 1024;            // slack to align the base to 1024
};

// tcgen05.mma chains (one thread).  All tiles are 128-byte-swizzled rows of 128 bytes; a
// 128-column (256-byte) row is split into two half tiles 16 KB apart.
template <int D>
__device__ __forceinline__ void issue_p(uint32_t tP, uint32_t q, uint32_t k) {
    constexpr uint32_t idesc = instr_desc_bf16(128, 128, false, false);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = (kk >> 2) * 16384u + (kk & 3) * 32u;
        mma_ss(tP, smem_desc(q + off, 16, 1024), smem_desc(k + off, 16, 1024), idesc, kk > 0);
    }
}
template <int D>
__device__ __forceinline__ void issue_qs(uint32_t tO, uint32_t q, uint32_t sb) {
    constexpr uint32_t idesc = instr_desc_bf16(128, D, false, true);
#pragma unroll
    for (int kk = 0; kk < D / 16; ++kk) {
        const uint32_t off = (kk >> 2) * 16384u + (kk & 3) * 32u;
        mma_ss(tO, smem_desc(q + off, 16, 1024), smem_desc(sb + kk * 2048u, D * 128u, 1024), idesc,
               kk > 0);
    }
}
template <int D>
__device__ __forceinline__ void issue_pv(uint32_t tO, uint32_t p, uint32_t v, bool acc_first) {
    constexpr uint32_t idesc = instr_desc_bf16(128, D, false, true);
#pragma unroll
    for (int kk = 0; kk < kChunk / 16; ++kk) {
        const uint32_t off = (kk >> 2) * 16384u + (kk & 3) * 32u;
        mma_ss(tO, smem_desc(p + off, 16, 1024), smem_desc(v + kk * 2048u, 16384, 1024), idesc,
               (kk > 0) || acc_first);
    }
}
template <int D>
__device__ __forceinline__ void issue_ktv(uint32_t tS, uint32_t k, uint32_t v, bool acc_first) {
    constexpr uint32_t idesc = instr_desc_bf16(D, D, true, true);
#pragma unroll
    for (int kk = 0; kk < kChunk / 16; ++kk)
        mma_ss(tS, smem_desc(k + kk * 2048u, 16384, 1024), smem_desc(v + kk * 2048u, 16384, 1024),
               idesc, (kk > 0) || acc_first);
}

enum { MODE_STATE = 0, MODE_CAUSAL = 1, MODE_READOUT = 2 };

template <int D, int MODE>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
              const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
              TcFwdParams p) {
    using L = Smem<D>;
    constexpr int NH = D / 64;                       // 64-column half tiles per row
    constexpr uint32_t kTmemCols = (D == 128) ? 512 : 256;
    constexpr uint32_t colS = 0, colO = D, colP = 2 * D;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gbase = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t bar_full0 = base + L::kOffBar, bar_full1 = bar_full0 + 8, bar_mma = bar_full0 + 16;
    const uint32_t tmem_slot = bar_full0 + 24;
    volatile uint32_t* tmem_slot_g = reinterpret_cast<volatile uint32_t*>(gbase + L::kOffBar + 24);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = blockIdx.x % p.n_groups, bh = blockIdx.x / p.n_groups;
    const int b = bh / p.H, h = bh % p.H;
    const int tok0 = g * p.group;
    const int tok1 = min(p.N, tok0 + p.group);
    const int n_chunks = (tok1 - tok0 + kChunk - 1) / kChunk;

    if (warp == 0) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    if (tid == 0) {
        mbar_init(bar_full0, 1); mbar_init(bar_full1, 1); mbar_init(bar_mma, 1);
        mbar_fence_init();
        fence_proxy_async();
        tma_prefetch_desc(&tmQ); tma_prefetch_desc(&tmK); tma_prefetch_desc(&tmV);
        tma_prefetch_desc(&tmO);
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
    auto stage_q = [&](int s) { return base + s * L::kStage; };
    auto stage_k = [&](int s) { return base + s * L::kStage + L::kTile; };
    auto stage_v = [&](int s) { return base + s * L::kStage + 2 * L::kTile; };

    auto issue_loads = [&](int c) {
        const int s = c & 1;
        const uint32_t bar = s ? bar_full1 : bar_full0;
        const int row = tok0 + c * kChunk;
        constexpr uint32_t n_tiles = (MODE == MODE_STATE) ? 2 : (MODE == MODE_CAUSAL ? 3 : 1);
        mbar_expect_tx(bar, n_tiles * L::kTile);
#pragma unroll
        for (int hh = 0; hh < NH; ++hh) {
            if (MODE != MODE_STATE) tma_load_3d(stage_q(s) + hh * 16384, &tmQ, bar, hh * 64, row, bh);
            if (MODE != MODE_READOUT) {
                tma_load_3d(stage_k(s) + hh * 16384, &tmK, bar, hh * 64, row, bh);
                tma_load_3d(stage_v(s) + hh * 16384, &tmV, bar, hh * 64, row, bh);
            }
        }
    };

    if (tid == 0 && n_chunks > 0) issue_loads(0);

    for (int c = 0; c < n_chunks; ++c) {
        const int s = c & 1;
        if (tid == 0 && c + 1 < n_chunks) {
            tma_store_wait_read0();  // the store that read stage s^1's V slot has drained
            issue_loads(c + 1);
        }
        bool ok = mbar_wait(s ? bar_full1 : bar_full0, (uint32_t)((c >> 1) & 1), kWaitTimeoutNs);
        if (__syncthreads_or(!ok)) { failed = true; break; }

        uint8_t* qs = gbase + s * L::kStage;
        uint8_t* ks = qs + L::kTile;
        uint8_t* vs = qs + 2 * L::kTile;
        float rq = 0.f;
        // Row norms (fp32): thread t owns token row t of the chunk.
        if (MODE != MODE_STATE) {
            float ss = 0.f;
#pragma unroll
            for (int ch = 0; ch < D / 8; ++ch) {
                uint4 w = *reinterpret_cast<const uint4*>(qs + (ch >> 3) * 16384 + swz(tid, ch & 7));
                const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float2 f = __bfloat1622float2(e[i]);
                    ss += f.x * f.x + f.y * f.y;
                }
            }
            rq = cfac / fmaxf(sqrtf(ss), kEps);
        }
        if (MODE != MODE_READOUT) {
            uint4 w[D / 8];
            float ss = 0.f;
#pragma unroll
            for (int ch = 0; ch < D / 8; ++ch) {
                w[ch] = *reinterpret_cast<const uint4*>(ks + (ch >> 3) * 16384 + swz(tid, ch & 7));
                const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w[ch]);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float2 f = __bfloat1622float2(e[i]);
                    ss += f.x * f.x + f.y * f.y;
                }
            }
            const float rk = 1.0f / fmaxf(sqrtf(ss), kEps);
#pragma unroll
            for (int ch = 0; ch < D / 8; ++ch) {
                const __nv_bfloat162* e = reinterpret_cast<const __nv_bfloat162*>(&w[ch]);
                uint4 o;
                uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    float2 f = __bfloat1622float2(e[i]);
                    ow[i] = pack_bf16(f.x * rk, f.y * rk);
                }
                *reinterpret_cast<uint4*>(ks + (ch >> 3) * 16384 + swz(tid, ch & 7)) = o;
            }
            fence_proxy_async();
        }
        tc_fence_before();
        __syncthreads();

        if (tid == 0) {
            tc_fence_after();
            if (MODE == MODE_CAUSAL) {
                issue_p<D>(tmem + colP, stage_q(s), stage_k(s));
                if (has_state) issue_qs<D>(tmem + colO, stage_q(s), sb);
                issue_ktv<D>(tmem + colS, stage_k(s), stage_v(s), has_state);
            } else if (MODE == MODE_STATE) {
                issue_ktv<D>(tmem + colS, stage_k(s), stage_v(s), has_state);
            } else {
                issue_qs<D>(tmem + colO, stage_q(s), sb);
            }
            tc_commit(bar_mma);
        }
        ok = mbar_wait(bar_mma, mma_phase, kWaitTimeoutNs);
        mma_phase ^= 1;
        if (__syncthreads_or(!ok)) { failed = true; break; }
        tc_fence_after();

        if (MODE == MODE_CAUSAL) {
            // Masked scores -> bf16 operand in the Q slot (Q is dead: both MMAs that read it
            // have completed).  Row i keeps columns j <= i (the diagonal stays, Eq. 6).
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
                        const float x0 = (col <= tid) ? __uint_as_float(r[i + j]) : 0.f;
                        const float x1 = (col + 1 <= tid) ? __uint_as_float(r[i + j + 1]) : 0.f;
                        ww[j >> 1] = pack_bf16(x0, x1);
                    }
                    const int col = c0 + i;
                    *reinterpret_cast<uint4*>(qs + (col >> 6) * 16384 + swz(tid, (col & 63) >> 3)) = w;
                }
            }
            // bf16 copy of the updated state for the next chunk's Q S product.
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
                issue_pv<D>(tmem + colO, stage_q(s), stage_v(s), has_state);
                tc_commit(bar_mma);
            }
            ok = mbar_wait(bar_mma, mma_phase, kWaitTimeoutNs);
            mma_phase ^= 1;
            if (__syncthreads_or(!ok)) { failed = true; break; }
            tc_fence_after();
        }
        has_state = true;

        if (MODE != MODE_STATE) {
            // Output rows: scale by c / ||q||, round to bf16, stage in the V slot, TMA store.
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 32) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + colO + c0, r);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; i += 8) {
                    uint4 w;
                    w.x = pack_bf16(__uint_as_float(r[i]) * rq, __uint_as_float(r[i + 1]) * rq);
                    w.y = pack_bf16(__uint_as_float(r[i + 2]) * rq, __uint_as_float(r[i + 3]) * rq);
                    w.z = pack_bf16(__uint_as_float(r[i + 4]) * rq, __uint_as_float(r[i + 5]) * rq);
                    w.w = pack_bf16(__uint_as_float(r[i + 6]) * rq, __uint_as_float(r[i + 7]) * rq);
                    const int col = c0 + i;
                    *reinterpret_cast<uint4*>(vs + (col >> 6) * 16384 + swz(tid, (col & 63) >> 3)) = w;
                }
            }
            fence_proxy_async();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
#pragma unroll
                for (int hh = 0; hh < NH; ++hh)
                    tma_store_3d(&tmO, stage_v(s) + hh * 16384, hh * 64, tok0 + c * kChunk, bh);
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

    if (failed) {
        if (tid == 0) atomicExch(p.status, 1);
        // Give outstanding loads a bounded chance to land before the CTA's shared memory
        // is released.
        if (tid == 0) {
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

}  // namespace

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
static cudaError_t launch_mode(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv,
                               const CUtensorMap& to, const TcFwdParams& p, int BH,
                               cudaStream_t st) {
    auto kern = tc_fwd_kernel<D, MODE>;
    static bool configured = false;
    if (!configured) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             Smem<D>::kDyn);
        if (e != cudaSuccess) return e;
        configured = true;
    }
    kern<<<dim3((unsigned)(BH * p.n_groups)), kTcThreads, Smem<D>::kDyn, st>>>(tq, tk, tv, to, p);
    note_launch();
    return cudaGetLastError();
}

cudaError_t launch_tc_fwd(int mode, const void* q, const void* k, const void* v, void* o,
                          const float* init, float* state_out, int* status, const float* m,
                          const float* seq_len, float seq_len_scalar, int B, int H, int N, int d,
                          int group, int n_groups, cudaStream_t st) {
    const int BH = B * H;
    CUtensorMap tq, tk, tv, to;
    // Unused operands still need a valid map: point them at a tensor that exists.
    const void* any = q ? q : k;
    if (!make_tile_map(&tq, q ? q : any, BH, N, d) || !make_tile_map(&tk, k ? k : any, BH, N, d) ||
        !make_tile_map(&tv, v ? v : any, BH, N, d) || !make_tile_map(&to, o ? o : any, BH, N, d))
        return cudaErrorInvalidValue;
    TcFwdParams p;
    p.init = init; p.state_out = state_out; p.status = status;
    p.m = m; p.seq_len = seq_len; p.seq_len_scalar = seq_len_scalar;
    p.H = H; p.N = N; p.group = group; p.n_groups = n_groups;
    if (d == 128) {
        if (mode == MODE_STATE) return launch_mode<128, MODE_STATE>(tq, tk, tv, to, p, BH, st);
        if (mode == MODE_CAUSAL) return launch_mode<128, MODE_CAUSAL>(tq, tk, tv, to, p, BH, st);
        return launch_mode<128, MODE_READOUT>(tq, tk, tv, to, p, BH, st);
    }
    if (d == 64) {
        if (mode == MODE_STATE) return launch_mode<64, MODE_STATE>(tq, tk, tv, to, p, BH, st);
        if (mode == MODE_CAUSAL) return launch_mode<64, MODE_CAUSAL>(tq, tk, tv, to, p, BH, st);
        return launch_mode<64, MODE_READOUT>(tq, tk, tv, to, p, BH, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace cott
