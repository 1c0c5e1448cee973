// fp32 SIMT kernels: the running-sum walk (Eq. 7 / Eq. 8), the scan over per-group partial
// states, the dm reduction and the recurrent decode step.  These serve fp32 I/O (tensor
// cores in TF32 cannot meet the fp32 tolerance) and every shape the tensor-core kernels do
// not cover.
#include "cott_internal.h"

namespace cott {

namespace {

constexpr int kThreads = 256;
constexpr int kTile = 16;  // tokens staged per shared-memory tile

template <typename T> __device__ __forceinline__ void load4(const T* p, float (&f)[4]);
template <> __device__ __forceinline__ void load4<float>(const float* p, float (&f)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <> __device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p,
                                                                 float (&f)[4]) {
    uint2 v = *reinterpret_cast<const uint2*>(p);
    __nv_bfloat162 lo = *reinterpret_cast<__nv_bfloat162*>(&v.x);
    __nv_bfloat162 hi = *reinterpret_cast<__nv_bfloat162*>(&v.y);
    f[0] = __low2float(lo); f[1] = __high2float(lo);
    f[2] = __low2float(hi); f[3] = __high2float(hi);
}
template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) {
    return __bfloat162float(v);
}
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
    return __float2bfloat16_rn(v);
}
template <typename T> __device__ __forceinline__ void store4(T* p, const float (&f)[4]);
template <> __device__ __forceinline__ void store4<float>(float* p, const float (&f)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p,
                                                                  const float (&f)[4]) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(f[0], f[1]);
    __nv_bfloat162 hi = __floats2bfloat162_rn(f[2], f[3]);
    uint2 v;
    v.x = *reinterpret_cast<uint32_t*>(&lo);
    v.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Stage rows [t0, t0+kTile) of one (b,h) slice (rows `sn` elements apart) as fp32; rows outside
// [lo,hi) become zero.
template <int D, typename T>
__device__ __forceinline__ void stage_tile(float (*dst)[D], const T* src, long long sn, int t0, int lo,
                                           int hi, int tid) {
    constexpr int V4 = D / 4;
    for (int i = tid; i < kTile * V4; i += kThreads) {
        int r = i / V4, c4 = i % V4;
        int t = t0 + r;
        float f[4] = {0.f, 0.f, 0.f, 0.f};
        if (t >= lo && t < hi) load4<T>(src + (size_t)t * sn + c4 * 4, f);
        *reinterpret_cast<float4*>(&dst[r][c4 * 4]) = make_float4(f[0], f[1], f[2], f[3]);
    }
}

// Apply the row treatment to a staged tile: one warp per row.
template <int D>
__device__ __forceinline__ void treat_rows(float (*tile)[D], int mode, float c, int warp,
                                           int lane) {
    if (mode == ROW_RAW) return;
    for (int r = warp; r < kTile; r += kThreads / 32) {
        float scale = c;
        if (mode == ROW_NORM) {
            float ss = 0.f;
            for (int e = lane; e < D; e += 32) ss += tile[r][e] * tile[r][e];
            ss = warp_sum(ss);
            scale = 1.0f / fmaxf(sqrtf(ss), kEps);
        }
        for (int e = lane; e < D; e += 32) tile[r][e] *= scale;
    }
}

template <int D, typename T>
__global__ void __launch_bounds__(kThreads) walk_kernel(WalkArgs w) {
    constexpr int NSPLIT = kThreads / D;  // threads sharing one state column
    constexpr int AR = D / NSPLIT;        // state rows owned by one thread
    __shared__ __align__(16) float xs[kTile][D];
    __shared__ __align__(16) float as[kTile][D];
    __shared__ __align__(16) float bs[kTile][D];
    __shared__ __align__(16) float part[kTile][NSPLIT][D];
    __shared__ float dm_red[kThreads / 32];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int g = blockIdx.x % w.n_groups;
    const int bh = blockIdx.x / w.n_groups;
    const int b = bh / w.H, h = bh % w.H;
    // (a packed batch: the rows of sequence b, one group)
    const int lo = w.cu_seqlens ? w.cu_seqlens[b] : g * w.group;
    const int hi = w.cu_seqlens ? w.cu_seqlens[b + 1] : min(w.N, lo + w.group);
    // (the launcher has resolved the layouts: strides are never all zero here)
    auto slice = [&](const RowLayout& l) { return (w.cu_seqlens ? (size_t)0 : (size_t)b * l.sb) + (size_t)h * l.sh; };
    const T* X = static_cast<const T*>(w.x) + slice(w.lx);
    const T* A = static_cast<const T*>(w.a) + slice(w.la);
    const T* Bv = static_cast<const T*>(w.bv) + slice(w.lbv);
    const T* P = w.proj ? static_cast<const T*>(w.proj) + slice(w.lproj) : nullptr;
    T* O = w.out ? static_cast<T*>(w.out) + slice(w.lout) : nullptr;

    const float s_b = w.seq_len ? w.seq_len[b]
                                : (w.seq_len_scalar > 0.f ? w.seq_len_scalar
                                                          : (float)(w.cu_seqlens ? max(hi - lo, 1) : w.N));
    const float c = stab_factor(w.m[h], s_b);

    const int col = tid % D, split = tid / D, a0 = split * AR;
    float S[AR];
    if (w.init) {
        const float* src = w.init + ((size_t)bh * w.n_groups + g) * D * D;
#pragma unroll
        for (int i = 0; i < AR; ++i) S[i] = src[(size_t)(a0 + i) * D + col];
    } else {
#pragma unroll
        for (int i = 0; i < AR; ++i) S[i] = 0.f;
    }

    float dm_acc = 0.f;
    const int n_tiles = (hi - lo + kTile - 1) / kTile;
    for (int it = 0; it < n_tiles; ++it) {
        const int tile_idx = w.reverse ? (n_tiles - 1 - it) : it;
        const int t0 = lo + tile_idx * kTile;
        __syncthreads();  // previous tile fully consumed
        stage_tile<D, T>(xs, X, w.lx.sn, t0, lo, hi, tid);
        stage_tile<D, T>(as, A, w.la.sn, t0, lo, hi, tid);
        stage_tile<D, T>(bs, Bv, w.lbv.sn, t0, lo, hi, tid);
        __syncthreads();
        treat_rows<D>(xs, w.mode_x, c, warp, lane);
        treat_rows<D>(as, w.mode_a, c, warp, lane);
        treat_rows<D>(bs, w.mode_b, c, warp, lane);
        __syncthreads();

        for (int s = 0; s < kTile; ++s) {
            const int tt = w.reverse ? (kTile - 1 - s) : s;
            const float bval = bs[tt][col];
            float acc = 0.f;
            if (w.update) {
#pragma unroll
                for (int i = 0; i < AR; i += 4) {
                    float4 av = *reinterpret_cast<const float4*>(&as[tt][a0 + i]);
                    S[i] += av.x * bval; S[i + 1] += av.y * bval;
                    S[i + 2] += av.z * bval; S[i + 3] += av.w * bval;
                }
            }
            if (w.write_out) {
#pragma unroll
                for (int i = 0; i < AR; i += 4) {
                    float4 xv = *reinterpret_cast<const float4*>(&xs[tt][a0 + i]);
                    acc += xv.x * S[i]; acc += xv.y * S[i + 1];
                    acc += xv.z * S[i + 2]; acc += xv.w * S[i + 3];
                }
                part[tt][split][col] = acc;
            }
        }
        if (!w.write_out) continue;
        __syncthreads();
        // Sum the partial read-outs of the NSPLIT thread groups into part[.][0][.].
        for (int i = tid; i < kTile * D; i += kThreads) {
            int r = i / D, e = i % D;
            float v = part[r][0][e];
#pragma unroll
            for (int sp = 1; sp < NSPLIT; ++sp) v += part[r][sp][e];
            part[r][0][e] = v;
        }
        if (w.epilogue != EPI_PLAIN) stage_tile<D, T>(xs, P, w.lproj.sn, t0, lo, hi, tid);  // xs is dead now
        __syncthreads();
        // Epilogue: one warp per row.
        for (int r = warp; r < kTile; r += kThreads / 32) {
            const int t = t0 + r;
            if (t >= hi) continue;
            float* row = part[r][0];
            if (w.epilogue == EPI_PROJ) {
                // dx = (dx^ - x^ <x^, dx^>) / ||x||, or dx^ / eps on the clamped branch
                float ss = 0.f, dp = 0.f;
                for (int e = lane; e < D; e += 32) {
                    ss += xs[r][e] * xs[r][e];
                    dp += xs[r][e] * row[e];
                }
                ss = warp_sum(ss); dp = warp_sum(dp);
                const float nrm = sqrtf(ss);
                const float rinv = 1.0f / fmaxf(nrm, kEps);
                const float coef = nrm > kEps ? dp * rinv * rinv : 0.f;  // <x^,dx^> * rinv
                for (int e = lane; e < D; e += 32) row[e] = (row[e] - xs[r][e] * coef) * rinv;
            } else if (w.epilogue == EPI_DV) {
                float dp = 0.f;
                for (int e = lane; e < D; e += 32) {
                    dp += xs[r][e] * row[e];
                    row[e] *= c;
                }
                dm_acc += dp;  // per-lane partial; summed over the warp at the end
            }
            __syncwarp();
            for (int e4 = lane; e4 < D / 4; e4 += 32) {
                float f[4] = {row[e4 * 4], row[e4 * 4 + 1], row[e4 * 4 + 2], row[e4 * 4 + 3]};
                store4<T>(O + (size_t)t * w.lout.sn + e4 * 4, f);
            }
        }
    }

    if (w.final_state) {
        float* dst = w.final_state +
                     (w.final_grouped ? ((size_t)bh * w.n_groups + g) : (size_t)bh) * D * D;
#pragma unroll
        for (int i = 0; i < AR; ++i) dst[(size_t)(a0 + i) * D + col] = S[i];
    }
    if (w.dm_partial) {
        dm_acc = warp_sum(dm_acc);
        if (lane == 0) dm_red[warp] = dm_acc;
        __syncthreads();
        if (tid == 0) {
            float t = 0.f;
            for (int i = 0; i < kThreads / 32; ++i) t += dm_red[i];
            w.dm_partial[(size_t)bh * w.n_groups + g] = t;
        }
    }
}

// Combine per-group partial states: exclusive prefix (forward), exclusive suffix (reverse
// time) or the total written to every group.  One thread per four consecutive state
// elements; groups are visited in batches whose loads are all issued before the first use.
__global__ void __launch_bounds__(256) scan_kernel(float* __restrict__ states,
                                                   float* __restrict__ total_out, int n_groups,
                                                   int dd, int mode, const float* scale_m,
                                                   const float* seq_len, float seq_len_scalar,
                                                   int H, int N, const float* __restrict__ init_in) {
    constexpr int kBatch = 8;
    const int e4 = blockIdx.x * blockDim.x + threadIdx.x;
    const int bh = blockIdx.y;
    if (e4 * 4 >= dd) return;
    float4* base = reinterpret_cast<float4*>(states + (size_t)bh * n_groups * dd) + e4;
    const size_t stride = (size_t)dd / 4;
    float4 run = make_float4(0.f, 0.f, 0.f, 0.f);
    // With scale_m the states being scanned are unscaled and the total is multiplied by c on
    // the way out; a caller's initial state (which contains c) enters divided by c.
    float c = 1.f;
    if (scale_m) {
        const float s_b = seq_len ? seq_len[bh / H]
                                  : (seq_len_scalar > 0.f ? seq_len_scalar : (float)N);
        c = stab_factor(scale_m[bh % H], s_b);
    }
    if (init_in) {
        const float4 v0 = reinterpret_cast<const float4*>(init_in + (size_t)bh * dd)[e4];
        const float ic = 1.0f / c;
        run = make_float4(v0.x * ic, v0.y * ic, v0.z * ic, v0.w * ic);
    }
    auto add = [](float4& a, const float4& b) { a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w; };
    if (mode == SCAN_TOTAL) {
        for (int g0 = 0; g0 < n_groups; g0 += kBatch) {
            float4 v[kBatch];
#pragma unroll
            for (int i = 0; i < kBatch; ++i)
                if (g0 + i < n_groups) v[i] = base[(size_t)(g0 + i) * stride];
#pragma unroll
            for (int i = 0; i < kBatch; ++i)
                if (g0 + i < n_groups) add(run, v[i]);
        }
        for (int g = 0; g < n_groups; ++g) base[(size_t)g * stride] = run;
    } else {
        const bool rev = mode == SCAN_SUFFIX;
        for (int g0 = 0; g0 < n_groups; g0 += kBatch) {
            float4 v[kBatch];
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const int g = rev ? n_groups - 1 - (g0 + i) : g0 + i;
                if (g0 + i < n_groups) v[i] = base[(size_t)g * stride];
            }
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const int g = rev ? n_groups - 1 - (g0 + i) : g0 + i;
                if (g0 + i < n_groups) {
                    base[(size_t)g * stride] = run;
                    add(run, v[i]);
                }
            }
        }
    }
    if (total_out) {
        if (scale_m) { run.x *= c; run.y *= c; run.z *= c; run.w *= c; }
        reinterpret_cast<float4*>(total_out + (size_t)bh * dd)[e4] = run;
    }
}

// dm_h = sum_b dc/dm * <dV', V>_{b,h},  dc/dm = -ln(s_b) sigma(m_h)(1-sigma(m_h)) c_{b,h}.
// Fixed summation order (deterministic).
__global__ void dm_finalize_kernel(const float* dm_partial, float* dm, const float* m,
                                   const float* seq_len, float seq_len_scalar, int B, int H,
                                   int n_groups, int N, const int* cu_seqlens) {
    const int h = blockIdx.x * blockDim.x + threadIdx.x;
    if (h >= H) return;
    const float sg = 1.0f / (1.0f + expf(-m[h]));
    float total = 0.f;
    for (int b = 0; b < B; ++b) {
        const float s_b = seq_len ? seq_len[b]
                                  : (seq_len_scalar > 0.f ? seq_len_scalar
                                                          : (float)(cu_seqlens ? max(cu_seqlens[b + 1] - cu_seqlens[b], 1) : N));
        const float ls = logf(s_b);
        const float c = expf(-sg * ls);
        float acc = 0.f;
        for (int g = 0; g < n_groups; ++g) acc += dm_partial[((size_t)b * H + h) * n_groups + g];
        total += acc * (-ls * sg * (1.0f - sg) * c);
    }
    dm[h] = total;
}

// Recurrent decode step (Eq. 8): SPLIT CTAs per (b,h), each owning D / SPLIT value columns of
// the fp32 state, which streams through once with 128-bit loads and stores, update and
// read-out fused.  Every thread first issues all loads of its state elements (the CTA's whole
// share is then in flight), and only then normalises q and k, so the row norms hide behind
// the memory latency.  The column split keeps the per-thread share small (more CTAs resident,
// a shorter last wave); every CTA normalises q and k for itself and owns its columns of o.
template <int D, int SPLIT, typename T>
__global__ void __launch_bounds__(kThreads) decode_kernel(const T* q, const T* k, const T* v,
                                                          float* state, T* o, int H,
                                                          const float* m, const float* seq_len,
                                                          float seq_len_scalar) {
    constexpr int DC = D / SPLIT;         // value columns of this CTA
    constexpr int V4 = DC / 4;            // float4 per state row share
    constexpr int RG = kThreads / V4;     // rows covered per sweep
    constexpr int NIT = D / RG;
    __shared__ float qh[D], kh[D], vp[DC];
    __shared__ __align__(16) float red[RG][DC];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int bh = blockIdx.x / SPLIT, col0 = (blockIdx.x % SPLIT) * DC;
    const int b = bh / H, h = bh % H;
    const int c4 = tid % V4, r0 = tid / V4;
    float4* S = reinterpret_cast<float4*>(state + (size_t)bh * D * D + col0);   // row stride D / 4
    float4 sv[NIT];
#pragma unroll
    for (int i = 0; i < NIT; ++i) sv[i] = S[(size_t)(r0 + i * RG) * (D / 4) + c4];

    const float s_b = seq_len ? seq_len[b] : seq_len_scalar;
    const float c = stab_factor(m[h], s_b);
    if (tid < D) {
        qh[tid] = to_f32<T>(q[(size_t)bh * D + tid]);
        kh[tid] = to_f32<T>(k[(size_t)bh * D + tid]);
        if (tid < DC) vp[tid] = to_f32<T>(v[(size_t)bh * D + col0 + tid]) * c;
    }
    __syncthreads();
    if (warp < 2) {
        float* row = warp == 0 ? qh : kh;
        float ss = 0.f;
        for (int e = lane; e < D; e += 32) ss += row[e] * row[e];
        ss = warp_sum(ss);
        const float r = 1.0f / fmaxf(sqrtf(ss), kEps);
        for (int e = lane; e < D; e += 32) row[e] *= r;
    }
    __syncthreads();
    const float4 vv = *reinterpret_cast<const float4*>(&vp[c4 * 4]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int i = 0; i < NIT; ++i) {
        const int a = r0 + i * RG;
        const float ka = kh[a], qa = qh[a];
        sv[i].x += ka * vv.x; sv[i].y += ka * vv.y; sv[i].z += ka * vv.z; sv[i].w += ka * vv.w;
        S[(size_t)a * (D / 4) + c4] = sv[i];
        acc.x += qa * sv[i].x; acc.y += qa * sv[i].y; acc.z += qa * sv[i].z; acc.w += qa * sv[i].w;
    }
    *reinterpret_cast<float4*>(&red[r0][c4 * 4]) = acc;
    __syncthreads();
    if (tid < DC) {
        float t = 0.f;
#pragma unroll
        for (int r = 0; r < RG; ++r) t += red[r][tid];
        o[(size_t)bh * D + col0 + tid] = from_f32<T>(t);
    }
}

template <typename T>
cudaError_t launch_walk_t(const WalkArgs& w, int BH, int d, cudaStream_t st) {
    dim3 grid((unsigned)(BH * w.n_groups));
    switch (d) {
        case 32: walk_kernel<32, T><<<grid, kThreads, 0, st>>>(w); break;
        case 64: walk_kernel<64, T><<<grid, kThreads, 0, st>>>(w); break;
        case 128: walk_kernel<128, T><<<grid, kThreads, 0, st>>>(w); break;
        default: return cudaErrorInvalidValue;
    }
    note_launch();
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_decode_t(const void* q, const void* k, const void* v, float* state, void* o,
                            int B, int H, int d, const float* m, const float* seq_len,
                            float seq_len_scalar, cudaStream_t st) {
    const unsigned BH = (unsigned)(B * H);
    const T *qq = (const T*)q, *kk = (const T*)k, *vv = (const T*)v;
    T* oo = (T*)o;
    switch (d) {
        case 32: decode_kernel<32, 1, T><<<BH, kThreads, 0, st>>>(qq, kk, vv, state, oo, H, m, seq_len, seq_len_scalar); break;
        case 64: decode_kernel<64, 1, T><<<BH, kThreads, 0, st>>>(qq, kk, vv, state, oo, H, m, seq_len, seq_len_scalar); break;
        case 128: decode_kernel<128, 2, T><<<2 * BH, kThreads, 0, st>>>(qq, kk, vv, state, oo, H, m, seq_len, seq_len_scalar); break;
        default: return cudaErrorInvalidValue;
    }
    note_launch();
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_walk_simt(const WalkArgs& w0, int BH, int d, cott_dtype dt, cudaStream_t st) {
    WalkArgs w = w0;   // resolve "all zero = dense [B,H,N,d]" once, on the host
    w.lx = resolve_layout(w0.lx, w0.H, w0.N, d); w.la = resolve_layout(w0.la, w0.H, w0.N, d);
    w.lbv = resolve_layout(w0.lbv, w0.H, w0.N, d); w.lproj = resolve_layout(w0.lproj, w0.H, w0.N, d);
    w.lout = resolve_layout(w0.lout, w0.H, w0.N, d);
    return dt == COTT_F32 ? launch_walk_t<float>(w, BH, d, st)
                          : launch_walk_t<__nv_bfloat16>(w, BH, d, st);
}

cudaError_t launch_scan(float* states, float* total_out, int BH, int n_groups, int d, int mode,
                        cudaStream_t st, const float* total_scale_m, const float* seq_len,
                        float seq_len_scalar, int H, int N, const float* init_in) {
    const int dd = d * d;
    dim3 grid((unsigned)((dd / 4 + 255) / 256), (unsigned)BH);
    scan_kernel<<<grid, 256, 0, st>>>(states, total_out, n_groups, dd, mode, total_scale_m, seq_len,
                                      seq_len_scalar, H, N, init_in);
    note_launch();
    return cudaGetLastError();
}

// out[h] = sum over the n slices of parts[i][h], in slice order (deterministic).
__global__ void sum_slices_kernel(const float* parts, float* out, int n, int H) {
    const int h = blockIdx.x * blockDim.x + threadIdx.x;
    if (h >= H) return;
    float acc = 0.f;
    for (int i = 0; i < n; ++i) acc += parts[(size_t)i * H + h];
    out[h] = acc;
}

cudaError_t launch_sum_slices(const float* parts, float* out, int n, int H, cudaStream_t st) {
    sum_slices_kernel<<<(H + 127) / 128, 128, 0, st>>>(parts, out, n, H);
    note_launch();
    return cudaGetLastError();
}

cudaError_t launch_dm_finalize(const float* dm_partial, float* dm, const float* m,
                               const float* seq_len, float seq_len_scalar, int B, int H,
                               int n_groups, int N, cudaStream_t st, const int* cu_seqlens) {
    dm_finalize_kernel<<<(H + 127) / 128, 128, 0, st>>>(dm_partial, dm, m, seq_len,
                                                        seq_len_scalar, B, H, n_groups, N, cu_seqlens);
    note_launch();
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Head sizes the tensor-core kernels run zero-padded (dk, dv <= their d): a caller's state
// [BH, dk, dv] enters and leaves through a padded [BH, d, d] copy in the workspace.
__global__ void pad_state_kernel(const float* __restrict__ src, float* __restrict__ dst, int dk, int dv, int d) {
    const size_t bh = blockIdx.y;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < d * d; i += gridDim.x * blockDim.x) {
        const int r = i / d, c = i - r * d;
        dst[bh * d * d + i] = (r < dk && c < dv) ? src[bh * dk * dv + (size_t)r * dv + c] : 0.f;
    }
}
__global__ void unpad_state_kernel(const float* __restrict__ src, float* __restrict__ dst, int dk, int dv, int d) {
    const size_t bh = blockIdx.y;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < dk * dv; i += gridDim.x * blockDim.x) {
        const int r = i / dv, c = i - r * dv;
        dst[bh * dk * dv + i] = src[bh * d * d + (size_t)r * d + c];
    }
}
// dst[bh][c][r] = src[bh][r][c] for square d x d states.
__global__ void transpose_state_kernel(const float* __restrict__ src, float* __restrict__ dst, int d) {
    const size_t bh = blockIdx.y;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < d * d; i += gridDim.x * blockDim.x) {
        const int r = i / d, c = i - r * d;
        dst[bh * d * d + (size_t)c * d + r] = src[bh * d * d + i];
    }
}
cudaError_t launch_transpose_state(const float* src, float* dst, int BH, int d, cudaStream_t st) {
    dim3 grid((unsigned)((d * d + 1023) / 1024), (unsigned)BH);
    transpose_state_kernel<<<grid, 256, 0, st>>>(src, dst, d);
    note_launch();
    return cudaGetLastError();
}
// dst = src (transposed if asked) times c[b,h] (scale_mode 1), divided by it (2) or as is (0):
// a caller's square state brought into the layout and scale a tensor-core stream starts from.
__global__ void state_prep_kernel(const float* __restrict__ src, float* __restrict__ dst, int d, int transpose, int scale_mode,
                                  const float* m, const float* seq_len, float seq_len_scalar, int H, int N) {
    const size_t bh = blockIdx.y;
    float f = 1.f;
    if (scale_mode) {
        const float s_b = seq_len ? seq_len[bh / H] : (seq_len_scalar > 0.f ? seq_len_scalar : (float)N);
        const float c = stab_factor(m[bh % H], s_b);
        f = scale_mode == 1 ? c : 1.0f / c;
    }
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < d * d; i += gridDim.x * blockDim.x) {
        const int r = i / d, c2 = i - r * d;
        dst[bh * d * d + (transpose ? (size_t)c2 * d + r : (size_t)i)] = src[bh * d * d + i] * f;
    }
}
cudaError_t launch_state_prep(const float* src, float* dst, int BH, int d, int transpose, int scale_mode, const float* m,
                              const float* seq_len, float seq_len_scalar, int H, int N, cudaStream_t st) {
    dim3 grid((unsigned)((d * d + 1023) / 1024), (unsigned)BH);
    state_prep_kernel<<<grid, 256, 0, st>>>(src, dst, d, transpose, scale_mode, m, seq_len, seq_len_scalar, H, N);
    note_launch();
    return cudaGetLastError();
}

// Backward of a segment through the three tensor-core walks: what the streams' totals give.
//   tq_total [d_v][d_k] = state_in^T + c V^T K^        (the dQ^ stream's final sum, scaled)
//   tk_total [d_v][d_k] = c (d_state_out + Q^^T dO)^T  (the dK^ stream's)
// With S = K^^T V and R = Q^^T dO of the segment:
//   d_state_in = d_state_out + R = tk_total^T / c
//   the dm sum over the query rows, <q^_i, dQ^_i>, contains q^_i^T (state_in / c) dO_i, which is no
//   derivative with respect to c, and lacks <d_state_out, S>:  T = T_q - <state_in / c, R> + <d_state_out, S>.
// One CTA per (b, h); the correction (and the dK^ stream's partial sums `fold`, if any) is added to
// dm_partial[bh * n_groups], which the dm finaliser sums afterwards.
__global__ void __launch_bounds__(256) segment_finish_kernel(const float* __restrict__ state_in, const float* __restrict__ d_state_out,
                                                             const float* __restrict__ tq_total, const float* __restrict__ tk_total,
                                                             float* __restrict__ d_state_in, float* dm_partial, const float* fold,
                                                             int n_groups, int d, const float* m, const float* seq_len,
                                                             float seq_len_scalar, int H, int N) {
    const size_t bh = blockIdx.x;
    const float s_b = seq_len ? seq_len[bh / H] : (seq_len_scalar > 0.f ? seq_len_scalar : (float)N);
    const float ic = 1.0f / stab_factor(m[bh % H], s_b);
    const size_t o = bh * (size_t)d * d;
    float acc = 0.f;
    for (int i = threadIdx.x; i < d * d; i += blockDim.x) {
        const int a = i / d, b = i - a * d;                    // element [a][b] of a [d_k][d_v] state
        const size_t t = o + (size_t)b * d + a;                // its place in a transposed total
        const float dsi = tk_total[t] * ic;                    // d_state_out + R
        const float dso = d_state_out ? d_state_out[o + i] : 0.f;
        const float sin = state_in ? state_in[o + i] : 0.f;
        if (d_state_in) d_state_in[o + i] = dsi;
        const float r = dsi - dso, sl = (tq_total[t] - sin) * ic;
        acc += dso * sl - sin * ic * r;
    }
    __shared__ float red[8];
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int w = 0; w < 8; ++w) t += red[w];
        float f = 0.f;
        if (fold) for (int g = 0; g < n_groups; ++g) f += fold[bh * n_groups + g];
        dm_partial[bh * n_groups] += t + f;
    }
}
cudaError_t launch_segment_finish(const float* state_in, const float* d_state_out, const float* tq_total, const float* tk_total,
                                  float* d_state_in, float* dm_partial, const float* fold, int BH, int n_groups, int d,
                                  const float* m, const float* seq_len, float seq_len_scalar, int H, int N, cudaStream_t st) {
    segment_finish_kernel<<<(unsigned)BH, 256, 0, st>>>(state_in, d_state_out, tq_total, tk_total, d_state_in, dm_partial, fold,
                                                        n_groups, d, m, seq_len, seq_len_scalar, H, N);
    note_launch();
    return cudaGetLastError();
}

cudaError_t launch_pad_state(const float* src, float* dst, int BH, int dk, int dv, int d, cudaStream_t st) {
    dim3 grid((unsigned)((d * d + 1023) / 1024), (unsigned)BH);
    pad_state_kernel<<<grid, 256, 0, st>>>(src, dst, dk, dv, d);
    note_launch();
    return cudaGetLastError();
}
cudaError_t launch_unpad_state(const float* src, float* dst, int BH, int dk, int dv, int d, cudaStream_t st) {
    dim3 grid((unsigned)((dk * dv + 1023) / 1024), (unsigned)BH);
    unpad_state_kernel<<<grid, 256, 0, st>>>(src, dst, dk, dv, d);
    note_launch();
    return cudaGetLastError();
}

// One step of Eq. 8 for any head sizes (dk keys, dv values, dv a multiple of 4): one CTA per
// (b, h); thread t owns the four state columns 4 (t % (dv/4)) .. +3 of the rows
// t / (dv/4), + 256 / (dv/4), ...: 128-bit state loads and stores, coalesced along a row; the
// per-column partial sums of o meet in shared memory.
//   S <- S + k^ (c v)^T ;  o = S^T q^      (update first, then observe)
template <typename T>
__global__ void __launch_bounds__(256) decode_generic_kernel(const T* __restrict__ q, const T* __restrict__ k,
                                                             const T* __restrict__ v, float* __restrict__ state,
                                                             T* __restrict__ o, int H, int dk, int dv,
                                                             const float* __restrict__ m, const float* __restrict__ seq_len,
                                                             float seq_len_scalar) {
    extern __shared__ float sm[];            // q^ [dk] | k^ [dk] | c v [dv] | partial o [slices][dv] | 2 norms
    float* qh = sm; float* kh = sm + dk; float* cv = kh + dk; float* part = cv + dv;
    const size_t bh = blockIdx.x;
    const int b = (int)(bh / H), h = (int)(bh % H), tid = threadIdx.x;
    const int cgs = dv / 4, slices = 256 / cgs;          // column groups, row slices (>= 1 since dv <= 1024)
    __shared__ float red[2][8];
    float sq = 0.f, sk = 0.f;
    for (int i = tid; i < dk; i += 256) {
        const float a = to_f32(q[bh * dk + i]), c2 = to_f32(k[bh * dk + i]);
        qh[i] = a; kh[i] = c2; sq = fmaf(a, a, sq); sk = fmaf(c2, c2, sk);
    }
    for (int off = 16; off; off >>= 1) { sq += __shfl_xor_sync(0xffffffffu, sq, off); sk += __shfl_xor_sync(0xffffffffu, sk, off); }
    if ((tid & 31) == 0) { red[0][tid >> 5] = sq; red[1][tid >> 5] = sk; }
    const float s_b = seq_len ? seq_len[b] : seq_len_scalar;
    const float cfac = stab_factor(m[h], s_b);
    for (int i = tid; i < dv; i += 256) cv[i] = cfac * to_f32(v[bh * dv + i]);
    __syncthreads();
    float nq = 0.f, nk = 0.f;
    for (int w = 0; w < 8; ++w) { nq += red[0][w]; nk += red[1][w]; }
    const float rq = 1.0f / fmaxf(sqrtf(nq), kEps), rk = 1.0f / fmaxf(sqrtf(nk), kEps);
    const int cg = tid % cgs, sl = tid / cgs;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (sl < slices) {
        const float4 vv = *reinterpret_cast<const float4*>(cv + 4 * cg);
        float4* S = reinterpret_cast<float4*>(state + bh * (size_t)dk * dv) + cg;
        for (int r = sl; r < dk; r += slices) {
            float4 x = S[(size_t)r * cgs];
            const float kr = kh[r] * rk, qr = qh[r] * rq;
            x.x = fmaf(kr, vv.x, x.x); x.y = fmaf(kr, vv.y, x.y); x.z = fmaf(kr, vv.z, x.z); x.w = fmaf(kr, vv.w, x.w);
            S[(size_t)r * cgs] = x;
            acc.x = fmaf(qr, x.x, acc.x); acc.y = fmaf(qr, x.y, acc.y); acc.z = fmaf(qr, x.z, acc.z); acc.w = fmaf(qr, x.w, acc.w);
        }
        *reinterpret_cast<float4*>(part + (size_t)sl * dv + 4 * cg) = acc;
    }
    __syncthreads();
    for (int i = tid; i < dv; i += 256) {
        float a = 0.f;
        for (int s2 = 0; s2 < slices; ++s2) a += part[(size_t)s2 * dv + i];
        o[bh * dv + i] = from_f32<T>(a);
    }
}

cudaError_t launch_decode_generic(const void* q, const void* k, const void* v, float* state, void* o,
                                  int B, int H, int dk, int dv, cott_dtype dt, const float* m,
                                  const float* seq_len, float seq_len_scalar, cudaStream_t st) {
    if (dk < 1 || dv < 4 || (dv & 3) || dv > 1024 || dk > 1024) return cudaErrorInvalidValue;
    const int cgs = dv / 4, slices = 256 / cgs;
    const size_t smem = sizeof(float) * ((size_t)2 * dk + dv + (size_t)slices * dv);
    const unsigned BH = (unsigned)(B * H);
    if (dt == COTT_F32)
        decode_generic_kernel<float><<<BH, 256, smem, st>>>((const float*)q, (const float*)k, (const float*)v, state,
                                                            (float*)o, H, dk, dv, m, seq_len, seq_len_scalar);
    else
        decode_generic_kernel<__nv_bfloat16><<<BH, 256, smem, st>>>((const __nv_bfloat16*)q, (const __nv_bfloat16*)k,
                                                                    (const __nv_bfloat16*)v, state, (__nv_bfloat16*)o, H,
                                                                    dk, dv, m, seq_len, seq_len_scalar);
    note_launch();
    return cudaGetLastError();
}

cudaError_t launch_decode(const void* q, const void* k, const void* v, float* state, void* o,
                          int B, int H, int d, cott_dtype dt, const float* m,
                          const float* seq_len, float seq_len_scalar, cudaStream_t st) {
    return dt == COTT_F32
               ? launch_decode_t<float>(q, k, v, state, o, B, H, d, m, seq_len, seq_len_scalar, st)
               : launch_decode_t<__nv_bfloat16>(q, k, v, state, o, B, H, d, m, seq_len,
                                                seq_len_scalar, st);
}

}  // namespace cott
