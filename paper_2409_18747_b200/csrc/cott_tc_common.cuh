// Helpers shared by the warp-specialised tensor-core kernels of cott_tc_bwd.cu and
// cott_tc_bidir.cu: the bounded mbarrier wait with its abort protocol, and a few small device
// functions.  Every kernel that uses them lays out its control block the same way: mbarriers in
// the first 512 bytes, then the tensor-memory slot (offset 512), the abort flag (516) and, three
// words behind it, the wait limit in units of 1024 SM cycles.
#pragma once
#include "cott_sm100.cuh"

namespace cott {
namespace tc {

using namespace sm100;

constexpr int kCtlTmemSlot = 512, kCtlAbort = 516;
constexpr uint32_t kDescHi = smem_desc_hi(1024);
#ifndef COTT_WAIT_HINT_NS
#define COTT_WAIT_HINT_NS 1000
#endif
constexpr uint32_t kWaitHintNs = COTT_WAIT_HINT_NS;   // a waiting thread may be parked this long per try

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Bounded wait that also gives up as soon as any thread of the CTA has given up.  The thread
// that gives up first leaves a record of where: bit 31 set, warp index in bits 16-20, byte
// offset of the barrier inside the barrier block in bits 4-13, parity in bit 0.
// (The loop is a function of its own, not inlined: these kernels have dozens of waits, and
// their code must stay small enough for the instruction caches -- several roles run different
// code on one SM at the same time.)
static __device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    const long long t0 = clock64();
    for (uint32_t it = 1;; ++it) {
        if (kWaitHintNs ? mbar_try_wait_hint(bar, parity, kWaitHintNs) : mbar_try_wait(bar, parity)) return true;
        if ((it & 15u) == 1) {
            if (*abort_flag) return false;
            if (clock64() - t0 > ((long long)abort_flag[3] << 10)) {
                const uint32_t bars = (uint32_t)__cvta_generic_to_shared((const void*)abort_flag) - (uint32_t)kCtlAbort;
                const uint32_t where = 0x80000000u | ((threadIdx.x >> 5) << 16) | (((bar - bars) & 0x3FFu) << 4) | (parity & 1u);
                atomicCAS(const_cast<int*>(abort_flag), 0, (int)where);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool wait_or_abort(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    return wait_slow(bar, parity, abort_flag);
}

__device__ __forceinline__ uint4 pack8(const uint32_t* r) {
    uint4 w;
    w.x = pack_bf16(__uint_as_float(r[0]), __uint_as_float(r[1]));
    w.y = pack_bf16(__uint_as_float(r[2]), __uint_as_float(r[3]));
    w.z = pack_bf16(__uint_as_float(r[4]), __uint_as_float(r[5]));
    w.w = pack_bf16(__uint_as_float(r[6]), __uint_as_float(r[7]));
    return w;
}

// x / max(||x||, eps) on one row of 64 bf16 values held in w[8] (eight 16-byte chunks), in
// packed bf16 arithmetic with the scale split in two bf16 terms (rn = hi + lo to 2^-17):
// round(x hi + round(x lo)) is x rn rounded once, up to a second rounding of the small term --
// two instructions per pair of elements instead of unpacking, two multiplies and a conversion.
// Returns the norm; *rn_out = 1 / max(norm, eps).
__device__ __forceinline__ float normalise_row64(uint4 (&w)[8], float eps, float* rn_out) {
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
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
    const float rn = 1.0f / fmaxf(nrm, eps);
    const __nv_bfloat16 hi = __float2bfloat16_rn(rn);
    const __nv_bfloat16 lo = __float2bfloat16_rn(rn - __bfloat162float(hi));
    const __nv_bfloat162 hi2 = __halves2bfloat162(hi, hi), lo2 = __halves2bfloat162(lo, lo);
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        __nv_bfloat162* e = reinterpret_cast<__nv_bfloat162*>(&w[j]);
#pragma unroll
        for (int i = 0; i < 4; ++i) e[i] = __hfma2(e[i], hi2, __hmul2(e[i], lo2));
    }
    *rn_out = rn;
    return nrm;
}

}  // namespace tc
}  // namespace cott
