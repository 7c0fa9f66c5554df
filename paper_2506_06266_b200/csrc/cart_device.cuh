// Device-side helpers shared by the kernels of libcart.so: mbarrier waits with a time limit, TMA tile
// loads, and small arithmetic wrappers.  Everything is internal (anonymous namespace per translation unit).
#ifndef CART_DEVICE_CUH_
#define CART_DEVICE_CUH_

#include <cuda_bf16.h>
#include <stdint.h>

#include "cart_internal.h"

namespace cart {
namespace {

constexpr uint64_t kWaitLimitNs = 2000000000ull;      // a wait gives up after about two seconds
constexpr long long kWaitLimitCycles = 4000000000ll;   // the same in SM cycles (2 s at 2 GHz, 3 s at 1.3 GHz)

// ---- small PTX wrappers ---------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ uint64_t global_timer_ns()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false if the block has given up (this wait ran out, or another warp's did).
// The limit is kept with the SM's cycle counter, which costs a few cycles to read and is first read
// after a thousand polls: a wait that is about to succeed never pays for time keeping.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          uint32_t *status, uint32_t code)
{
    if (mbar_try_wait(bar, parity)) return true;
    uint32_t spins = 0;
    long long t0 = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 0x3FFu) == 0) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) {
                t0 = now | 1;
            } else if (now - t0 > kWaitLimitCycles) {
                *abort_flag = 1;
                atomicOr(status, code);
                return false;
            }
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tmap, int32_t x, int32_t y,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// The same with an L2 eviction-priority hint (a policy made by l2_evict_first_policy()).
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap *tmap, int32_t x, int32_t y,
                                                 uint32_t bar, uint64_t policy)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}
// Data that is read once per launch (a request's own KV stream) should leave L2 first.
__device__ __forceinline__ uint64_t l2_evict_first_policy()
{
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    return policy;
}
// Programmatic dependent launch.  The decode kernels are launched so that the next kernel on the
// stream may become resident while this one drains: every block says at once that dependents may be
// scheduled, and a dependent thread waits for the full completion (and memory visibility) of the
// kernels before it only when it first needs what they may have written.
__device__ __forceinline__ void pdl_launch_dependents()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
}
// a word another kernel on the stream has written (not through the read-only path)
__device__ __forceinline__ uint32_t ld_volatile_u32(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ float fast_exp2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
// Log-sum-exp merge of the partials of one split row group (softmax over a union of token sets is
// the lse-weighted mix of the softmaxes over the sets, from Eq. 1): slots mi.slot_begin .. slot_end-1
// hold normalised fp32 outputs [slot][G][128] and base-2 lse values [slot][kMaxGroup].  Called by
// `nthreads` threads of one block with tid = 0 .. nthreads-1; the caller has fenced.  An item is one
// query row times four output dims; a thread works on up to kItems items at once and on kSlots slots
// at a time, so that kItems * kSlots independent 16-byte loads are in flight (a lone warp: 4 x 2; a
// block with a thread per item: 1 x 8).
template <int kItems, int kSlots>
__device__ __forceinline__ void merge_row_group(const cart_merge_item mi, int G, const float *part_o,
                                                const float *part_lse2, void *out, float *lse, int tid,
                                                int nthreads)
{
    const uint32_t n = mi.slot_end - mi.slot_begin;
    const int total = G * 32;
    for (int base = tid; base < total; base += kItems * nthreads) {
        const float *lp[kItems];
        const float4 *op4[kItems];
        float M[kItems], L[kItems];
        float4 a[kItems];
        bool on[kItems];
#pragma unroll
        for (int k = 0; k < kItems; ++k) {
            const int idx = base + k * nthreads;
            on[k] = idx < total;
            const int r = on[k] ? idx >> 5 : 0, quad = idx & 31;
            lp[k] = part_lse2 + (size_t)mi.slot_begin * kMaxGroup + r;
            op4[k] = reinterpret_cast<const float4 *>(part_o + ((size_t)mi.slot_begin * G + r) * kHeadDim) + quad;
            M[k] = -INFINITY;
            L[k] = 0.f;
            a[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (uint32_t c0 = 0; c0 < n; c0 += 8) {  // eight slots' lse values in flight per item
            float lv[kItems][8];
#pragma unroll
            for (int k = 0; k < kItems; ++k)
#pragma unroll
                for (uint32_t j = 0; j < 8; ++j)
                    lv[k][j] = (on[k] && c0 + j < n) ? __ldcg(lp[k] + (size_t)(c0 + j) * kMaxGroup) : -INFINITY;
#pragma unroll
            for (int k = 0; k < kItems; ++k)
#pragma unroll
                for (uint32_t j = 0; j < 8; ++j) M[k] = fmaxf(M[k], lv[k][j]);
        }
        for (uint32_t c0 = 0; c0 < n; c0 += kSlots) {
            float lv[kItems][kSlots];
            float4 v[kItems][kSlots];
#pragma unroll
            for (int k = 0; k < kItems; ++k) {
#pragma unroll
                for (uint32_t j = 0; j < kSlots; ++j) {
                    const bool in = on[k] && c0 + j < n;
                    lv[k][j] = in ? __ldcg(lp[k] + (size_t)(c0 + j) * kMaxGroup) : -INFINITY;
                    v[k][j] = in ? __ldcg(op4[k] + (size_t)(c0 + j) * G * (kHeadDim / 4)) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
#pragma unroll
            for (int k = 0; k < kItems; ++k) {
#pragma unroll
                for (uint32_t j = 0; j < kSlots; ++j) {
                    const float wgt = on[k] ? fast_exp2(lv[k][j] - M[k]) : 0.f;  // 0 for the slots past the end
                    L[k] += wgt;
                    a[k].x += wgt * v[k][j].x;
                    a[k].y += wgt * v[k][j].y;
                    a[k].z += wgt * v[k][j].z;
                    a[k].w += wgt * v[k][j].w;
                }
            }
        }
#pragma unroll
        for (int k = 0; k < kItems; ++k) {
            const int idx = base + k * nthreads;
            if (!on[k]) continue;
            const int r = idx >> 5, quad = idx & 31;
            const float inv = 1.f / L[k];
            const size_t orow = (size_t)mi.row_group * G + r;
            uint2 packed;
            packed.x = pack_bf16(a[k].x * inv, a[k].y * inv);
            packed.y = pack_bf16(a[k].z * inv, a[k].w * inv);
            *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(out) + orow * kHeadDim + 4 * quad) = packed;
            if (quad == 0 && lse) lse[orow] = (M[k] + log2f(L[k])) * 0.6931471805599453f;
        }
    }
}

}  // namespace
}  // namespace cart
#endif
