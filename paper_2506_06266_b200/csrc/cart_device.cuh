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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          uint32_t *status, uint32_t code)
{
    if (mbar_try_wait(bar, parity)) return true;
    if (*abort_flag) return false;
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 0xFFu) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
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
// `nthreads` threads of one block with tid = 0 .. nthreads-1; the caller has fenced.
__device__ __forceinline__ void merge_row_group(const cart_merge_item mi, int G, const float *part_o,
                                                const float *part_lse2, void *out, float *lse, int tid,
                                                int nthreads)
{
    for (int idx = tid; idx < G * 64; idx += nthreads) {
        const int r = idx >> 6, dpair = idx & 63;
        float M = -INFINITY;
        for (uint32_t c = mi.slot_begin; c < mi.slot_end; ++c)
            M = fmaxf(M, __ldcg(part_lse2 + (size_t)c * kMaxGroup + r));
        float L = 0.f, a0 = 0.f, a1 = 0.f;
        for (uint32_t c = mi.slot_begin; c < mi.slot_end; ++c) {
            const float wgt = fast_exp2(__ldcg(part_lse2 + (size_t)c * kMaxGroup + r) - M);
            const float2 v = __ldcg(reinterpret_cast<const float2 *>(part_o + ((size_t)c * G + r) * kHeadDim + 2 * dpair));
            L += wgt;
            a0 += wgt * v.x;
            a1 += wgt * v.y;
        }
        const float inv = 1.f / L;
        const size_t orow = (size_t)mi.row_group * G + r;
        __nv_bfloat162 *op = reinterpret_cast<__nv_bfloat162 *>(reinterpret_cast<__nv_bfloat16 *>(out) + orow * kHeadDim + 2 * dpair);
        *op = __floats2bfloat162_rn(a0 * inv, a1 * inv);
        if (dpair == 0 && lse) lse[orow] = (M + log2f(L)) * 0.6931471805599453f;
    }
}

}  // namespace
}  // namespace cart
#endif
