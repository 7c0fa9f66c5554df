// Shared-segment decode attention for sm_100a: the dense part of the path.
//
// When many requests of a batch attend to the same stored Cartridge (one Cartridge serving many
// users, Sec. 1 / Sec. 3.3 of the paper; pool members composed by many requests, Sec. 5.4), the scores
// of all their query heads against one K tile are one matrix product, and so is the weighted sum of
// the V tile.  This kernel evaluates Eq. 1 restricted to a run of 128-token tiles of such a segment
// for up to 128 query rows at once (row i * G + h = head h of the M-tile's i-th reader) on the
// tcgen05 tensor cores, so the tile is fetched once per 128 rows instead of once per request:
//
//   producer warps  TMA loads of K tiles (warp 0, three stages) and V tiles (warp 2, two stages), 128 tokens
//                   x 128 dims, 128-byte swizzle, completion on mbarriers
//   MMA warp        one thread issues  S = Q K^T  (128 x 128 x 128, both operands from shared memory,
//                   accumulator in tensor memory) and  O += P V  (A operand P from tensor memory, V from
//                   shared memory, accumulating in tensor memory over the warpgroup's tiles of the unit);
//                   tcgen05.commit signals mbarriers
//   2 x 4 softmax  two warpgroups take alternate tiles (warpgroup w owns S buffer w and accumulator w).
//   warps           Thread r of a warpgroup owns query row r: reads S from tensor memory (two loads in
//                   flight), keeps a reference maximum and the sum of an online softmax over its
//                   warpgroup's tiles in fp32, and writes P = 2^(s - m) as bf16 pairs back over the first
//                   half of the S buffer (tcgen05.st).  The reference maximum only moves when a row's
//                   maximum has grown by more than 2^8 (then the warp rescales its lanes of the accumulator
//                   in tensor memory); sum and accumulator always refer to the same reference, so the
//                   result is exact.  At the end of a unit the warpgroups read their accumulators and
//                   combine their states through shared memory.
//
// S (with P in it) is double-buffered in tensor memory and each warpgroup has its own accumulator
// (4 x 128 columns), so the products of tile t+1 run while the softmax of tile t does.  At the end of a
// unit every row is written as a
// normalised fp32 partial (o, lse); the partials of a (request, KV head) row group are merged by
// log-sum-exp either by the block that delivers the last one -- this kernel's or the stream kernel's --
// or, when the batch has more split row groups than blocks, by a merge kernel that runs afterwards.
//
// Every wait is bounded; on expiry the block raises a flag in the device status word, stops issuing
// work, waits (bounded) for what is in flight, frees its tensor memory and returns.
#include <cuda_bf16.h>

#include "cart_device.cuh"
#include "cart_internal.h"

namespace cart {
namespace {

constexpr int kShTile = kShareTileTokens;             // tokens per tile = N of the score product
constexpr uint32_t kShBlock = 128u * 128u;            // 128 rows x 128 bytes: one swizzled block (64 bf16 wide)
constexpr uint32_t kShTileBytes = 2u * kShBlock;      // 128 x 128 bf16
constexpr int kKStages = 3;                           // K tiles in flight (each ring has its own producer warp)
constexpr int kVStages = 2;
constexpr int kShThreads = 384;                       // utility warpgroup (K producer, MMA, V producer, 1 idle) + 2 softmax warpgroups
// Registers per thread after the warpgroups have re-divided the block's allocation (384 x 168): the
// utility warps need few, the softmax threads hold a 128-float accumulator at the end of a unit.  4 x 32 x 40 + 8 x 32 x 232
// = 64512 registers, and per SM sub-partition 1 utility + 2 softmax warps = 16128 of its 16384.
constexpr int kRegsUtility = 40;
constexpr int kRegsSoftmax = 232;
constexpr int kSoftmaxThreads = 128;                  // one softmax warpgroup
constexpr uint32_t kTmemCols = 512;                   // S0 S1 (scores, then P), O0 O1 (accumulators): 128 fp32 columns each
constexpr float kRescaleStep = 8.f;                   // how far a row's maximum may outgrow its reference (base-2 units)

// shared-memory layout (offsets from a 1024-byte aligned base)
constexpr uint32_t kOffQ = 0;
constexpr uint32_t kOffX = kOffQ + kShTileBytes;       // with Q: the 64 KB scratch of a unit's end
constexpr uint32_t kOffK = kOffX + kShTileBytes;
constexpr uint32_t kOffV = kOffK + kKStages * kShTileBytes;
constexpr uint32_t kOffBar = kOffV + kVStages * kShTileBytes;
constexpr uint32_t kOffMisc = kOffBar + 32 * 8;        // room for 32 barriers (22 used); then: tmem address, abort flag, unit flag
constexpr uint32_t kOffFlags = kOffMisc + 16;          // one word per reader: "merge this row group"
constexpr uint32_t kOffComb = kOffFlags + 128 * 4;     // running maximum and sum of the second warpgroup's rows
constexpr uint32_t kShSmemUsed = kOffComb + 2 * 128 * 4;
constexpr uint32_t kShSmemBytes = kShSmemUsed + 1024;  // slack to align the base
static_assert(kShSmemBytes <= 232448, "shared memory budget of one sm_100 block exceeded");

enum Bar : int {
    kBarKFull = 0,   // [kKStages] TMA -> MMA
    kBarKEmpty = 3,  // [kKStages] MMA (commit) -> TMA
    kBarVFull = 6,   // [kVStages]
    kBarVEmpty = 8,  // [kVStages]
    kBarSFull = 10,  // [2] MMA (commit) -> softmax
    kBarSFree = 12,  // [2] MMA (commit of P V: the probabilities live in the S buffer) -> MMA
    kBarPReady = 14, // [2] softmax -> MMA          (4 arrivals: one per warp of the warpgroup)
    kBarOFull = 16,  // [2] MMA (commit of P V) -> softmax: the accumulator holds the product
    kBarQReady = 20, // softmax -> MMA              (8 arrivals: every softmax warp)
    kBarDrain = 21,  // MMA (commit) -> MMA, on the way out
};
static_assert(kBarKEmpty - kBarKFull >= kKStages && kBarVFull - kBarKEmpty >= kKStages &&
              kBarVEmpty - kBarVFull >= kVStages && kBarSFull - kBarVEmpty >= kVStages, "barrier indices overlap");

// ---- tcgen05 wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle.  lbo / sbo in bytes.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo)
{
    uint64_t d = (uint64_t)((saddr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;  // descriptor version of this architecture
    d |= 2ull << 61;  // layout type: 128-byte swizzle
    return d;
}
// Instruction descriptor, kind::f16: fp32 accumulator, bf16 A and B, M = 128, N = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescS = kIdesc;                  // A (Q) and B (K tile) both K-major
constexpr uint32_t kIdescPV = kIdesc | (1u << 16);    // B (V tile) is MN-major: dims contiguous

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The same with the A operand in tensor memory (lane = row, 8 columns of bf16 pairs per 16-wide step).
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Writes 16 consecutive 32-bit columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&w)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "r"(w[0]), "r"(w[1]), "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7]), "r"(w[8]), "r"(w[9]),
        "r"(w[10]), "r"(w[11]), "r"(w[12]), "r"(w[13]), "r"(w[14]), "r"(w[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 32 consecutive 32-bit columns of this thread's tensor-memory lane, in two steps, so that several
// loads can be in flight and arithmetic can run under them: tmem_ld32_issue starts a load, tmem_ld_wait waits for all loads issued so far; the registers named
// in the wait are only then valid (naming them keeps the compiler from reading them earlier).
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
        "%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait(uint32_t (&r)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                   "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                   "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :
                 : "memory");
}
__device__ __forceinline__ void softmax_bar()  // the first softmax warpgroup
{
    asm volatile("bar.sync 2, %0;" ::"n"(kSoftmaxThreads) : "memory");
}
__device__ __forceinline__ void softmax_bar_both()  // both softmax warpgroups
{
    asm volatile("bar.sync 3, %0;" ::"n"(2 * kSoftmaxThreads) : "memory");
}

// "The kernels before this one on the stream are complete and their writes visible."  Alone, that is
// griddepcontrol.wait.  Side by side with the stream kernel (launched just before, resident at the same
// time) it is a flag that the stream kernel's block 0 sets after its own griddepcontrol.wait: waiting for
// the stream kernel itself would put the two kernels one after the other again.  All of the stream
// kernel's blocks are resident before this kernel is launched (a dependent launch happens once every
// block of the kernel before has started), so the flag is on its way; the wait is bounded all the same.
// Called by one lane per warp; the others follow through __syncwarp.
__device__ __forceinline__ bool wait_for_prior_kernels(const SharedParams &p, volatile uint32_t *abort_flag)
{
    if (p.ready_flag == nullptr) {
        pdl_wait();
        return true;
    }
    uint32_t spins = 0;
    long long t0 = 0;
    for (;;) {
        uint32_t v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p.ready_flag) : "memory");
        if ((int32_t)(v - p.seq) >= 0) return true;
        if ((++spins & 0xFFu) == 0) {
            if (*abort_flag) return false;
            const long long now = clock64();
            if (t0 == 0) {
                t0 = now | 1;
            } else if (now - t0 > kWaitLimitCycles) {
                *abort_flag = 1;
                atomicOr(p.status, kStatusTimeoutConsumer);
                return false;
            }
        }
    }
}

__global__ void __launch_bounds__(kShThreads, 1)
cart_shared_kernel(const __grid_constant__ CUtensorMap tmap, const SharedParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    auto bar = [&](int i) { return base + kOffBar + (uint32_t)i * 8u; };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + kOffMisc);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    volatile uint32_t *unit_ok = tmem_slot + 2;
    volatile uint32_t *flags = reinterpret_cast<volatile uint32_t *>(smem + kOffFlags);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    pdl_launch_dependents();

    if (threadIdx.x == 0) {
        for (int i = 0; i < kKStages; ++i) {
            mbar_init(bar(kBarKFull + i), 1);
            mbar_init(bar(kBarKEmpty + i), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(kBarVFull + i), 1);
            mbar_init(bar(kBarVEmpty + i), 1);
            mbar_init(bar(kBarSFull + i), 1);
            mbar_init(bar(kBarSFree + i), 1);
            mbar_init(bar(kBarOFull + i), 1);
            mbar_init(bar(kBarPReady + i), 4);
        }
        mbar_init(bar(kBarQReady), 8);
        mbar_init(bar(kBarDrain), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        // the whole tensor memory of the SM: one block per SM runs this kernel (shared memory sees to that)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + kOffMisc),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    // The plan is in place before any of these kernels starts.  Shared tiles of stored Cartridges are only
    // ever written by copies and may be fetched at once; shared tiles in suffix storage (prefill: the part
    // of the suffix that a group of rows has in common, units marked CART_UNIT_SUFFIX) may have been
    // written by the kernel before this one, so the producers wait for the kernels before them ahead of
    // the first such unit.  The queries, the partial slots and the tickets may still be in use by those
    // kernels too: the softmax warps wait before they read a query.
    const uint32_t unit_begin = p.unit_cta_begin[blockIdx.x];
    const uint32_t unit_end = p.unit_cta_begin[blockIdx.x + 1];

    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsUtility));
        if (warp == 0 || warp == 2) {
            // ================= producers: warp 0 feeds the K ring, warp 2 the V ring ========================
            // (separate threads, so that a K tile is requested the moment its stage is free, whatever the
            //  V ring is waiting for)
            if (lane == 0) {
                const bool is_v = warp == 2;
                const int full0 = is_v ? kBarVFull : kBarKFull, empty0 = is_v ? kBarVEmpty : kBarKEmpty;
                const uint32_t ring = base + (is_v ? kOffV : kOffK);
                const uint32_t nst = is_v ? (uint32_t)kVStages : (uint32_t)kKStages;
                asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap)) : "memory");
                uint32_t tt = 0;
                bool ok = true;
                bool waited = false;
                for (uint32_t ui = unit_begin; ui < unit_end && ok; ++ui) {
                    const cart_shared_unit u = p.units[ui];
                    if (!waited && (u.flags & CART_UNIT_SUFFIX)) {
                        ok = wait_for_prior_kernels(p, abort_flag);
                        if (!ok) break;
                        waited = true;
                    }
                    const uint32_t row0 = (is_v ? u.v_row : u.k_row) + (uint32_t)p.layer * u.layer_stride;
                    for (uint32_t t = 0; t < u.n_tiles; ++t, ++tt) {
                        const int st = (int)(tt % nst);
                        const uint32_t par = (tt / nst) & 1u;
                        const int32_t y = (int32_t)(row0 + t * kShTile);
                        ok = mbar_wait(bar(empty0 + st), par ^ 1u, abort_flag, p.status, kStatusTimeoutProducer);
                        if (!ok) break;
                        const uint32_t dst = ring + (uint32_t)st * kShTileBytes;
                        mbar_expect_tx(bar(full0 + st), kShTileBytes);
                        // a block of the tile = 128 rows x 64 dims = two boxes of 64 rows
                        tma_load_2d(dst, &tmap, 0, y, bar(full0 + st));
                        tma_load_2d(dst + kShBlock / 2, &tmap, 0, y + 64, bar(full0 + st));
                        tma_load_2d(dst + kShBlock, &tmap, 64, y, bar(full0 + st));
                        tma_load_2d(dst + kShBlock + kShBlock / 2, &tmap, 64, y + 64, bar(full0 + st));
                    }
                }
                if (!ok) {
                    // gave up: wait (bounded) for the copies still in flight before the block leaves
                    for (uint32_t u2 = (tt > nst ? tt - nst : 0u); u2 <= tt; ++u2) {
                        const int st = (int)(u2 % nst);
                        const uint32_t par = (u2 / nst) & 1u;
                        const uint64_t t0 = global_timer_ns();
                        while (!mbar_try_wait(bar(full0 + st), par) && global_timer_ns() - t0 < kWaitLimitNs) {}
                    }
                }
            }
            __syncwarp();
        } else if (warp == 1) {
            // ================= MMA issuer ===================================================================
            if (lane == 0) {
                const uint32_t q_lo = base + kOffQ;
                uint32_t tt0 = 0;   // tiles of earlier units
                uint32_t nunit = 0;
                bool ok = true;
                // S(tt) = Q K^T into S buffer tt & 1
                auto issue_s = [&](uint32_t tt) -> bool {
                    const int st = (int)(tt & 1u);
                    const uint32_t par = (tt >> 1) & 1u;
                    const uint32_t kst = tt % (uint32_t)kKStages, kpar = (tt / (uint32_t)kKStages) & 1u;
                    if (!mbar_wait(bar(kBarKFull + (int)kst), kpar, abort_flag, p.status, kStatusTimeoutMma)) return false;
                    if (!mbar_wait(bar(kBarSFree + st), par ^ 1u, abort_flag, p.status, kStatusTimeoutMma)) return false;
                    tc_fence_after();
                    const uint32_t k_lo = base + kOffK + kst * kShTileBytes;
                    // the operands' descriptors differ from step to step only in the start address field
                    // (units of 16 bytes): the next 16 dims are 32 bytes on, the second 64-dim block kShBlock on
                    const uint64_t a0 = umma_desc(q_lo, 16, 1024), b0 = umma_desc(k_lo, 16, 1024);
                    const uint32_t d_s = tmem + (uint32_t)st * 128u;
    #pragma unroll
                    for (uint32_t k = 0; k < 8; ++k) {  // 16 dims per instruction
                        const uint64_t off16 = (uint64_t)(((k >> 2) * kShBlock + (k & 3u) * 32u) >> 4);
                        umma_bf16(d_s, a0 + off16, b0 + off16, kIdescS, k);
                    }
                    umma_commit(bar(kBarSFull + st));
                    umma_commit(bar(kBarKEmpty + (int)kst));
                    return true;
                };
                // O += P V into the accumulator of warpgroup tt & 1; `first`: the warpgroup's first tile of the unit
                auto issue_pv = [&](uint32_t tt, bool first) -> bool {
                    const int st = (int)(tt & 1u);
                    const uint32_t par = (tt >> 1) & 1u;
                    if (!mbar_wait(bar(kBarVFull + st), par, abort_flag, p.status, kStatusTimeoutMma)) return false;
                    if (!mbar_wait(bar(kBarPReady + st), par, abort_flag, p.status, kStatusTimeoutMma)) return false;
                    tc_fence_after();
                    const uint32_t v_lo = base + kOffV + (uint32_t)st * kShTileBytes;
                    // P: the A operand comes from tensor memory, where the softmax warps left it in the first
                    // 64 columns of the S buffer (two bf16 per column, 16 tokens = 8 columns per step).
                    // V: tokens are rows of 128 bytes (8-token groups 1024 bytes apart, 16 tokens = 2048 bytes
                    // per step); the two 64-dim blocks of the tile are kShBlock bytes apart.
                    const uint64_t b0 = umma_desc(v_lo, kShBlock, 1024);
                    const uint32_t p_tm = tmem + (uint32_t)st * 128u;
                    const uint32_t d_o = tmem + 256u + (uint32_t)st * 128u;
    #pragma unroll
                    for (uint32_t k = 0; k < 8; ++k)  // 16 tokens per instruction
                        umma_bf16_ts(d_o, p_tm + 8u * k, b0 + (uint64_t)(k * 128u), kIdescPV, (first && k == 0u) ? 0u : 1u);
                    umma_commit(bar(kBarOFull + st));
                    umma_commit(bar(kBarVEmpty + st));
                    umma_commit(bar(kBarSFree + st));  // the S buffer (and the P in it) may be overwritten
                    return true;
                };
                for (uint32_t ui = unit_begin; ui < unit_end && ok; ++ui, ++nunit) {
                    const uint32_t n = p.units[ui].n_tiles;
                    ok = mbar_wait(bar(kBarQReady), nunit & 1u, abort_flag, p.status, kStatusTimeoutMma);
                    if (!ok) break;
                    tc_fence_after();
                    ok = issue_s(tt0);
                    for (uint32_t t = 0; t < n && ok; ++t) {
                        if (t + 1 < n) ok = issue_s(tt0 + t + 1);
                        if (ok) ok = issue_pv(tt0 + t, t < 2u);
                    }
                    tt0 += n;
                }
                // products still in flight must finish before the tensor memory is given back
                umma_commit(bar(kBarDrain));
                const uint64_t t0 = global_timer_ns();
                while (!mbar_try_wait(bar(kBarDrain), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
            }
            __syncwarp();
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        // ================= softmax / epilogue warps ====================================================
        const int G = p.group;
        const int wg = (warp - 4) >> 2;       // softmax warpgroup 0 or 1: owns the tiles with (index & 1) == wg
        const int sw = warp & 3;              // the tensor-memory lanes this warp may read: 32 sw .. 32 sw + 31
        const int row = 32 * sw + lane;       // query row of the M-tile = tensor-memory lane
        const int tid = row;                  // index among the 128 threads of the warpgroup
        const uint32_t lane_addr = tmem + ((uint32_t)(32 * sw) << 16);
        const __nv_bfloat16 *q = reinterpret_cast<const __nv_bfloat16 *>(p.q);
        const uint32_t swz = (uint32_t)(row & 7);
        float *comb_ml = reinterpret_cast<float *>(smem + kOffComb); // [2][128 rows]
        uint32_t tt0 = 0;
        bool alive = true;
        bool waited = false;  // for the kernels before this one on the stream
        float o_acc[128];
        // the warp's lanes must stay together (the tensor-memory loads are warp-wide): a wait fails for
        // all of them or for none
        auto warp_wait = [&](uint32_t b, uint32_t parity) -> bool {
            return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag, p.status, kStatusTimeoutConsumer));
        };
        const uint32_t s_addr = lane_addr + (uint32_t)wg * 128u;
        const uint32_t o_addr = lane_addr + 256u + (uint32_t)wg * 128u;

        for (uint32_t ui = unit_begin; ui < unit_end && alive; ++ui) {
            const cart_shared_unit u = p.units[ui];
            const int i_reader = row / G, h = row - i_reader * G;
            const bool valid = (uint32_t)i_reader < u.n_readers;
            uint32_t entry = 0, batch = 0, slot = 0;
            if (valid) {
                entry = u.reader_begin + (uint32_t)i_reader;
                batch = p.readers[entry];
                slot = p.reader_slot[(size_t)entry * p.n_kv_heads + u.kv_head] + u.chunk;  // where this row's partial goes
            }
            // ---- this row's query into shared memory, in the swizzled K-major operand layout; each
            //      warpgroup copies one 64-dim half -------------------------------------------------
            if (!waited) {
                bool ok0 = true;
                if (lane == 0) ok0 = wait_for_prior_kernels(p, abort_flag);
                alive = __all_sync(0xffffffffu, ok0);
                waited = true;
            }
            {
                const uint4 *src = reinterpret_cast<const uint4 *>(
                    q + ((size_t)batch * p.n_q_heads + (size_t)u.kv_head * G + h) * kHeadDim) + 8 * wg;
                const uint32_t qrow = base + kOffQ + (uint32_t)wg * kShBlock + (uint32_t)row * 128u;
                uint4 v[8];
#pragma unroll
                for (uint32_t c = 0; c < 8; ++c) v[c] = valid ? __ldg(src + c) : make_uint4(0u, 0u, 0u, 0u);  // all in flight
#pragma unroll
                for (uint32_t c = 0; c < 8; ++c) {
                    const uint32_t a = qrow + ((c ^ swz) << 4);
                    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(v[c].x), "r"(v[c].y), "r"(v[c].z),
                                 "r"(v[c].w)
                                 : "memory");
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarQReady));
            }
            // m_run: the reference maximum that l_run and the warpgroup's accumulator in tensor memory refer to.
            // It only moves when a row's maximum has outgrown it by more than kRescaleStep (base 2); until then
            // probabilities may exceed 1 (by at most that factor), which bf16 and the fp32 sums hold easily.
            float m_run = -INFINITY, l_run = 0.f;

            // this warpgroup's tiles of the unit: those whose block-wide index is congruent to wg mod 2
            bool have_prev = false;
            uint32_t prev_tt = 0;
            for (uint32_t t = ((uint32_t)wg ^ tt0) & 1u; t < u.n_tiles; t += 2) {
                const uint32_t tt = tt0 + t;
                const uint32_t par = (tt >> 1) & 1u;
                alive = warp_wait(bar(kBarSFull + wg), par);
                if (!alive) break;
                tc_fence_after();
                // pass 1: the row's maximum over the tile
                float mx = -INFINITY;
#pragma unroll
                for (int c2 = 0; c2 < 2; ++c2) {  // two loads of 32 columns in flight
                    uint32_t a[32], b[32];
                    tmem_ld32_issue(s_addr + (uint32_t)c2 * 64u, a);
                    tmem_ld32_issue(s_addr + (uint32_t)c2 * 64u + 32u, b);
                    tmem_ld_wait(a);
                    tmem_ld_wait(b);
#pragma unroll
                    for (int k = 0; k < 32; ++k) mx = fmaxf(mx, fmaxf(__uint_as_float(a[k]), __uint_as_float(b[k])));
                }
                mx *= p.scale_log2;
                if (!have_prev) {
                    m_run = mx;
                } else if (__any_sync(0xffffffffu, mx > m_run + kRescaleStep)) {
                    // a row of this warp has outgrown its reference: every row moves up to its maximum and the
                    // warp rescales its lanes of the accumulator (tensor-memory accesses are warp-wide, so the
                    // warp decides together; the other rows' factors are 1 or close to it)
                    const float m_new = fmaxf(m_run, mx);
                    const float f = fast_exp2(m_run - m_new);
                    m_run = m_new;
                    l_run *= f;
                    // the product of this warpgroup's previous tile must have landed first
                    alive = warp_wait(bar(kBarOFull + wg), (prev_tt >> 1) & 1u);
                    if (!alive) break;
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        uint32_t o[32];
                        tmem_ld32_issue(o_addr + (uint32_t)c * 32u, o);
                        tmem_ld_wait(o);
#pragma unroll
                        for (int k = 0; k < 32; ++k) o[k] = __float_as_uint(__uint_as_float(o[k]) * f);
                        tmem_st16(o_addr + (uint32_t)c * 32u, reinterpret_cast<const uint32_t(&)[16]>(o[0]));
                        tmem_st16(o_addr + (uint32_t)c * 32u + 16u, reinterpret_cast<const uint32_t(&)[16]>(o[16]));
                    }
                    // (these stores are waited for with those of P below, before the MMA warp hears of the tile)
                }
                const float m_new = m_run;
                // pass 2: probabilities, as bf16 pairs, back into tensor memory over the first half of the
                // scores they came from (32 scores are read, then 16 columns behind the read position are
                // written): the A operand of the second product
                float psum = 0.f;
                {
                    uint32_t buf[2][32];  // the load of the next 32 scores runs under the arithmetic on these
                    tmem_ld32_issue(s_addr, buf[0]);
                    tmem_ld_wait(buf[0]);
#pragma unroll
                    for (int c4 = 0; c4 < 4; ++c4) {
                        uint32_t(&v)[32] = buf[c4 & 1];
                        if (c4 < 3) tmem_ld32_issue(s_addr + (uint32_t)(c4 + 1) * 32u, buf[(c4 + 1) & 1]);
                        uint32_t w[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float p0 = fast_exp2(fmaf(__uint_as_float(v[2 * j]), p.scale_log2, -m_new));
                            const float p1 = fast_exp2(fmaf(__uint_as_float(v[2 * j + 1]), p.scale_log2, -m_new));
                            psum += p0 + p1;
                            w[j] = pack_bf16(p0, p1);  // the even token in the low half
                        }
                        tmem_st16(s_addr + (uint32_t)c4 * 16u, w);
                        if (c4 < 3) tmem_ld_wait(buf[(c4 + 1) & 1]);
                    }
                }
                l_run += psum;
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPReady + wg));
                prev_tt = tt;
                have_prev = true;
            }
            // the warpgroup's share of the unit's output, out of tensor memory
            if (alive && have_prev) {
                alive = warp_wait(bar(kBarOFull + wg), (prev_tt >> 1) & 1u);
                if (alive) {
                    tc_fence_after();
#pragma unroll
                    for (int c2 = 0; c2 < 2; ++c2) {  // two loads of 32 columns in flight
                        uint32_t a[32], b[32];
                        tmem_ld32_issue(o_addr + (uint32_t)c2 * 64u, a);
                        tmem_ld32_issue(o_addr + (uint32_t)c2 * 64u + 32u, b);
                        tmem_ld_wait(a);
                        tmem_ld_wait(b);
#pragma unroll
                        for (int k = 0; k < 32; ++k) {
                            o_acc[c2 * 64 + k] = __uint_as_float(a[k]);
                            o_acc[c2 * 64 + 32 + k] = __uint_as_float(b[k]);
                        }
                    }
                    tc_fence_before();
                }
            } else {
#pragma unroll
                for (int d = 0; d < 128; ++d) o_acc[d] = 0.f;
            }
            tt0 += u.n_tiles;

            // ---- combine the two warpgroups' states of each row and write the partials ------------------
            // All products of the unit are complete once both warpgroups have taken their last O, so the P
            // buffers can serve as scratch: row r lives at r * 512 bytes, its 16-byte quad q at position
            // q ^ (r & 31), which keeps both the row-per-lane and the quad-per-lane accesses free of bank
            // conflicts.
            softmax_bar_both();
            uint8_t *comb = smem + kOffQ;   // the query buffer and the block behind it: 64 KB
            const uint32_t rsw = (uint32_t)(row & 31);
            if (wg == 1) {
#pragma unroll
                for (uint32_t q4 = 0; q4 < 32; ++q4)
                    *reinterpret_cast<float4 *>(comb + (size_t)row * 512 + ((q4 ^ rsw) << 4)) =
                        make_float4(o_acc[4 * q4], o_acc[4 * q4 + 1], o_acc[4 * q4 + 2], o_acc[4 * q4 + 3]);
                comb_ml[row] = m_run;
                comb_ml[128 + row] = l_run;
            }
            softmax_bar_both();
            if (wg == 0) {
                const float m1 = comb_ml[row], l1 = comb_ml[128 + row];
                const float M = fmaxf(m_run, m1);   // finite: the unit has at least one tile
                const float w0 = fast_exp2(m_run - M), w1 = fast_exp2(m1 - M);
                const float l = l_run * w0 + l1 * w1;
                const float inv = 1.f / l;
                const float c0 = w0 * inv, c1 = w1 * inv;
#pragma unroll
                for (uint32_t q0 = 0; q0 < 32; q0 += 8) {  // eight loads in flight, then eight stores
                    float4 v[8];
#pragma unroll
                    for (uint32_t j = 0; j < 8; ++j)
                        v[j] = *reinterpret_cast<const float4 *>(comb + (size_t)row * 512 + (((q0 + j) ^ rsw) << 4));
#pragma unroll
                    for (uint32_t j = 0; j < 8; ++j) {
                        const uint32_t q4 = q0 + j;
                        *reinterpret_cast<float4 *>(comb + (size_t)row * 512 + ((q4 ^ rsw) << 4)) =
                            make_float4(o_acc[4 * q4] * c0 + v[j].x * c1, o_acc[4 * q4 + 1] * c0 + v[j].y * c1,
                                        o_acc[4 * q4 + 2] * c0 + v[j].z * c1, o_acc[4 * q4 + 3] * c0 + v[j].w * c1);
                    }
                }
                uint32_t dst_row = 0xFFFFFFFFu;  // row of part_o ([slot][G] flattened) this query row goes to
                if (alive && valid) {
                    dst_row = slot * (uint32_t)G + (uint32_t)h;
                    p.part_lse2[(size_t)slot * kMaxGroup + h] = M + log2f(l);
                }
                flags[row] = dst_row;
            }
            softmax_bar_both();
            // both warpgroups copy the normalised rows out, a warp writing one 512-byte row per instruction
            {
                const uint32_t *dst_rows = reinterpret_cast<const uint32_t *>(smem + kOffFlags);
                const uint32_t q4 = (uint32_t)lane;                       // a warp = one row per pass
                const uint32_t r0 = (uint32_t)(wg * 4 + (warp & 3));      // 8 softmax warps, 16 rows each
#pragma unroll
                for (uint32_t rb = 0; rb < 16; rb += 8) {  // eight rows' loads in flight, then their stores
                    uint32_t dst[8];
                    float4 v[8];
#pragma unroll
                    for (uint32_t j = 0; j < 8; ++j) {
                        const uint32_t r = r0 + 8u * (rb + j);
                        dst[j] = dst_rows[r];
                        v[j] = *reinterpret_cast<const float4 *>(comb + (size_t)r * 512 + ((q4 ^ (r & 31u)) << 4));
                    }
#pragma unroll
                    for (uint32_t j = 0; j < 8; ++j)
                        if (dst[j] != 0xFFFFFFFFu)
                            reinterpret_cast<float4 *>(p.part_o + (size_t)dst[j] * kHeadDim)[q4] = v[j];
                }
            }
            if (p.tickets) __threadfence();  // publish the partials before the tickets
            softmax_bar_both();

            // ---- arrival tickets (when no merge kernel follows) -------------------------------------------
            if (wg == 0) {
                // one thread decides for all whether the block is still in business, so that all softmax
                // threads leave the unit loop together
                if (tid == 0) *unit_ok = (*abort_flag == 0u) ? 1u : 0u;
                if (p.tickets && tid < 128 / G) {
                    uint32_t mine = 0;
                    if (*abort_flag == 0u && (uint32_t)tid < u.n_readers) {
                        // thread tid speaks for reader tid (rows tid * G .. tid * G + G - 1): the block that
                        // delivers the last partial of the reader's row group merges it
                        const uint32_t e2 = u.reader_begin + (uint32_t)tid;
                        const uint32_t mg = p.reader_merge[(size_t)e2 * p.n_kv_heads + u.kv_head];
                        const cart_merge_item mi = p.merges[mg];
                        const uint32_t seen = atomicAdd(&p.tickets[mg], 1u);
                        if (seen + 1u == mi.slot_end - mi.slot_begin) mine = mg + 1u;
                    }
                    flags[tid] = mine;
                }
                softmax_bar();
                for (uint32_t r = 0; p.tickets && *unit_ok != 0u && r < u.n_readers; ++r) {
                    const uint32_t f = flags[r];
                    if (f == 0) continue;
                    __threadfence();
                    merge_row_group<1, 4>(p.merges[f - 1u], G, p.part_o, p.part_lse2, p.out, p.lse, tid, kSoftmaxThreads);
                    if (tid == 0) p.tickets[f - 1u] = 0;  // ready for the next launch
                }
            }
            softmax_bar_both();  // scratch, flags and unit_ok may be rewritten by the next unit from here on
            alive = *unit_ok != 0u;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    // Side by side: this kernel must not complete before the stream kernel does, because the kernel after
    // this one takes this kernel's completion for that of everything before it.
    if (p.ready_flag != nullptr && threadIdx.x == 0) pdl_wait();
}

}  // namespace

cudaError_t prepare_shared_kernel()
{
    return cudaFuncSetAttribute(cart_shared_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kShSmemBytes);
}

cudaError_t launch_shared(const CUtensorMap &tmap, const SharedParams &p, int grid, cudaStream_t s)
{
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg = pdl_config(grid, kShThreads, kShSmemBytes, s, &attr);
    return cudaLaunchKernelEx(&cfg, cart_shared_kernel, tmap, p);
}

}  // namespace cart
