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
//                   accumulator in tensor memory) one tile ahead of the softmax, and, per half x of the tile's
//                   tokens,  O_x += P_x V_x  (A operand P_x from tensor memory, V from shared memory, one
//                   accumulator per half for the whole unit); tcgen05.commit signals mbarriers
//   2 x 4 softmax   both warpgroups work on every tile: thread (w, r) owns query row r (tensor-memory
//   warps           lane r) and the 64 score columns (tokens) of half w.  It reads its 64 scores once and writes
//                   P = 2^(s - m) as bf16 pairs over its own half of the score buffer (tcgen05.st).  Each half
//                   of the tokens keeps a reference m, a sum and an accumulator of its own, so the two
//                   warpgroups never wait for each other inside a unit: a half's P V product is issued when its
//                   probabilities are there, and the warpgroups drift apart instead of meeting at the
//                   exponential unit every tile (one accumulator and a per-tile exchange of maxima through
//                   shared memory took 12 % longer per tile).  A reference only moves when the row's maximum
//                   has outgrown it by more than 2^8 (then the warpgroup rescales its accumulator in tensor
//                   memory); sum and accumulator always refer to the same reference, so the result is exact.
//                   At the end of a unit the owners trade references and sums, each mixes its 64 output dims
//                   from both accumulators by log-sum-exp weights, and the row leaves as a normalised fp32
//                   partial (or, for a chain's last unit, as the bf16 output).
//
// Tensor memory: two score buffers (S0 S1, with P inside) and the two accumulators, 128 fp32 columns each.
// The score product of tile t+1 is complete or in flight while the softmax of tile t runs, and the one of tile
// t+2 is queued right behind the P V products of tile t (the tensor pipe runs one thread's products in order),
// so neither side waits for the other's latency: the tile rate is set by the tensor pipe (16 instructions per
// tile) or by the exponentials (128 x 128 per tile), whichever is slower.
// The partials of a (request, KV head) row group are merged by log-sum-exp either by the block that
// delivers the last one -- this kernel's or the stream kernel's -- or, when the batch has more split row
// groups than blocks, by a merge kernel that runs afterwards.
//
// Every wait is bounded; on expiry the block raises a flag in the device status word, stops issuing
// work, waits (bounded) for what is in flight, frees its tensor memory and returns.
#include <cuda_bf16.h>

#include "cart_device.cuh"
#include "cart_internal.h"
#include "cart_tc.cuh"

namespace cart {
namespace {

constexpr int kShTile = kShareTileTokens;             // tokens per tile = N of the score product
constexpr uint32_t kShBlock = 128u * 128u;            // 128 rows x 128 bytes: one swizzled block (64 bf16 wide)
constexpr uint32_t kShTileBytes = 2u * kShBlock;      // 128 x 128 bf16
constexpr int kKStages = 3;                           // K tiles in flight (each ring has its own producer warp)
constexpr int kVStages = 2;
constexpr int kSBufs = 2;                             // score buffers in tensor memory
constexpr int kShThreads = 384;                       // utility warpgroup (K producer, MMA, V producer, 1 idle) + 2 softmax warpgroups
// Registers per thread after the warpgroups have re-divided the block's allocation (384 x 168): the
// utility warps need few, a softmax thread holds 64 scores and 32 packed probabilities.  4 x 32 x 40 + 8 x 32 x 232
// = 64512 registers, and per SM sub-partition 1 utility + 2 softmax warps = 16128 of its 16384.
constexpr int kRegsUtility = 40;
constexpr int kRegsSoftmax = 232;
constexpr int kSoftmaxThreads = 128;                  // one softmax warpgroup
constexpr uint32_t kTmemCols = 512;                   // S0 S1 (scores, then P), O_a O_b (accumulators): 128 fp32 columns each
constexpr uint32_t kTmemO = 2u * 128u;                // first column of the accumulators (one per softmax warpgroup)
constexpr float kRescaleStep = 8.f;                   // how far a row's maximum may outgrow its reference (base-2 units)

// shared-memory layout (offsets from a 1024-byte aligned base)
constexpr uint32_t kOffQ = 0;                          // two query buffers
constexpr uint32_t kOffK = kOffQ + 2u * kShTileBytes;
constexpr uint32_t kOffV = kOffK + kKStages * kShTileBytes;
constexpr uint32_t kOffBar = kOffV + kVStages * kShTileBytes;
constexpr uint32_t kOffMisc = kOffBar + 32 * 8;        // room for 32 barriers; then: tmem address, abort flag, unit flag
constexpr uint32_t kOffFlags = kOffMisc + 16;          // one word per reader: "merge this row group"
// what the two owners of a row tell each other at a unit's end: their references, then their sums (fp32 [half][row];
// one after the other through the same kilobyte: shared memory has no room for both at once)
constexpr uint32_t kOffXchg = kOffFlags + 128 * 4;
constexpr uint32_t kShSmemUsed = kOffXchg + 2 * 128 * 4;
constexpr uint32_t kShSmemBytes = kShSmemUsed + 1024;  // slack to align the base
static_assert(kShSmemBytes <= 232448, "shared memory budget of one sm_100 block exceeded");

enum Bar : int {
    kBarKFull = 0,   // [kKStages] TMA -> MMA
    kBarKEmpty = 3,  // [kKStages] MMA (commit of the score product) -> K producer
    kBarVFull = 6,   // [kVStages]
    kBarVEmpty = 8,  // [kVStages]
    kBarSFull = 10,  // [kSBufs] MMA (commit) -> softmax
    kBarSFree = 13,  // [kSBufs] MMA (commit of P V) -> softmax: the accumulator holds the products up to this tile
    kBarPReady = 16, // [kSBufs][2] softmax -> MMA: a warpgroup's half of the probabilities  (4 arrivals: one per warp)
    kBarQReady = 20, // [2] softmax -> MMA: a unit's query rows are in their buffer  (8 arrivals: one per softmax warp)
    kBarDrain = 24,  // MMA (commit) -> MMA, on the way out
};
static_assert(kBarKEmpty - kBarKFull >= kKStages && kBarVFull - kBarKEmpty >= kKStages &&
              kBarVEmpty - kBarVFull >= kVStages && kBarSFull - kBarVEmpty >= kVStages &&
              kBarSFree - kBarSFull >= kSBufs && kBarPReady - kBarSFree >= kSBufs && kBarQReady - kBarPReady >= 2 * kSBufs,
              "barrier indices overlap");

// Instruction descriptor, kind::f16: fp32 accumulator, bf16 A and B, M = 128, N = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescS = kIdesc;                  // A (Q) and B (K tile) both K-major
constexpr uint32_t kIdescPV = kIdesc | (1u << 16);    // B (V tile) is MN-major: dims contiguous

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
        if (v == 1u) return true;
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

// kChains: the kernel also understands chained, masked and directly written units (CART_UNIT_CONT / _HOLD / _MASKED /
// _DIRECT: the forward of training attention).  The decode and prefill plans never contain them, and their
// instantiation carries none of that code in its tile loop.
template <bool kChains>
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
    // The plan is in place before any of these kernels starts: read it at once.
    const uint32_t unit_begin = p.unit_cta_begin[blockIdx.x];
    const uint32_t unit_end = p.unit_cta_begin[blockIdx.x + 1];
    // ... as far as the first unit and, for the softmax threads, the batch index of the row's reader: these
    // dependent loads run under the set-up below (and, in a sequence of dependent launches, under the tail
    // of the kernel before)
    cart_shared_unit u_first{};
    uint32_t first_batch = 0;
    if (unit_begin < unit_end) {
        u_first = p.units[unit_begin];
        const uint32_t r0 = (threadIdx.x & 127u) / (uint32_t)p.group;
        // (in a plan of chains reader entry t is query row t: the table is not consulted, one dependent read less)
        if (threadIdx.x >= 128u && r0 < u_first.n_readers)
            first_batch = kChains ? u_first.reader_begin + r0 : p.readers[u_first.reader_begin + r0];
    }

    if (threadIdx.x == 0) {
        for (int i = 0; i < kKStages; ++i) {
            mbar_init(bar(kBarKFull + i), 1);
            mbar_init(bar(kBarKEmpty + i), 1);
        }
        for (int i = 0; i < kVStages; ++i) {
            mbar_init(bar(kBarVFull + i), 1);
            mbar_init(bar(kBarVEmpty + i), 1);
        }
        for (int i = 0; i < kSBufs; ++i) {
            mbar_init(bar(kBarSFull + i), 1);
            mbar_init(bar(kBarSFree + i), 1);
            mbar_init(bar(kBarPReady + 2 * i), 4);
            mbar_init(bar(kBarPReady + 2 * i + 1), 4);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(kBarQReady + i), 8);
        }
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

    // Shared tiles of stored Cartridges are only ever written by copies and may be fetched at once; shared
    // tiles in suffix storage (prefill: the part of the suffix that a group of rows has in common, units
    // marked CART_UNIT_SUFFIX) may have been written by the kernel before this one, so the producers wait
    // for the kernels before them ahead of the first such unit.  The queries, the partial slots and the
    // tickets may still be in use by those kernels too: the softmax warps wait before they read a query, and
    // nothing is written before the first scores exist.

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
                    // Paged suffix storage: a 128-token tile is two pages of 64 tokens, entries u.k_row + 2 t and
                    // + 2 t + 1 of the page list; inside a page the head's K block is at u.v_row, its V block 64
                    // rows later.  The entries of the next tile are read while this tile's stage is waited for.
                    const bool paged = (u.flags & CART_UNIT_PAGED) != 0u;
                    const uint32_t in_page = (uint32_t)p.layer * u.layer_stride + u.v_row + (is_v ? 64u : 0u);
                    uint32_t pg0 = 0, pg1 = 0;
                    if (paged) {
                        pg0 = __ldg(p.pages + u.k_row);
                        pg1 = __ldg(p.pages + u.k_row + 1u);
                    }
                    for (uint32_t t = 0; t < u.n_tiles; ++t, ++tt) {
                        const int st = (int)(tt % nst);
                        const uint32_t par = (tt / nst) & 1u;
                        const int32_t y = paged ? (int32_t)(pg0 + in_page) : (int32_t)(row0 + t * kShTile);
                        const int32_t y2 = paged ? (int32_t)(pg1 + in_page) : y + 64;
                        if (paged && t + 1u < u.n_tiles) {
                            pg0 = __ldg(p.pages + u.k_row + 2u * (t + 1u));
                            pg1 = __ldg(p.pages + u.k_row + 2u * (t + 1u) + 1u);
                        }
                        ok = mbar_wait(bar(empty0 + st), par ^ 1u, abort_flag, p.status, kStatusTimeoutProducer);
                        if (!ok) break;
                        const uint32_t dst = ring + (uint32_t)st * kShTileBytes;
                        mbar_expect_tx(bar(full0 + st), kShTileBytes);
                        // a block of the tile = 128 rows x 64 dims = two boxes of 64 rows
                        tma_load_2d(dst, &tmap, 0, y, bar(full0 + st));
                        tma_load_2d(dst + kShBlock / 2, &tmap, 0, y2, bar(full0 + st));
                        tma_load_2d(dst + kShBlock, &tmap, 64, y, bar(full0 + st));
                        tma_load_2d(dst + kShBlock + kShBlock / 2, &tmap, 64, y2, bar(full0 + st));
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
            // All lanes walk the loop and wait together; lane 0 issues.
            const uint32_t issue = lane == 0 ? 1u : 0u;
            bool ok = true;
            auto wait_all = [&](int b, uint32_t parity) -> bool {
                return __all_sync(0xffffffffu, mbar_wait(bar(b), parity, abort_flag, p.status, kStatusTimeoutMma));
            };
            // Two cursors walk the block's tiles in order: `qk` names the next score product to issue (it
            // runs two tiles ahead), `pv` the next P V product.  tt = tile index counted over the block.
            struct Cursor { uint32_t ui, t, n, unit_no, cont; };  // unit_no counts the units that bring their own query rows
            auto tiles_of = [&](uint32_t ui) { return ui < unit_end ? p.units[ui].n_tiles : 0u; };
            auto cont_of = [&](uint32_t ui) {
                return kChains && ui < unit_end ? (uint32_t)(p.units[ui].flags & CART_UNIT_CONT) : 0u;
            };
            Cursor qk{unit_begin, 0u, tiles_of(unit_begin), 0u, cont_of(unit_begin)}, pv = qk;
            auto advance = [&](Cursor &c) {
                if (++c.t == c.n) {
                    ++c.ui;
                    c.t = 0;
                    c.n = tiles_of(c.ui);
                    c.cont = cont_of(c.ui);
                    if (c.cont == 0u) ++c.unit_no;   // (a unit that continues a chain keeps its rows and their query buffer)
                }
            };
            uint32_t total = 0;
            for (uint32_t ui = unit_begin; ui < unit_end; ++ui) total += p.units[ui].n_tiles;
            // S(tt) = Q K^T into score buffer tt % 2.  The buffer last held the probabilities of tile tt - 2,
            // read by that tile's P V products, which this thread issued earlier: the tensor pipe executes one
            // thread's products in the order of issue, so no completion has to be waited for here.
            auto issue_s = [&](uint32_t tt) -> bool {
                const uint32_t sb = tt % (uint32_t)kSBufs;
                const uint32_t kst = tt % (uint32_t)kKStages, kpar = (tt / (uint32_t)kKStages) & 1u;
                const uint32_t qb = qk.unit_no & 1u;
                if (qk.t == 0u && qk.cont == 0u && !wait_all(kBarQReady + (int)qb, (qk.unit_no >> 1) & 1u)) return false;
                if (!wait_all(kBarKFull + (int)kst, kpar)) return false;
                tc_fence_after();
                const uint32_t q_lo = base + kOffQ + qb * kShTileBytes;
                const uint32_t k_lo = base + kOffK + kst * kShTileBytes;
                // the operands' descriptors differ from step to step only in the start address field
                // (units of 16 bytes): the next 16 dims are 32 bytes on, the second 64-dim block kShBlock on
                const uint64_t a0 = umma_desc(q_lo, 16, 1024), b0 = umma_desc(k_lo, 16, 1024);
                const uint32_t d_s = tmem + sb * 128u;
#pragma unroll
                for (uint32_t k = 0; k < 8; ++k) {  // 16 dims per instruction
                    const uint64_t off16 = (uint64_t)(((k >> 2) * kShBlock + (k & 3u) * 32u) >> 4);
                    umma_bf16(d_s, a0 + off16, b0 + off16, kIdescS, k, issue);
                }
                // the softmax warps hear that the scores are there, the K producer that its stage is free
                umma_commit(bar(kBarSFull + (int)sb), issue);
                umma_commit(bar(kBarKEmpty + (int)kst), issue);
                advance(qk);
                return true;
            };
            // O_x += P_x V_x for both halves x of the tile's tokens (O_x = P_x V_x for a unit's first tile): each softmax
            // warpgroup owns 64 tokens of every tile, with a reference, a sum and an accumulator of its own, so
            // its half of the product goes out as soon as its probabilities are there, whatever the other does
            auto issue_pv = [&](uint32_t tt) -> bool {
                const uint32_t sb = tt % (uint32_t)kSBufs, spar = (tt / (uint32_t)kSBufs) & 1u;
                const uint32_t vst = tt % (uint32_t)kVStages, vpar = (tt / (uint32_t)kVStages) & 1u;
                if (!wait_all(kBarVFull + (int)vst, vpar)) return false;
                if (!wait_all(kBarPReady + 2 * (int)sb, spar)) return false;
                tc_fence_after();
                const uint32_t v_lo = base + kOffV + vst * kShTileBytes;
                // P: the A operand comes from tensor memory, where the softmax warps left it inside the
                // score buffer: two bf16 per column, 16 tokens = 8 columns per step; tokens 0-63 in columns
                // 0-31 (written by the first warpgroup over its own scores), tokens 64-127 in columns 64-95.
                // V: tokens are rows of 128 bytes (8-token groups 1024 bytes apart, 16 tokens = 2048 bytes
                // per step); the two 64-dim blocks of the tile are kShBlock bytes apart.
                const uint64_t b0 = umma_desc(v_lo, kShBlock, 1024);
                const uint32_t p_tm = tmem + sb * 128u;
                const uint32_t d_o = tmem + kTmemO;
                const bool first = pv.t == 0u && pv.cont == 0u;  // (a unit that continues a chain adds to its accumulators)
#pragma unroll
                for (uint32_t k = 0; k < 4; ++k)  // 16 tokens per instruction
                    umma_bf16_ts(d_o, p_tm + 8u * k, b0 + (uint64_t)(k * 128u), kIdescPV, (first && k == 0u) ? 0u : 1u, issue);
                if (!wait_all(kBarPReady + 2 * (int)sb + 1, spar)) return false;
                tc_fence_after();
#pragma unroll
                for (uint32_t k = 4; k < 8; ++k)
                    umma_bf16_ts(d_o + 128u, p_tm + 64u + 8u * (k - 4u), b0 + (uint64_t)(k * 128u), kIdescPV,
                                 (first && k == 4u) ? 0u : 1u, issue);
                umma_commit(bar(kBarVEmpty + (int)vst), issue);
                umma_commit(bar(kBarSFree + (int)sb), issue);  // the accumulator holds the products up to this tile
                advance(pv);
                return true;
            };
            if (total > 0u) ok = issue_s(0u);
            if (ok && total > 1u) ok = issue_s(1u);
            for (uint32_t tt = 0; tt < total && ok; ++tt) {
                // The scores of tile tt + 1 are in the other buffer already (or on the pipe), so the softmax of that
                // tile starts the moment this tile's is over; the score product two tiles on reuses this tile's
                // buffer and is queued right behind this tile's P V products.
                ok = issue_pv(tt);
                if (ok && tt + 2u < total) ok = issue_s(tt + 2u);
            }
            // products still in flight must finish before the tensor memory is given back
            umma_commit(bar(kBarDrain), issue);
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(bar(kBarDrain), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
            __syncwarp();
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        // ================= softmax / epilogue warps ====================================================
        const int G = p.group;
        const int wg = (warp - 4) >> 2;       // which 64 score columns (tokens) of every tile this thread owns
        const int sw = warp & 3;              // the tensor-memory lanes this warp may read: 32 sw .. 32 sw + 31
        const int row = 32 * sw + lane;       // query row of the M-tile = tensor-memory lane
        const int tid = row;                  // index among the 128 threads of the warpgroup
        const uint32_t lane_addr = tmem + ((uint32_t)(32 * sw) << 16);
        const uint32_t col0 = 64u * (uint32_t)wg;
        float *xchg = reinterpret_cast<float *>(smem + kOffXchg);           // [half][row]
        uint32_t tt = 0;      // tiles of the block so far
        bool alive = true;    // false once the block has given up: work is skipped, barriers are still met
        // the warp's lanes must stay together (the tensor-memory loads are warp-wide): a wait fails for
        // all of them or for none
        auto warp_wait = [&](uint32_t b, uint32_t parity) -> bool {
            return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag, p.status, kStatusTimeoutConsumer));
        };
        const uint32_t o_addr = lane_addr + kTmemO + 128u * (uint32_t)wg;   // this warpgroup's accumulator: 128 columns

        // Query rows.  Thread (w, r) copies the 64-dim half w of row r (head r % G of the M-tile's reader r / G)
        // into the unit's query buffer, in the swizzled K-major operand layout: block w, row r, 16-byte chunk c
        // at position c ^ (r % 8).  Rows past the unit's readers are zeros.  Unit number n of the block uses
        // buffer n & 1.  The first unit's rows are fetched at once; the rows of unit n + 1 are requested after
        // the first tile of unit n and stored a tile later, when the loads have landed (all products of unit
        // n - 1, the buffer's last readers, were complete before the first scores of unit n arrived).
        const int i_reader = row / G, h = row - i_reader * G;
        const __nv_bfloat16 *q = reinterpret_cast<const __nv_bfloat16 *>(p.q);
        // The copies are cp.async (global to shared memory without passing through registers: 32 registers held over a
        // tile's arithmetic were what made this loop spill); load_q requests a unit's rows into buffer `buf`, store_q
        // waits for them and tells the MMA warp.
        auto q_src = [&](uint32_t kv_head, uint32_t batch) {   // this thread's 128 bytes of a unit's query rows
            return reinterpret_cast<const uint8_t *>(q + ((size_t)batch * p.n_q_heads + (size_t)kv_head * G + h) * kHeadDim) + 128 * wg;
        };
        auto load_q = [&](const uint8_t *src, bool on, uint32_t buf) {
            const uint32_t qrow = base + kOffQ + buf * kShTileBytes + (uint32_t)wg * kShBlock + (uint32_t)row * 128u;
            const uint32_t swz = (uint32_t)(row & 7);
#pragma unroll
            for (uint32_t c = 0; c < 8; ++c)   // (size 0: zeros are written instead)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(qrow + ((c ^ swz) << 4)),
                             "l"(on ? src + 16u * c : reinterpret_cast<const uint8_t *>(q)), "r"(on ? 16u : 0u)
                             : "memory");
        };
        auto store_q = [&](uint32_t buf) {
            asm volatile("cp.async.wait_all;" ::: "memory");
            fence_async_smem();   // these writes before the tensor core's reads of the operand
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarQReady + (int)buf));
        };
        cart_shared_unit u{}, u_next{};
        u = u_first;
        if (unit_begin + 1u < unit_end) u_next = p.units[unit_begin + 1u];
        {
            // the first unit's queries: everything up to the rows themselves is part of the plan
            const bool on = unit_begin < unit_end && (uint32_t)i_reader < u.n_readers;
            const uint32_t batch = first_batch;
            bool ok0 = true;
            if (lane == 0) ok0 = wait_for_prior_kernels(p, abort_flag);
            alive = __all_sync(0xffffffffu, ok0);  // (from here on the partial slots and the tickets are this kernel's too)
            if (unit_begin < unit_end) {
                load_q(q_src(u.kv_head, batch), on && alive, 0u);
                store_q(0u);
            }
        }

        float m_run = -INFINITY, l_run = 0.f;
        bool fresh = true;   // no tile of the chain has been seen yet
        uint32_t unit_no = 0;   // counts the units that bring their own query rows (not those that continue a chain)
        for (uint32_t ui = unit_begin; ui < unit_end; ++ui) {
            if (ui != unit_begin) {
                u = u_next;
                u_next = cart_shared_unit{};
                if (ui + 1u < unit_end) u_next = p.units[ui + 1u];
            }
            const bool brings_rows = !kChains || !(u.flags & CART_UNIT_CONT);
            if (brings_rows && ui != unit_begin) ++unit_no;
            // the next unit with rows of its own (the units of a chain in between reuse this one's)
            bool has_next = false;
            cart_shared_unit uq{};
            if (brings_rows) {
                // (in a plan with chains the unit says how many units on the next chain begins)
                const uint32_t uj = kChains ? ui + (u.reserved ? u.reserved : (unit_end - ui)) : ui + 1u;
                has_next = uj < unit_end;
                if (has_next) uq = uj == ui + 1u ? u_next : p.units[uj];
            }
            const bool valid = (uint32_t)i_reader < u.n_readers;
            // (in a plan with chains uq is a load in flight here, and the reader's batch index one more: they are looked
            //  at a tile later, so that nothing waits for them at the start of a chain)
            bool valid_next = false;
            uint32_t batch_next = 0;
            if (!kChains && has_next) {
                valid_next = (uint32_t)i_reader < uq.n_readers;
                if (valid_next) batch_next = p.readers[uq.reader_begin + (uint32_t)i_reader];
            }
            // the tiles after which the next unit's rows are requested and stored: in a plan with chains the request
            // hangs on the read of the next chain's first unit issued above, which gets a tile's time
            const uint32_t t_load = kChains ? (u.n_tiles > 1u ? 1u : 0u) : 0u;
            const uint32_t t_store = kChains ? (u.n_tiles > 3u ? 3u : u.n_tiles - 1u) : (u.n_tiles > 1u ? 1u : 0u);
            const bool direct = kChains && (u.flags & CART_UNIT_DIRECT) != 0u, hold = kChains && (u.flags & CART_UNIT_HOLD) != 0u;
            const bool masked = kChains && (u.flags & CART_UNIT_MASKED) != 0u;
            uint32_t slot = 0;   // where this row's partial goes, or (direct) its query row: needed at the unit's end
            if (valid && !hold)
                slot = direct ? u.reader_begin + (uint32_t)i_reader
                              : p.reader_slot[(size_t)(u.reader_begin + (uint32_t)i_reader) * p.n_kv_heads + u.kv_head] + u.chunk;
            // m_run: the reference that l_run and the accumulator in tensor memory refer to, the same for both
            // owners of the row.  It only moves when the row's maximum has outgrown it by more than
            // kRescaleStep (base 2); until then probabilities may exceed 1 (by at most that factor), which
            // bf16 and the fp32 sums hold easily.  l_run: the sum over this thread's columns.  A unit that
            // continues the one before it (a chain over the same rows) inherits all three.
            if (!kChains || !(u.flags & CART_UNIT_CONT)) {
                m_run = -INFINITY;
                l_run = 0.f;
                fresh = true;
            }
            // masked run: the last key of the run this row sees (-1: none)
            int32_t limit = 0x7FFFFFFF;
            if (masked) {
                const int32_t lb = u.lim_base + i_reader;
                limit = (uint32_t)i_reader < u.tr_hi ? (lb < u.lim_cap ? lb : u.lim_cap) : -1;
            }

            for (uint32_t t = 0; t < u.n_tiles; ++t, ++tt) {
                const uint32_t sb = tt % (uint32_t)kSBufs, spar = (tt / (uint32_t)kSBufs) & 1u;
                const uint32_t s_addr = lane_addr + sb * 128u + col0;
                uint32_t s[64];
                float mx = -INFINITY;
                bool all_on = true;
                if (alive) alive = warp_wait(bar(kBarSFull + (int)sb), spar);
                if (alive) {
                    tc_fence_after();
                    tmem_ld32_issue(s_addr, reinterpret_cast<uint32_t(&)[32]>(s[0]));
                    tmem_ld32_issue(s_addr + 32u, reinterpret_cast<uint32_t(&)[32]>(s[32]));
                    tmem_ld_wait(reinterpret_cast<uint32_t(&)[32]>(s[0]));
                    tmem_ld_wait(reinterpret_cast<uint32_t(&)[32]>(s[32]));
                    // keys of this thread's columns: kidx0 .. kidx0 + 63 of the run; all of them seen unless masked
                    const int32_t kidx0 = (int32_t)(t * (uint32_t)kShTile + col0);
                    all_on = !masked || kidx0 + 63 <= limit;
                    if (all_on) {
#pragma unroll
                        for (int k = 0; k < 64; k += 2) mx = fmaxf(mx, fmaxf(__uint_as_float(s[k]), __uint_as_float(s[k + 1])));
                    } else {
                        // (what lies past a row's limit may be anything, NaN included: it is left out of the maximum
                        //  and replaced by -inf, which the exponential below turns into a probability of zero)
#pragma unroll
                        for (int k = 0; k < 64; ++k) {
                            if (kidx0 + k <= limit) mx = fmaxf(mx, __uint_as_float(s[k]));
                            else s[k] = 0xFF800000u;
                        }
                    }
                    mx *= p.scale_log2;
                }
                // the row's maximum over this warpgroup's 64 tokens: the two halves of a tile keep references, sums and
                // accumulators of their own and only meet at the unit's end, so neither waits for the other per tile
                if (!alive) continue;
                const float m_tile = mx;
                if (fresh) {
                    m_run = m_tile;
                    fresh = false;
                } else if (__any_sync(0xffffffffu, m_tile > m_run + kRescaleStep)) {
                    // a row of this warp has outgrown its reference: every row of the warp moves up to its
                    // maximum and rescales its lane of the warpgroup's accumulator (tensor-memory accesses are
                    // warp-wide, so the warp decides together; the other rows' factors are 1 or close to it)
                    const float m_new = fmaxf(m_run, m_tile);
                    // (a row of a masked run may not have seen a key yet: its reference stays at -inf, factor 1)
                    const float f = m_new == -INFINITY ? 1.f : fast_exp2(m_run - m_new);
                    m_run = m_new;
                    l_run *= f;
                    // The product of the tile before must have landed first.  Its completion is read from the
                    // barrier of the score buffer it used: a barrier that completes once per tile could be two
                    // phases behind this warp (the tensor pipe also holds score products queued ahead), which a
                    // parity cannot tell from none; a score buffer's barrier is at most one behind.
                    alive = warp_wait(bar(kBarSFree + (int)((tt - 1u) % (uint32_t)kSBufs)), ((tt - 1u) / (uint32_t)kSBufs) & 1u);
                    if (!alive) continue;
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
                // probabilities of this thread's 64 tokens, as bf16 pairs (the even token in the low half), written
                // over the first 32 columns of the scores they came from: the A operand of the second product
                float psum0 = 0.f, psum1 = 0.f;
                // (a row of a masked run that has not seen a key yet has no reference: all its scores are -inf here)
                const float m_use = kChains && m_run == -INFINITY ? 0.f : m_run;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t w[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(s[32 * c + 2 * j]), p.scale_log2, -m_use));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(s[32 * c + 2 * j + 1]), p.scale_log2, -m_use));
                        psum0 += p0;
                        psum1 += p1;
                        w[j] = pack_bf16(p0, p1);
                    }
                    tmem_st16(s_addr + (uint32_t)c * 16u, w);
                }
                l_run += psum0 + psum1;
                if (masked && t + 1u == u.n_tiles && (uint32_t)(u.lim_cap + 1) < u.n_tiles * (uint32_t)kShTile) {
                    // The run ends inside this tile.  The rows behind its last key hold whatever follows in memory;
                    // their probabilities are zero, but 0 * NaN would poison the product, so those rows of the V tile
                    // are cleared before the MMA warp hears of the tile.
                    const uint32_t vst = tt % (uint32_t)kVStages, vpar = (tt / (uint32_t)kVStages) & 1u;
                    alive = warp_wait(bar(kBarVFull + (int)vst), vpar);
                    if (!alive) continue;
                    const uint32_t first_bad = (uint32_t)(u.lim_cap + 1) - t * (uint32_t)kShTile;   // 1 .. 127
                    const uint32_t v_lo = base + kOffV + vst * kShTileBytes;
                    // (this warpgroup's product reads the rows of its own 64 tokens only, and clears those)
                    const uint32_t r_lo = first_bad > 64u * (uint32_t)wg ? first_bad : 64u * (uint32_t)wg, r_hi = 64u * (uint32_t)wg + 64u;
                    for (uint32_t x = (uint32_t)tid; r_lo < r_hi && x < (r_hi - r_lo) * 16u; x += (uint32_t)kSoftmaxThreads) {
                        const uint32_t r = r_lo + x / 16u, c = x % 16u;
                        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(v_lo + (c >> 3) * kShBlock + r * 128u + ((c & 7u) << 4)),
                                     "r"(0u)
                                     : "memory");
                    }
                    fence_async_smem();
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPReady + 2 * (int)sb + wg));
                if (has_next) {
                    if (kChains && t == 0u) {
                        valid_next = (uint32_t)i_reader < uq.n_readers;
                        if (valid_next) batch_next = uq.reader_begin + (uint32_t)i_reader;
                    }
                    if (t == t_load) load_q(q_src(uq.kv_head, batch_next), valid_next, (unit_no + 1u) & 1u);
                    if (t == t_store) store_q((unit_no + 1u) & 1u);
                }
            }

            // ---- the unit's rows leave as normalised partials -------------------------------------------
            // (unless the next unit continues the same rows: then the state simply stays)
            if (hold) continue;
            // The two halves of the row's keys meet here: the owners trade references and sums, and each writes 64 of
            // the row's 128 output dims, mixed from both accumulators by log-sum-exp weights (in a fixed order, so
            // the result does not depend on timing).  o[k]: the unnormalised output, l: the sum it is divided by,
            // m_all: the reference both refer to.
            uint32_t o[64];
            if (alive) alive = warp_wait(bar(kBarSFree + (int)((tt - 1u) % (uint32_t)kSBufs)), ((tt - 1u) / (uint32_t)kSBufs) & 1u);
            softmax_bar_both();  // the exchange area is free: the unit before has been read
            xchg[wg * 128 + row] = m_run;
            softmax_bar_both();
            float2 theirs;
            theirs.x = xchg[(wg ^ 1) * 128 + row];
            softmax_bar_both();
            xchg[wg * 128 + row] = l_run;
            softmax_bar_both();
            theirs.y = xchg[(wg ^ 1) * 128 + row];
            const float m_all = fmaxf(m_run, theirs.x);
            // (a half that saw no key has reference -inf and weight 0; a row that saw none at all has l = 0)
            const float w_mine = m_all == -INFINITY ? 0.f : fast_exp2(m_run - m_all);
            const float w_theirs = m_all == -INFINITY ? 0.f : fast_exp2(theirs.x - m_all);
            const float w_a = wg == 0 ? w_mine : w_theirs, w_b = wg == 0 ? w_theirs : w_mine;
            const float l = w_a * (wg == 0 ? l_run : theirs.y) + w_b * (wg == 0 ? theirs.y : l_run);
            if (alive) {
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t a[32], b[32];
                    tmem_ld32_issue(lane_addr + kTmemO + col0 + 32u * (uint32_t)c, a);
                    tmem_ld32_issue(lane_addr + kTmemO + 128u + col0 + 32u * (uint32_t)c, b);
                    tmem_ld_wait(a);
                    tmem_ld_wait(b);
#pragma unroll
                    for (int k = 0; k < 32; ++k)
                        o[32 * c + k] = __float_as_uint(w_a * __uint_as_float(a[k]) + w_b * __uint_as_float(b[k]));
                }
                tc_fence_before();
            }
            if (alive && valid && direct) {
                // the chain covered the row's whole cache: the final output, rounded to bf16, and the lse
                const float inv = 1.f / l;
                const size_t orow = (size_t)slot * p.n_q_heads + (size_t)u.kv_head * G + h;
                __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.out) + orow * kHeadDim + col0;
#pragma unroll
                for (int c16 = 0; c16 < 4; ++c16) {   // 32 bytes per store (see the partials below)
                    uint32_t w[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        w[j] = pack_bf16(__uint_as_float(o[16 * c16 + 2 * j]) * inv, __uint_as_float(o[16 * c16 + 2 * j + 1]) * inv);
                    asm volatile("st.global.v8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst + 16 * c16), "r"(w[0]), "r"(w[1]),
                                 "r"(w[2]), "r"(w[3]), "r"(w[4]), "r"(w[5]), "r"(w[6]), "r"(w[7])
                                 : "memory");
                }
                if (wg == 0 && p.lse) p.lse[orow] = (m_all + log2f(l)) * 0.6931471805599453f;
            } else if (alive && valid) {
                // (a row that saw no key of the unit -- all of them beyond its causal limit -- leaves an empty partial:
                //  zeros with lse = -inf, which the merge gives no weight)
                const float inv = l > 0.f ? 1.f / l : 0.f;
                // 32 bytes per store: a thread writes a row by itself, so every store of a warp touches 32 rows, and
                // 16-byte stores fill only half of each 32-byte sector they touch
                float *dst = p.part_o + ((size_t)slot * G + h) * kHeadDim + col0;
#pragma unroll
                for (int q8 = 0; q8 < 8; ++q8)
                    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(dst + 8 * q8),
                                 "f"(__uint_as_float(o[8 * q8]) * inv), "f"(__uint_as_float(o[8 * q8 + 1]) * inv),
                                 "f"(__uint_as_float(o[8 * q8 + 2]) * inv), "f"(__uint_as_float(o[8 * q8 + 3]) * inv),
                                 "f"(__uint_as_float(o[8 * q8 + 4]) * inv), "f"(__uint_as_float(o[8 * q8 + 5]) * inv),
                                 "f"(__uint_as_float(o[8 * q8 + 6]) * inv), "f"(__uint_as_float(o[8 * q8 + 7]) * inv)
                                 : "memory");
                if (wg == 0) p.part_lse2[(size_t)slot * kMaxGroup + h] = l > 0.f ? m_all + log2f(l) : -INFINITY;
            }
            // (the exchange area is written next behind the first barrier of the next unit's end: nothing to wait for here)
            if (p.tickets == nullptr || direct) continue;

            // ---- arrival tickets (when no merge kernel follows) -------------------------------------------
            __threadfence();  // publish the partials before the tickets
            softmax_bar_both();
            if (wg == 0) {
                // one thread decides for all whether the block is still in business
                if (tid == 0) *unit_ok = (*abort_flag == 0u) ? 1u : 0u;
                if (tid < 128 / G) {
                    uint32_t won = 0;
                    if (*abort_flag == 0u && (uint32_t)tid < u.n_readers) {
                        // thread tid speaks for reader tid (rows tid * G .. tid * G + G - 1): the block that
                        // delivers the last partial of the reader's row group merges it
                        const uint32_t e2 = u.reader_begin + (uint32_t)tid;
                        const uint32_t mg = p.reader_merge[(size_t)e2 * p.n_kv_heads + u.kv_head];
                        const cart_merge_item mi = p.merges[mg];
                        const uint32_t seen = atomicAdd(&p.tickets[mg], 1u);
                        if (seen + 1u == mi.slot_end - mi.slot_begin) won = mg + 1u;
                    }
                    flags[tid] = won;
                }
                softmax_bar();
                for (uint32_t r = 0; *unit_ok != 0u && r < u.n_readers; ++r) {
                    const uint32_t f = flags[r];
                    if (f == 0) continue;
                    __threadfence();
                    merge_row_group<1, 4>(p.merges[f - 1u], G, p.part_o, p.part_lse2, p.out, p.lse, tid, kSoftmaxThreads);
                    if (tid == 0) p.tickets[f - 1u] = 0;  // ready for the next launch
                }
            }
            softmax_bar_both();  // flags, unit_ok and the exchange area may be rewritten by the next unit from here on
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
    if (p.ready_flag != nullptr && threadIdx.x == 0) {
        pdl_wait();
        // every block has read the flag by the time it gets here; the last one clears it (and the count) for the next
        // pair, whose stream kernel sets it only after this kernel is complete
        if (atomicAdd(p.ready_flag + 1, 1u) == gridDim.x - 1u) {
            p.ready_flag[1] = 0u;
            p.ready_flag[0] = 0u;
        }
    }
}

}  // namespace

cudaError_t prepare_shared_kernel()
{
    cudaError_t e = cudaFuncSetAttribute(cart_shared_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kShSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(cart_shared_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kShSmemBytes);
}

cudaError_t launch_shared(const CUtensorMap &tmap, const SharedParams &p, int grid, cudaStream_t s, bool chains)
{
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg = pdl_config(grid, kShThreads, kShSmemBytes, s, &attr);
    return chains ? cudaLaunchKernelEx(&cfg, cart_shared_kernel<true>, tmap, p)
                  : cudaLaunchKernelEx(&cfg, cart_shared_kernel<false>, tmap, p);
}

}  // namespace cart
