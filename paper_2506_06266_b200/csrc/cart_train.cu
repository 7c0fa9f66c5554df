// Training-time attention over a shared trainable Cartridge, backward pass, for sm_100a.
//
// Self-Study (Sec. 4 of the paper) trains a Cartridge Z -- p key and p value vectors per layer and KV head, the
// parameterisation of Sec. 3.2 -- by back-propagating through causal attention of many short conversations over
// [Z ; own tokens]; Sec. 6 names shared-prefix attention kernels as what would make that training cheaper.  The
// forward is Eq. 1 of Sec. 2.3 with Z as the prefix and runs on the decode kernels (the conversations' tokens are
// rows that share Z).  This file holds the backward.  With P the probabilities of the forward (recomputed from the
// scores and the saved log-sum-exp), dO the gradient of the output and D_i = <dO_i, O_i>:
//
//     dV_j = sum_i P_ij dO_i        dP_ij = <dO_i, V_j>        dS_ij = scale * P_ij (dP_ij - D_i)
//     dK_j = sum_i dS_ij q_i        dq_i  = sum_j dS_ij K_j
//
// where i runs over the query rows (token, head) that see key j: all rows of all conversations for a key of Z --
// which is how the gradient of Z comes to be summed over every reader -- and the rows of the same conversation at
// or after the key's position for a conversation's own key.
//
// One thread block owns a tile of 128 keys of one KV head and walks over the row tiles that see it (128 rows =
// 128 / G tokens x the G heads of the group).  Everything is computed key-major, so that the gradients of the
// tile's keys and values accumulate in tensor memory over all row tiles and are written once:
//
//     S^T  = K Q^T        (tcgen05.mma, 128 keys x 128 rows, K and Q tiles K-major in shared memory)
//     dP^T = V dO^T
//     thread (w, j) owns key j (tensor-memory lane j) and the rows 64 w .. 64 w + 63 of the row tile: it turns
//     S^T into P^T = 2^(S^T * scale * log2 e - lse_i * log2 e) and dP^T into dS^T, masks what the key does not
//     see, and writes both back over their own columns as bf16 pairs, dS^T also to shared memory;
//     dV  += P^T dO       (A operand from tensor memory, dO tile as the MN-major B operand)
//     dK  += dS^T Q
//     dQ_part = dS K      (dS from shared memory as an MN-major A operand, into the columns S^T held)
//     the same threads, now as row owners, put dQ_part into shared memory (the row tile's Q and dO stage, spent by
//     then) and a bulk tensor reduction adds it into dq.
//
// Tensor memory: S^T / P^T / dQ_part, dP^T / dS^T, the dV accumulator, the dK accumulator: 4 x 128 columns.
// The tensor pipe executes one thread's instructions in the order of issue, which orders dV += P^T dO before the
// product that overwrites P^T.  All gradients are accumulated into zero-initialised fp32 tensors by additions in the
// memory system (every key tile adds into dq; several blocks share a Cartridge tile when its rows are split), so the
// last bits depend on the order of arrival.  Every wait is bounded, as in the other kernels.
#include <cuda_bf16.h>

#include "cart_device.cuh"
#include "cart_internal.h"
#include "cart_tc.cuh"

namespace cart {
namespace {

constexpr uint32_t kTBlock = 128u * 128u;         // 128 rows x 128 bytes: one swizzled block (64 bf16 wide)
constexpr uint32_t kTTile = 2u * kTBlock;         // 128 x 128 bf16
constexpr int kTrThreads = 384;                   // utility warpgroup (producer, MMA, 2 idle) + 2 compute warpgroups
constexpr int kTrRegsUtility = 96;
constexpr int kTrRegsCompute = 176;
constexpr uint32_t kTrTmemCols = 512;
constexpr uint32_t kTmS = 0, kTmDP = 128, kTmDV = 256, kTmDK = 384;

constexpr uint32_t kTrOffK = 0;
constexpr uint32_t kTrOffV = kTrOffK + kTTile;
constexpr uint32_t kTrOffQ = kTrOffV + kTTile;          // two stages
constexpr uint32_t kTrOffDO = kTrOffQ + 2u * kTTile;    // two stages
constexpr uint32_t kTrOffDS = kTrOffDO + 2u * kTTile;
constexpr uint32_t kTrOffLD = kTrOffDS + kTTile;        // [stage][128] (lse * log2 e, D) per row
constexpr uint32_t kTrOffTok = kTrOffLD + 2u * 128u * 8u;  // [128] token offset of row i inside its row tile (i / G)
constexpr uint32_t kTrOffBar = kTrOffTok + 128u;
constexpr uint32_t kTrOffMisc = kTrOffBar + 16u * 8u;   // tensor-memory address, abort flag
constexpr uint32_t kTrOffItem = kTrOffMisc + 16u;       // the block's work item (read by every warp, all through the loop)
constexpr uint32_t kTrSmemUsed = kTrOffItem + 64u;
static_assert(sizeof(TrainItem) == 64, "the work item's copy in shared memory is 64 bytes");
constexpr uint32_t kTrSmemBytes = 232448u;              // all of it: what is left over is the room to align the base
static_assert(kTrSmemUsed <= kTrSmemBytes, "shared memory budget of one sm_100 block exceeded");

enum TrBar : int {
    kTbKV = 0,       // TMA -> all: the key tile's K and V are in shared memory
    kTbQFull = 1,    // [2] TMA + producer warp (2 arrivals) -> MMA, compute: a row tile's Q, dO, lse and D
    kTbQEmpty = 3,   // [2] compute (2 arrivals: one per warpgroup, once its dq reduction has left the stage) -> producer
    kTbSFull = 5,    // MMA (commit) -> compute: S^T and dP^T
    kTbPReady = 6,   // compute (8 arrivals) -> MMA: P^T, dS^T in tensor memory, dS in shared memory
    kTbDQFull = 7,   // MMA (commit) -> compute: dQ_part (and the accumulators up to this row tile)
    kTbTmFree = 8,   // compute (8 arrivals) -> MMA: dQ_part has been read
    kTbDrain = 9,
};

constexpr uint32_t kIdKK = umma_idesc_bf16(128, 128, false, false);   // both operands K-major
constexpr uint32_t kIdTsMn = umma_idesc_bf16(128, 128, false, true);  // A from tensor memory, B MN-major
constexpr uint32_t kIdMnMn = umma_idesc_bf16(128, 128, true, true);   // both MN-major

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tmap, int32_t x, int32_t y, int32_t z,
                                            uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z), "r"(bar)
        : "memory");
}

// Adds a box of fp32 from shared memory into global memory (dq as [T][Hq][128], boxes of 128 / G tokens x G heads x
// 32 dims): the additions happen in the memory system, one instruction per box instead of one atomic per 16 bytes.
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap *tmap, uint32_t src, int32_t x, int32_t y, int32_t z)
{
    asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(z), "r"(src)
                 : "memory");
}

// D_i = <dout_i, out_i> per query row: one warp per row of 128 bf16 pairs.
__global__ void __launch_bounds__(256) cart_train_delta_kernel(const TrainDeltaParams p)
{
    const int row = (int)(blockIdx.x * 8u + (threadIdx.x >> 5));
    const int lane = (int)(threadIdx.x & 31u);
    if (row >= p.n_rows) return;
    const uint2 a = reinterpret_cast<const uint2 *>(p.out)[(size_t)row * 32 + lane];
    const uint2 b = reinterpret_cast<const uint2 *>(p.dout)[(size_t)row * 32 + lane];
    const float2 a0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&a.x));
    const float2 a1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&a.y));
    const float2 b0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&b.x));
    const float2 b1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&b.y));
    float s = a0.x * b0.x + a0.y * b0.y + a1.x * b1.x + a1.y * b1.y;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) p.delta[row] = s;
}

__global__ void __launch_bounds__(kTrThreads, 1)
cart_train_bwd_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap_q,
                      const __grid_constant__ CUtensorMap tmap_do, const __grid_constant__ CUtensorMap tmap_dq,
                      const TrainBwdParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    if (base - raw + kTrSmemUsed > kTrSmemBytes) {  // (the base is expected to be aligned already)
        if (threadIdx.x == 0) atomicOr(p.status, kStatusTimeoutConsumer);
        return;
    }
    uint8_t *smem = smem_raw + (base - raw);
    auto bar = [&](int i) { return base + kTrOffBar + (uint32_t)i * 8u; };
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + kTrOffMisc);
    volatile uint32_t *abort_flag = tmem_slot + 1;
    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    // The item lives in shared memory: the warps with few registers would otherwise keep its fields in local memory
    // and wait for them, row tile after row tile.
    if (threadIdx.x < 16)
        reinterpret_cast<uint32_t *>(smem + kTrOffItem)[threadIdx.x] =
            reinterpret_cast<const uint32_t *>(p.items + blockIdx.x)[threadIdx.x];
    __syncthreads();
    const TrainItem &it = *reinterpret_cast<const TrainItem *>(smem + kTrOffItem);
    const int G = p.group;
    const uint32_t tpt = 128u / (uint32_t)G;          // tokens per row tile
    const uint32_t rows_valid = tpt * (uint32_t)G;    // rows of a row tile that exist (128 unless G does not divide it)
    const uint32_t n_it = it.rt_end - it.rt_begin;

    if (threadIdx.x == 0) {
        mbar_init(bar(kTbKV), 1);
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(kTbQFull + i), 2);
            mbar_init(bar(kTbQEmpty + i), 2);
        }
        mbar_init(bar(kTbSFull), 1);
        mbar_init(bar(kTbPReady), 8);
        mbar_init(bar(kTbDQFull), 1);
        mbar_init(bar(kTbTmFree), 8);
        mbar_init(bar(kTbDrain), 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + kTrOffMisc),
                     "r"(kTrTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (threadIdx.x >= 128 && threadIdx.x < 256) {
        // row i of a row tile is head i % G of the tile's token i / G
        reinterpret_cast<uint8_t *>(smem + kTrOffTok)[threadIdx.x - 128] = (uint8_t)((threadIdx.x - 128u) / (uint32_t)G);
    }
    if (rows_valid < 128u) {
        // rows that no box ever fills (G does not divide 128) must read as zeros: both stages of Q and dO
        const uint32_t per_tile = (128u - rows_valid) * 16u;  // 16-byte chunks: 2 blocks x 8 per row
        for (uint32_t x = threadIdx.x; x < 4u * per_tile; x += kTrThreads) {
            const uint32_t tile = x / per_tile, y = x % per_tile;
            const uint32_t r = rows_valid + y / 16u, c = y % 16u;
            const uint32_t a = base + kTrOffQ + tile * kTTile + (c >> 3) * kTBlock + r * 128u + ((c & 7u) << 4);
            asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp < 4) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kTrRegsUtility));
        if (warp == 0) {
            // ================= producer ====================================================================
            bool ok = true;
            if (lane == 0) {
                asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap)) : "memory");
                asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_q)) : "memory");
                asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_do)) : "memory");
                asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_dq)) : "memory");
                // the key tile: 128 keys x 128 dims of K and of V, each as four boxes of 64 rows x 64 dims
                mbar_expect_tx(bar(kTbKV), 2u * kTTile);
                const int32_t ky = (int32_t)(it.k_row + (uint32_t)p.layer * it.layer_stride);
                const int32_t vy = (int32_t)(it.v_row + (uint32_t)p.layer * it.layer_stride);
#pragma unroll
                for (uint32_t b = 0; b < 4; ++b) {
                    const uint32_t off = (b >> 1) * kTBlock + (b & 1u) * (kTBlock / 2u);
                    tma_load_2d(base + kTrOffK + off, &tmap, (int32_t)((b >> 1) * 64u), ky + (int32_t)((b & 1u) * 64u), bar(kTbKV));
                    tma_load_2d(base + kTrOffV + off, &tmap, (int32_t)((b >> 1) * 64u), vy + (int32_t)((b & 1u) * 64u), bar(kTbKV));
                }
            }
            for (uint32_t i = 0; i < n_it && ok; ++i) {
                const uint32_t st = i & 1u, par = (i >> 1) & 1u;
                const uint32_t rt = it.rt_begin + (it.rt_first - it.rt_begin + i) % n_it;
                bool ok0 = true;
                if (lane == 0) ok0 = mbar_wait(bar(kTbQEmpty + (int)st), par ^ 1u, abort_flag, p.status, kStatusTimeoutProducer);
                ok = __shfl_sync(0xffffffffu, (int)ok0, 0) != 0;
                if (!ok) break;
                if (lane == 0) {
                    mbar_expect_tx(bar(kTbQFull + (int)st), 4u * rows_valid * 128u);
                    const int32_t y = (int32_t)(it.kv_head * (uint32_t)G), z = (int32_t)(rt * tpt);
                    const uint32_t qd = base + kTrOffQ + st * kTTile, dd = base + kTrOffDO + st * kTTile;
                    tma_load_3d(qd, &tmap_q, 0, y, z, bar(kTbQFull + (int)st));
                    tma_load_3d(qd + kTBlock, &tmap_q, 64, y, z, bar(kTbQFull + (int)st));
                    tma_load_3d(dd, &tmap_do, 0, y, z, bar(kTbQFull + (int)st));
                    tma_load_3d(dd + kTBlock, &tmap_do, 64, y, z, bar(kTbQFull + (int)st));
                }
                // lse (in base-2 units) and D of the tile's rows
                float2 *ld = reinterpret_cast<float2 *>(smem + kTrOffLD) + st * 128u;
#pragma unroll
                for (uint32_t k = 0; k < 4; ++k) {
                    const uint32_t r = (uint32_t)lane + 32u * k;
                    const uint32_t tk = rt * tpt + r / (uint32_t)G, h = r % (uint32_t)G;
                    float2 v = make_float2(0.f, 0.f);
                    if (r < rows_valid && tk < (uint32_t)p.n_tokens) {
                        const size_t idx = (size_t)tk * p.n_q_heads + it.kv_head * (uint32_t)G + h;
                        v = make_float2(__ldg(p.lse + idx) * 1.4426950408889634f, __ldg(p.delta + idx));
                    }
                    ld[r] = v;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kTbQFull + (int)st));
            }
        } else if (warp == 1) {
            // ================= MMA issuer: all lanes walk the loop, lane 0 issues ==========================
            const uint32_t issue = lane == 0 ? 1u : 0u;
            auto wait_all = [&](int b, uint32_t parity) -> bool {
                return __all_sync(0xffffffffu, mbar_wait(bar(b), parity, abort_flag, p.status, kStatusTimeoutMma));
            };
            bool ok = wait_all(kTbKV, 0u);
            const uint32_t k_lo = base + kTrOffK, v_lo = base + kTrOffV, ds_lo = base + kTrOffDS;
            for (uint32_t i = 0; i < n_it && ok; ++i) {
                const uint32_t st = i & 1u, par = (i >> 1) & 1u;
                const uint32_t q_lo = base + kTrOffQ + st * kTTile, do_lo = base + kTrOffDO + st * kTTile;
                ok = wait_all(kTbQFull + (int)st, par);
                if (ok && i > 0u) ok = wait_all(kTbTmFree, (i - 1u) & 1u);
                if (!ok) break;
                tc_fence_after();
                {
                    // S^T = K Q^T and dP^T = V dO^T: K-major operands, the next 16 dims are 32 bytes on, the second
                    // 64-dim block kTBlock on
                    const uint64_t ak = umma_desc(k_lo, 16, 1024), av = umma_desc(v_lo, 16, 1024);
                    const uint64_t bq = umma_desc(q_lo, 16, 1024), bd = umma_desc(do_lo, 16, 1024);
#pragma unroll
                    for (uint32_t k = 0; k < 8; ++k) {
                        const uint64_t off16 = (uint64_t)(((k >> 2) * kTBlock + (k & 3u) * 32u) >> 4);
                        umma_bf16(tmem + kTmS, ak + off16, bq + off16, kIdKK, k, issue);
                    }
#pragma unroll
                    for (uint32_t k = 0; k < 8; ++k) {
                        const uint64_t off16 = (uint64_t)(((k >> 2) * kTBlock + (k & 3u) * 32u) >> 4);
                        umma_bf16(tmem + kTmDP, av + off16, bd + off16, kIdKK, k, issue);
                    }
                    umma_commit(bar(kTbSFull), issue);
                }
                ok = wait_all(kTbPReady, i & 1u);
                if (!ok) break;
                tc_fence_after();
                {
                    // dV += P^T dO, dK += dS^T Q: A from tensor memory (bf16 pairs, 16 rows = 8 columns per step; rows
                    // 0-63 of the tile in columns 0-31 of the buffer, rows 64-127 in columns 64-95), B = the dO / Q
                    // tile as it lies in shared memory, rows 128 bytes apart: MN-major, 16 rows = 2048 bytes per step
                    const uint64_t bdo = umma_desc(do_lo, kTBlock, 1024), bq = umma_desc(q_lo, kTBlock, 1024);
#pragma unroll
                    for (uint32_t k = 0; k < 8; ++k)
                        umma_bf16_ts(tmem + kTmDV, tmem + kTmS + (k < 4u ? 8u * k : 64u + 8u * (k - 4u)),
                                     bdo + (uint64_t)(k * 128u), kIdTsMn, (i == 0u && k == 0u) ? 0u : 1u, issue);
#pragma unroll
                    for (uint32_t k = 0; k < 8; ++k)
                        umma_bf16_ts(tmem + kTmDK, tmem + kTmDP + (k < 4u ? 8u * k : 64u + 8u * (k - 4u)),
                                     bq + (uint64_t)(k * 128u), kIdTsMn, (i == 0u && k == 0u) ? 0u : 1u, issue);
                    // dQ_part = dS K over the columns that held S^T and P^T (the tensor pipe runs this thread's
                    // products in order, so P^T has been consumed): dS [key][row] and K [key][dim] both MN-major
                    const uint64_t ads = umma_desc(ds_lo, kTBlock, 1024), bk = umma_desc(k_lo, kTBlock, 1024);
#pragma unroll
                    for (uint32_t k = 0; k < 8; ++k)
                        umma_bf16(tmem + kTmS, ads + (uint64_t)(k * 128u), bk + (uint64_t)(k * 128u), kIdMnMn, k, issue);
                    umma_commit(bar(kTbDQFull), issue);  // (the stage's Q and dO tiles have been consumed with it)
                }
            }
            umma_commit(bar(kTbDrain), issue);
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(bar(kTbDrain), 0) && global_timer_ns() - t0 < kWaitLimitNs) {}
            __syncwarp();
        }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kTrRegsCompute));
        // ================= compute warps ===================================================================
        const int wg = (warp - 4) >> 2;
        const int sw = warp & 3;
        const uint32_t j = (uint32_t)(32 * sw + lane);         // key of the tile (S^T lane) and, for dQ_part, row
        const uint32_t col0 = 64u * (uint32_t)wg;
        const uint32_t lane_addr = tmem + ((uint32_t)(32 * sw) << 16);
        const uint8_t *tokoff = reinterpret_cast<const uint8_t *>(smem + kTrOffTok);
        const float sl2 = p.scale * 1.4426950408889634f;
        const uint32_t n_keys = it.n_keys, rt_begin = it.rt_begin, rt_first = it.rt_first, kv_head = it.kv_head;
        const uint32_t causal = it.causal, key_tok0 = it.key_tok0;
        const bool key_valid = j < n_keys;
        // key j is seen by the rows of tokens lo .. hi - 1
        const uint32_t lo = causal ? key_tok0 + j : 0u, hi = it.tok_end;
        bool alive = true;
        auto warp_wait = [&](int b, uint32_t parity) -> bool {
            return __all_sync(0xffffffffu, mbar_wait(bar(b), parity, abort_flag, p.status, kStatusTimeoutConsumer));
        };
        alive = warp_wait(kTbKV, 0u);
        if (alive && n_keys < 128u) {
            // keys past the tile's end hold whatever follows in the arena; dS is zero there, but 0 * NaN would poison
            // dQ_part = dS K, so those rows of K are cleared (dS K reads them as the B operand)
            const uint32_t n_bad = 128u - n_keys;
            for (uint32_t x = threadIdx.x - 128u; x < n_bad * 16u; x += 256u) {
                const uint32_t r = n_keys + x / 16u, c = x % 16u;
                const uint32_t a = base + kTrOffK + (c >> 3) * kTBlock + r * 128u + ((c & 7u) << 4);
                asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        }
        for (uint32_t i = 0; i < n_it; ++i) {
            const uint32_t st = i & 1u;
            const uint32_t rt = rt_begin + (rt_first - rt_begin + i) % n_it;
            const uint32_t tok0 = rt * tpt;
            const float2 *ld = reinterpret_cast<const float2 *>(smem + kTrOffLD) + st * 128u;
            // a Cartridge tile whose keys all exist against a row tile whose rows all exist needs no mask
            const bool full = !causal && n_keys == 128u && rows_valid == 128u && tok0 + tpt <= hi;
            if (alive) alive = warp_wait(kTbQFull + (int)st, (i >> 1) & 1u);   // the row tile's lse and D are in shared memory
            if (alive) alive = warp_wait(kTbSFull, i & 1u);
            if (alive) {
                tc_fence_after();
#pragma unroll
                for (uint32_t half = 0; half < 2; ++half) {
                    uint32_t s[32], d[32], w[16], x[16];
                    const uint32_t c_base = col0 + 32u * half;
                    tmem_ld32_issue(lane_addr + kTmS + c_base, s);
                    tmem_ld32_issue(lane_addr + kTmDP + c_base, d);
                    tmem_ld_wait(s);
                    tmem_ld_wait(d);
#pragma unroll
                    for (uint32_t c = 0; c < 32; c += 2) {
                        float pv[2], dv[2];
#pragma unroll
                        for (uint32_t e = 0; e < 2; ++e) {
                            const uint32_t r = c_base + c + e;            // row of the row tile
                            const float2 l = ld[r];
                            bool on = true;
                            if (!full) {
                                const uint32_t tk = tok0 + tokoff[r];
                                on = key_valid && r < rows_valid && tk >= lo && tk < hi;
                            }
                            const float pr = on ? fast_exp2(fmaf(__uint_as_float(s[c + e]), sl2, -l.x)) : 0.f;
                            pv[e] = pr;
                            // (what the key does not see may hold anything, NaN included: it is left out, not weighted by 0)
                            dv[e] = on ? pr * (__uint_as_float(d[c + e]) - l.y) * p.scale : 0.f;
                        }
                        w[c >> 1] = pack_bf16(pv[0], pv[1]);
                        x[c >> 1] = pack_bf16(dv[0], dv[1]);
                    }
                    // bf16 pairs back over the first half of the columns they came from
                    tmem_st16(lane_addr + kTmS + col0 + 16u * half, w);
                    tmem_st16(lane_addr + kTmDP + col0 + 16u * half, x);
                    // dS for dQ_part = dS K: key j's row of the [key][row] tile, rows 64 w .. 64 w + 63 are block w
                    const uint32_t row_addr = base + kTrOffDS + (uint32_t)wg * kTBlock + j * 128u;
#pragma unroll
                    for (uint32_t c8 = 0; c8 < 4; ++c8) {
                        const uint32_t a = row_addr + (((4u * half + c8) ^ (j & 7u)) << 4);
                        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(a), "r"(x[4 * c8]), "r"(x[4 * c8 + 1]),
                                     "r"(x[4 * c8 + 2]), "r"(x[4 * c8 + 3])
                                     : "memory");
                    }
                }
                tmem_st_wait();
                tc_fence_before();
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kTbPReady));
            }
            if (alive) alive = warp_wait(kTbDQFull, i & 1u);
            if (alive) {
                tc_fence_after();
                // dQ_part: this thread now owns ROW j of the row tile (tensor-memory lane j), dims col0 .. col0 + 63.  The
                // row goes to shared memory -- the stage's Q tile (first warpgroup) or dO tile (second), which the
                // products no longer need -- as two blocks of 128 rows x 32 dims with the 128-byte swizzle, and one
                // thread per warpgroup has the memory system add the blocks into dq: rows of tokens past the end of
                // the batch are clipped by the tensor map, rows the key tile does not reach hold zeros.
                const uint32_t stage_lo = base + (wg == 0 ? kTrOffQ : kTrOffDO) + st * kTTile;
#pragma unroll
                for (uint32_t half = 0; half < 2; ++half) {
                    uint32_t v[32];
                    tmem_ld32_issue(lane_addr + kTmS + col0 + 32u * half, v);
                    tmem_ld_wait(v);
                    const uint32_t row_addr = stage_lo + half * kTBlock + j * 128u;
#pragma unroll
                    for (uint32_t c8 = 0; c8 < 8; ++c8)
                        asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(row_addr + ((c8 ^ (j & 7u)) << 4)),
                                     "r"(v[4 * c8]), "r"(v[4 * c8 + 1]), "r"(v[4 * c8 + 2]), "r"(v[4 * c8 + 3])
                                     : "memory");
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kTbTmFree));
            }
            // the warpgroup's rows are all in shared memory: one thread sends them off and, once they have been read,
            // gives the stage back to the producer (the barrier is met by every warp, also by one that has given up)
            if (wg == 0) asm volatile("bar.sync 5, 128;" ::: "memory");
            else asm volatile("bar.sync 6, 128;" ::: "memory");
            if (alive && sw == 0 && lane == 0) {
                const uint32_t stage_lo = base + (wg == 0 ? kTrOffQ : kTrOffDO) + st * kTTile;
                const int32_t y = (int32_t)(kv_head * (uint32_t)G), z = (int32_t)tok0;
                tma_reduce_add_3d(&tmap_dq, stage_lo, (int32_t)col0, y, z);
                tma_reduce_add_3d(&tmap_dq, stage_lo + kTBlock, (int32_t)col0 + 32, y, z);
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                mbar_arrive(bar(kTbQEmpty + (int)st));
            }
        }
        // the key tile's gradients: lane j = key j, dims col0 .. col0 + 63 of dV and dK (complete with the last dQ_part)
        if (alive && n_it > 0u) {
            float *gv = (it.is_z ? p.dzv : p.dv) + ((size_t)it.dst_row + (size_t)j * it.dst_stride) * kHeadDim + col0;
            float *gk = (it.is_z ? p.dzk : p.dk) + ((size_t)it.dst_row + (size_t)j * it.dst_stride) * kHeadDim + col0;
#pragma unroll
            for (uint32_t half = 0; half < 2; ++half) {
                uint32_t a[32], b[32];   // (the loads are warp-wide: every lane takes part, valid keys store)
                tmem_ld32_issue(lane_addr + kTmDV + col0 + 32u * half, a);
                tmem_ld32_issue(lane_addr + kTmDK + col0 + 32u * half, b);
                tmem_ld_wait(a);
                tmem_ld_wait(b);
                if (key_valid) {
#pragma unroll
                    for (uint32_t q4 = 0; q4 < 8; ++q4) {
                        atomicAdd(reinterpret_cast<float4 *>(gv + 32u * half) + q4,
                                  make_float4(__uint_as_float(a[4 * q4]), __uint_as_float(a[4 * q4 + 1]),
                                              __uint_as_float(a[4 * q4 + 2]), __uint_as_float(a[4 * q4 + 3])));
                        atomicAdd(reinterpret_cast<float4 *>(gk + 32u * half) + q4,
                                  make_float4(__uint_as_float(b[4 * q4]), __uint_as_float(b[4 * q4 + 1]),
                                              __uint_as_float(b[4 * q4 + 2]), __uint_as_float(b[4 * q4 + 3])));
                    }
                }
            }
        }
        tc_fence_before();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTrTmemCols) : "memory");
    }
}

}  // namespace

cudaError_t prepare_train_kernels()
{
    return cudaFuncSetAttribute(cart_train_bwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTrSmemBytes);
}

cudaError_t launch_train_delta(const TrainDeltaParams &p, cudaStream_t s)
{
    const int grid = (p.n_rows + 7) / 8;
    cart_train_delta_kernel<<<grid, 256, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_train_bwd(const CUtensorMap &tmap, const CUtensorMap &tmap_q, const CUtensorMap &tmap_do,
                             const CUtensorMap &tmap_dq, const TrainBwdParams &p, int n_items, cudaStream_t s)
{
    cart_train_bwd_kernel<<<n_items, kTrThreads, kTrSmemBytes, s>>>(tmap, tmap_q, tmap_do, tmap_dq, p);
    return cudaGetLastError();
}

}  // namespace cart
