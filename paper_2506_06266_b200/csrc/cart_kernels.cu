// sm_100a kernels of libcart.so: split-KV decode attention over [Cartridge(s) ; suffix] with the
// log-sum-exp merge of split row groups, and the KV append / extend scatters.
//
// Decode kernel in one paragraph.  One persistent block per SM walks its list of work items (runs
// of 64-token tiles of one KV segment of one (request, KV head) row group).  A producer warp streams
// K and V tiles from HBM into a ring of shared-memory stages with TMA (cp.async.bulk.tensor, 128-byte
// swizzle, completion on mbarriers); each stage has its own consumer warp, which takes whole tiles.  In a
// fused decode step one more warp writes the requests' new tokens into their suffixes and tells the
// producer, which fetches a tile that ends with such a token only afterwards.  A
// consumer multiplies the group's G query heads (padded to the 16 rows of an m16n8k16 bf16 MMA, so
// a K/V tile is read once per group) with the tile, keeps an fp32 online softmax (running max, sum,
// rescaled output) in registers, and multiplies the probabilities with V.  At the end of a row-group
// piece every warp deposits its state in shared memory and moves on; a warp of its own combines the
// six states and writes either the final bf16 output + lse (piece = whole row group) or an fp32
// partial; the block that delivers the last partial of a split row group merges them (an arrival
// ticket per split row group, no waiting), unless a merge kernel follows.
// Arithmetic follows Eq. 1 of the paper evaluated at the last position; the split and the merge use
// that a softmax over a union of token sets is the lse-weighted mix of the softmaxes over the sets.
#include <cuda_bf16.h>

#include "cart_internal.h"
#include "cart_device.cuh"

namespace cart {
namespace {

constexpr int kStages = 6;
// One consumer warp per stage: warp w is the only reader of stage w, so its waits on that stage's
// barriers follow one another round by round.  (With several warps sharing a stage, a warp two
// rounds ahead would mistake an older completed phase for its own: an mbarrier only tells the
// current phase from the one before.)
constexpr int kConsumerWarps = kStages;
constexpr int kConsumerThreads = kConsumerWarps * 32;
constexpr int kThreads = kConsumerThreads + 96;      // + the producer warp + the append warp + the combine warp
constexpr uint32_t kHalfBytes = kTileTokens * 128;    // 64 tokens x 64 dims of bf16
constexpr uint32_t kTileBytes = 2 * kHalfBytes;       // K or V tile: 64 tokens x 128 dims
constexpr uint32_t kStageBytes = 2 * kTileBytes;      // K tile then V tile
constexpr uint32_t kEdgeRows = kEdgeBoxRows;           // rows of the small box that ragged tiles are fetched in
constexpr uint32_t kEdgeBoxBytes = kEdgeRows * 128;    // kEdgeRows tokens x 64 dims of bf16
static_assert(kEdgeRows % 16 == 0 && kTileTokens % kEdgeRows == 0,
              "an edge box must hold whole 8-row swizzle groups and whole 16-token steps of the P V product");
constexpr int kScratchStride = 132;                   // floats per scratch row (128 + pad)
constexpr uint32_t kScratchOBytes = kConsumerWarps * kMaxGroup * kScratchStride * 4;
constexpr uint32_t kScratchMLBytes = 2 * kConsumerWarps * kMaxGroup * 2 * 4;  // two buffers
constexpr uint32_t kBarrierBytes = (3 * kStages + 4) * 8;
constexpr uint32_t kSmemUsed = kStages * kStageBytes + kScratchOBytes + kScratchMLBytes + kBarrierBytes + 16;  // + flags
constexpr uint32_t kSmemBytes = kSmemUsed + 1024;     // slack to align the stages to 1024 bytes
static_assert(kSmemBytes <= 232448, "shared memory budget of one sm_100 block exceeded");

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr)
                 : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr)
                 : "memory");
}
// D += A(16x16, row) * B(16x8, col); rows 8..15 of A are zero here, so a1 = a3 = 0.
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

// Online-softmax state of one warp for one row-group piece.  Thread (lane) owns query row lane/4
// (valid when < G) and, per 8-wide column tile, columns 2*(lane%4) and 2*(lane%4)+1.
struct WarpState {
    float o[16][4];  // output accumulator, 16 tiles of 8 dims; [.][2..3] belong to the zero rows 8..15
    float m;         // running maximum of the scaled scores (base-2 units)
    float l;         // this thread's share of the running sum of 2^(score - m)
};

// One 64-token tile: scores, online softmax update, probabilities times V.
__device__ __forceinline__ void process_tile(WarpState &st, const uint32_t (&qa0)[8], const uint32_t (&qa2)[8],
                                             uint32_t kbase, uint32_t vbase, uint32_t full_k, uint32_t full_v,
                                             uint32_t parity, int valid, float scale_log2, int lane,
                                             volatile uint32_t *abort_flag, uint32_t *status, bool &ok)
{
    const int l7 = lane & 7;
    const int lm = lane >> 3;
    // (the MMA and ldmatrix instructions below are warp-wide: a wait fails for all lanes or for none)
    ok = __all_sync(0xffffffffu, mbar_wait(full_k, parity, abort_flag, status, kStatusTimeoutConsumer));
    if (!ok) return;

    // ---- S = Q K^T : 16 (padded heads) x 64 tokens, fp32 ------------------------------------
    float s[8][4];
#pragma unroll
    for (int j = 0; j < 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
#pragma unroll
    for (int kp = 0; kp < 4; ++kp) {  // 32 dims per step
#pragma unroll
        for (int j = 0; j < 8; ++j) {  // 8 tokens per column tile
            const uint32_t addr = kbase + (uint32_t)(kp >> 1) * kHalfBytes + (uint32_t)(8 * j + l7) * 128u +
                                  (uint32_t)(((4 * (kp & 1) + lm) ^ l7) << 4);
            uint32_t b0, b1, b2, b3;
            ldmatrix_x4(addr, b0, b1, b2, b3);
            mma_bf16(s[j], qa0[2 * kp], qa2[2 * kp], b0, b1);
            mma_bf16(s[j], qa0[2 * kp + 1], qa2[2 * kp + 1], b2, b3);
        }
    }

    // ---- online softmax on the valid rows (c0, c1 of every column tile) ------------------------
    const int col0 = 2 * (lane & 3);
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        float x0 = s[j][0] * scale_log2, x1 = s[j][1] * scale_log2;
        if (valid < kTileTokens) {  // ragged last tile of a segment: tokens >= valid do not exist
            if (8 * j + col0 >= valid) x0 = -INFINITY;
            if (8 * j + col0 + 1 >= valid) x1 = -INFINITY;
        }
        s[j][0] = x0;
        s[j][1] = x1;
        mx = fmaxf(mx, fmaxf(x0, x1));
    }
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(st.m, mx);
    const float alpha = fast_exp2(st.m - m_new);  // 0 on the first tile (st.m = -inf)
    st.m = m_new;
    float psum = 0.f;
    uint32_t pa0[4], pa2[4];  // probabilities as the A operand of the second MMA, 16 tokens per step
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        const float p00 = fast_exp2(s[2 * t][0] - m_new), p01 = fast_exp2(s[2 * t][1] - m_new);
        const float p10 = fast_exp2(s[2 * t + 1][0] - m_new), p11 = fast_exp2(s[2 * t + 1][1] - m_new);
        psum += (p00 + p01) + (p10 + p11);
        pa0[t] = pack_bf16(p00, p01);
        pa2[t] = pack_bf16(p10, p11);
    }
    st.l = st.l * alpha + psum;
#pragma unroll
    for (int d = 0; d < 16; ++d) {
        st.o[d][0] *= alpha;
        st.o[d][1] *= alpha;
    }

    // ---- O += P V ---------------------------------------------------------------------------------
    ok = __all_sync(0xffffffffu, mbar_wait(full_v, parity, abort_flag, status, kStatusTimeoutConsumer));
    if (!ok) return;
    int ksteps = 4;
    if (valid < kTileTokens) {
        // Rows past the segment's end hold whatever follows it in memory.  Their probability is zero,
        // but 0 * NaN would poison the sum, so clear the rows that the last 16-token step still reads.
        ksteps = (valid + 15) >> 4;
        const int row_end = ksteps << 4;
        for (int idx = lane; idx < (row_end - valid) * 16; idx += 32) {
            const int r = valid + (idx >> 4), c = idx & 15;
            const uint32_t a = vbase + (uint32_t)(c >> 3) * kHalfBytes + (uint32_t)r * 128u + (uint32_t)((c & 7) << 4);
            asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(a), "r"(0u) : "memory");
        }
        __syncwarp();
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
        if (t < ksteps) {
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {  // two 8-dim column tiles per load
                const uint32_t addr = vbase + (uint32_t)(dp >> 2) * kHalfBytes +
                                      (uint32_t)(16 * t + 8 * (lm & 1) + l7) * 128u +
                                      (uint32_t)(((2 * (dp & 3) + (lm >> 1)) ^ l7) << 4);
                uint32_t b0, b1, b2, b3;
                ldmatrix_x4_trans(addr, b0, b1, b2, b3);
                mma_bf16(st.o[2 * dp], pa0[t], pa2[t], b0, b1);
                mma_bf16(st.o[2 * dp + 1], pa0[t], pa2[t], b2, b3);
            }
        }
    }
    if (valid < kTileTokens) {
        // the zeroing above wrote through the generic proxy; order it before the next TMA write
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
}

__global__ void __launch_bounds__(kThreads, 1)
cart_decode_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap_edge,
                   const DecodeParams p)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    const uint32_t stages = base;
    float *scratch_o = reinterpret_cast<float *>(smem + kStages * kStageBytes);
    float *scratch_ml = reinterpret_cast<float *>(smem + kStages * kStageBytes + kScratchOBytes);
    const uint32_t bars = base + kStages * kStageBytes + kScratchOBytes + kScratchMLBytes;
    volatile uint32_t *abort_flag =
        reinterpret_cast<volatile uint32_t *>(smem + kStages * kStageBytes + kScratchOBytes + kScratchMLBytes + kBarrierBytes);
    volatile uint32_t *arrivals = abort_flag + 1;   // [2]: see append_count ([0], [1] unused)
    auto full_k = [&](int s) { return bars + (uint32_t)s * 8u; };
    auto full_v = [&](int s) { return bars + (uint32_t)(kStages + s) * 8u; };
    auto empty = [&](int s) { return bars + (uint32_t)(2 * kStages + s) * 8u; };
    auto scratch_free = [&](uint32_t b) { return bars + (uint32_t)(3 * kStages) * 8u + b * 8u; };
    auto deposited = [&](uint32_t b) { return bars + (uint32_t)(3 * kStages + 2) * 8u + b * 8u; };
    // [1] how many of the block's new tokens (in work-list order) are in the arena: append warp -> producer
    const uint32_t append_count = smem_u32(const_cast<uint32_t *>(arrivals + 2));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    pdl_launch_dependents();

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_k(s), 1);
            mbar_init(full_v(s), 1);
            mbar_init(empty(s), 1);
        }
        mbar_init(scratch_free(0), 1);
        mbar_init(scratch_free(1), 1);
        mbar_init(deposited(0), kConsumerWarps);
        mbar_init(deposited(1), kConsumerWarps);
        *abort_flag = 0;
        arrivals[0] = 0;
        arrivals[1] = 0;
        arrivals[2] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const uint32_t item_begin = p.cta_begin[blockIdx.x];
    const uint32_t item_end = p.cta_begin[blockIdx.x + 1];

    if (warp == kConsumerWarps) {
        // ================= producer: the warp walks the items together, lane 0 feeds the ring =========
        if (lane == 0) {
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap)) : "memory");
            asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&tmap_edge)) : "memory");
        }
        uint32_t t = 0;  // tiles issued by this block so far
        bool ok = true;
        const uint64_t stream_once = l2_evict_first_policy();  // a tile is read once per launch: let it leave L2 first
        // Until the kernels before this one on the stream are known to be complete, only tiles that
        // none of them can have written are fetched: the tiles of stored Cartridges, which only copies
        // write.  Suffix storage (items marked CART_ITEM_SUFFIX) is written by kernels -- the append and
        // extend kernels, and the fused append of an earlier decode step, which may be the kernel right
        // before this one -- so the first suffix tile is fetched only after griddepcontrol.wait.
        bool waited = false;
        uint32_t grow = p.grow;
        bool grow_known = p.grow_ctr == nullptr;  // else the count lives in memory that a kernel before this one advances
        uint32_t tails_seen = 0;  // tiles met so far that end with a new token
        // The next work item is requested while the copies of this one are issued: read at the item's start, it
        // held the ring back by a memory round trip per item, which short row groups cannot spare.
        cart_work_item w_next{};
        if (item_begin < item_end) w_next = p.items[item_begin];
        for (uint32_t it = item_begin; it < item_end && ok; ++it) {
            cart_work_item w = w_next;
            if (it + 1 < item_end) w_next = p.items[it + 1];
            if (w.flags & CART_ITEM_TAIL) {
                if (!grow_known) {  // (read at the first item that needs it: the Cartridge tiles before are fetched meanwhile)
                    if (!waited) {
                        pdl_wait();
                        waited = true;
                    }
                    grow = ld_volatile_u32(p.grow_ctr);
                    grow_known = true;
                }
                w.n_tok += grow;  // tokens appended since the plan was built
            }
            const uint32_t k_row = w.k_row + (uint32_t)p.layer * w.layer_stride;
            const uint32_t v_row = w.v_row + (uint32_t)p.layer * w.layer_stride;
            const uint32_t ntiles = (w.n_tok + kTileTokens - 1) / kTileTokens;
            // Paged suffix (Sec. 3.3: per-user KV caches of any length): tile j of the item is page w.k_row + j of the
            // batch's page list.  Lane l holds the base row of the page of tile 32 c + l, fetched 32 tiles at a time.
            const bool paged = (w.flags & CART_ITEM_PAGED) != 0u;
            const uint32_t in_page = (uint32_t)p.layer * w.layer_stride + w.v_row;  // the head's K block inside a page
            uint32_t page_row = 0;
            for (uint32_t j = 0; j < ntiles; ++j, ++t) {
                if (paged && (j & 31u) == 0u) page_row = j + (uint32_t)lane < ntiles ? __ldg(p.pages + w.k_row + j + (uint32_t)lane) : 0u;
                const uint32_t page_base = __shfl_sync(0xffffffffu, page_row, (int)(j & 31u)) + in_page;
                const int s = (int)(t % kStages);
                const uint32_t round = t / kStages;
                bool ok0 = true;
                if (lane == 0) ok0 = mbar_wait(empty(s), (round & 1u) ^ 1u, abort_flag, p.status, kStatusTimeoutProducer);
                ok = __shfl_sync(0xffffffffu, (int)ok0, 0) != 0;
                if (!ok) break;
                if (!waited && (w.flags & CART_ITEM_SUFFIX)) {
                    pdl_wait();
                    waited = true;
                }
                if (p.k_new != nullptr && (w.flags & CART_ITEM_TAIL) && j + 1 == ntiles) {
                    // Fused append: this tile ends with the request's new token, which the append warp writes.
                    // It works through the block's list far ahead of the producer.
                    ++tails_seen;
                    bool ok1 = true;
                    if (lane == 0) {
                        uint32_t spins = 0;
                        long long t0 = 0;
                        for (;;) {
                            uint32_t done;
                            asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(done) : "r"(append_count) : "memory");
                            if (done >= tails_seen) break;
                            if ((++spins & 0x3FFu) == 0) {  // bounded like every other wait of the kernel
                                if (*abort_flag) { ok1 = false; break; }
                                const long long now = clock64();
                                if (t0 == 0) {
                                    t0 = now | 1;
                                } else if (now - t0 > kWaitLimitCycles) {
                                    *abort_flag = 1;
                                    atomicOr(p.status, kStatusTimeoutProducer);
                                    ok1 = false;
                                    break;
                                }
                            }
                        }
                    }
                    ok = __shfl_sync(0xffffffffu, (int)ok1, 0) != 0;
                    if (!ok) break;
                    // (the append warp has ordered its generic-proxy stores before the TMA reads that follow its
                    // release: the proxy fence is on the writer's side, off the path of the copies)
                }
                {
                    // The tile's four boxes (K and V, each as two 64-dim halves) are requested by four lanes in
                    // one instruction: a copy instruction costs the issuing thread about a hundred cycles,
                    // and one thread issuing all of them one after the other is what limits the tile rate of
                    // a block when the batch is made of many short runs.
                    const uint32_t kdst = stages + (uint32_t)s * kStageBytes;
                    const uint32_t is_v = ((uint32_t)lane >> 1) & 1u, hi = (uint32_t)lane & 1u;
                    const uint32_t dst = kdst + is_v * kTileBytes + hi * kHalfBytes;
                    const int32_t y = paged ? (int32_t)(page_base + is_v * (uint32_t)kTileTokens)
                                            : (int32_t)((is_v ? v_row : k_row) + j * kTileTokens);
                    const uint32_t bar = is_v ? full_v(s) : full_k(s);
                    const uint32_t valid = min((uint32_t)kTileTokens, w.n_tok - j * kTileTokens);
                    // Ragged last tile of a segment with at most kEdgeRows tokens: only one small box per half
                    // is fetched (the consumers read no row past the 16-row step that holds the last token),
                    // not the rows that follow the segment in memory.  A small box is a whole number of 8-row
                    // swizzle groups, so the tile's layout is unchanged.  (Boxes of 16 rows save more bytes
                    // but cost up to three times the copy instructions.)
                    const bool edge = p.edge_boxes != 0u && valid <= kEdgeRows;
                    static_assert(2 * kEdgeRows == kTileTokens, "a ragged tile is fetched as one small box or whole");
                    if (lane < 4) {
                        if (hi == 0u) mbar_expect_tx(bar, edge ? 2u * kEdgeBoxBytes : kTileBytes);
                        tma_load_2d_hint(dst, edge ? &tmap_edge : &tmap, (int32_t)(hi * 64u), y, bar, stream_once);
                    }
                }
            }
        }
        if (!ok && lane == 0) {
            // Gave up: no new copies are issued; wait (bounded) for those still in flight so that
            // none lands in shared memory after the block has gone.
            const uint32_t issued = t;
            for (uint32_t u = (issued > (uint32_t)kStages ? issued - kStages : 0u); u < issued; ++u) {
                const int s = (int)(u % kStages);
                const uint32_t par = (u / kStages) & 1u;
                const uint64_t t0 = global_timer_ns();
                while (!mbar_try_wait(full_k(s), par) && global_timer_ns() - t0 < kWaitLimitNs) {}
                while (!mbar_try_wait(full_v(s), par) && global_timer_ns() - t0 < kWaitLimitNs) {}
            }
        }
        return;
    }

    if (warp == kConsumerWarps + 1) {
        // ================= append warp (decode phase of Sec. 2.3, fused) ===============================
        // Writes the new token of every request whose cache ends in this block's work list to the end of
        // its suffix -- K row by lanes 0-15, V row by lanes 16-31, 256 bytes each -- and then tells the
        // producer, which fetches the tiles that hold these rows only afterwards.  No other block reads
        // them in this launch.  Doing this on a warp of its own keeps the producer issuing copies.
        if (p.k_new != nullptr) {
            const uint32_t c = (uint32_t)lane & 15u;
            bool waited = false;
            const uint4 *new_rows = reinterpret_cast<const uint4 *>(lane < 16 ? p.k_new : p.v_new);
            uint32_t n_done = 0;
            uint32_t grow = p.grow;
            if (p.grow_ctr != nullptr) {
                pdl_wait();
                waited = true;
                grow = ld_volatile_u32(p.grow_ctr);
            }
            for (uint32_t base_it = item_begin; base_it < item_end; base_it += 32u) {
                const uint32_t mine = base_it + (uint32_t)lane;
                cart_work_item a{};
                if (mine < item_end) a = p.items[mine];
                uint32_t tails = __ballot_sync(0xffffffffu, (a.flags & CART_ITEM_TAIL) != 0u);
                if (!waited) {
                    pdl_wait();  // k_new and v_new come from the kernels before (the plan does not: it is read above)
                    waited = true;
                }
                while (tails) {
                    // up to four requests at a time, their loads in flight together; the very first one alone,
                    // so that the producer does not wait long for it at the start of a launch
                    uint4 val[4];
                    size_t dst[4];
                    int n = 0;
                    const int batch = n_done == 0u ? 1 : 4;
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        if (tails && u < batch) {
                            const int src_lane = __ffs((int)tails) - 1;
                            tails &= tails - 1u;
                            const uint32_t a_k = __shfl_sync(0xffffffffu, a.k_row, src_lane);
                            const uint32_t a_v = __shfl_sync(0xffffffffu, a.v_row, src_lane);
                            const uint32_t row0 = lane < 16 ? a_k : a_v;
                            const uint32_t a_ls = __shfl_sync(0xffffffffu, a.layer_stride, src_lane);
                            const uint32_t a_n = __shfl_sync(0xffffffffu, a.n_tok, src_lane) + grow;
                            const uint32_t a_rg = __shfl_sync(0xffffffffu, a.row_group, src_lane);
                            const uint32_t a_fl = __shfl_sync(0xffffffffu, a.flags, src_lane);
                            val[u] = __ldg(new_rows + (size_t)a_rg * 16 + c);
                            if (a_fl & CART_ITEM_PAGED) {
                                // the page that holds the item's last token, then the head's K or V block in it
                                const uint32_t page = __ldg(p.pages + a_k + ((a_n - 1u) / (uint32_t)kTileTokens));
                                dst[u] = ((size_t)page + (size_t)p.layer * a_ls + a_v + (lane < 16 ? 0u : (uint32_t)kTileTokens) +
                                          ((a_n - 1u) % (uint32_t)kTileTokens)) * 16 + c;
                            } else {
                                dst[u] = ((size_t)row0 + (size_t)p.layer * a_ls + (a_n - 1u)) * 16 + c;
                            }
                            n = u + 1;
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (u < n) reinterpret_cast<uint4 *>(p.arena)[dst[u]] = val[u];
                    __threadfence();  // the rows are in memory before the producer hears of them
                    asm volatile("fence.proxy.async;" ::: "memory");  // ... and before the TMA reads it then issues
                    __syncwarp();
                    n_done += (uint32_t)n;
                    if (lane == 0)
                        asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(append_count), "r"(n_done) : "memory");
                }
            }
        }
        return;
    }

    if (warp == kConsumerWarps + 2) {
        // ================= combine warp ================================================================
        // At the end of a row-group piece every consumer warp deposits its online-softmax state in shared
        // memory and goes straight on to its tiles of the next piece; this warp combines the six states
        // and writes the piece -- the final bf16 output and lse when the piece is the whole row group,
        // else a normalised fp32 partial followed by the arrival ticket and, if it was the last one, the
        // merge.  On a consumer warp the combine (about a microsecond of dependent shared-memory reads)
        // held up that warp's ring stage, and the producer, which refills the stages in order, with it.
        pdl_wait();  // out, the partial slots and the tickets belong to the kernels before until they are done
        const int G = p.group;
        const uint32_t nbuf = G <= kMaxGroup / 2 ? 2u : 1u;
        const int rows_buf = G <= kMaxGroup / 2 ? kMaxGroup / 2 : kMaxGroup;
        uint32_t piece = 0;
        cart_work_item w_next{};
        if (item_begin < item_end) w_next = p.items[item_begin];
        for (uint32_t it = item_begin; it < item_end; ++it) {
            const cart_work_item w = w_next;
            if (it + 1 < item_end) w_next = p.items[it + 1];
            if (!(w.flags & CART_ITEM_END)) continue;
            const uint32_t b = piece % nbuf, use = piece / nbuf;
            ++piece;
            if (!__all_sync(0xffffffffu, mbar_wait(deposited(b), use & 1u, abort_flag, p.status, kStatusTimeoutConsumer)))
                return;
            const float *buf_o = scratch_o + (size_t)b * kConsumerWarps * rows_buf * kScratchStride;
            const float *buf_ml = scratch_ml + (size_t)b * kConsumerWarps * kMaxGroup * 2;
            const int quad = lane;  // four output dims per lane
#pragma unroll 2
            for (int r = 0; r < G; ++r) {
                float mw[kConsumerWarps], lw[kConsumerWarps];
                float4 v[kConsumerWarps];
                float M = -INFINITY;
#pragma unroll
                for (int wv = 0; wv < kConsumerWarps; ++wv) {  // all loads of the row in flight together
                    mw[wv] = buf_ml[(wv * kMaxGroup + r) * 2];
                    lw[wv] = buf_ml[(wv * kMaxGroup + r) * 2 + 1];
                    v[wv] = *reinterpret_cast<const float4 *>(buf_o + ((size_t)wv * rows_buf + r) * kScratchStride + 4 * quad);
                }
#pragma unroll
                for (int wv = 0; wv < kConsumerWarps; ++wv) M = fmaxf(M, mw[wv]);
                float L = 0.f;
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int wv = 0; wv < kConsumerWarps; ++wv) {
                    if (mw[wv] == -INFINITY) continue;  // that warp had no tile of the piece (its slot holds old data)
                    const float wgt = fast_exp2(mw[wv] - M);
                    L += wgt * lw[wv];
                    a.x += wgt * v[wv].x;
                    a.y += wgt * v[wv].y;
                    a.z += wgt * v[wv].z;
                    a.w += wgt * v[wv].w;
                }
                const float inv = 1.f / L;
                const float lse2 = M + log2f(L);
                if (w.flags & CART_ITEM_DIRECT) {
                    const size_t orow = (size_t)w.row_group * G + r;
                    uint2 packed;
                    packed.x = pack_bf16(a.x * inv, a.y * inv);
                    packed.y = pack_bf16(a.z * inv, a.w * inv);
                    *reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(p.out) + orow * kHeadDim + 4 * quad) = packed;
                    if (quad == 0 && p.lse) p.lse[orow] = lse2 * 0.6931471805599453f;
                } else {
                    float4 *pp = reinterpret_cast<float4 *>(p.part_o + ((size_t)w.slot * G + r) * kHeadDim) + quad;
                    *pp = make_float4(a.x * inv, a.y * inv, a.z * inv, a.w * inv);
                    if (quad == 0) p.part_lse2[(size_t)w.slot * kMaxGroup + r] = lse2;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(scratch_free(b));  // the buffer may be refilled from here on
            if (!(w.flags & CART_ITEM_DIRECT) && p.tickets != nullptr) {
                // Split row group: the block whose piece arrives last merges all pieces.  Nobody waits.
                __threadfence();  // publish the partial before the ticket
                __syncwarp();
                const cart_merge_item mi = p.merges[w.merge];
                uint32_t mine = 0;
                if (lane == 0) mine = (atomicAdd(&p.tickets[w.merge], 1u) + 1u == mi.slot_end - mi.slot_begin) ? 1u : 0u;
                mine = __shfl_sync(0xffffffffu, mine, 0);
                if (mine) {
                    __threadfence();
                    merge_row_group<4, 2>(mi, G, p.part_o, p.part_lse2, p.out, p.lse, lane, 32);
                    __syncwarp();
                    if (lane == 0) p.tickets[w.merge] = 0;  // ready for the next launch
                }
            }
        }
        return;
    }

    // ===================== consumers ==============================================================
    pdl_wait();  // q, the partial slots and the tickets belong to the kernels before until they are done
    if (p.ready_flag != nullptr && blockIdx.x == 0 && threadIdx.x == 0)  // tell the kernel that runs beside this one
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p.ready_flag), "r"(1u) : "memory");
    const uint32_t grow = p.grow_ctr != nullptr ? ld_volatile_u32(p.grow_ctr) : p.grow;
    const int G = p.group;
    const int row = lane >> 2;  // query head inside the group that this thread's c0/c1 belong to
    const __nv_bfloat16 *q = reinterpret_cast<const __nv_bfloat16 *>(p.q);
    WarpState st;
    uint32_t qa0[8], qa2[8];
    uint32_t t = 0;       // tiles seen by this block so far (same count as the producer's)
    bool alive = true;    // false once the block has given up
    // The combine scratch holds the six warps' states of a piece.  With G <= 4 it fits twice, and
    // consecutive pieces alternate between the halves; larger groups use it as one buffer.
    const uint32_t nbuf = G <= kMaxGroup / 2 ? 2u : 1u;
    const int rows_buf = G <= kMaxGroup / 2 ? kMaxGroup / 2 : kMaxGroup;
    uint32_t piece = 0;   // pieces this block has finished

    for (uint32_t it = item_begin; it < item_end; ++it) {
        cart_work_item w = p.items[it];
        if (w.flags & CART_ITEM_TAIL) w.n_tok += grow;
        if (w.flags & CART_ITEM_BEGIN) {
            st.m = -INFINITY;
            st.l = 0.f;
#pragma unroll
            for (int d = 0; d < 16; ++d) st.o[d][0] = st.o[d][1] = st.o[d][2] = st.o[d][3] = 0.f;
            if (row < G) {
                const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
                    q + ((size_t)w.row_group * G + row) * kHeadDim);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    qa0[kk] = __ldg(qrow + kk * 8 + (lane & 3));
                    qa2[kk] = __ldg(qrow + kk * 8 + 4 + (lane & 3));
                }
            } else {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) qa0[kk] = qa2[kk] = 0u;
            }
        }
        const uint32_t ntiles = (w.n_tok + kTileTokens - 1) / kTileTokens;
        // this warp takes the tiles that land in its own stage: block-wide tile index = warp (mod stages)
        uint32_t j = (uint32_t)((warp + kStages - (int)(t % kStages)) % kStages);
        for (; j < ntiles; j += kStages) {
            if (!alive) break;
            const uint32_t tt = t + j;
            const int s = warp;
            const uint32_t parity = (tt / kStages) & 1u;
            const uint32_t kbase = stages + (uint32_t)s * kStageBytes;
            const int valid = min((int)kTileTokens, (int)(w.n_tok - j * kTileTokens));
            bool ok;
            process_tile(st, qa0, qa2, kbase, kbase + kTileBytes, full_k(s), full_v(s), parity, valid,
                         p.scale_log2, lane, abort_flag, p.status, ok);
            if (!ok) { alive = false; break; }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty(s));
        }
        t += ntiles;

        if (w.flags & CART_ITEM_END) {
            // ---- hand this warp's state of the piece to the combine warp ------------------------------
            // No block-wide barrier: a warp that has deposited goes straight on to its tiles of the next
            // piece.  Pieces alternate between the scratch buffers; a buffer is free again once the
            // combine of the piece that used it before is done.
            const uint32_t b = piece % nbuf, use = piece / nbuf;
            ++piece;
            if (alive && use > 0)
                alive = __all_sync(0xffffffffu, mbar_wait(scratch_free(b), (use - 1u) & 1u, abort_flag, p.status,
                                                          kStatusTimeoutConsumer));
            if (!alive) continue;
            float lsum = st.l;
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 1);
            lsum += __shfl_xor_sync(0xffffffffu, lsum, 2);
            float *buf_o = scratch_o + (size_t)b * kConsumerWarps * rows_buf * kScratchStride;
            float *buf_ml = scratch_ml + (size_t)b * kConsumerWarps * kMaxGroup * 2;
            if (row < G) {
                float *so = buf_o + ((size_t)warp * rows_buf + row) * kScratchStride + 2 * (lane & 3);
#pragma unroll
                for (int d = 0; d < 16; ++d)
                    *reinterpret_cast<float2 *>(so + 8 * d) = make_float2(st.o[d][0], st.o[d][1]);
                if ((lane & 3) == 0) {
                    buf_ml[(warp * kMaxGroup + row) * 2 + 0] = st.m;   // -inf if the warp had no tile of the piece
                    buf_ml[(warp * kMaxGroup + row) * 2 + 1] = lsum;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(deposited(b));  // (release) the combine warp takes it from here
        }
    }
}

// Merges split row groups after the decode kernels, one block per row group.  Used instead of the
// in-kernel arrival tickets when a batch has more split row groups than blocks (every reader of a
// shared Cartridge is one).
__global__ void __launch_bounds__(128) cart_merge_kernel(const MergeParams p)
{
    pdl_launch_dependents();
    // (the plan was uploaded before the kernels whose partials are merged here were launched: its entry is read
    //  while those kernels still run, one memory round trip less behind them)
    const cart_merge_item mi = p.merges[blockIdx.x];
    pdl_wait();  // the partials come from the kernels before
    merge_row_group<1, 8>(mi, p.group, p.part_o, p.part_lse2, p.out, p.lse, (int)threadIdx.x, 128);
}

// One block per request: copy the new token's K and V rows (Hkv x 256 bytes each) to the suffix end.
__global__ void __launch_bounds__(128) cart_append_kernel(const __grid_constant__ AppendParams p)
{
    const int i = blockIdx.x;
    const AppendEntry e = p.e[i];
    const int chunks = p.n_kv_heads * 16;  // 16-byte chunks per tensor
    uint4 *arena = reinterpret_cast<uint4 *>(p.arena);
    const uint4 *ks = reinterpret_cast<const uint4 *>(p.k_new) + (size_t)i * chunks;
    const uint4 *vs = reinterpret_cast<const uint4 *>(p.v_new) + (size_t)i * chunks;
    for (int c = threadIdx.x; c < 2 * chunks; c += blockDim.x) {
        const bool is_v = c >= chunks;
        const int cc = is_v ? c - chunks : c;
        const int h = cc >> 4, part = cc & 15;
        const size_t row = (size_t)(is_v ? e.v_row : e.k_row) + (size_t)h * e.head_stride;
        arena[row * 16 + part] = is_v ? vs[cc] : ks[cc];
    }
}

// Advances the count of tokens appended since the plan was built (one decode step of a recorded loop is over).
__global__ void cart_advance_kernel(uint32_t *ctr)
{
    pdl_launch_dependents();
    pdl_wait();  // the kernels before still read the old value
    if (threadIdx.x == 0 && blockIdx.x == 0) *ctr = *ctr + 1u;
}

// Token-major [T][Hkv][128] -> head-major suffix rows; one thread per 16-byte chunk.
__global__ void __launch_bounds__(256) cart_extend_kernel(const ExtendParams p)
{
    // launched as a dependent of the kernel before it: its blocks are placed while that kernel drains, and wait
    // here for it (k and v may be its output, and its tiles may still cover the rows written below)
    pdl_launch_dependents();
    pdl_wait();
    const size_t chunks = (size_t)p.n_tokens * p.n_kv_heads * 16;
    uint4 *arena = reinterpret_cast<uint4 *>(p.arena);
    const uint4 *ks = reinterpret_cast<const uint4 *>(p.k);
    const uint4 *vs = reinterpret_cast<const uint4 *>(p.v);
    for (size_t c = (size_t)blockIdx.x * blockDim.x + threadIdx.x; c < 2 * chunks;
         c += (size_t)gridDim.x * blockDim.x) {
        const bool is_v = c >= chunks;
        const size_t cc = is_v ? c - chunks : c;
        const int part = (int)(cc & 15);
        const size_t th = cc >> 4;  // token * Hkv + head
        const size_t tok = th / p.n_kv_heads, h = th % p.n_kv_heads;
        const size_t row = (size_t)(is_v ? p.v_row : p.k_row) + h * p.head_stride + tok;
        arena[row * 16 + part] = is_v ? vs[cc] : ks[cc];
    }
}

}  // namespace

size_t decode_smem_bytes() { return kSmemBytes; }
int decode_threads() { return kThreads; }

cudaError_t prepare_kernels()
{
    return cudaFuncSetAttribute(cart_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
}

cudaError_t launch_decode(const CUtensorMap &tmap, const CUtensorMap &tmap_edge, const DecodeParams &p, int grid,
                          cudaStream_t s)
{
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg = pdl_config(grid, kThreads, kSmemBytes, s, &attr);
    return cudaLaunchKernelEx(&cfg, cart_decode_kernel, tmap, tmap_edge, p);
}

cudaError_t launch_merge(const MergeParams &p, int n_merges, cudaStream_t s)
{
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg = pdl_config(n_merges, 128, 0, s, &attr);
    return cudaLaunchKernelEx(&cfg, cart_merge_kernel, p);
}

cudaError_t launch_advance(uint32_t *ctr, cudaStream_t s)
{
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg = pdl_config(1, 32, 0, s, &attr);
    return cudaLaunchKernelEx(&cfg, cart_advance_kernel, ctr);
}

cudaError_t launch_append(const AppendParams &p, cudaStream_t s)
{
    cart_append_kernel<<<p.n, 128, 0, s>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_extend(const ExtendParams &p, cudaStream_t s)
{
    const size_t chunks = 2ull * (size_t)p.n_tokens * p.n_kv_heads * 16;
    int grid = (int)((chunks + 255) / 256);
    if (grid > 148 * 8) grid = 148 * 8;
    if (grid < 1) grid = 1;
    cudaLaunchAttribute attr;
    const cudaLaunchConfig_t cfg = pdl_config(grid, 256, 0, s, &attr);
    return cudaLaunchKernelEx(&cfg, cart_extend_kernel, p);
}

}  // namespace cart
