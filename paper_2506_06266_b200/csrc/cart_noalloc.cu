// cart_decode_attention_static: decode attention for callers that cannot allocate.
//
// The context-based entry points need an arena from the caller and pinned host staging from
// cart_create.  Some callers can do neither: code running inside a memory-pool region where
// cudaMalloc / cudaHostAlloc would synchronise the device or break the pool's accounting, plug-ins
// that are handed tensors by a host framework but may not call its allocator, and start-up or
// health-check paths that run before any allocator exists.  For them this file keeps the split-KV
// kernels' scratch (work list and split partials) in a fixed device array that is part of the
// library image, and the host copy of the work list in a fixed host array.
#include <cstring>

#include "cart.h"
#include "cart_internal.h"

namespace {

using namespace cart;

constexpr int kNaMaxCta = 256;                                  // persistent blocks used at most
constexpr int kNaMaxRowGroups = CART_STATIC_MAX_ROW_GROUPS;     // n_reqs * n_kv_heads
constexpr int kNaItemsCap = kNaMaxRowGroups + kNaMaxCta;
constexpr int kNaSlotsCap = 2 * kNaMaxCta;
constexpr int kNaMaxDevices = 64;

constexpr size_t kOffStatus = 0;
constexpr size_t kOffTickets = 256;
constexpr size_t kOffCtaBegin = kOffTickets + (size_t)kNaMaxCta * 4;
constexpr size_t kOffMerges = kOffCtaBegin + ((kNaMaxCta + 1) * 4 + 255) / 256 * 256;
constexpr size_t kOffItems = kOffMerges + (size_t)kNaMaxCta * sizeof(cart_merge_item);
constexpr size_t kOffPartO = kOffItems + (size_t)kNaItemsCap * sizeof(cart_work_item);
constexpr size_t kOffPartLse = kOffPartO + (size_t)kNaSlotsCap * kMaxGroup * kHeadDim * 4;
constexpr size_t kScratchBytes = kOffPartLse + (size_t)kNaSlotsCap * kMaxGroup * 4;
static_assert(kOffItems % 256 == 0 && kOffPartO % 256 == 0 && kOffPartLse % 256 == 0, "scratch regions are 256-byte aligned");
static_assert(kScratchBytes <= CART_STATIC_SCRATCH_BYTES, "the stated scratch size must cover the layout");

// The scratch itself.  Every GPU that loads the library holds these bytes until the process exits.
// In host code this name is only a handle for cudaGetSymbolAddress, never a device address.
static __device__ __align__(256) unsigned char g_static_scratch[CART_STATIC_SCRATCH_BYTES];

// Host copy of the plan region [cta_begin | merges | items] (what gets uploaded each call).
alignas(256) unsigned char g_host_plan[kOffPartO - kOffCtaBegin];

struct DeviceSetup {
    bool done = false;
    unsigned char *scratch = nullptr;  // device address of g_static_scratch on this device
    int n_cta = 0;
    void *encode_fn = nullptr;
};
DeviceSetup g_setup[kNaMaxDevices];

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Once per device, with that device current: resolve the scratch's device address, raise the decode
// kernel's shared-memory limit, look up the SM count and the tensor-map encoder.
cart_status setup_device(int device, DeviceSetup **out)
{
    DeviceSetup &s = g_setup[device];
    if (!s.done) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return CART_ERR_CUDA;
        if (prepare_kernels() != cudaSuccess) return CART_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 1)
            return CART_ERR_CUDA;
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
            !fn || qres != cudaDriverEntryPointSuccess)
            return CART_ERR_CUDA;
        s.scratch = static_cast<unsigned char *>(ptr);
        s.n_cta = sms < kNaMaxCta ? sms : kNaMaxCta;
        s.encode_fn = fn;
        s.done = true;
    }
    *out = &s;
    return CART_OK;
}

}  // namespace

extern "C" cart_status cart_decode_attention_static(const void *q, const void *kv, int32_t n_reqs, int32_t n_q_heads,
                                                    int32_t n_kv_heads, int32_t n_tokens, float softmax_scale,
                                                    void *out, float *lse, int32_t device, void *stream)
{
    if (!q || !kv || !out || (reinterpret_cast<uintptr_t>(q) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u) ||
        (reinterpret_cast<uintptr_t>(kv) & 255u) || (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)) ||
        n_reqs < 1 || n_tokens < 1 || !(softmax_scale >= 0.f) || device < 0 || device >= kNaMaxDevices)
        return CART_ERR_INVALID_ARG;
    if (n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads != 0 || n_q_heads / n_kv_heads > kMaxGroup)
        return CART_ERR_SHAPE;
    if ((int64_t)n_reqs * n_kv_heads > kNaMaxRowGroups) return CART_ERR_CAPACITY;  // beyond the fixed scratch
    const uint64_t rows_one = (uint64_t)n_reqs * n_kv_heads * (uint64_t)n_tokens;    // rows of K (and of V)
    if (2 * rows_one >= (1ull << 31)) return CART_ERR_CAPACITY;
    int current = -1;
    if (cudaGetDevice(&current) != cudaSuccess) return CART_ERR_CUDA;
    if (current != device) return CART_ERR_INVALID_ARG;  // set-up and launches need `device` current

    DeviceSetup *su = nullptr;
    cart_status st = setup_device(device, &su);
    if (st != CART_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);

    // The caller's buffer [K block | V block] as rows of 128 bf16; rows past its end read as zero.
    alignas(64) CUtensorMap tmap;
    const cuuint64_t gdim[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)(2 * rows_one)};
    const cuuint64_t gstride[1] = {(cuuint64_t)kRowBytes};
    const cuuint32_t box[2] = {64u, (cuuint32_t)kTileTokens};
    const cuuint32_t estride[2] = {1u, 1u};
    if (reinterpret_cast<EncodeFn>(su->encode_fn)(&tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(kv),
                                                  gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                  CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return CART_ERR_CUDA;

    // Plan: every request is one segment of n_tokens rows per KV head; built into the fixed host array.
    cart_plan_seg seg[CART_STATIC_MAX_ROW_GROUPS];
    int32_t seg_begin[CART_STATIC_MAX_ROW_GROUPS + 1];
    for (int32_t i = 0; i < n_reqs; ++i) {
        seg[i].k_row = (uint32_t)((uint64_t)i * n_kv_heads * (uint64_t)n_tokens);
        seg[i].v_row = (uint32_t)(rows_one + (uint64_t)i * n_kv_heads * (uint64_t)n_tokens);
        seg[i].head_stride = (uint32_t)n_tokens;
        seg[i].layer_stride = 0;
        seg[i].n_tok = (uint32_t)n_tokens;
        seg[i].flags = CART_SEG_SUFFIX;  // the caller's buffer: a kernel earlier on the stream may have written it
        seg_begin[i] = i;
    }
    seg_begin[n_reqs] = n_reqs;
    unsigned char *hp = g_host_plan;
    int32_t n_items = 0, n_merges = 0, n_cta_used = 0, n_slots = 0;
    int64_t total_tiles = 0;
    st = cart_plan_build(seg, seg_begin, n_reqs, n_kv_heads, su->n_cta, kTileTokens,
                         reinterpret_cast<cart_work_item *>(hp + (kOffItems - kOffCtaBegin)), kNaItemsCap, &n_items,
                         reinterpret_cast<uint32_t *>(hp), reinterpret_cast<cart_merge_item *>(hp + (kOffMerges - kOffCtaBegin)),
                         kNaMaxCta, &n_merges, &n_cta_used, &n_slots, &total_tiles);
    if (st != CART_OK) return st;
    if (n_slots > kNaSlotsCap) return CART_ERR_CAPACITY;

    // The scratch keeps the previous call's contents.  The status word and the arrival tickets must
    // start at zero; the plan region is overwritten here and every partial slot that is read is
    // written first.
    unsigned char *sc = su->scratch;
    if (cudaMemsetAsync(sc + kOffStatus, 0, kOffCtaBegin, s) != cudaSuccess) return CART_ERR_CUDA;
    const size_t plan_bytes = (kOffItems - kOffCtaBegin) + (size_t)n_items * sizeof(cart_work_item);
    if (cudaMemcpyAsync(sc + kOffCtaBegin, hp, plan_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return CART_ERR_CUDA;

    DecodeParams dp;
    dp.cta_begin = reinterpret_cast<const uint32_t *>(sc + kOffCtaBegin);
    dp.items = reinterpret_cast<const cart_work_item *>(sc + kOffItems);
    dp.q = q;
    dp.out = out;
    dp.lse = lse;
    dp.part_o = reinterpret_cast<float *>(sc + kOffPartO);
    dp.part_lse2 = reinterpret_cast<float *>(sc + kOffPartLse);
    dp.merges = reinterpret_cast<const cart_merge_item *>(sc + kOffMerges);
    dp.tickets = reinterpret_cast<uint32_t *>(sc + kOffTickets);
    dp.status = reinterpret_cast<uint32_t *>(sc + kOffStatus);
    dp.layer = 0;
    dp.group = n_q_heads / n_kv_heads;
    const float scale = softmax_scale > 0.f ? softmax_scale : 0.08838834764831845f;  // 1/sqrt(128)
    dp.scale_log2 = scale * 1.4426950408889634f;
    if (launch_decode(tmap, tmap, dp, n_cta_used, s) != cudaSuccess) return CART_ERR_CUDA;  // whole tiles only
    return CART_OK;
}
