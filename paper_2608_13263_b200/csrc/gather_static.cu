// vtoken_gather_logical_noalloc: the logical gather for callers that must not allocate.
//
// Same kernels as vtoken_gather_logical; the only difference is where the scratch lives: a
// fixed array in this library's device image instead of buffers from vtoken_create.  The
// array exists once per GPU that loads the library, is shared by every call and keeps the
// previous call's contents, so the words that must start at zero are cleared on the stream
// at the top of each call.
#include <mutex>

#include <cstring>

#include "common.cuh"

namespace {

constexpr int32_t NOALLOC_MAX_REQUESTS = 4096;
constexpr int64_t NOALLOC_MAX_TOKENS = 262144;

// layout: [0,256) counts + row total | live counts per request part | source slot of each output row
constexpr size_t OFF_COUNTS = 0;
constexpr size_t OFF_TOTAL = 64;
constexpr size_t OFF_REQ_N = 256;
constexpr size_t OFF_SRC = OFF_REQ_N + sizeof(int32_t) * NOALLOC_MAX_REQUESTS * VTK_PLAN_PARTS;
constexpr size_t SCRATCH_BYTES = OFF_SRC + sizeof(int32_t) * NOALLOC_MAX_TOKENS;

}  // namespace

static __device__ __align__(256) unsigned char vtk_noalloc_scratch[SCRATCH_BYTES];

namespace {

// Per-device set-up.  In host code the array's name above is only a handle for the runtime,
// not an address a kernel can use; the device address is asked for once per device (with
// that device current) and kept here.
constexpr int MAX_DEVICES = 64;
struct DeviceSlot {
    bool ready;
    unsigned char *scratch;   // device address of vtk_noalloc_scratch on this device
    int num_sms;
};
DeviceSlot g_slots[MAX_DEVICES];
std::mutex g_slots_mutex;

int device_slot(DeviceSlot **out, int *cuda_err)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) { *cuda_err = (int)e; return VTOKEN_ECUDA; }
    if (dev < 0 || dev >= MAX_DEVICES) return VTOKEN_EINVAL;
    std::lock_guard<std::mutex> lock(g_slots_mutex);
    DeviceSlot &s = g_slots[dev];
    if (!s.ready) {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, vtk_noalloc_scratch);
        if (e != cudaSuccess || p == nullptr) { *cuda_err = (int)e; return VTOKEN_ECUDA; }
        int sms = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) { *cuda_err = (int)e; return VTOKEN_ECUDA; }
        s.scratch = (unsigned char *)p;
        s.num_sms = sms;
        s.ready = true;
    }
    *out = &s;
    return VTOKEN_OK;
}

}  // namespace

extern "C" int vtoken_gather_logical_noalloc(const void *k_pool, const void *v_pool, int32_t num_layers,
                                             int32_t num_blocks, int32_t block_size, int64_t row_bytes,
                                             int64_t layer_stride_bytes, const int32_t *num_requests,
                                             int32_t max_requests, const int32_t *tt_offsets,
                                             const int32_t *tt_slots, const uint8_t *keep, const uint8_t *select,
                                             int32_t layer_begin, int32_t layer_end, void *out_k, void *out_v,
                                             int64_t out_capacity_tokens, int32_t *out_offsets,
                                             uint32_t *error_flags, void *cuda_stream)
{
    if (!k_pool || !v_pool || !num_requests || !tt_offsets || !tt_slots || !out_k || !out_v || !out_offsets)
        return VTOKEN_EINVAL;
    if (num_layers < 1 || num_blocks < 1 || block_size < 1 || row_bytes < 16 || row_bytes % 16 != 0) return VTOKEN_EINVAL;
    if (layer_begin < 0 || layer_end > num_layers || layer_begin >= layer_end) return VTOKEN_EINVAL;
    if (max_requests < 1 || out_capacity_tokens < 0) return VTOKEN_EINVAL;
    const int64_t slots = (int64_t)num_blocks * block_size;
    if (slots >= (int64_t)INT32_MAX) return VTOKEN_EINVAL;
    const int64_t stride = layer_stride_bytes ? layer_stride_bytes : slots * row_bytes;
    if (stride < slots * row_bytes || stride % 16 != 0) return VTOKEN_EINVAL;
    if (((uintptr_t)k_pool | (uintptr_t)v_pool | (uintptr_t)out_k | (uintptr_t)out_v) & 15) return VTOKEN_EINVAL;
    // the fixed scratch bounds the problem: say so instead of overrunning it
    if (max_requests > NOALLOC_MAX_REQUESTS || out_capacity_tokens > NOALLOC_MAX_TOKENS) return VTOKEN_ECAPACITY;

    DeviceSlot *slot = nullptr;
    int cuda_err = 0;
    int rc = device_slot(&slot, &cuda_err);
    if (rc != VTOKEN_OK) return rc;

    // a context that lives on this stack frame and points into the fixed scratch
    vtoken_ctx ctx;
    memset(&ctx, 0, sizeof(ctx));
    ctx.cfg.num_layers = num_layers;
    ctx.cfg.num_blocks = num_blocks;
    ctx.cfg.block_size = block_size;
    ctx.cfg.k_pool = const_cast<void *>(k_pool);
    ctx.cfg.v_pool = const_cast<void *>(v_pool);
    ctx.cfg.max_requests = max_requests;
    ctx.cfg.max_tokens = NOALLOC_MAX_TOKENS;
    ctx.row_bytes = row_bytes;
    ctx.layer_stride = stride;
    ctx.slots_per_layer = slots;
    ctx.num_sms = slot->num_sms;
    ctx.counts = reinterpret_cast<vtoken_counts *>(slot->scratch + OFF_COUNTS);
    ctx.rt_counts = ctx.counts;
    ctx.g_total = reinterpret_cast<int32_t *>(slot->scratch + OFF_TOTAL);
    ctx.part_n = reinterpret_cast<int32_t *>(slot->scratch + OFF_REQ_N);
    ctx.g_src = reinterpret_cast<int32_t *>(slot->scratch + OFF_SRC);

    cudaStream_t st = (cudaStream_t)cuda_stream;
    // flags and the row total are accumulated by the kernels: they must start at zero
    if (cudaMemsetAsync(slot->scratch, 0, OFF_REQ_N, st) != cudaSuccess) return VTOKEN_ECUDA;
    rc = vtk_launch_gather(&ctx, num_requests, tt_offsets, tt_slots, keep, select, layer_begin, layer_end, out_k,
                           out_v, out_capacity_tokens, out_offsets, st);
    if (rc != VTOKEN_OK) return rc;
    if (error_flags) {
        if (cudaMemcpyAsync(error_flags, &ctx.rt_counts->error_flags, sizeof(uint32_t), cudaMemcpyDeviceToDevice, st) !=
            cudaSuccess)
            return VTOKEN_ECUDA;
    }
    return VTOKEN_OK;
}
