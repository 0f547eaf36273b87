// Harness kernels (separate library, not part of the repack path): the deterministic K/V pool
// fill, a whole-pool verifier against an origin map, and a bandwidth-bound decode-read proxy.
//
// The fill is the counter-based generator documented in the workloads module:
//   counter = ((kv * L + layer) * slots_per_layer + slot) * row_elems + elem
//   h = splitmix64(counter + seed * GOLDEN);  s = sum of the four 16-bit fields of h
//   value = bf16_rne(float(s - 131070) * FILL_SCALE)
// Integer arithmetic, one exact int->float conversion and one float multiply: bit-identical
// to the numpy implementation.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ uint64_t splitmix64(uint64_t x)
{
    x += 0x9E3779B97F4A7C15ull;
    x ^= x >> 30;
    x *= 0xBF58476D1CE4E5B9ull;
    x ^= x >> 27;
    x *= 0x94D049BB133111EBull;
    x ^= x >> 31;
    return x;
}

__device__ __forceinline__ uint16_t fill_value(uint64_t counter, uint64_t seed)
{
    const uint64_t h = splitmix64(counter + seed * 0x9E3779B97F4A7C15ull);
    const int s = (int)(h & 0xFFFF) + (int)((h >> 16) & 0xFFFF) + (int)((h >> 32) & 0xFFFF) + (int)(h >> 48);
    const float x = __fmul_rn((float)(s - 131070), __uint_as_float(0x37ddb3d7u));   // FILL_SCALE
    const uint32_t bits = __float_as_uint(x);
    return (uint16_t)((bits + 0x7FFFu + ((bits >> 16) & 1u)) >> 16);
}

// 8 elements (16 bytes) per thread
__global__ void fill_kernel(uint8_t *pool, int kv, int L, int layer_begin, int layer_end, int64_t slots_per_layer,
                            int row_elems, int64_t layer_stride, uint64_t seed)
{
    const int64_t vec_per_layer = slots_per_layer * row_elems / 8;
    const int64_t total = vec_per_layer * (layer_end - layer_begin);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int layer = layer_begin + (int)(i / vec_per_layer);
        const int64_t e0 = (i % vec_per_layer) * 8;
        const uint64_t c0 = ((uint64_t)(kv * L + layer) * (uint64_t)slots_per_layer) * (uint64_t)row_elems + (uint64_t)e0;
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k)
            w[k] = (uint32_t)fill_value(c0 + 2 * k, seed) | ((uint32_t)fill_value(c0 + 2 * k + 1, seed) << 16);
        *reinterpret_cast<uint4 *>(pool + (int64_t)(layer - layer_begin) * layer_stride + e0 * 2) =
            make_uint4(w[0], w[1], w[2], w[3]);
    }
}

// Address-encoding fill (a debugging aid): every 8 bytes of a row say where the row was filled --
// low word = slot, high word = pool (bit 31), layer (bits 16..30), index of the 8-byte group in the row
// (bits 0..15) -- so that a row found in the wrong place names the place it came from.
__global__ void fill_address_kernel(uint8_t *pool, int kv, int layer_begin, int layer_end, int64_t slots_per_layer,
                                    int row_elems, int64_t layer_stride)
{
    const int groups = row_elems / 4;                     // 8-byte groups per row
    const int64_t per_layer = slots_per_layer * groups;
    const int64_t total = per_layer * (layer_end - layer_begin);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int layer = layer_begin + (int)(i / per_layer);
        const int64_t r = i % per_layer;
        const uint32_t slot = (uint32_t)(r / groups), g = (uint32_t)(r % groups);
        const uint32_t hi = ((uint32_t)kv << 31) | ((uint32_t)layer << 16) | g;
        *reinterpret_cast<uint2 *>(pool + (int64_t)(layer - layer_begin) * layer_stride + r * 8) = make_uint2(slot, hi);
    }
}

// Every slot s of every layer must hold the fill of slot origin[s] (origin[s] == s: untouched).
__global__ void verify_kernel(const uint8_t *pool, int kv, int L, int64_t slots_per_layer, int row_elems,
                              int64_t layer_stride, uint64_t seed, const int32_t *origin,
                              unsigned long long *mismatches)
{
    const int vec_per_row = row_elems / 8;
    const int64_t vec_per_layer = slots_per_layer * vec_per_row;
    const int64_t total = vec_per_layer * L;
    unsigned long long bad = 0;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (int64_t)gridDim.x * blockDim.x) {
        const int layer = (int)(i / vec_per_layer);
        const int64_t r = i % vec_per_layer;
        const int64_t slot = r / vec_per_row;
        const int e0 = (int)(r % vec_per_row) * 8;
        const int64_t from = origin[slot];
        const uint64_t c0 = ((uint64_t)(kv * L + layer) * (uint64_t)slots_per_layer + (uint64_t)from) * (uint64_t)row_elems + (uint64_t)e0;
        const uint4 got = *reinterpret_cast<const uint4 *>(pool + (int64_t)layer * layer_stride + (slot * row_elems + e0) * 2);
        const uint32_t g[4] = {got.x, got.y, got.z, got.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t want = (uint32_t)fill_value(c0 + 2 * k, seed) | ((uint32_t)fill_value(c0 + 2 * k + 1, seed) << 16);
            bad += (want != g[k]);
        }
    }
    for (int d = 16; d > 0; d >>= 1) bad += __shfl_down_sync(0xffffffffu, bad, d);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(mismatches, bad);
}

// Decode-read proxy: reads every allocated block of every request through the block tables,
// K and V, all layers, and XOR-folds each request's bytes into a 64-bit checksum.  Work item
// = (request block entry, pool, layer); one CTA per item at a time, persistent grid.
__global__ void __launch_bounds__(256) decode_read_kernel(const uint8_t *k_pool, const uint8_t *v_pool,
                                                          const int32_t *bt_offsets, const int32_t *bt_blocks,
                                                          const int32_t *bt_owner, int32_t total_blocks, int L,
                                                          int64_t block_bytes, int64_t layer_stride,
                                                          unsigned long long *checksums)
{
    const int64_t items = (int64_t)total_blocks * 2 * L;
    const int vecs = (int)(block_bytes / 16);
    for (int64_t it = blockIdx.x; it < items; it += gridDim.x) {
        const int slab = (int)(it / total_blocks);            // slab-major like the repack
        const int e = (int)(it % total_blocks);
        const uint8_t *pool = slab < L ? k_pool : v_pool;
        const int layer = slab < L ? slab : slab - L;
        const uint4 *p = reinterpret_cast<const uint4 *>(pool + (int64_t)layer * layer_stride + (int64_t)bt_blocks[e] * block_bytes);
        unsigned long long x = 0;
        for (int c = threadIdx.x; c < vecs; c += 256 * 4) {
            uint4 v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) v[k] = (c + 256 * k < vecs) ? __ldcs(p + c + 256 * k) : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int k = 0; k < 4; ++k)
                x ^= ((unsigned long long)(v[k].x ^ v[k].z) << 32) | (unsigned long long)(v[k].y ^ v[k].w);
        }
        for (int d = 16; d > 0; d >>= 1) x ^= __shfl_down_sync(0xffffffffu, x, d);
        if ((threadIdx.x & 31) == 0 && x) atomicXor(&checksums[bt_owner[e]], x);
    }
}

// SMs of the current device (queried once per process and device; grids are multiples of it)
int sm_count()
{
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 1;
        cached[dev] = n;
    }
    return cached[dev];
}

}  // namespace

extern "C" {

// Fills layers [layer_begin, layer_end) of pool kv (0 = K, 1 = V).  `dst` points at the first
// filled layer (so a single slab can be regenerated into a scratch buffer).  DEVICE memory.
int vth_fill(void *dst, int kv, int num_layers, int layer_begin, int layer_end, int64_t slots_per_layer,
             int row_elems, int64_t layer_stride_bytes, uint64_t seed, void *stream)
{
    if (!dst || row_elems % 8 != 0 || layer_begin < 0 || layer_end > num_layers || layer_begin >= layer_end) return -1;
    if (layer_stride_bytes == 0) layer_stride_bytes = slots_per_layer * row_elems * 2;
    fill_kernel<<<sm_count() * 16, 256, 0, (cudaStream_t)stream>>>((uint8_t *)dst, kv, num_layers, layer_begin, layer_end,
                                                            slots_per_layer, row_elems, layer_stride_bytes, seed);
    return cudaGetLastError() == cudaSuccess ? 0 : -3;
}

// Address-encoding fill of layers [layer_begin, layer_end) of pool kv; row_elems a multiple of 4, at most
// 65536 groups per row and 32768 layers.
int vth_fill_address(void *dst, int kv, int num_layers, int layer_begin, int layer_end, int64_t slots_per_layer,
                     int row_elems, int64_t layer_stride_bytes, void *stream)
{
    if (!dst || row_elems % 4 != 0 || row_elems / 4 > 65536 || num_layers > 32768 || layer_begin < 0 ||
        layer_end > num_layers || layer_begin >= layer_end)
        return -1;
    if (layer_stride_bytes == 0) layer_stride_bytes = slots_per_layer * row_elems * 2;
    fill_address_kernel<<<sm_count() * 16, 256, 0, (cudaStream_t)stream>>>((uint8_t *)dst, kv, layer_begin, layer_end,
                                                                        slots_per_layer, row_elems, layer_stride_bytes);
    return cudaGetLastError() == cudaSuccess ? 0 : -3;
}

// Adds to *mismatches (DEVICE, zeroed by the caller) the number of 32-bit words of pool kv that
// differ from fill(origin[slot]).  origin: DEVICE int32 [slots_per_layer].
int vth_verify(const void *pool, int kv, int num_layers, int64_t slots_per_layer, int row_elems,
               int64_t layer_stride_bytes, uint64_t seed, const int32_t *origin, uint64_t *mismatches, void *stream)
{
    if (!pool || !origin || !mismatches || row_elems % 8 != 0) return -1;
    if (layer_stride_bytes == 0) layer_stride_bytes = slots_per_layer * row_elems * 2;
    verify_kernel<<<sm_count() * 16, 256, 0, (cudaStream_t)stream>>>((const uint8_t *)pool, kv, num_layers, slots_per_layer,
                                                              row_elems, layer_stride_bytes, seed, origin,
                                                              (unsigned long long *)mismatches);
    return cudaGetLastError() == cudaSuccess ? 0 : -3;
}

// bt_owner: DEVICE int32 [total_blocks], request index of each block-table entry.
// checksums: DEVICE uint64 [R], zeroed by the caller.
int vth_decode_read(const void *k_pool, const void *v_pool, const int32_t *bt_offsets, const int32_t *bt_blocks,
                    const int32_t *bt_owner, int32_t total_blocks, int num_layers, int64_t block_bytes,
                    int64_t layer_stride_bytes, uint64_t *checksums, int ctas, void *stream)
{
    if (!k_pool || !v_pool || !bt_blocks || !bt_owner || !checksums || block_bytes % 16 != 0) return -1;
    if (ctas <= 0) ctas = sm_count() * 8;
    decode_read_kernel<<<ctas, 256, 0, (cudaStream_t)stream>>>((const uint8_t *)k_pool, (const uint8_t *)v_pool,
                                                               bt_offsets, bt_blocks, bt_owner, total_blocks, num_layers,
                                                               block_bytes, layer_stride_bytes,
                                                               (unsigned long long *)checksums);
    return cudaGetLastError() == cudaSuccess ? 0 : -3;
}

}  // extern "C"
