// Shared device/host helpers of the GLANCE round library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "glance.h"

namespace glance {

typedef __nv_bfloat16 bf16;

constexpr int kPage = 64;        // tokens per KV page (one 64-key attention tile = one page)
constexpr int kMaxTreeN = 128;   // verify rows per sequence, root included
constexpr int kMaxTopk = 16;
constexpr int kMaxBlock = 16;

// Paged KV pool geometry: element (layer, page, kv, kv_head, slot, dim), row-major.
struct KvGeom {
    int n_pages, n_kv_heads, head_dim, max_pages_per_seq;
    __host__ __device__ size_t layer_stride() const {
        return (size_t)n_pages * 2 * n_kv_heads * kPage * head_dim;
    }
    // offset (in elements) of row `slot` of (page, kv, head) inside one layer
    __host__ __device__ size_t row(int page, int kv, int head, int slot) const {
        return ((((size_t)page * 2 + kv) * n_kv_heads + head) * kPage + slot) * head_dim;
    }
};

// Per-pass row bookkeeping written by the setup kernels and read by every later kernel of the pass.
struct RowMeta {
    int32_t *seq;     // [R] sequence of the row
    int32_t *pos;     // [R] rotary position, -1 for a padding row
    long long *kvrow; // [R] element offset of the row's K slot (kv head 0) inside a pool layer, -1 = none
    const double *inv_freq;  // [d/2] theta^(-2i/d), computed in double on the host
    float *rope_cos;  // [R][d/2]
    float *rope_sin;  // [R][d/2]
};

__device__ __forceinline__ void set_status(int32_t *status, int32_t code) {
    atomicCAS(status, 0, code);
}

// order-preserving map float -> uint32 (larger float -> larger key)
__device__ __forceinline__ uint32_t float_key(float f) {
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
    uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(u);
}
// (value desc, id asc) packed so that a plain unsigned max picks the winner
__device__ __forceinline__ unsigned long long pack_val_id(float v, int id) {
    return ((unsigned long long)float_key(v) << 32) | (uint32_t)(~(uint32_t)id);
}
__device__ __forceinline__ int unpack_id(unsigned long long k) { return (int)(~(uint32_t)(k & 0xffffffffu)); }
__device__ __forceinline__ float unpack_val(unsigned long long k) { return key_float((uint32_t)(k >> 32)); }

__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        unsigned long long w = __shfl_xor_sync(0xffffffffu, v, o);
        v = w > v ? w : v;
    }
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

}  // namespace glance
