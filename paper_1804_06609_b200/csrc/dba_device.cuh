// Small device helpers: ordering keys, logit loads, warp/block reductions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace dba {

constexpr unsigned kFullMask = 0xffffffffu;

// Programmatic dependent launch: the kernels of successive steps follow one another on a stream.  A kernel
// launched with launch_after() may start while its predecessor is still running; it must not touch what the
// predecessor produces (or still reads and this kernel writes) before grid_dependency_wait() returns, which
// is when the predecessor has finished and its writes are visible.  allow_dependents() lets the successor's
// blocks be scheduled as soon as there is room for them.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void allow_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float neg_inf() { return __int_as_float(0xff800000); }

// Monotone map float -> uint32 (larger float, larger integer).  -0.0 is folded onto +0.0 first so that
// the integer order agrees with floating-point comparison on equal values.
__device__ __forceinline__ uint32_t ord32(float x) {
    uint32_t u = __float_as_uint(x + 0.0f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float unord32(uint32_t o) {
    uint32_t u = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
    return __uint_as_float(u);
}
// Key of a row entry: larger key = better = (value descending, index ascending).
__device__ __forceinline__ uint64_t row_key(float x, int idx) {
    return ((uint64_t)ord32(x) << 32) | (uint32_t)(0xffffffffu - (uint32_t)idx);
}
__device__ __forceinline__ float row_key_val(uint64_t key) { return unord32((uint32_t)(key >> 32)); }
__device__ __forceinline__ int row_key_idx(uint64_t key) { return (int)(0xffffffffu - (uint32_t)key); }

template <typename T>
__device__ __forceinline__ float load_logit(const T* p);
template <>
__device__ __forceinline__ float load_logit<float>(const float* p) { return __ldg(p); }
template <>
__device__ __forceinline__ float load_logit<__nv_bfloat16>(const __nv_bfloat16* p) {
    return __uint_as_float(((uint32_t)__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
}
__device__ __forceinline__ float load_logit_dyn(const void* base, int dtype, int64_t i) {
    return dtype == 0 ? load_logit<float>((const float*)base + i)
                      : load_logit<__nv_bfloat16>((const __nv_bfloat16*)base + i);
}

// score(h, w) = fl32(fl32(x - lse) + parent): two separately rounded operations.
__device__ __forceinline__ float cell_score(float x, float lse, float parent) {
    return __fadd_rn(__fsub_rn(x, lse), parent);
}

// "a better than b" for beam cells: higher score first, then lower flat index.
__device__ __forceinline__ bool cell_better(float sa, int fa, float sb, int fb) {
    return sa > sb || (sa == sb && fa < fb);
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFullMask, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {   // fixed butterfly: same result on every lane
#pragma unroll
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(kFullMask, v, o);
    return v;
}
__device__ __forceinline__ uint64_t warp_max_u64(uint64_t v) {
#pragma unroll
    for (int o = 16; o; o >>= 1) {
        uint64_t t = __shfl_xor_sync(kFullMask, v, o);
        v = t > v ? t : v;
    }
    return v;
}

}  // namespace dba
