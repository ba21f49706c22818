// Shared device/host helpers of the CMPQ CUDA library (sm_100a).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cmpq.h"

namespace cmpq {

// Exact widening of a 16-bit storage pattern to fp32.
template <int DT>
__device__ __forceinline__ float widen16(uint16_t h) {
    if (DT == CMPQ_BF16) {
        return __uint_as_float(static_cast<uint32_t>(h) << 16);
    } else {
        return __half2float(__ushort_as_half(h));
    }
}

// Two packed 16-bit values (little endian: .x is the low half) to two floats.
template <int DT>
__device__ __forceinline__ float2 widen16x2(uint32_t w) {
    if (DT == CMPQ_BF16) {
        return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    } else {
        __half2 h = *reinterpret_cast<__half2*>(&w);
        return __half22float2(h);
    }
}

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Number of SMs of the current device (queried once per device and cached).
int sm_count();

// Raises a kernel's dynamic shared-memory limit to `bytes` once per device (the limit is an upper bound, so
// callers pass the largest amount any launch of the kernel can ask for); later calls on the same device return
// at once.  `done` is the caller's flag array for this kernel, one entry per device.
template <class Kernel>
inline bool raise_smem_limit_once(Kernel kern, size_t bytes, bool (&done)[64]) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (dev >= 0 && dev < 64 && done[dev]) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return false;
    if (dev >= 0 && dev < 64) done[dev] = true;
    return true;
}

// Converts the last CUDA launch error into a status.
inline cmpq_status launch_status() {
    return cudaGetLastError() == cudaSuccess ? CMPQ_OK : CMPQ_ERR_CUDA;
}

// Bump allocator over the caller's workspace (256-byte granules).
struct Workspace {
    char* base;
    size_t size;
    size_t used;
    Workspace(void* p, size_t n) : base(static_cast<char*>(p)), size(n), used(0) {}
    template <typename T>
    T* take(size_t count) {
        size_t bytes = round_up(count * sizeof(T), 256);
        T* out = reinterpret_cast<T*>(base + used);
        used += bytes;
        return out;
    }
    bool ok() const { return used <= size; }
};

// Work-space layouts, shared by cmpq_workspace_bytes and the entry points.
size_t stats_ws_bytes(int64_t d_in);
size_t alloc_ws_bytes(int64_t d_in);
size_t outliers_ws_bytes(int64_t d_in, int64_t d_out);
size_t quantize_ws_bytes(int64_t d_in, int64_t d_out);
size_t pack_ws_bytes(int64_t d_in, int64_t d_out);
size_t protect_quantize_ws_bytes(int64_t d_in, int64_t d_out);
size_t quantize_packed_ws_bytes(int64_t d_in, int64_t d_out);
size_t protect_quantize_pack_ws_bytes(int64_t d_in, int64_t d_out);
size_t matvec_ws_bytes(int64_t d_in, int64_t d_out);
size_t by_column_ws_bytes(int64_t d_out);

}  // namespace cmpq
