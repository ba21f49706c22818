// Stored formats of the per-channel look-up tables (Section 5.1, memory usage: the tables are kept
// in FP16 -- 16 bits per centroid, about 0.03 bit per weight at 4096 weights per channel -- and a
// variant keeps 4 bits per centroid, below 0.01 bit per weight).
//
// FP16: round to nearest even.  4 bit: the uniform quantizer of Section 3 with N = 4 over the K
// centroids of a channel, between the channel's smallest and largest centroid (each rounded to FP16
// and stored with the codes); every step is a single fp32 operation, nothing is fused.
// One thread per channel: the tables are 64 bytes per channel, the work is negligible.
#include "common.cuh"

namespace cmpq {

__device__ __forceinline__ float half_bits_to_float(uint16_t h) { return __half2float(__ushort_as_half(h)); }

__global__ void lut_store_f16_kernel(const float* __restrict__ lut, const uint8_t* __restrict__ bits, int64_t d_in,
                                     uint16_t* __restrict__ out) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= d_in * CMPQ_LUT_STRIDE) return;
    const int64_t i = t / CMPQ_LUT_STRIDE;
    const int k = (int)(t % CMPQ_LUT_STRIDE);
    const int c = bits[i];
    const int K = c == 2 ? 4 : (c == 3 ? 8 : 16);
    out[t] = k < K ? __half_as_ushort(__float2half_rn(lut[t])) : (uint16_t)0;
}

__global__ void lut_load_f16_kernel(const uint16_t* __restrict__ in, int64_t n, float* __restrict__ lut) {
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < n) lut[t] = half_bits_to_float(in[t]);
}

__global__ void lut_store_u4_kernel(const float* __restrict__ lut, const uint8_t* __restrict__ bits, int64_t d_in,
                                    uint8_t* __restrict__ out) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= d_in) return;
    const int c = bits[i];
    const int K = c == 2 ? 4 : (c == 3 ? 8 : 16);
    float v[16];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float4 f = reinterpret_cast<const float4*>(lut + i * CMPQ_LUT_STRIDE)[q];
        v[4 * q] = f.x; v[4 * q + 1] = f.y; v[4 * q + 2] = f.z; v[4 * q + 3] = f.w;
    }
    float lo = v[0], hi = v[0];
#pragma unroll
    for (int k = 1; k < 16; ++k) {
        if (k < K) {
            if (v[k] < lo) lo = v[k];
            if (v[k] > hi) hi = v[k];
        }
    }
    const uint16_t lo16 = __half_as_ushort(__float2half_rn(lo)), hi16 = __half_as_ushort(__float2half_rn(hi));
    const float flo = half_bits_to_float(lo16), fhi = half_bits_to_float(hi16);
    const float D = __fdiv_rn(__fsub_rn(fhi, flo), 15.0f);
    uint32_t w0 = 0, w1 = 0;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        uint32_t code = 0;
        if (k < K && D > 0.0f) {
            const float r = rintf(__fdiv_rn(__fsub_rn(v[k], flo), D));  // half to even
            code = r < 0.0f ? 0u : (r > 15.0f ? 15u : (uint32_t)r);
        }
        if (k < 8) w0 |= code << (4 * k); else w1 |= code << (4 * (k - 8));
    }
    uint32_t* o = reinterpret_cast<uint32_t*>(out + i * CMPQ_LUT_U4_BYTES);  // 12 bytes per channel: word aligned
    o[0] = w0;
    o[1] = w1;
    o[2] = (uint32_t)lo16 | ((uint32_t)hi16 << 16);
}

__global__ void lut_load_u4_kernel(const uint8_t* __restrict__ in, const uint8_t* __restrict__ bits, int64_t d_in,
                                   float* __restrict__ lut) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= d_in) return;
    const int c = bits[i];
    const int K = c == 2 ? 4 : (c == 3 ? 8 : 16);
    const uint32_t* o = reinterpret_cast<const uint32_t*>(in + i * CMPQ_LUT_U4_BYTES);
    const uint32_t w0 = o[0], w1 = o[1], ends = o[2];
    const float flo = half_bits_to_float((uint16_t)(ends & 0xffffu)), fhi = half_bits_to_float((uint16_t)(ends >> 16));
    const float D = __fdiv_rn(__fsub_rn(fhi, flo), 15.0f);
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        const uint32_t code = ((k < 8 ? w0 >> (4 * k) : w1 >> (4 * (k - 8)))) & 15u;
        lut[i * CMPQ_LUT_STRIDE + k] = k < K ? __fadd_rn(flo, __fmul_rn((float)code, D)) : 0.0f;
    }
}

}  // namespace cmpq

using namespace cmpq;

extern "C" size_t cmpq_lut_bytes(cmpq_lut_format fmt, int64_t d_in) {
    if (d_in < 1 || d_in > CMPQ_MAX_D_IN) return 0;
    switch (fmt) {
        case CMPQ_LUT_F32: return (size_t)d_in * CMPQ_LUT_STRIDE * 4;
        case CMPQ_LUT_F16: return (size_t)d_in * CMPQ_LUT_STRIDE * 2;
        case CMPQ_LUT_U4: return (size_t)d_in * CMPQ_LUT_U4_BYTES;
    }
    return 0;
}

extern "C" cmpq_status cmpq_store_lut(const float* lut, const uint8_t* bits, int64_t d_in, cmpq_lut_format fmt,
                                      void* stored, void* stream) {
    if (!lut || !bits || !stored || d_in < 1 || d_in > CMPQ_MAX_D_IN) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(lut, 16) || !aligned_to(stored, 4)) return CMPQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t n = d_in * CMPQ_LUT_STRIDE;
    if (fmt == CMPQ_LUT_F16)
        lut_store_f16_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(lut, bits, d_in, static_cast<uint16_t*>(stored));
    else if (fmt == CMPQ_LUT_U4)
        lut_store_u4_kernel<<<(unsigned)((d_in + 127) / 128), 128, 0, st>>>(lut, bits, d_in, static_cast<uint8_t*>(stored));
    else
        return CMPQ_ERR_INVALID_ARG;
    return launch_status();
}

extern "C" cmpq_status cmpq_load_lut(const void* stored, cmpq_lut_format fmt, const uint8_t* bits, int64_t d_in,
                                     float* lut, void* stream) {
    if (!stored || !bits || !lut || d_in < 1 || d_in > CMPQ_MAX_D_IN) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(lut, 4) || !aligned_to(stored, 4)) return CMPQ_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t n = d_in * CMPQ_LUT_STRIDE;
    if (fmt == CMPQ_LUT_F16)
        lut_load_f16_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(static_cast<const uint16_t*>(stored), n, lut);
    else if (fmt == CMPQ_LUT_U4)
        lut_load_u4_kernel<<<(unsigned)((d_in + 127) / 128), 128, 0, st>>>(static_cast<const uint8_t*>(stored), bits, d_in, lut);
    else
        return CMPQ_ERR_INVALID_ARG;
    return launch_status();
}

extern "C" double cmpq_table_bits_per_weight(const uint8_t* bits_host, int64_t d_in, int64_t d_out, cmpq_lut_format fmt,
                                             int count_grid_ends) {
    if (!bits_host || d_in < 1 || d_out < 1) return 0.0;
    const double per_centroid = fmt == CMPQ_LUT_F32 ? 32.0 : (fmt == CMPQ_LUT_F16 ? 16.0 : 4.0);
    double total = 0.0;
    for (int64_t i = 0; i < d_in; ++i) {
        const int c = bits_host[i];
        const int K = c == 2 ? 4 : (c == 3 ? 8 : 16);
        total += 4.0 + K * per_centroid + ((fmt == CMPQ_LUT_U4 && count_grid_ends) ? 32.0 : 0.0);
    }
    return total / ((double)d_in * (double)d_out);
}
