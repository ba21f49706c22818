// Bit-packing of CMPQ codes (storage accounting of Section 5.1; the inference scheme of
// Section 6 multiplies one sub-matrix per precision, hence channels are grouped by bit width).
//
// HBM-bound: one byte read and bits/8 bytes written per weight.  A thread turns 32 codes
// (two 128-bit loads) into 2, 3 or 4 consecutive 32-bit words, so a warp reads 1 KiB and writes
// a contiguous 256 to 512 bytes.  Every channel of a segment has the same length in words, so
// its offset is segment base + (number of earlier channels of that width) * words.
#include "common.cuh"

namespace cmpq {

constexpr int kPackThreads = 256;

size_t pack_ws_bytes(int64_t d_in, int64_t) {
    return round_up((size_t)d_in * sizeof(int64_t), 256);
}

// Single block: segment sizes, perm, row_off (segment order) and word_off (by channel id).
__global__ void __launch_bounds__(1024)
pack_layout_kernel(const uint8_t* __restrict__ bits, int64_t d_in, int64_t d_out,
                   int64_t* __restrict__ row_off, int32_t* __restrict__ perm,
                   int64_t* __restrict__ seg_rows, int64_t* __restrict__ word_off) {
    __shared__ int warp_tot[3][32];
    __shared__ long long seg_count[3];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    // pass 1: channels per width
    long long cnt[3] = {0, 0, 0};
    for (int64_t i = threadIdx.x; i < d_in; i += blockDim.x) {
        int c = bits[i];
        cnt[0] += c == 2; cnt[1] += c == 3; cnt[2] += c == 4;
    }
    if (threadIdx.x < 3) seg_count[threadIdx.x] = 0;
    __syncthreads();
#pragma unroll
    for (int s = 0; s < 3; ++s) {
        long long v = cnt[s];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0 && v) atomicAdd((unsigned long long*)&seg_count[s], (unsigned long long)v);
    }
    __syncthreads();
    long long words[3], seg_base[3], seg_word_base[3];
    long long rb = 0, wb = 0;
#pragma unroll
    for (int s = 0; s < 3; ++s) {
        words[s] = (d_out * (s + 2) + 31) / 32;
        seg_base[s] = rb;
        seg_word_base[s] = wb;
        rb += seg_count[s];
        wb += seg_count[s] * words[s];
    }
    if (threadIdx.x < 3) seg_rows[threadIdx.x] = seg_count[threadIdx.x];
    if (threadIdx.x == 0) row_off[d_in] = wb;
    // pass 2: position of every channel among the channels of its width (ascending id)
    long long seen[3] = {0, 0, 0};
    for (int64_t base = 0; base < d_in; base += blockDim.x) {
        int64_t i = base + threadIdx.x;
        int c = i < d_in ? bits[i] : 0;
        int excl[3];
        __syncthreads();
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            unsigned m = __ballot_sync(0xffffffffu, c == s + 2);
            excl[s] = __popc(m & ((1u << lane) - 1));
            if (lane == 0) warp_tot[s][warp] = __popc(m);
        }
        __syncthreads();
        long long tot[3] = {0, 0, 0};
#pragma unroll
        for (int s = 0; s < 3; ++s) {
            int before = 0, all = 0;
            for (int w = 0; w < nwarps; ++w) {
                int t = warp_tot[s][w];
                if (w < warp) before += t;
                all += t;
            }
            excl[s] += before;
            tot[s] = all;
        }
        if (i < d_in && c >= 2 && c <= 4) {
            int s = c - 2;
            long long pos = seen[s] + excl[s];
            long long r = seg_base[s] + pos;
            long long off = seg_word_base[s] + pos * words[s];
            perm[r] = (int32_t)i;
            row_off[r] = off;
            word_off[i] = off;
        }
#pragma unroll
        for (int s = 0; s < 3; ++s) seen[s] += tot[s];
    }
}

// One thread packs 32 consecutive codes of one channel.
__global__ void __launch_bounds__(kPackThreads)
pack_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ bits, int64_t d_out,
            const int64_t* __restrict__ word_off, uint32_t* __restrict__ packed, int vec_ok) {
    const int64_t row = blockIdx.x;
    const int64_t g = (int64_t)blockIdx.y * blockDim.x + threadIdx.x;  // group of 32 codes
    const int64_t j0 = g * 32;
    if (j0 >= d_out) return;
    const int c = bits[row];
    const uint8_t* src = codes + row * d_out + j0;
    const int cnt = (int)min((int64_t)32, d_out - j0);
    uint32_t b[8];  // 32 code bytes, little endian
    if (vec_ok && cnt == 32) {
        uint4 v0 = __ldcs(reinterpret_cast<const uint4*>(src));
        uint4 v1 = __ldcs(reinterpret_cast<const uint4*>(src) + 1);
        b[0] = v0.x; b[1] = v0.y; b[2] = v0.z; b[3] = v0.w;
        b[4] = v1.x; b[5] = v1.y; b[6] = v1.z; b[7] = v1.w;
    } else {
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            uint32_t w = 0;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                int j = q * 4 + t;
                if (j < cnt) w |= (uint32_t)src[j] << (8 * t);
            }
            b[q] = w;
        }
    }
    // 128-bit little-endian bit stream of the 32 codes, c bits each
    unsigned long long lo = 0, hi = 0;
    const uint32_t cmask = (1u << c) - 1u;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        unsigned long long code = (b[j >> 2] >> (8 * (j & 3))) & cmask;
        int pos = j * c;
        if (pos < 64) {
            lo |= code << pos;
            if (pos + c > 64) hi |= code >> (64 - pos);
        } else {
            hi |= code << (pos - 64);
        }
    }
    uint32_t* dst = packed + word_off[row] + g * c;
    const int nwords = (cnt * c + 31) / 32;
    uint32_t w[4] = {(uint32_t)lo, (uint32_t)(lo >> 32), (uint32_t)hi, (uint32_t)(hi >> 32)};
#pragma unroll
    for (int t = 0; t < 4; ++t)
        if (t < nwords) dst[t] = w[t];
}

}  // namespace cmpq

using namespace cmpq;

extern "C" int64_t cmpq_packed_words(const uint8_t* bits_host, int64_t d_in, int64_t d_out) {
    int64_t words = 0;
    if (!bits_host) return 0;
    for (int64_t i = 0; i < d_in; ++i) words += (d_out * bits_host[i] + 31) / 32;
    return words;
}

extern "C" cmpq_status cmpq_pack(const uint8_t* codes, const uint8_t* bits, int64_t d_in, int64_t d_out,
                                 uint32_t* packed, int64_t* row_off, int32_t* perm, int64_t* seg_rows,
                                 void* ws, size_t ws_bytes, void* stream) {
    if (!codes || !bits || !packed || !row_off || !perm || !seg_rows) return CMPQ_ERR_INVALID_ARG;
    if (d_in < 1 || d_in > CMPQ_MAX_D_IN || d_out < 1 || d_out > CMPQ_MAX_D_OUT) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(packed, 4) || !aligned_to(row_off, 8) || !aligned_to(perm, 4) || !aligned_to(seg_rows, 8))
        return CMPQ_ERR_INVALID_ARG;
    if (!ws || !aligned_to(ws, 256) || ws_bytes < pack_ws_bytes(d_in, d_out)) return CMPQ_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int64_t* word_off = static_cast<int64_t*>(ws);
    pack_layout_kernel<<<1, 1024, 0, st>>>(bits, d_in, d_out, row_off, perm, seg_rows, word_off);
    const int64_t groups = (d_out + 31) / 32;
    dim3 grid((unsigned)d_in, (unsigned)((groups + kPackThreads - 1) / kPackThreads));
    const int vec_ok = aligned_to(codes, 16) && (d_out % 16 == 0);
    pack_kernel<<<grid, kPackThreads, 0, st>>>(codes, bits, d_out, word_off, packed, vec_ok);
    return launch_status();
}
