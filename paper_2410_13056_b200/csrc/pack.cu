// Bit-packing of CMPQ codes (storage accounting of Section 5.1; the inference scheme of
// Section 6 multiplies one sub-matrix per precision, hence channels are grouped by bit width).
//
// HBM-bound: one byte read and bits/8 bytes written per weight.  A thread turns 32 codes
// (two 128-bit loads) into 2, 3 or 4 consecutive 32-bit words, so a warp reads 1 KiB and writes
// a contiguous 256 to 512 bytes.  Every channel of a segment has the same length in words, so
// its offset is segment base + (number of earlier channels of that width) * words.
#include "common.cuh"
#include "pack_bits.cuh"

namespace cmpq {

constexpr int kPackThreads = 256;

size_t pack_ws_bytes(int64_t d_in, int64_t) {
    return round_up((size_t)d_in * sizeof(int64_t), 256);
}

__global__ void __launch_bounds__(1024)
pack_layout_kernel(const uint8_t* __restrict__ bits, int64_t d_in, int64_t d_out,
                   int64_t* __restrict__ row_off, int32_t* __restrict__ perm,
                   int64_t* __restrict__ seg_rows, int64_t* __restrict__ word_off) {
    __shared__ unsigned long long warp_tot[32];
    pack_layout_block(bits, d_in, d_out, row_off, perm, seg_rows, word_off, warp_tot);
}

// One thread packs 32 consecutive codes of one channel into C consecutive words.
__global__ void __launch_bounds__(kPackThreads)
pack_kernel(const uint8_t* __restrict__ codes, const uint8_t* __restrict__ bits, int64_t d_out,
            const int64_t* __restrict__ word_off, uint32_t* __restrict__ packed, int vec_ok) {
    const int64_t row = blockIdx.x;
    const int64_t g = (int64_t)blockIdx.y * blockDim.x + threadIdx.x;  // group of 32 codes
    const int64_t j0 = g * 32;
    if (j0 >= d_out) return;
    const int c = bits[row];
    if (c < 2 || c > 4) return;  // not a width of the method: the layout gave this row no words
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
    uint32_t w[4];
    if (c == 2) pack32<2>(b, w);
    else if (c == 3) pack32<3>(b, w);
    else pack32<4>(b, w);
    uint32_t* dst = packed + word_off[row] + g * c;
    const int nwords = (cnt * c + 31) / 32;
#pragma unroll
    for (int t = 0; t < 4; ++t)
        if (t < nwords) dst[t] = w[t];
}

// Layout of the packed segments from the widths alone: row_off / perm / seg_rows (outputs of cmpq_pack) and
// word_off[i] = first word of channel i (d_in int64 of scratch).
cmpq_status launch_pack_layout(const uint8_t* bits, int64_t d_in, int64_t d_out, int64_t* row_off, int32_t* perm,
                               int64_t* seg_rows, int64_t* word_off, cudaStream_t st) {
    pack_layout_kernel<<<1, 1024, 0, st>>>(bits, d_in, d_out, row_off, perm, seg_rows, word_off);
    return launch_status();
}

cmpq_status launch_pack_codes(const uint8_t* codes, const uint8_t* bits, int64_t d_in, int64_t d_out,
                              const int64_t* word_off, uint32_t* packed, cudaStream_t st) {
    const int64_t groups = (d_out + 31) / 32;
    dim3 grid((unsigned)d_in, (unsigned)((groups + kPackThreads - 1) / kPackThreads));
    const int vec_ok = aligned_to(codes, 16) && (d_out % 16 == 0);
    pack_kernel<<<grid, kPackThreads, 0, st>>>(codes, bits, d_out, word_off, packed, vec_ok);
    return launch_status();
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
    const cmpq_status s = launch_pack_layout(bits, d_in, d_out, row_off, perm, seg_rows, word_off, st);
    if (s != CMPQ_OK) return s;
    return launch_pack_codes(codes, bits, d_in, d_out, word_off, packed, st);
}
