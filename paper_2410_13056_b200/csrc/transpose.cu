// Layout conversion for weights stored the way deep-learning frameworks store a linear layer,
// [d_out][d_in] (output-major), into the layout the paper's notation implies and this library works in:
// W in R^{d_in x d_out}, row i = the d_out weights of input channel i (Section 3.2.1).
// HBM bound: 2 bytes read and 2 bytes written per weight.  64 x 64 tiles go through shared memory so that
// both the reads and the writes are contiguous rows (128 bytes per warp and row; 32-bit accesses when the
// alignment allows, single elements otherwise).
#include "common.cuh"

namespace cmpq {

constexpr int kTrTile = 64;
constexpr int kTrThreads = 256;

// dst[c][r] = src[r][c] for a [rows][cols] source; 16-bit elements moved as raw patterns.
__global__ void __launch_bounds__(kTrThreads)
transpose16_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t cols, int64_t ld_src,
                   uint16_t* __restrict__ dst, int64_t ld_dst) {
    __shared__ uint16_t tile[kTrTile][kTrTile + 2];  // pad: column reads hit different banks
    const int64_t r0 = (int64_t)blockIdx.y * kTrTile, c0 = (int64_t)blockIdx.x * kTrTile;
    const int tx = threadIdx.x % kTrTile, ty = threadIdx.x / kTrTile;  // 64 x 4
#pragma unroll
    for (int k = 0; k < kTrTile; k += kTrThreads / kTrTile) {
        const int64_t r = r0 + ty + k, c = c0 + tx;
        if (r < rows && c < cols) tile[ty + k][tx] = src[r * ld_src + c];
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kTrTile; k += kTrThreads / kTrTile) {
        const int64_t c = c0 + ty + k, r = r0 + tx;
        if (r < rows && c < cols) dst[c * ld_dst + r] = tile[tx][ty + k];
    }
}

// The same tile with 32-bit accesses on both sides (two adjacent elements per thread and access), for
// sources and destinations whose rows start on 4-byte boundaries and whose extents are even: a warp then
// reads and writes 128 contiguous bytes per row, twice the bytes in flight of the element-wise kernel.
__global__ void __launch_bounds__(kTrThreads)
transpose16_pairs_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t cols, int64_t ld_src,
                         uint16_t* __restrict__ dst, int64_t ld_dst) {
    __shared__ uint16_t tile[kTrTile][kTrTile + 2];
    const int64_t r0 = (int64_t)blockIdx.y * kTrTile, c0 = (int64_t)blockIdx.x * kTrTile;
    const int tx = threadIdx.x % 32, ty = threadIdx.x / 32;  // 32 pairs x 8 rows
#pragma unroll
    for (int k = 0; k < kTrTile; k += kTrThreads / 32) {
        const int64_t r = r0 + ty + k, c = c0 + 2 * tx;
        if (r < rows && c < cols) {  // cols is even: the pair is inside
            const uint32_t v = __ldcs(reinterpret_cast<const uint32_t*>(src + r * ld_src + c));
            *reinterpret_cast<uint32_t*>(&tile[ty + k][2 * tx]) = v;
        }
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kTrTile; k += kTrThreads / 32) {
        const int64_t c = c0 + ty + k, r = r0 + 2 * tx;
        if (r < rows && c < cols) {  // rows is even
            const uint32_t v = (uint32_t)tile[2 * tx][ty + k] | ((uint32_t)tile[2 * tx + 1][ty + k] << 16);
            __stcs(reinterpret_cast<uint32_t*>(dst + c * ld_dst + r), v);
        }
    }
}

}  // namespace cmpq

using namespace cmpq;

extern "C" cmpq_status cmpq_transpose16(const void* src, int64_t rows, int64_t cols, int64_t ld_src, void* dst,
                                        int64_t ld_dst, void* stream) {
    if (!src || !dst || rows < 1 || cols < 1 || ld_src < cols || ld_dst < rows) return CMPQ_ERR_INVALID_ARG;
    if (rows > CMPQ_MAX_D_IN || cols > CMPQ_MAX_D_IN) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(src, 2) || !aligned_to(dst, 2)) return CMPQ_ERR_INVALID_ARG;
    dim3 grid((unsigned)((cols + kTrTile - 1) / kTrTile), (unsigned)((rows + kTrTile - 1) / kTrTile));
    const bool pairs = aligned_to(src, 4) && aligned_to(dst, 4) && rows % 2 == 0 && cols % 2 == 0 && ld_src % 2 == 0 &&
                       ld_dst % 2 == 0;
    if (pairs)
        transpose16_pairs_kernel<<<grid, kTrThreads, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const uint16_t*>(src), rows, cols, ld_src, static_cast<uint16_t*>(dst), ld_dst);
    else
        transpose16_kernel<<<grid, kTrThreads, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const uint16_t*>(src), rows, cols, ld_src, static_cast<uint16_t*>(dst), ld_dst);
    return launch_status();
}
