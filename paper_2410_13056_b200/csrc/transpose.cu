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

// The same tile with 128-bit accesses on both sides, for sources and destinations whose rows start on 16-byte
// boundaries and whose extents are multiples of 8.  A thread loads two groups of eight elements of a source
// row and writes them into shared memory as they are; group g of tile row r is kept in slot g ^ (r / 8), so
// that afterwards the 32 lanes of a warp -- eight row blocks times four column pairs -- read 32 different
// banks.  Each thread then reads the same column pair from eight consecutive tile rows (eight 32-bit words),
// separates the two columns with byte permutes and stores eight elements of two destination rows: a warp
// writes four whole 128-byte lines per store.
__global__ void __launch_bounds__(kTrThreads)
transpose16_wide_kernel(const uint16_t* __restrict__ src, int64_t rows, int64_t cols, int64_t ld_src,
                        uint16_t* __restrict__ dst, int64_t ld_dst) {
    __shared__ uint4 tile[kTrTile][kTrTile / 8];
    const int64_t r0 = (int64_t)blockIdx.y * kTrTile, c0 = (int64_t)blockIdx.x * kTrTile;
    const int t = threadIdx.x;
    {
        const int g = t & 7, r = t >> 3;  // 8 groups x 32 rows, twice
        uint4 v[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int64_t rr = r0 + r + 32 * h, cc = c0 + 8 * g;
            v[h] = make_uint4(0u, 0u, 0u, 0u);
            if (rr < rows && cc < cols) v[h] = __ldcs(reinterpret_cast<const uint4*>(src + rr * ld_src + cc));
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) tile[r + 32 * h][g ^ ((r + 32 * h) >> 3)] = v[h];
    }
    __syncthreads();
    const int lane = t & 31, warp = t >> 5;
    const int rb = lane & 7;               // block of eight tile rows = eight consecutive elements of a destination row
    const int w = warp * 4 + (lane >> 3);  // column pair of the tile (0..31)
    const uint32_t* words = reinterpret_cast<const uint32_t*>(&tile[0][0]);
    uint32_t a[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) a[i] = words[((rb * 8 + i) * 8 + ((w >> 2) ^ rb)) * 4 + (w & 3)];
    const int64_t rr = r0 + 8 * rb, cc = c0 + 2 * w;
    if (rr < rows && cc < cols) {  // extents are multiples of 8: both columns and all eight rows are inside
        const uint4 lo = make_uint4(__byte_perm(a[0], a[1], 0x5410), __byte_perm(a[2], a[3], 0x5410),
                                    __byte_perm(a[4], a[5], 0x5410), __byte_perm(a[6], a[7], 0x5410));
        const uint4 hi = make_uint4(__byte_perm(a[0], a[1], 0x7632), __byte_perm(a[2], a[3], 0x7632),
                                    __byte_perm(a[4], a[5], 0x7632), __byte_perm(a[6], a[7], 0x7632));
        __stcs(reinterpret_cast<uint4*>(dst + cc * ld_dst + rr), lo);
        __stcs(reinterpret_cast<uint4*>(dst + (cc + 1) * ld_dst + rr), hi);
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
    const bool wide = aligned_to(src, 16) && aligned_to(dst, 16) && rows % 8 == 0 && cols % 8 == 0 && ld_src % 8 == 0 &&
                      ld_dst % 8 == 0;
    if (wide)
        transpose16_wide_kernel<<<grid, kTrThreads, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const uint16_t*>(src), rows, cols, ld_src, static_cast<uint16_t*>(dst), ld_dst);
    else if (pairs)
        transpose16_pairs_kernel<<<grid, kTrThreads, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const uint16_t*>(src), rows, cols, ld_src, static_cast<uint16_t*>(dst), ld_dst);
    else
        transpose16_kernel<<<grid, kTrThreads, 0, static_cast<cudaStream_t>(stream)>>>(
            static_cast<const uint16_t*>(src), rows, cols, ld_src, static_cast<uint16_t*>(dst), ld_dst);
    return launch_status();
}
