// Measurement aids of the library: an arithmetic-throughput probe and kernel resource queries.
//
// The brute-force K-means assignment (Section 3: every weight goes to its nearest centroid) costs one
// fp32 subtract and one compare/select per (weight, centroid) pair.  The probe below executes exactly
// that mix -- d = v - c; best = min(best, |d|) -- on register operands only, in independent chains, so
// its rate is the ceiling the fp32 pipes of this GPU give to any all-pairs assignment kernel at the
// clocks of the moment.  Nothing here is on the quantization path.
#include "common.cuh"

namespace cmpq {

constexpr int kProbeChains = 8;    // independent dependency chains per thread
constexpr int kProbeCentroids = 16;

__constant__ float probe_centroids[kProbeCentroids] = {-0.9f, -0.7f, -0.55f, -0.4f, -0.3f, -0.2f, -0.1f, -0.03f,
                                                       0.02f,  0.09f, 0.17f,  0.28f, 0.41f, 0.52f, 0.66f, 0.88f};

// Every thread carries kProbeChains running minima through `rounds` rounds of the 16 centroids:
// best = min(best, |best - c|).  Each evaluation depends on the one before it in its chain, so no round
// can be hoisted or merged, and the chains of a thread are independent of each other.
__global__ void __launch_bounds__(256, 4)
alu_probe_kernel(int rounds, float seed, float* __restrict__ sink) {
    float best[kProbeChains];
#pragma unroll
    for (int u = 0; u < kProbeChains; ++u) best[u] = 1.0f + seed * (float)(threadIdx.x * kProbeChains + u + 1);
    for (int r = 0; r < rounds; ++r) {
#pragma unroll
        for (int k = 0; k < kProbeCentroids; ++k) {
            const float c = probe_centroids[k];
#pragma unroll
            for (int u = 0; u < kProbeChains; ++u) best[u] = fminf(best[u], fabsf(best[u] - c));
        }
    }
    float total = 0.f;
#pragma unroll
    for (int u = 0; u < kProbeChains; ++u) total += best[u];
    if (total < 0.f) sink[blockIdx.x * blockDim.x + threadIdx.x] = total;  // never true: distances are >= 0
}

// kernels of other translation units whose resources can be asked for
const void* stats_kernel_address();        // stats.cu
const void* lloyd_table_kernel_address();  // lloyd_hist.cu

static const void* kernel_address(cmpq_kernel k) {
    switch (k) {
        case CMPQ_KERNEL_STATS_PARTIAL_VEC_BF16: return stats_kernel_address();
        case CMPQ_KERNEL_LLOYD_TABLE_BF16_4096: return lloyd_table_kernel_address();
    }
    return nullptr;
}

}  // namespace cmpq

using namespace cmpq;

extern "C" cmpq_status cmpq_alu_probe(int rounds, int blocks, float* sink, unsigned long long* evaluations,
                                      void* stream) {
    if (rounds < 1 || rounds > (1 << 24) || blocks < 1 || blocks > (1 << 20) || !sink) return CMPQ_ERR_INVALID_ARG;
    alu_probe_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(rounds, 1.0e-3f, sink);
    if (evaluations)
        *evaluations = (unsigned long long)rounds * kProbeCentroids * kProbeChains * 256ull * (unsigned long long)blocks;
    return launch_status();
}

extern "C" cmpq_status cmpq_kernel_resources(cmpq_kernel k, int* registers, int* static_smem_bytes) {
    const void* fn = kernel_address(k);
    if (!fn) return CMPQ_ERR_INVALID_ARG;
    cudaFuncAttributes attr;
    if (cudaFuncGetAttributes(&attr, fn) != cudaSuccess) return CMPQ_ERR_CUDA;
    if (registers) *registers = attr.numRegs;
    if (static_smem_bytes) *static_smem_bytes = (int)attr.sharedSizeBytes;
    return CMPQ_OK;
}
