// Allocation-free variant of the activation statistic.
//
// Some callers of this library must not, or cannot, obtain device memory while they run: code
// that executes inside another framework's memory plan and may not disturb its allocator, code
// on a latency-critical path where cudaMalloc's implicit device synchronisation is not
// acceptable, and plug-ins that are handed input and output buffers and nothing else.  For them
// the partial sums of the column reduction live in a fixed array that is part of the library
// image instead of a caller-supplied work space.  The array exists once per GPU that loads the
// library, from load until the process exits.
#include <mutex>

#include "common.cuh"

namespace cmpq {

// defined in stats.cu
cmpq_status launch_collect_stats(const void* X, cmpq_dtype dt, int64_t n_tokens, int64_t d_in,
                                 int64_t ldx, double* sumsq, double* partial, int64_t row_blocks,
                                 cudaStream_t st);
int64_t stats_row_blocks(int64_t d_in, int64_t n_tokens);

constexpr int64_t kStaticScratchDoubles = 262144;  // 2 MiB
constexpr int kMaxDevices = 64;

static __device__ __align__(256) double g_stats_scratch[kStaticScratchDoubles];

// In host code g_stats_scratch is only a handle for the runtime; the address a kernel can use
// is asked for once per device, with that device current.
static double* scratch_address_for_current_device(cmpq_status* status) {
    static std::mutex lock;
    static double* address[kMaxDevices] = {nullptr};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        *status = CMPQ_ERR_CUDA;
        return nullptr;
    }
    std::lock_guard<std::mutex> guard(lock);
    if (!address[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_stats_scratch) != cudaSuccess || !p) {
            *status = CMPQ_ERR_CUDA;
            return nullptr;
        }
        address[dev] = static_cast<double*>(p);
    }
    *status = CMPQ_OK;
    return address[dev];
}

}  // namespace cmpq

using namespace cmpq;

extern "C" cmpq_status cmpq_collect_stats_static(const void* X, cmpq_dtype dt, int64_t n_tokens,
                                                 int64_t d_in, int64_t ldx, double* sumsq,
                                                 void* stream) {
    if (!sumsq || n_tokens < 0 || d_in < 1 || ldx < d_in) return CMPQ_ERR_INVALID_ARG;
    if (dt != CMPQ_F16 && dt != CMPQ_BF16) return CMPQ_ERR_INVALID_ARG;
    if (n_tokens > 0 && !X) return CMPQ_ERR_INVALID_ARG;
    if (!aligned_to(X, 2) || !aligned_to(sumsq, 8)) return CMPQ_ERR_INVALID_ARG;
    if (d_in > CMPQ_STATIC_MAX_D_IN) return CMPQ_ERR_UNSUPPORTED;  // beyond the built-in scratch
    if (n_tokens == 0) return CMPQ_OK;
    cmpq_status s;
    double* partial = scratch_address_for_current_device(&s);
    if (s != CMPQ_OK) return s;
    // every block of the launch overwrites its own 256 partials and the combine step reads
    // exactly those, so nothing left in the array by an earlier call is ever read
    const int64_t padded_cols = (d_in + 255) / 256 * 256;
    int64_t rb = stats_row_blocks(d_in, n_tokens);
    if (rb <= 0) return CMPQ_ERR_CUDA;
    const int64_t cap = kStaticScratchDoubles / padded_cols;
    if (rb > cap) rb = cap;
    return launch_collect_stats(X, dt, n_tokens, d_in, ldx, sumsq, partial, rb,
                                static_cast<cudaStream_t>(stream));
}
