// Host-only helpers of the C ABI.
#include "common.cuh"

using namespace cmpq;

extern "C" size_t cmpq_workspace_bytes(cmpq_op op, int64_t d_in, int64_t d_out) {
    if (d_in < 1 || d_in > CMPQ_MAX_D_IN) return 0;
    switch (op) {
        case CMPQ_OP_COLLECT_STATS: return stats_ws_bytes(d_in);
        case CMPQ_OP_ALLOCATE_BITS: return alloc_ws_bytes(d_in);
        case CMPQ_OP_EXTRACT_OUTLIERS:
            if (d_out < 1 || d_out > CMPQ_MAX_D_OUT) return 0;
            return outliers_ws_bytes(d_in, d_out);
        case CMPQ_OP_QUANTIZE_LAYER:
            if (d_out < 1 || d_out > CMPQ_MAX_D_OUT) return 0;
            return quantize_ws_bytes(d_in, d_out);
        case CMPQ_OP_PACK:
            if (d_out < 1 || d_out > CMPQ_MAX_D_OUT) return 0;
            return pack_ws_bytes(d_in, d_out);
        case CMPQ_OP_PROTECT_AND_QUANTIZE:
            if (d_out < 1 || d_out > CMPQ_MAX_D_OUT) return 0;
            return protect_quantize_ws_bytes(d_in, d_out);
        case CMPQ_OP_OUTLIERS_BY_COLUMN:
            if (d_out < 1 || d_out > CMPQ_MAX_D_OUT) return 0;
            return by_column_ws_bytes(d_out);
        case CMPQ_OP_MATVEC:
            if (d_out < 1 || d_out > CMPQ_MAX_D_OUT) return 0;
            return matvec_ws_bytes(d_in, d_out);
        case CMPQ_OP_QUANTIZE_LAYER_PACKED:
            if (d_out < 1 || d_out > CMPQ_MAX_D_OUT) return 0;
            return quantize_packed_ws_bytes(d_in, d_out);
        case CMPQ_OP_PROTECT_QUANTIZE_PACK:
            if (d_out < 1 || d_out > CMPQ_MAX_D_OUT) return 0;
            return protect_quantize_pack_ws_bytes(d_in, d_out);
    }
    return 0;
}

extern "C" const char* cmpq_status_string(cmpq_status s) {
    switch (s) {
        case CMPQ_OK: return "ok";
        case CMPQ_ERR_INVALID_ARG: return "invalid argument";
        case CMPQ_ERR_UNSUPPORTED: return "unsupported argument combination";
        case CMPQ_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case CMPQ_ERR_CUDA: return "CUDA runtime error";
        case CMPQ_ERR_INTERNAL: return "internal error";
        case CMPQ_ERR_NONFINITE: return "an input held a NaN or an infinity";
    }
    return "unknown status";
}
