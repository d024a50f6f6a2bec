// Entry points that launch no kernel: status strings, version, workspace sizing.
#include <cstdio>

#include "pq_common.cuh"

extern "C" const char *pq_status_string(pq_status s) {
    switch (s) {
        case PQ_OK: return "ok";
        case PQ_ERR_NULL: return "a required pointer is NULL";
        case PQ_ERR_SHAPE: return "size out of range or not divisible as required";
        case PQ_ERR_ALIGN: return "pointer or leading dimension misaligned";
        case PQ_ERR_FORMAT: return "unsupported quantization format or scale layout";
        case PQ_ERR_WORKSPACE: return "workspace missing or too small";
        case PQ_ERR_CUDA: return "CUDA runtime error";
        case PQ_ERR_TIMEOUT: return "a bounded device-side wait expired";
    }
    return "unknown status";
}

extern "C" int pq_version(void) { return 1; }

// Last CUDA failure seen by this host thread, as text: "<cuda error name>: <call> (line N)".
static thread_local char g_last_error[256] = "";

void pq_note_cuda_error(cudaError_t err, const char *what, int line) {
    snprintf(g_last_error, sizeof(g_last_error), "%s: %.180s (line %d)", cudaGetErrorName(err), what, line);
}

extern "C" const char *pq_last_error_detail(void) { return g_last_error; }

static size_t round256(size_t b) { return (b + 255) / 256 * 256; }

extern "C" size_t pq_workspace_bytes(int op, int64_t rows, int64_t K, int64_t N, int P) {
    (void)N;
    if (K <= 0) return 0;
    const int64_t chunks = rows > 0 ? pq_ceil_div(rows, PQ_CHUNK_ROWS) : 0;
    const int64_t slabs = rows > 0 ? pq_ceil_div(rows, PQ_SLAB_ROWS) : 0;
    switch (op) {
        case PQ_OP_CALIB_STATS: return round256(static_cast<size_t>(slabs) * K * (sizeof(double) + sizeof(float)));
        case PQ_OP_SELECT_PERM: return round256(static_cast<size_t>(P > 0 ? P : 1) * K * sizeof(uint64_t));
        case PQ_OP_GROUP_ERROR: {
            // fp32 chunk partials of P candidate orders, or fp64 slab sums of the original order
            const size_t by_chunk = static_cast<size_t>(chunks) * (P > 0 ? P : 1) * (K / 16 + 1) * sizeof(float);
            const size_t by_slab = static_cast<size_t>(slabs) * (K / 16 + 1) * sizeof(double);
            return round256(by_chunk > by_slab ? by_chunk : by_slab);
        }
        case PQ_OP_QUANT_WEIGHT: return 256;
        case PQ_OP_GEMM: return 256;
        case PQ_OP_OUTPUT_ERROR: return round256(static_cast<size_t>(slabs) * K * sizeof(double));
        default: return 0;
    }
}
