// Channel statistics of the calibration pass (second moments of Assumption 3.1 / Sec. 3.3 and
// the absmax behind the tensor scale), plus the small reductions derived from them.
//
// pq_calib_stats is a streaming read of the tensor (2 bytes per element): every thread owns 8
// adjacent channels (one 16-byte load per row) of one 16-row chunk, issues the chunk's loads at
// once and adds the squares in row order, so the fp32 partial of a (chunk, channel) pair is
// produced by one thread in row order.  Partials go to the workspace; a second small kernel folds
// them (and the per-chunk absmax) into the totals in ascending chunk order.  No atomics anywhere.
#include <mutex>

#include "pq_common.cuh"

namespace {

constexpr int kStatsThreads = 128;  // 128 threads x 8 channels = 1024 channels per block

__device__ __forceinline__ void stats_row(const uint4 &v, float (&s)[8], float (&a)[8]) {
    float x[8];
    pq::unpack8(v, x);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        s[i] = __fmaf_rn(x[i], x[i], s[i]);
        a[i] = fmaxf(a[i], fabsf(x[i]));
    }
}

__global__ void __launch_bounds__(kStatsThreads)
calib_stats_partial(const uint16_t *__restrict__ T, int64_t rows, int64_t K, int64_t ld,
                    float *__restrict__ part /*[chunks, K]*/, float *__restrict__ part_max /*[chunks, K]*/) {
    const int64_t col = (static_cast<int64_t>(blockIdx.y) * kStatsThreads + threadIdx.x) * 8;
    if (col >= K) return;
    const int64_t chunk = blockIdx.x;
    const int64_t r0 = chunk * PQ_CHUNK_ROWS;
    const int n = static_cast<int>(min(static_cast<int64_t>(PQ_CHUNK_ROWS), rows - r0));
    const uint16_t *p = T + r0 * ld + col;

    float s[8], a[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] = 0.0f, a[i] = 0.0f;

    if (n == PQ_CHUNK_ROWS) {
        uint4 v[PQ_CHUNK_ROWS];
#pragma unroll
        for (int u = 0; u < PQ_CHUNK_ROWS; ++u) v[u] = __ldcs(reinterpret_cast<const uint4 *>(p + static_cast<int64_t>(u) * ld));
#pragma unroll
        for (int u = 0; u < PQ_CHUNK_ROWS; ++u) stats_row(v[u], s, a);
    } else {
        for (int t = 0; t < n; ++t) stats_row(__ldcs(reinterpret_cast<const uint4 *>(p + static_cast<int64_t>(t) * ld)), s, a);
    }
    float4 *dst = reinterpret_cast<float4 *>(part + chunk * K + col);
    dst[0] = make_float4(s[0], s[1], s[2], s[3]);
    dst[1] = make_float4(s[4], s[5], s[6], s[7]);
    float4 *dmax = reinterpret_cast<float4 *>(part_max + chunk * K + col);
    dmax[0] = make_float4(a[0], a[1], a[2], a[3]);
    dmax[1] = make_float4(a[4], a[5], a[6], a[7]);
}

__global__ void tensor_scale_kernel(const float *__restrict__ amax, int64_t K, float *ts) {
    __shared__ float red[32];
    float a = 0.0f;
    for (int64_t i = threadIdx.x; i < K; i += blockDim.x) a = fmaxf(a, amax[i]);
    for (int m = 16; m; m >>= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, m));
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < static_cast<int>(blockDim.x >> 5); ++w) a = fmaxf(a, red[w]);
        *ts = (a == 0.0f) ? 1.0f : __fdiv_rn(a, 2688.0f);
    }
}

// lambda[s] = 1 / (sequential fp64 sum of side s), one thread per side.
__global__ void error_weights_kernel(const double *__restrict__ sa, const double *__restrict__ sw,
                                     int64_t K, double *lambda) {
    const double *src = threadIdx.x == 0 ? sa : sw;
    double s = 0.0;
    for (int64_t i = 0; i < K; ++i) s = __dadd_rn(s, src[i]);
    lambda[threadIdx.x] = __ddiv_rn(1.0, s);
}

}  // namespace

extern "C" pq_status pq_calib_stats(const void *T, int64_t rows, int64_t K, int64_t ld,
                                    double *sumsq, float *amax, void *ws, size_t ws_bytes,
                                    void *stream) {
    PQ_REQUIRE(T && sumsq && amax, PQ_ERR_NULL);
    PQ_REQUIRE(rows > 0 && K > 0 && K % 8 == 0 && ld >= K, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(T) && ld % 8 == 0 && pq_aligned16(amax), PQ_ERR_ALIGN);
    const size_t need = pq_workspace_bytes(PQ_OP_CALIB_STATS, rows, K, 0, 0);
    PQ_REQUIRE(ws && ws_bytes >= need, PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);
    const int64_t chunks = pq_ceil_div(rows, PQ_CHUNK_ROWS);
    PQ_REQUIRE(chunks < (1ll << 31) && K <= 65535ll * kStatsThreads * 8, PQ_ERR_SHAPE);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    dim3 grid(static_cast<unsigned>(chunks), static_cast<unsigned>(pq_ceil_div(K, kStatsThreads * 8)));
    float *part = static_cast<float *>(ws), *part_max = part + chunks * K;
    calib_stats_partial<<<grid, kStatsThreads, 0, st>>>(static_cast<const uint16_t *>(T), rows, K, ld, part, part_max);
    pq::fold_partials<true><<<static_cast<unsigned>(pq_ceil_div(K, 32)), pq::kFoldThreads, 0, st>>>(part, part_max, chunks,
                                                                                                    K, sumsq, amax);
    return pq_launch_status();
}

extern "C" pq_status pq_tensor_scale(const float *amax, int64_t K, float *ts, void *stream) {
    PQ_REQUIRE(amax && ts, PQ_ERR_NULL);
    PQ_REQUIRE(K > 0, PQ_ERR_SHAPE);
    tensor_scale_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(amax, K, ts);
    return pq_launch_status();
}

extern "C" pq_status pq_error_weights(const double *sumsq_a, const double *sumsq_w, int64_t K,
                                      double *lambda, void *stream) {
    PQ_REQUIRE(sumsq_a && sumsq_w && lambda, PQ_ERR_NULL);
    PQ_REQUIRE(K > 0, PQ_ERR_SHAPE);
    error_weights_kernel<<<1, 2, 0, static_cast<cudaStream_t>(stream)>>>(sumsq_a, sumsq_w, K, lambda);
    return pq_launch_status();
}

// ---------------------------------------------------------------- statistics without a caller workspace
// Scratch for pq_calib_stats_static: part of the library image, so every GPU that loads the
// library holds these bytes until the process exits.
constexpr size_t kStaticStatsScratchBytes = 8u << 20;
static __device__ __align__(256) unsigned char g_static_stats_scratch[kStaticStatsScratchBytes];

extern "C" size_t pq_calib_stats_static_max_bytes(void) { return kStaticStatsScratchBytes; }

extern "C" pq_status pq_calib_stats_static(const void *T, int64_t rows, int64_t K, int64_t ld, double *sumsq,
                                           float *amax, void *stream) {
    PQ_REQUIRE(rows > 0 && K > 0, PQ_ERR_SHAPE);
    // sizes first: this needs no CUDA call, so an oversized request fails the same way everywhere
    PQ_REQUIRE(pq_workspace_bytes(PQ_OP_CALIB_STATS, rows, K, 0, 0) <= kStaticStatsScratchBytes, PQ_ERR_WORKSPACE);
    // In host code the array's name is only a handle; the device address has to be asked for,
    // once per device, with that device current.
    constexpr int kMaxDevices = 64;
    static std::mutex lock;
    static void *scratch[kMaxDevices] = {};
    int dev = -1;
    PQ_CUDA_OK(cudaGetDevice(&dev));
    PQ_REQUIRE(dev >= 0 && dev < kMaxDevices, PQ_ERR_CUDA);
    void *ptr = nullptr;
    {
        std::lock_guard<std::mutex> guard(lock);
        if (!scratch[dev]) {
            void *p = nullptr;
            PQ_CUDA_OK(cudaGetSymbolAddress(&p, g_static_stats_scratch));
            scratch[dev] = p;
        }
        ptr = scratch[dev];
    }
    return pq_calib_stats(T, rows, K, ld, sumsq, amax, ptr, kStaticStatsScratchBytes, stream);
}
