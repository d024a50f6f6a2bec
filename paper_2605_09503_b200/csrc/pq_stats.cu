// Channel statistics of the calibration pass (second moments of Assumption 3.1 / Sec. 3.3 and
// the absmax behind the tensor scale), plus the small reductions derived from them.
//
// pq_calib_stats is a streaming read of the tensor (2 bytes per element).  A block of 8 warps owns
// one 128-row slab x 256 channels: warp w takes the slab's w-th 16-row chunk, each lane 8 adjacent
// channels (one 16-byte load per row, the chunk's 16 loads in flight together) and adds the squares
// in row order in fp32.  The eight chunk partials of a channel meet in shared memory, where one
// thread per channel adds them in fp64 in chunk order; the slab sums (and slab absmax) go to the
// workspace, 12 bytes per channel per 128 rows.  A second small kernel, launched as a programmatic
// dependent, adds the slab sums to the totals in slab order.  No atomics anywhere.
#include <mutex>

#include "pq_common.cuh"

namespace {

constexpr int kStatsThreads = 256;                                // 8 warps = the 8 chunks of a slab
constexpr int kStatsCols = 256;                                   // 32 lanes x 8 channels
constexpr int kSlabChunks = PQ_SLAB_ROWS / PQ_CHUNK_ROWS;
static_assert(kSlabChunks * 32 == kStatsThreads, "one warp per chunk of the slab");

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
calib_stats_slab(const uint16_t *__restrict__ T, int64_t rows, int64_t K, int64_t ld,
                 double *__restrict__ slab_sum /*[slabs, K]*/, float *__restrict__ slab_max /*[slabs, K]*/) {
    __shared__ __align__(16) float sum_s[kSlabChunks][kStatsCols];
    __shared__ __align__(16) float max_s[kSlabChunks][kStatsCols];
    pq::dependents_may_launch();
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t col0 = static_cast<int64_t>(blockIdx.y) * kStatsCols;
    const int64_t col = col0 + lane * 8;
    const int64_t slab = blockIdx.x;
    const int64_t r0 = slab * PQ_SLAB_ROWS + w * PQ_CHUNK_ROWS;
    const int64_t left = rows - r0;
    const int n = left >= PQ_CHUNK_ROWS ? PQ_CHUNK_ROWS : (left > 0 ? static_cast<int>(left) : 0);

    float s[8], a[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] = 0.0f, a[i] = 0.0f;
    if (col < K) {
        const uint16_t *p = T + r0 * ld + col;
        if (n == PQ_CHUNK_ROWS) {
            uint4 v[PQ_CHUNK_ROWS];
#pragma unroll
            for (int u = 0; u < PQ_CHUNK_ROWS; ++u) v[u] = __ldcs(reinterpret_cast<const uint4 *>(p + static_cast<int64_t>(u) * ld));
#pragma unroll
            for (int u = 0; u < PQ_CHUNK_ROWS; ++u) stats_row(v[u], s, a);
        } else {
            for (int t = 0; t < n; ++t) stats_row(__ldcs(reinterpret_cast<const uint4 *>(p + static_cast<int64_t>(t) * ld)), s, a);
        }
    }
    float4 *ds = reinterpret_cast<float4 *>(&sum_s[w][lane * 8]);
    ds[0] = make_float4(s[0], s[1], s[2], s[3]);
    ds[1] = make_float4(s[4], s[5], s[6], s[7]);
    float4 *dm = reinterpret_cast<float4 *>(&max_s[w][lane * 8]);
    dm[0] = make_float4(a[0], a[1], a[2], a[3]);
    dm[1] = make_float4(a[4], a[5], a[6], a[7]);
    __syncthreads();
    // one thread per channel: the slab's chunk partials in chunk order, from zero (a chunk past
    // the last row contributes +0.0, which leaves the sum unchanged)
    const int c = threadIdx.x;
    if (col0 + c < K) {
        double acc = 0.0;
        float m = 0.0f;
#pragma unroll
        for (int k = 0; k < kSlabChunks; ++k) {
            acc = __dadd_rn(acc, static_cast<double>(sum_s[k][c]));
            m = fmaxf(m, max_s[k][c]);
        }
        slab_sum[slab * K + col0 + c] = acc;
        slab_max[slab * K + col0 + c] = m;
    }
}

// First moments (plain column sums) with the same slab / chunk walk: fp32 additions in row order
// inside a chunk, the slab's eight chunk partials in fp64 from zero.
__global__ void __launch_bounds__(kStatsThreads)
calib_sum_slab(const uint16_t *__restrict__ T, int64_t rows, int64_t K, int64_t ld, double *__restrict__ slab_sum) {
    __shared__ __align__(16) float sum_s[kSlabChunks][kStatsCols];
    pq::dependents_may_launch();
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t col0 = static_cast<int64_t>(blockIdx.y) * kStatsCols;
    const int64_t col = col0 + lane * 8;
    const int64_t slab = blockIdx.x;
    const int64_t r0 = slab * PQ_SLAB_ROWS + w * PQ_CHUNK_ROWS;
    const int64_t left = rows - r0;
    const int n = left >= PQ_CHUNK_ROWS ? PQ_CHUNK_ROWS : (left > 0 ? static_cast<int>(left) : 0);
    float s[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] = 0.0f;
    if (col < K) {
        const uint16_t *p = T + r0 * ld + col;
        uint4 v[PQ_CHUNK_ROWS];
#pragma unroll
        for (int u = 0; u < PQ_CHUNK_ROWS; ++u)
            v[u] = u < n ? __ldcs(reinterpret_cast<const uint4 *>(p + static_cast<int64_t>(u) * ld)) : make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int u = 0; u < PQ_CHUNK_ROWS; ++u) {
            if (u < n) {  // a row past the end must not even add +0.0: -0.0 + 0.0 would change a sign
                float x[8];
                pq::unpack8(v[u], x);
#pragma unroll
                for (int i = 0; i < 8; ++i) s[i] = __fadd_rn(s[i], x[i]);
            }
        }
    }
    float4 *ds = reinterpret_cast<float4 *>(&sum_s[w][lane * 8]);
    ds[0] = make_float4(s[0], s[1], s[2], s[3]);
    ds[1] = make_float4(s[4], s[5], s[6], s[7]);
    __syncthreads();
    const int c = threadIdx.x;
    if (col0 + c < K) {
        double acc = 0.0;
#pragma unroll
        for (int k = 0; k < kSlabChunks; ++k) acc = __dadd_rn(acc, static_cast<double>(sum_s[k][c]));
        slab_sum[slab * K + col0 + c] = acc;
    }
}

// Output-side calibration error: the same slab / chunk walk over the fp32 difference of two
// tensors (fp32 reference, bf16 quantized-layer output): 6 bytes per element, streaming.  A lane
// owns 8 adjacent columns; eight rows (two 16-byte loads of the reference and one of the output per
// row) are in flight at a time, the rows of a chunk are added in order.
constexpr int kDiffRows = 8;

__device__ __forceinline__ void diff_row(const float4 &r0, const float4 &r1, const uint4 &q, float (&s)[8]) {
    float y[8];
    pq::unpack8(q, y);
    const float ref[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float d = __fsub_rn(ref[i], y[i]);
        s[i] = __fmaf_rn(d, d, s[i]);
    }
}

__global__ void __launch_bounds__(kStatsThreads)
output_error_slab(const float *__restrict__ Yref, int64_t ld_ref, const uint16_t *__restrict__ Yq, int64_t ld_q,
                  int64_t rows, int64_t N, double *__restrict__ slab_sum /*[slabs, N]*/) {
    __shared__ __align__(16) float sum_s[kSlabChunks][kStatsCols];
    pq::dependents_may_launch();
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t col0 = static_cast<int64_t>(blockIdx.y) * kStatsCols;
    const int64_t col = col0 + lane * 8;
    const int64_t slab = blockIdx.x;
    const int64_t r0 = slab * PQ_SLAB_ROWS + w * PQ_CHUNK_ROWS;
    const int64_t left = rows - r0;
    const int n = left >= PQ_CHUNK_ROWS ? PQ_CHUNK_ROWS : (left > 0 ? static_cast<int>(left) : 0);

    float s[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) s[i] = 0.0f;
    if (col < N) {
        const float *pr = Yref + r0 * ld_ref + col;
        const uint16_t *yq_row = Yq + r0 * ld_q + col;
        for (int t0 = 0; t0 < n; t0 += kDiffRows) {
            float4 a[kDiffRows], b[kDiffRows];
            uint4 q[kDiffRows];
#pragma unroll
            for (int u = 0; u < kDiffRows; ++u) {
                if (t0 + u < n) {
                    const float4 *src = reinterpret_cast<const float4 *>(pr + static_cast<int64_t>(t0 + u) * ld_ref);
                    a[u] = __ldcs(src), b[u] = __ldcs(src + 1);
                    q[u] = __ldcs(reinterpret_cast<const uint4 *>(yq_row + static_cast<int64_t>(t0 + u) * ld_q));
                }
            }
#pragma unroll
            for (int u = 0; u < kDiffRows; ++u)
                if (t0 + u < n) diff_row(a[u], b[u], q[u], s);
        }
    }
    float4 *ds = reinterpret_cast<float4 *>(&sum_s[w][lane * 8]);
    ds[0] = make_float4(s[0], s[1], s[2], s[3]);
    ds[1] = make_float4(s[4], s[5], s[6], s[7]);
    __syncthreads();
    // one thread per column: the slab's chunk partials in chunk order, from zero
    const int c = threadIdx.x;
    if (col0 + c < N) {
        double acc = 0.0;
#pragma unroll
        for (int k = 0; k < kSlabChunks; ++k) acc = __dadd_rn(acc, static_cast<double>(sum_s[k][c]));
        slab_sum[slab * N + col0 + c] = acc;
    }
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

// lambda[s] = 1 / (sequential fp64 sum of side s in ascending channel order), one warp per side: the lanes
// fetch 1024 values at a time into shared memory (coalesced), lane 0 adds them in order.
__global__ void __launch_bounds__(64) error_weights_kernel(const double *__restrict__ sa, const double *__restrict__ sw,
                                                           int64_t K, double *lambda) {
    __shared__ double stage[2][1024];
    const int side = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const double *src = side == 0 ? sa : sw;
    double s = 0.0;
    for (int64_t i0 = 0; i0 < K; i0 += 1024) {
        const int n = static_cast<int>(K - i0 < 1024 ? K - i0 : 1024);
        for (int j = lane; j < n; j += 32) stage[side][j] = src[i0 + j];
        __syncwarp();
        if (lane == 0)
            for (int j = 0; j < n; ++j) s = __dadd_rn(s, stage[side][j]);
        __syncwarp();
    }
    if (lane == 0) lambda[side] = __ddiv_rn(1.0, s);
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
    const int64_t slabs = pq_ceil_div(rows, PQ_SLAB_ROWS);
    PQ_REQUIRE(slabs < (1ll << 31) && K <= 65535ll * kStatsCols, PQ_ERR_SHAPE);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    dim3 grid(static_cast<unsigned>(slabs), static_cast<unsigned>(pq_ceil_div(K, kStatsCols)));
    double *slab_sum = static_cast<double *>(ws);
    float *slab_max = reinterpret_cast<float *>(slab_sum + slabs * K);
    calib_stats_slab<<<grid, kStatsThreads, 0, st>>>(static_cast<const uint16_t *>(T), rows, K, ld, slab_sum, slab_max);
    PQ_CUDA_OK((pq::launch_fold<double, 1, true>(slab_sum, slab_max, slabs, K, sumsq, amax, st)));
    return pq_launch_status();
}

extern "C" pq_status pq_calib_sum(const void *T, int64_t rows, int64_t K, int64_t ld, double *sum, void *ws,
                                  size_t ws_bytes, void *stream) {
    PQ_REQUIRE(T && sum, PQ_ERR_NULL);
    PQ_REQUIRE(rows > 0 && K > 0 && K % 8 == 0 && ld >= K, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(T) && ld % 8 == 0, PQ_ERR_ALIGN);
    PQ_REQUIRE(ws && ws_bytes >= pq_workspace_bytes(PQ_OP_CALIB_STATS, rows, K, 0, 0), PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);
    const int64_t slabs = pq_ceil_div(rows, PQ_SLAB_ROWS);
    PQ_REQUIRE(slabs < (1ll << 31) && K <= 65535ll * kStatsCols, PQ_ERR_SHAPE);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    dim3 grid(static_cast<unsigned>(slabs), static_cast<unsigned>(pq_ceil_div(K, kStatsCols)));
    double *slab_sum = static_cast<double *>(ws);
    calib_sum_slab<<<grid, kStatsThreads, 0, st>>>(static_cast<const uint16_t *>(T), rows, K, ld, slab_sum);
    PQ_CUDA_OK((pq::launch_fold<double, 1, false>(slab_sum, nullptr, slabs, K, sum, nullptr, st)));
    return pq_launch_status();
}

extern "C" pq_status pq_output_error(const float *Yref, int64_t ld_ref, const void *Yq, int64_t ld_q, int64_t rows,
                                     int64_t N, double *err, void *ws, size_t ws_bytes, void *stream) {
    PQ_REQUIRE(Yref && Yq && err, PQ_ERR_NULL);
    PQ_REQUIRE(rows > 0 && N > 0 && N % 8 == 0 && ld_ref >= N && ld_q >= N, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(Yref) && ld_ref % 4 == 0 && pq_aligned16(Yq) && ld_q % 8 == 0, PQ_ERR_ALIGN);
    const size_t need = pq_workspace_bytes(PQ_OP_OUTPUT_ERROR, rows, N, 0, 0);
    PQ_REQUIRE(ws && ws_bytes >= need, PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);
    const int64_t slabs = pq_ceil_div(rows, PQ_SLAB_ROWS);
    PQ_REQUIRE(slabs < (1ll << 31) && N <= 65535ll * kStatsCols, PQ_ERR_SHAPE);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    dim3 grid(static_cast<unsigned>(slabs), static_cast<unsigned>(pq_ceil_div(N, kStatsCols)));
    double *slab_sum = static_cast<double *>(ws);
    output_error_slab<<<grid, kStatsThreads, 0, st>>>(Yref, ld_ref, static_cast<const uint16_t *>(Yq), ld_q, rows, N,
                                                      slab_sum);
    PQ_CUDA_OK((pq::launch_fold<double, 1, false>(slab_sum, nullptr, slabs, N, err, nullptr, st)));
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
    error_weights_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(sumsq_a, sumsq_w, K, lambda);
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
