// Calibration quantization error per candidate order and group column (Eq. 3), the quantity
// the candidate selection (Sec. 3.3) and the acceptance rule (Eq. 10) compare.
//
// Work decomposition mirrors the arithmetic definition: a TEAM of group/8 adjacent lanes owns
// one (order, group column) pair for one 16-row chunk and walks the chunk's rows in order,
// adding each row's group error to an fp32 partial.  Partials go to the workspace
// [chunk][order][group column]; a second kernel folds them into the fp64 totals in ascending
// chunk order.  No floating-point atomics.
//
//   original order (perms == NULL): rows are read straight from global memory with coalesced
//     16-byte loads -- a pure streaming pass, bound by HBM bandwidth.
//   candidate orders: one block per (chunk, order); rows are staged in shared memory a few at a
//     time (coalesced) and the lanes gather their eight channels from there, so the tensor is
//     fetched from HBM once per chunk and served from L2 to the other orders' blocks.
#include "pq_common.cuh"

namespace {

constexpr int kErrThreads = 256;

template <int KIND, int TEAM>
__device__ __forceinline__ float group_sse_lane(const float (&x)[8], float ts, float Qf) {
    const float amax = pq::team_max<TEAM>(pq::absmax8(x));
    float q[8], d;
    if (KIND == 0) {
        uint32_t sf8;
        float r;
        pq::nvfp4_scale(amax, ts, sf8, d, r);
        pq::e2m1x8_to_f32(pq::nvfp4_codes(x, r), q);
    } else {
        float r;
        pq::int_scale(amax, Qf, d, r);
        pq::int_levels(x, r, Qf, q);
    }
    return pq::team_sum<TEAM>(pq::run_sse(x, q, d));
}

// ---------------------------------------------------------------- original order
constexpr int kDirectThreads = 128;

template <int KIND, int TEAM>
__global__ void __launch_bounds__(kDirectThreads)
group_error_direct(const uint16_t *__restrict__ T, int64_t rows, int64_t K, int64_t ld,
                   const float *__restrict__ ts_ptr, float Qf, float *__restrict__ part /*[chunks, K/g]*/) {
    const int64_t oct = static_cast<int64_t>(blockIdx.y) * kDirectThreads + threadIdx.x;
    const bool live = oct * 8 < K;  // K % (8*TEAM) == 0, so a team is live or dead as a whole
    const int64_t chunk = blockIdx.x;
    const int64_t r0 = chunk * PQ_CHUNK_ROWS;
    const int n = static_cast<int>(min(static_cast<int64_t>(PQ_CHUNK_ROWS), rows - r0));
    const float ts = (KIND == 0) ? __ldg(ts_ptr) : 1.0f;
    const uint16_t *p = T + r0 * ld + (live ? oct * 8 : 0);
    const uint4 zero = make_uint4(0, 0, 0, 0);
    float acc = 0.0f;
    if (n == PQ_CHUNK_ROWS) {
        // all of the chunk's loads first, then the per-row errors (independent of one another),
        // then the row-ordered sum
        uint4 v[PQ_CHUNK_ROWS];
#pragma unroll
        for (int u = 0; u < PQ_CHUNK_ROWS; ++u)
            v[u] = live ? __ldcs(reinterpret_cast<const uint4 *>(p + static_cast<int64_t>(u) * ld)) : zero;
        float e[PQ_CHUNK_ROWS];
#pragma unroll
        for (int u = 0; u < PQ_CHUNK_ROWS; ++u) {
            float x[8];
            pq::unpack8(v[u], x);
            e[u] = group_sse_lane<KIND, TEAM>(x, ts, Qf);
        }
#pragma unroll
        for (int u = 0; u < PQ_CHUNK_ROWS; ++u) acc = __fadd_rn(acc, e[u]);
    } else {
        for (int t = 0; t < n; ++t) {
            float x[8];
            pq::unpack8(live ? __ldcs(reinterpret_cast<const uint4 *>(p + static_cast<int64_t>(t) * ld)) : zero, x);
            acc = __fadd_rn(acc, group_sse_lane<KIND, TEAM>(x, ts, Qf));
        }
    }
    if (live && (oct % TEAM) == 0) part[chunk * (K / (8 * TEAM)) + oct / TEAM] = acc;
}

// ---------------------------------------------------------------- candidate orders
constexpr int kMaxOctPerThread = 8;  // 256 threads x 8 octets x 8 channels = 16384 channels

template <int KIND, int TEAM>
__global__ void __launch_bounds__(kErrThreads)
group_error_gather(const uint16_t *__restrict__ T, int64_t rows, int64_t K, int64_t ld,
                   const float *__restrict__ ts_ptr, float Qf, const int32_t *__restrict__ perms, int P,
                   int sub_rows, float *__restrict__ part /*[chunks, P, K/g]*/) {
    extern __shared__ __align__(16) uint16_t rows_s[];  // [sub_rows][K]
    const int64_t chunk = blockIdx.x;
    const int p = blockIdx.y;
    const int32_t *perm = perms + static_cast<int64_t>(p) * K;
    const int oct_per_row = static_cast<int>(K >> 3);
    const int64_t r0 = chunk * PQ_CHUNK_ROWS;
    const int n = static_cast<int>(min(static_cast<int64_t>(PQ_CHUNK_ROWS), rows - r0));
    const float ts = (KIND == 0) ? __ldg(ts_ptr) : 1.0f;

    // this thread's octets: o = threadIdx.x + i * kErrThreads; channel indices packed 2 x 16 bit
    uint32_t ch[kMaxOctPerThread][4];
    float acc[kMaxOctPerThread];
#pragma unroll
    for (int i = 0; i < kMaxOctPerThread; ++i) {
        acc[i] = 0.0f;
        const int o = threadIdx.x + i * kErrThreads;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            uint32_t lo = 0, hi = 0;
            if (o < oct_per_row) {
                lo = static_cast<uint32_t>(perm[o * 8 + 2 * w]);
                hi = static_cast<uint32_t>(perm[o * 8 + 2 * w + 1]);
            }
            ch[i][w] = lo | (hi << 16);
        }
    }

    for (int s0 = 0; s0 < n; s0 += sub_rows) {
        const int ns = min(sub_rows, n - s0);
        __syncthreads();
        for (int idx = threadIdx.x; idx < ns * oct_per_row; idx += kErrThreads) {
            const int rr = idx / oct_per_row, o = idx - rr * oct_per_row;
            reinterpret_cast<uint4 *>(rows_s)[idx] =
                __ldg(reinterpret_cast<const uint4 *>(T + (r0 + s0 + rr) * ld) + o);
        }
        __syncthreads();
        for (int rr = 0; rr < ns; ++rr) {
            const uint16_t *row = rows_s + static_cast<int64_t>(rr) * K;
#pragma unroll
            for (int i = 0; i < kMaxOctPerThread; ++i) {
                if (i * kErrThreads >= oct_per_row) break;  // uniform over the block
                const bool live = threadIdx.x + i * kErrThreads < oct_per_row;
                float x[8];
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    x[2 * w] = live ? pq::bf16_bits_to_f32(row[ch[i][w] & 0xFFFFu]) : 0.0f;
                    x[2 * w + 1] = live ? pq::bf16_bits_to_f32(row[ch[i][w] >> 16]) : 0.0f;
                }
                acc[i] = __fadd_rn(acc[i], group_sse_lane<KIND, TEAM>(x, ts, Qf));
            }
        }
    }
    const int64_t Kg = K / (8 * TEAM);
#pragma unroll
    for (int i = 0; i < kMaxOctPerThread; ++i) {
        const int o = threadIdx.x + i * kErrThreads;
        if (o < oct_per_row && (o % TEAM) == 0) part[(chunk * P + p) * Kg + o / TEAM] = acc[i];
    }
}

template <int KIND, int TEAM>
pq_status launch(const uint16_t *T, int64_t rows, int64_t K, int64_t ld, const float *ts, float Qf,
                 const int32_t *perms, int P, float *part, cudaStream_t st) {
    const int64_t chunks = pq_ceil_div(rows, PQ_CHUNK_ROWS);
    if (!perms) {
        dim3 grid(static_cast<unsigned>(chunks), static_cast<unsigned>(pq_ceil_div(K / 8, kDirectThreads)));
        group_error_direct<KIND, TEAM><<<grid, kDirectThreads, 0, st>>>(T, rows, K, ld, ts, Qf, part);
        return pq_launch_status();
    }
    int sub_rows = static_cast<int>((96 * 1024) / (K * 2));
    if (sub_rows > 16) sub_rows = 16;
    if (sub_rows < 1) sub_rows = 1;
    const size_t smem = static_cast<size_t>(sub_rows) * K * 2;
    if (smem > 48 * 1024)
        PQ_CUDA_OK(cudaFuncSetAttribute(group_error_gather<KIND, TEAM>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    dim3 grid(static_cast<unsigned>(chunks), static_cast<unsigned>(P));
    group_error_gather<KIND, TEAM><<<grid, kErrThreads, smem, st>>>(T, rows, K, ld, ts, Qf, perms, P, sub_rows, part);
    return pq_launch_status();
}

}  // namespace

extern "C" pq_status pq_group_error(const void *T, int64_t rows, int64_t K, int64_t ld, pq_format fmt,
                                    const float *ts, const int32_t *perms, int P, double *err, void *ws,
                                    size_t ws_bytes, void *stream) {
    PQ_REQUIRE(T && err, PQ_ERR_NULL);
    PQ_REQUIRE(fmt.kind == 0 || fmt.kind == 1, PQ_ERR_FORMAT);
    const int group = fmt.kind == 0 ? 16 : fmt.group;
    if (fmt.kind == 1) {
        PQ_REQUIRE(fmt.bits >= 2 && fmt.bits <= 8, PQ_ERR_FORMAT);
        PQ_REQUIRE(group == 16 || group == 32 || group == 64 || group == 128, PQ_ERR_FORMAT);
    } else {
        PQ_REQUIRE(ts, PQ_ERR_NULL);
    }
    PQ_REQUIRE(rows > 0 && K > 0 && K % group == 0 && K <= 16384 && ld >= K, PQ_ERR_SHAPE);
    PQ_REQUIRE(P >= 1 && P <= 8 && (perms || P == 1), PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(T) && ld % 8 == 0, PQ_ERR_ALIGN);
    const int64_t chunks = pq_ceil_div(rows, PQ_CHUNK_ROWS);
    PQ_REQUIRE(chunks < (1ll << 31), PQ_ERR_SHAPE);
    PQ_REQUIRE(ws && ws_bytes >= pq_workspace_bytes(PQ_OP_GROUP_ERROR, rows, K, 0, P), PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint16_t *t = static_cast<const uint16_t *>(T);
    float *part = static_cast<float *>(ws);
    const float Qf = fmt.kind == 1 ? static_cast<float>((1 << (fmt.bits - 1)) - 1) : 0.0f;
    pq_status rc;
    if (fmt.kind == 0) {
        rc = launch<0, 2>(t, rows, K, ld, ts, Qf, perms, P, part, st);
    } else {
        switch (group) {
            case 16: rc = launch<1, 2>(t, rows, K, ld, ts, Qf, perms, P, part, st); break;
            case 32: rc = launch<1, 4>(t, rows, K, ld, ts, Qf, perms, P, part, st); break;
            case 64: rc = launch<1, 8>(t, rows, K, ld, ts, Qf, perms, P, part, st); break;
            default: rc = launch<1, 16>(t, rows, K, ld, ts, Qf, perms, P, part, st); break;
        }
    }
    if (rc != PQ_OK) return rc;
    const int64_t n = static_cast<int64_t>(P) * (K / group);
    pq::fold_partials<false><<<static_cast<unsigned>(pq_ceil_div(n, 32)), pq::kFoldThreads, 0, st>>>(part, nullptr, chunks, n,
                                                                                                     err, nullptr);
    return pq_launch_status();
}
