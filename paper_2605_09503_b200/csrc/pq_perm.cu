// Sort candidates of the joint second-moment criterion (Eq. 9, Prop. 3.2) and the
// selection / acceptance rule (Eq. 10).
//
// Sorting is done by rank counting: position of channel i = number of channels that precede
// it under the total order (key descending, channel ascending).  K <= 16384, so the K^2
// comparisons of one candidate are a few hundred million integer compares spread over the
// whole GPU -- latency-trivial next to the calibration passes, free of shared-memory size
// limits, and the result is unique, hence identical to any comparison sort.
// Keys are 64-bit patterns that order like the doubles they stand for: a non-negative double orders
// like its own bits; a signed one after flipping all bits of a negative value and the sign bit of
// the others.
#include "pq_common.cuh"

namespace {

// keys[j*K + i] = bit pattern of (a_i)^j (w_i)^(J-j), multiplied left to right in fp64.
__global__ void perm_keys(const double *__restrict__ sa, double rows_a, const double *__restrict__ sw,
                          double rows_w, int64_t K, int J, unsigned long long *__restrict__ keys) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= K) return;
    const double a = __ddiv_rn(sa[i], rows_a);
    const double w = __ddiv_rn(sw[i], rows_w);
    for (int j = 0; j <= J; ++j) {
        double key = 1.0;
        for (int f = 0; f < j; ++f) key = __dmul_rn(key, a);
        for (int f = 0; f < J - j; ++f) key = __dmul_rn(key, w);
        keys[static_cast<int64_t>(j) * K + i] = static_cast<unsigned long long>(__double_as_longlong(key));
    }
}

// keys[i] = bit pattern of the channel's absmax widened to fp64 (exact; non-negative).
__global__ void absmax_keys(const float *__restrict__ amax, int64_t K, unsigned long long *__restrict__ keys) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < K) keys[i] = static_cast<unsigned long long>(__double_as_longlong(static_cast<double>(fabsf(amax[i]))));
}

// keys[i] = sortable pattern of var_i = sumsq_i / rows - (sum_i / rows)^2 in fp64 (two divisions, one
// multiplication, one subtraction); the value may be slightly negative for a constant channel.
__global__ void variance_keys(const double *__restrict__ sum, const double *__restrict__ sumsq, double rows, int64_t K,
                              unsigned long long *__restrict__ keys) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i >= K) return;
    const double mean = __ddiv_rn(sum[i], rows);
    const double second = __ddiv_rn(sumsq[i], rows);
    const double var = __dadd_rn(__dsub_rn(second, __dmul_rn(mean, mean)), 0.0);  // + 0.0: a zero is +0
    const long long bits = __double_as_longlong(var);
    keys[i] = bits < 0 ? ~static_cast<unsigned long long>(bits) : static_cast<unsigned long long>(bits) | (1ull << 63);
}

// keys[i] = bit pattern of a non-negative fp64 value
__global__ void plain_keys(const double *__restrict__ v, int64_t K, unsigned long long *__restrict__ keys) {
    const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (i < K) keys[i] = static_cast<unsigned long long>(__double_as_longlong(fabs(v[i])));
}

constexpr int kRankThreads = 256;

// Four neighbouring lanes share a channel: each counts the keys of a quarter of every tile that precede the
// channel's, the four counts are added by shuffles (integers: any order).  A block ranks 64 channels.
constexpr int kRankShare = 4, kRankChannels = kRankThreads / kRankShare;

__global__ void __launch_bounds__(kRankThreads)
perm_rank(const unsigned long long *__restrict__ keys, int64_t K, int32_t *__restrict__ perms, int deal_groups, int group) {
    __shared__ unsigned long long tile[kRankThreads];
    const int j = blockIdx.y;
    const unsigned long long *kj = keys + static_cast<int64_t>(j) * K;
    const int sub = threadIdx.x % kRankShare;
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kRankChannels + threadIdx.x / kRankShare;
    const unsigned long long mine = (i < K) ? kj[i] : 0ull;
    int rank = 0;
    for (int64_t base = 0; base < K; base += kRankThreads) {
        const int64_t l = base + threadIdx.x;
        __syncthreads();
        tile[threadIdx.x] = (l < K) ? kj[l] : 0ull;
        __syncthreads();
        // the whole tile, unrolled: a slot past the end holds key 0 at an index above every channel, which
        // precedes nothing ("other precedes mine": larger key, or equal key and lower channel index)
#pragma unroll 16
        for (int u = sub; u < kRankThreads; u += kRankShare) {
            const unsigned long long other = tile[u];
            rank += (other > mine) || (other == mine && base + u < i);
        }
    }
#pragma unroll
    for (int m = 1; m < kRankShare; m <<= 1) rank += __shfl_xor_sync(0xFFFFFFFFu, rank, m);
    // deal_groups == 0: the channel of rank r is read at position r; otherwise the sorted channels are dealt
    // to deal_groups groups in turn: rank r goes to group r % deal_groups, slot r / deal_groups
    const int64_t pos = deal_groups ? static_cast<int64_t>(rank % deal_groups) * group + rank / deal_groups : rank;
    if (i < K && sub == 0) perms[static_cast<int64_t>(j) * K + pos] = static_cast<int32_t>(i);
}

// One thread per order p = 0..P sums its error rows; thread 0 then applies Eq. 10.
__global__ void accept_kernel(const double *__restrict__ ex, const double *__restrict__ ew,
                              const double *__restrict__ lambda, int P, int64_t Kg, double tau,
                              int32_t *best, int32_t *accept, double *E_out) {
    __shared__ double E[32];
    const int p = threadIdx.x;
    if (p <= P) {
        const double lx = lambda ? lambda[0] : 1.0, lw = lambda ? lambda[1] : 1.0;
        double sx = 0.0, sw = 0.0;
        for (int64_t k = 0; k < Kg; ++k) sx = __dadd_rn(sx, ex[p * Kg + k]);
        for (int64_t k = 0; k < Kg; ++k) sw = __dadd_rn(sw, ew[p * Kg + k]);
        E[p] = __dadd_rn(__dmul_rn(lx, sx), __dmul_rn(lw, sw));
        if (E_out) E_out[p] = E[p];
    }
    __syncthreads();
    if (p == 0) {
        int b = 1;
        for (int q = 2; q <= P; ++q)
            if (E[q] < E[b]) b = q;
        const double gain = __dadd_rn(E[0], -E[b]);
        const double need = __dmul_rn(tau, E[0]);
        *best = b;
        *accept = (gain > need) ? 1 : 0;
    }
}

}  // namespace

extern "C" pq_status pq_select_perm(const double *sumsq_a, int64_t rows_a, const double *sumsq_w,
                                    int64_t rows_w, int64_t K, int J, int32_t *perms, void *ws,
                                    size_t ws_bytes, void *stream) {
    PQ_REQUIRE(sumsq_a && sumsq_w && perms, PQ_ERR_NULL);
    PQ_REQUIRE(K > 0 && K <= 16384 && J >= 1 && J <= 16 && rows_a > 0 && rows_w > 0, PQ_ERR_SHAPE);
    const size_t need = pq_workspace_bytes(PQ_OP_SELECT_PERM, 0, K, 0, J + 1);
    PQ_REQUIRE(ws && ws_bytes >= need, PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long *keys = static_cast<unsigned long long *>(ws);
    perm_keys<<<static_cast<unsigned>(pq_ceil_div(K, 128)), 128, 0, st>>>(
        sumsq_a, static_cast<double>(rows_a), sumsq_w, static_cast<double>(rows_w), K, J, keys);
    dim3 grid(static_cast<unsigned>(pq_ceil_div(K, kRankChannels)), static_cast<unsigned>(J + 1));
    perm_rank<<<grid, kRankThreads, 0, st>>>(keys, K, perms, 0, 0);
    return pq_launch_status();
}

extern "C" pq_status pq_order_by_absmax(const float *amax, int64_t K, int32_t *perm, void *ws, size_t ws_bytes,
                                        void *stream) {
    PQ_REQUIRE(amax && perm, PQ_ERR_NULL);
    PQ_REQUIRE(K > 0 && K <= 16384, PQ_ERR_SHAPE);
    PQ_REQUIRE(ws && ws_bytes >= pq_workspace_bytes(PQ_OP_SELECT_PERM, 0, K, 0, 1), PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long *keys = static_cast<unsigned long long *>(ws);
    absmax_keys<<<static_cast<unsigned>(pq_ceil_div(K, 128)), 128, 0, st>>>(amax, K, keys);
    perm_rank<<<dim3(static_cast<unsigned>(pq_ceil_div(K, kRankChannels)), 1), kRankThreads, 0, st>>>(keys, K, perm, 0, 0);
    return pq_launch_status();
}

extern "C" pq_status pq_order_by_variance(const double *sum, const double *sumsq, int64_t rows, int64_t K, int32_t *perm,
                                          void *ws, size_t ws_bytes, void *stream) {
    PQ_REQUIRE(sum && sumsq && perm, PQ_ERR_NULL);
    PQ_REQUIRE(K > 0 && K <= 16384 && rows > 0, PQ_ERR_SHAPE);
    PQ_REQUIRE(ws && ws_bytes >= pq_workspace_bytes(PQ_OP_SELECT_PERM, 0, K, 0, 1), PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long *keys = static_cast<unsigned long long *>(ws);
    variance_keys<<<static_cast<unsigned>(pq_ceil_div(K, 128)), 128, 0, st>>>(sum, sumsq, static_cast<double>(rows), K, keys);
    perm_rank<<<dim3(static_cast<unsigned>(pq_ceil_div(K, kRankChannels)), 1), kRankThreads, 0, st>>>(keys, K, perm, 0, 0);
    return pq_launch_status();
}

extern "C" pq_status pq_order_round_robin(const double *sumsq, int64_t K, int group, int32_t *perm, void *ws,
                                          size_t ws_bytes, void *stream) {
    PQ_REQUIRE(sumsq && perm, PQ_ERR_NULL);
    PQ_REQUIRE(K > 0 && K <= 16384 && group > 0 && K % group == 0, PQ_ERR_SHAPE);
    PQ_REQUIRE(ws && ws_bytes >= pq_workspace_bytes(PQ_OP_SELECT_PERM, 0, K, 0, 1), PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned long long *keys = static_cast<unsigned long long *>(ws);
    plain_keys<<<static_cast<unsigned>(pq_ceil_div(K, 128)), 128, 0, st>>>(sumsq, K, keys);
    perm_rank<<<dim3(static_cast<unsigned>(pq_ceil_div(K, kRankChannels)), 1), kRankThreads, 0, st>>>(
        keys, K, perm, static_cast<int>(K / group), group);
    return pq_launch_status();
}

extern "C" pq_status pq_accept(const double *err_x, const double *err_w, const double *lambda, int P,
                               int64_t Kg, double tau, int32_t *best, int32_t *accept, double *E,
                               void *stream) {
    PQ_REQUIRE(err_x && err_w && best && accept, PQ_ERR_NULL);
    PQ_REQUIRE(P >= 1 && P <= 31 && Kg > 0, PQ_ERR_SHAPE);
    accept_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(err_x, err_w, lambda, P, Kg, tau,
                                                                  best, accept, E);
    return pq_launch_status();
}
