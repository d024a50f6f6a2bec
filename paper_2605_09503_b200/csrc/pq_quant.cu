// NVFP4 quantizers (runtime activations, offline permuted weights) and the integer fake-quant
// of Eq. 1-2.
//
// All three are streaming kernels bound by HBM bandwidth: a thread owns 8 adjacent channels
// (one 16-byte load), the TEAM = group/8 lanes that share a group reduce the absmax with
// xor-shuffles, every lane then derives the group scale redundantly and converts its own
// eight values.  A warp reads 512 contiguous bytes per load instruction and writes 128
// contiguous bytes of codes; the scale bytes of four adjacent groups are merged into one
// 32-bit store (the four bytes are adjacent in both scale layouts).
//
// The permuted variants (weights, fake-quant with a gather) stage each row in shared memory
// with coalesced 16-byte loads and gather from there, so global memory is still read once.
#include "pq_common.cuh"

namespace {

constexpr int kQuantThreads = 256;

// ---------------------------------------------------------------- activations (no gather)
// Index space: octets (8 channels) of the tensor padded to rows_pad rows; padding rows only
// write zero scale bytes (tensor-core layout), never codes.  Each warp walks the index space in
// steps of 32 octets; two independent steps are in flight per iteration (loads issued first).
struct OctetRef {
    int64_t row, oct;
    bool in_range, live;
};

__device__ __forceinline__ OctetRef locate(int64_t idx, int64_t total, int64_t oct_per_row, int64_t rows,
                                           bool small) {
    OctetRef o;
    o.in_range = idx < total;
    if (!o.in_range) {
        o.row = 0, o.oct = 0, o.live = false;
        return o;
    }
    if (small) {  // 32-bit division when the index space allows it
        const uint32_t r = static_cast<uint32_t>(idx) / static_cast<uint32_t>(oct_per_row);
        o.row = r;
        o.oct = static_cast<uint32_t>(idx) - r * static_cast<uint32_t>(oct_per_row);
    } else {
        o.row = idx / oct_per_row;
        o.oct = idx - o.row * oct_per_row;
    }
    o.live = o.row < rows;
    return o;
}

template <int SF_LAYOUT>
__device__ __forceinline__ void quant_octet(const OctetRef &o, const uint4 &v, float ts, int64_t K,
                                            int64_t kb4, bool words, uint8_t *__restrict__ codes,
                                            uint8_t *__restrict__ sf) {
    float x[8];
    pq::unpack8(v, x);
    const float amax = pq::team_max<2>(pq::absmax8(x));
    uint32_t sf8;
    float d, r;
    pq::nvfp4_scale(amax, ts, sf8, d, r);
    const uint32_t c = pq::nvfp4_codes(x, r);
    if (o.live) __stcs(reinterpret_cast<uint32_t *>(codes + o.row * (K >> 1) + o.oct * 4), c);
    // collect the scale bytes of 4 adjacent groups (lanes l, l+2, l+4, l+6) into lane l
    uint32_t word = sf8;
    word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 2) << 8;
    word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 4) << 16;
    word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 6) << 24;
    if (!o.in_range) return;
    const int64_t g = o.oct >> 1;
    if (SF_LAYOUT == PQ_SF_TCGEN05) {
        if ((threadIdx.x & 7) == 0)
            *reinterpret_cast<uint32_t *>(sf + pq::sf_tc_offset(o.row, g, kb4)) = word;
    } else if (o.live) {
        if (words) {
            if ((threadIdx.x & 7) == 0) *reinterpret_cast<uint32_t *>(sf + o.row * (K >> 4) + g) = word;
        } else if ((o.oct & 1) == 0) {
            sf[o.row * (K >> 4) + g] = static_cast<uint8_t>(sf8);
        }
    }
}

template <int SF_LAYOUT>
__global__ void __launch_bounds__(kQuantThreads)
quant_nvfp4_kernel(const uint16_t *__restrict__ X, int64_t rows, int64_t rows_pad, int64_t K,
                   int64_t ld, const float *__restrict__ ts_ptr, uint8_t *__restrict__ codes,
                   uint8_t *__restrict__ sf) {
    const float ts = __ldg(ts_ptr);
    const int64_t oct_per_row = K >> 3;
    const int64_t total = rows_pad * oct_per_row;
    const bool small = total < (1ll << 31);
    const int64_t kb4 = (K + 63) >> 6;
    const bool words = (K & 63) == 0;  // four groups per 32-bit scale store
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kQuantThreads;
    // every lane of a warp iterates the same number of times so the shuffles stay convergent
    const int64_t warp_first = (static_cast<int64_t>(blockIdx.x) * kQuantThreads + threadIdx.x) & ~31ll;
    const int lane = threadIdx.x & 31;
    const uint4 zero = make_uint4(0, 0, 0, 0);
    for (int64_t base = warp_first; base < total; base += 2 * stride) {
        const OctetRef a = locate(base + lane, total, oct_per_row, rows, small);
        const OctetRef b = locate(base + stride + lane, total, oct_per_row, rows, small);
        const uint4 va = a.live ? __ldcs(reinterpret_cast<const uint4 *>(X + a.row * ld + a.oct * 8)) : zero;
        const uint4 vb = b.live ? __ldcs(reinterpret_cast<const uint4 *>(X + b.row * ld + b.oct * 8)) : zero;
        quant_octet<SF_LAYOUT>(a, va, ts, K, kb4, words, codes, sf);
        if (base + stride < total) quant_octet<SF_LAYOUT>(b, vb, ts, K, kb4, words, codes, sf);
    }
}

// ---------------------------------------------------------------- weights
__global__ void amax_all_kernel(const uint16_t *__restrict__ W, int64_t rows, int64_t K, int64_t ld,
                                unsigned int *__restrict__ amax_bits) {
    const int64_t oct_per_row = K >> 3;
    const int64_t total = rows * oct_per_row;
    float a = 0.0f;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total;
         idx += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t row = idx / oct_per_row, oct = idx - row * oct_per_row;
        float x[8];
        pq::unpack8(__ldg(reinterpret_cast<const uint4 *>(W + row * ld + oct * 8)), x);
        a = fmaxf(a, pq::absmax8(x));
    }
    for (int m = 16; m; m >>= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, m));
    if ((threadIdx.x & 31) == 0 && a > 0.0f) atomicMax(amax_bits, __float_as_uint(a));
}

__global__ void weight_scale_kernel(const unsigned int *__restrict__ amax_bits, float *ts) {
    const float a = __uint_as_float(*amax_bits);
    *ts = (a == 0.0f) ? 1.0f : __fdiv_rn(a, 2688.0f);
}

// Resolve which order to apply: `table` is either one order [K] (select == NULL) or the
// candidate table with {best, accept} on the device.  Returns NULL for the original order.
__device__ __forceinline__ const int32_t *resolve_perm(const int32_t *table, const int32_t *select,
                                                       int64_t K) {
    if (select == nullptr) return table;
    const int32_t best = select[0], accept = select[1];
    return accept ? table + static_cast<int64_t>(best - 1) * K : nullptr;
}

// One block per row: stage the row in shared memory, gather by the order, quantize.
template <int SF_LAYOUT>
__global__ void __launch_bounds__(kQuantThreads)
quant_nvfp4_gather_kernel(const uint16_t *__restrict__ W, int64_t rows, int64_t K, int64_t ld,
                          const int32_t *__restrict__ table, const int32_t *__restrict__ select,
                          const float *__restrict__ ts_ptr, uint8_t *__restrict__ codes,
                          uint8_t *__restrict__ sf) {
    extern __shared__ __align__(16) uint16_t row_s[];
    const int32_t *perm = resolve_perm(table, select, K);
    const float ts = *ts_ptr;
    const int64_t kb4 = (K + 63) >> 6;
    const int oct_per_row = static_cast<int>(K >> 3);
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        __syncthreads();
        for (int o = threadIdx.x; o < oct_per_row; o += kQuantThreads)
            reinterpret_cast<uint4 *>(row_s)[o] = __ldg(reinterpret_cast<const uint4 *>(W + row * ld) + o);
        __syncthreads();
        for (int base = 0; base < oct_per_row; base += kQuantThreads) {
            const int oct = base + threadIdx.x;
            const bool live = oct < oct_per_row;
            float x[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int j = oct * 8 + i;
                const int ch = live ? (perm ? perm[j] : j) : 0;
                x[i] = live ? pq::bf16_bits_to_f32(row_s[ch]) : 0.0f;
            }
            const float amax = pq::team_max<2>(pq::absmax8(x));
            uint32_t sf8;
            float d, r;
            pq::nvfp4_scale(amax, ts, sf8, d, r);
            const uint32_t c = pq::nvfp4_codes(x, r);
            if (!live) continue;
            *reinterpret_cast<uint32_t *>(codes + row * (K >> 1) + oct * 4) = c;
            if ((oct & 1) == 0) {
                const int64_t g = oct >> 1;
                if (SF_LAYOUT == PQ_SF_TCGEN05) sf[pq::sf_tc_offset(row, g, kb4)] = static_cast<uint8_t>(sf8);
                else sf[row * (K >> 4) + g] = static_cast<uint8_t>(sf8);
            }
        }
    }
}

// Zero the scale bytes of the padding rows of the tensor-core layout.
__global__ void sf_zero_pad_kernel(uint8_t *sf, int64_t rows, int64_t rows_pad, int64_t K) {
    const int64_t kb4 = (K + 63) >> 6;
    const int64_t cols = kb4 * 4;
    const int64_t total = (rows_pad - rows) * cols;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total;
         idx += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t row = rows + idx / cols, col = idx % cols;
        sf[pq::sf_tc_offset(row, col, kb4)] = 0;
    }
}

// ---------------------------------------------------------------- integer fake-quant
template <int TEAM>
__device__ __forceinline__ uint4 fakequant8(const float (&x)[8], float Qf) {
    const float amax = pq::team_max<TEAM>(pq::absmax8(x));
    float s, r, z[8];
    pq::int_scale(amax, Qf, s, r);
    pq::int_levels(x, r, Qf, z);
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const uint32_t lo = __bfloat16_as_ushort(__float2bfloat16_rn(__fmul_rn(z[2 * i], s)));
        const uint32_t hi = __bfloat16_as_ushort(__float2bfloat16_rn(__fmul_rn(z[2 * i + 1], s)));
        w[i] = lo | (hi << 16);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}

template <int TEAM>
__global__ void __launch_bounds__(kQuantThreads)
fakequant_int_kernel(const uint16_t *__restrict__ T, int64_t rows, int64_t K, int64_t ld, float Qf,
                     uint16_t *__restrict__ out, int64_t ldo) {
    const int64_t oct_per_row = K >> 3;
    const int64_t total = rows * oct_per_row;
    const int64_t stride = static_cast<int64_t>(gridDim.x) * kQuantThreads;
    const int64_t warp_first = (static_cast<int64_t>(blockIdx.x) * kQuantThreads + threadIdx.x) & ~31ll;
    for (int64_t base = warp_first; base < total; base += stride) {
        const int64_t idx = base + (threadIdx.x & 31);
        const bool live = idx < total;
        const int64_t row = live ? idx / oct_per_row : 0;
        const int64_t oct = live ? idx - row * oct_per_row : 0;
        float x[8];
        if (live) {
            pq::unpack8(__ldcs(reinterpret_cast<const uint4 *>(T + row * ld + oct * 8)), x);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = 0.0f;
        }
        const uint4 o = fakequant8<TEAM>(x, Qf);
        if (live) __stcs(reinterpret_cast<uint4 *>(out + row * ldo + oct * 8), o);
    }
}

template <int TEAM>
__global__ void __launch_bounds__(kQuantThreads)
fakequant_int_gather_kernel(const uint16_t *__restrict__ T, int64_t rows, int64_t K, int64_t ld,
                            const int32_t *__restrict__ perm, float Qf, uint16_t *__restrict__ out,
                            int64_t ldo) {
    extern __shared__ __align__(16) uint16_t row_s[];
    const int oct_per_row = static_cast<int>(K >> 3);
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        __syncthreads();
        for (int o = threadIdx.x; o < oct_per_row; o += kQuantThreads)
            reinterpret_cast<uint4 *>(row_s)[o] = __ldg(reinterpret_cast<const uint4 *>(T + row * ld) + o);
        __syncthreads();
        for (int base = 0; base < oct_per_row; base += kQuantThreads) {
            const int oct = base + threadIdx.x;
            const bool live = oct < oct_per_row;
            float x[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) x[i] = live ? pq::bf16_bits_to_f32(row_s[perm[oct * 8 + i]]) : 0.0f;
            const uint4 o = fakequant8<TEAM>(x, Qf);
            if (live) *reinterpret_cast<uint4 *>(out + row * ldo + oct * 8) = o;
        }
    }
}

__global__ void sf_to_linear_kernel(const uint8_t *__restrict__ src, int64_t rows, int64_t K,
                                    uint8_t *__restrict__ dst) {
    const int64_t cols = K >> 4, kb4 = (K + 63) >> 6;
    const int64_t total = rows * cols;
    for (int64_t idx = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; idx < total;
         idx += static_cast<int64_t>(gridDim.x) * blockDim.x)
        dst[idx] = src[pq::sf_tc_offset(idx / cols, idx % cols, kb4)];
}

int grid_for(int64_t work_items, int threads, int per_sm) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int64_t want = pq_ceil_div(work_items, threads);
    const int64_t cap = static_cast<int64_t>(sms) * per_sm;
    return static_cast<int>(want < cap ? (want > 0 ? want : 1) : cap);
}

template <typename Kern>
pq_status allow_smem(Kern kern, size_t bytes) {
    if (bytes > 48 * 1024)
        PQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(bytes)));
    return PQ_OK;
}

}  // namespace

extern "C" size_t pq_sf_bytes(int64_t rows, int64_t K, int sf_layout) {
    if (rows <= 0 || K <= 0 || K % 16 != 0) return 0;
    if (sf_layout == PQ_SF_LINEAR) return static_cast<size_t>(rows * (K / 16));
    if (sf_layout == PQ_SF_TCGEN05) return static_cast<size_t>(pq_ceil_div(rows, 128) * pq_ceil_div(K, 64) * 512);
    return 0;
}

extern "C" pq_status pq_quant_act_nvfp4(const void *X, int64_t M, int64_t K, int64_t ld,
                                        const float *ts_x, uint8_t *codes, uint8_t *sf, int sf_layout,
                                        void *stream) {
    PQ_REQUIRE(X && ts_x && codes && sf, PQ_ERR_NULL);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || sf_layout == PQ_SF_TCGEN05, PQ_ERR_FORMAT);
    PQ_REQUIRE(M > 0 && K > 0 && K % 16 == 0 && ld >= K, PQ_ERR_SHAPE);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || K % 64 == 0, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(X) && ld % 8 == 0 && pq_aligned16(codes) && pq_aligned16(sf), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint16_t *x = static_cast<const uint16_t *>(X);
    if (sf_layout == PQ_SF_TCGEN05) {
        const int64_t rows_pad = pq_ceil_div(M, 128) * 128;
        const int grid = grid_for(rows_pad * (K / 8), kQuantThreads, 16);
        quant_nvfp4_kernel<PQ_SF_TCGEN05><<<grid, kQuantThreads, 0, st>>>(x, M, rows_pad, K, ld, ts_x, codes, sf);
    } else {
        const int grid = grid_for(M * (K / 8), kQuantThreads, 16);
        quant_nvfp4_kernel<PQ_SF_LINEAR><<<grid, kQuantThreads, 0, st>>>(x, M, M, K, ld, ts_x, codes, sf);
    }
    return pq_launch_status();
}

extern "C" pq_status pq_quant_weight(const void *Wt, int64_t N, int64_t K, int64_t ld,
                                     const int32_t *perm, const int32_t *perm_select, uint8_t *codes,
                                     uint8_t *sf, int sf_layout, float *ts_w, void *ws, size_t ws_bytes,
                                     void *stream) {
    PQ_REQUIRE(Wt && codes && sf && ts_w, PQ_ERR_NULL);
    PQ_REQUIRE(perm || !perm_select, PQ_ERR_NULL);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || sf_layout == PQ_SF_TCGEN05, PQ_ERR_FORMAT);
    PQ_REQUIRE(N > 0 && K > 0 && K % 16 == 0 && K <= 16384 && ld >= K, PQ_ERR_SHAPE);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || K % 64 == 0, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(Wt) && ld % 8 == 0 && pq_aligned16(codes) && pq_aligned16(sf), PQ_ERR_ALIGN);
    PQ_REQUIRE(ws && ws_bytes >= pq_workspace_bytes(PQ_OP_QUANT_WEIGHT, N, K, 0, 0), PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint16_t *w = static_cast<const uint16_t *>(Wt);
    unsigned int *amax_bits = static_cast<unsigned int *>(ws);
    PQ_CUDA_OK(cudaMemsetAsync(amax_bits, 0, sizeof(unsigned int), st));
    amax_all_kernel<<<grid_for(N * (K / 8), 256, 8), 256, 0, st>>>(w, N, K, ld, amax_bits);
    weight_scale_kernel<<<1, 1, 0, st>>>(amax_bits, ts_w);
    if (!perm) return pq_quant_act_nvfp4(Wt, N, K, ld, ts_w, codes, sf, sf_layout, stream);

    const size_t smem = static_cast<size_t>(K) * 2;
    const int grid = static_cast<int>(N < 148 * 8 ? N : 148 * 8);
    if (sf_layout == PQ_SF_TCGEN05) {
        const int64_t rows_pad = pq_ceil_div(N, 128) * 128;
        if (rows_pad > N) sf_zero_pad_kernel<<<64, 256, 0, st>>>(sf, N, rows_pad, K);
        if (allow_smem(quant_nvfp4_gather_kernel<PQ_SF_TCGEN05>, smem) != PQ_OK) return PQ_ERR_CUDA;
        quant_nvfp4_gather_kernel<PQ_SF_TCGEN05><<<grid, kQuantThreads, smem, st>>>(
            w, N, K, ld, perm, perm_select, ts_w, codes, sf);
    } else {
        if (allow_smem(quant_nvfp4_gather_kernel<PQ_SF_LINEAR>, smem) != PQ_OK) return PQ_ERR_CUDA;
        quant_nvfp4_gather_kernel<PQ_SF_LINEAR><<<grid, kQuantThreads, smem, st>>>(
            w, N, K, ld, perm, perm_select, ts_w, codes, sf);
    }
    return pq_launch_status();
}

extern "C" pq_status pq_fakequant_int(const void *T, int64_t rows, int64_t K, int64_t ld, pq_format fmt,
                                      const int32_t *perm, void *out, int64_t ldo, void *stream) {
    PQ_REQUIRE(T && out, PQ_ERR_NULL);
    PQ_REQUIRE(fmt.kind == 1 && fmt.bits >= 2 && fmt.bits <= 8, PQ_ERR_FORMAT);
    PQ_REQUIRE(fmt.group == 16 || fmt.group == 32 || fmt.group == 64 || fmt.group == 128, PQ_ERR_FORMAT);
    PQ_REQUIRE(rows > 0 && K > 0 && K % fmt.group == 0 && ld >= K && ldo >= K, PQ_ERR_SHAPE);
    PQ_REQUIRE(!perm || K <= 16384, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(T) && pq_aligned16(out) && ld % 8 == 0 && ldo % 8 == 0, PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint16_t *t = static_cast<const uint16_t *>(T);
    uint16_t *o = static_cast<uint16_t *>(out);
    const float Qf = static_cast<float>((1 << (fmt.bits - 1)) - 1);
    const size_t smem = static_cast<size_t>(K) * 2;
    const int grid_g = static_cast<int>(rows < 148 * 8 ? rows : 148 * 8);
    const int grid = grid_for(rows * (K / 8), kQuantThreads, 16);
#define PQ_FQ_CASE(TEAM)                                                                              \
    if (perm) {                                                                                       \
        if (allow_smem(fakequant_int_gather_kernel<TEAM>, smem) != PQ_OK) return PQ_ERR_CUDA;         \
        fakequant_int_gather_kernel<TEAM><<<grid_g, kQuantThreads, smem, st>>>(t, rows, K, ld, perm, Qf, o, ldo); \
    } else {                                                                                          \
        fakequant_int_kernel<TEAM><<<grid, kQuantThreads, 0, st>>>(t, rows, K, ld, Qf, o, ldo);        \
    }
    switch (fmt.group) {
        case 16: PQ_FQ_CASE(2) break;
        case 32: PQ_FQ_CASE(4) break;
        case 64: PQ_FQ_CASE(8) break;
        default: PQ_FQ_CASE(16) break;
    }
#undef PQ_FQ_CASE
    return pq_launch_status();
}

extern "C" pq_status pq_sf_to_linear(const uint8_t *sf_tc, int64_t rows, int64_t K, uint8_t *sf_linear,
                                     void *stream) {
    PQ_REQUIRE(sf_tc && sf_linear, PQ_ERR_NULL);
    PQ_REQUIRE(rows > 0 && K > 0 && K % 64 == 0, PQ_ERR_SHAPE);
    sf_to_linear_kernel<<<grid_for(rows * (K / 16), 256, 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        sf_tc, rows, K, sf_linear);
    return pq_launch_status();
}
