// NVFP4 quantizers (runtime activations, offline permuted weights) and the integer fake-quant
// of Eq. 1-2.
//
// All three are streaming kernels bound by HBM bandwidth.  The activation quantizer gives a thread a
// whole 16-channel group (one 32-byte load, no shuffles; a warp reads 1 KB of a row per instruction
// and writes 256 contiguous bytes of codes).  The fake-quant kernels give a thread 8 adjacent
// channels (one 16-byte load); the TEAM = group/8 lanes that share a group reduce the absmax with
// xor-shuffles, every lane then derives the group scale redundantly and converts its own values.
//
// The permuted variants (weights, fake-quant with a gather) stage each row in shared memory
// with coalesced 16-byte loads and gather from there, so global memory is still read once.  For
// NVFP4 and rows of up to 6400 channels the gather runs in the fused producer's kernel (pq_norm.cu,
// four rows per warp sharing indices and gathers) with its normalization compiled out.
#include "pq_common.cuh"

namespace {

constexpr int kQuantThreads = 256;
constexpr int kTileRows = 8;                    // blocks of the streaming kernels: 32 lanes along K x 8 rows
// The activation quantizer comes in two block shapes: 8 warps (best alone) and 4 warps, one per SM
// sub-partition at 32 registers, which is what fits on an SM beside a GEMM CTA (batched linear path).
constexpr int kActThreads = 32 * kTileRows;
constexpr unsigned kGridYMax = 65535;

// Row block of a (x = column chunk, y/z = row block) grid; y alone is limited to 65535 blocks.
__device__ __forceinline__ int64_t row_block_index() {
    return static_cast<int64_t>(blockIdx.z) * kGridYMax + blockIdx.y;
}
inline dim3 tile_grid(int64_t col_chunks, int64_t row_blocks) {
    const int64_t z = pq_ceil_div(row_blocks, kGridYMax);
    return dim3(static_cast<unsigned>(col_chunks), static_cast<unsigned>(row_blocks < kGridYMax ? row_blocks : kGridYMax),
                static_cast<unsigned>(z));
}

// ---------------------------------------------------------------- activations (no gather)
// One thread per 16-channel group: a 32-byte load (one 256-bit instruction when the tensor is
// 32-byte aligned), the group's absmax (on the bf16 pairs), scale and codes in registers (packed fp32
// multiplies), an 8-byte store of codes and a one-byte store of the scale.  The index space covers the rows padded to a multiple of 128
// in the tensor-core layout; padding rows only write zero scale bytes.  A block owns 8 (or 4) rows x 32
// consecutive groups (a warp = 1 KB of one row), so no thread divides anything.
template <bool WIDE>
__device__ __forceinline__ void load_group(const uint16_t *p, uint4 &lo, uint4 &hi) {
    if (WIDE) {
        asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                     : "=r"(lo.x), "=r"(lo.y), "=r"(lo.z), "=r"(lo.w), "=r"(hi.x), "=r"(hi.y), "=r"(hi.z), "=r"(hi.w)
                     : "l"(p));
    } else {
        lo = __ldcs(reinterpret_cast<const uint4 *>(p));
        hi = __ldcs(reinterpret_cast<const uint4 *>(p) + 1);
    }
}

#ifndef PQ_ACT_ROWS
#define PQ_ACT_ROWS 1
#endif
constexpr int kActRows = PQ_ACT_ROWS;  // rows per thread: their loads are issued together

// 32 registers per thread (eight 256-thread blocks per SM): all 2048 thread slots of an SM carry a load
template <int SF_LAYOUT, bool WIDE, int kActTileRows>
__global__ void __launch_bounds__(kActThreads, 2048 / kActThreads)
quant_nvfp4_kernel(const uint16_t *__restrict__ X, int64_t rows, int64_t rows_pad, int64_t K,
                   int64_t ld, const float *__restrict__ ts_ptr, uint8_t *__restrict__ codes,
                   uint8_t *__restrict__ sf) {
    const uint32_t gpr = static_cast<uint32_t>(K >> 4);  // groups per row
    const uint32_t g = blockIdx.x * 32u + threadIdx.x;
    const int64_t row0 = row_block_index() * (kActTileRows * kActRows) + threadIdx.y;
    // This kernel is launched as a programmatic dependent of whatever precedes it in the stream:
    // its blocks may become resident while that kernel's last blocks run, and wait here until it
    // has completed and its writes are visible (ordinary stream order from here on).  In turn a
    // programmatic dependent of this kernel (the GEMM of pq_linear_w4a4) may begin its set-up now;
    // it waits for this grid to complete before reading the results.
    pq::wait_for_prior_grid();
    pq::dependents_may_launch();
    const float ts = __ldg(ts_ptr);

    uint4 lo[kActRows], hi[kActRows];
#pragma unroll
    for (int i = 0; i < kActRows; ++i) {
        const int64_t row = row0 + i * kActTileRows;
        lo[i] = make_uint4(0, 0, 0, 0), hi[i] = lo[i];
        if (row < rows && g < gpr) load_group<WIDE>(X + row * ld + static_cast<int64_t>(g) * 16, lo[i], hi[i]);
    }
#pragma unroll
    for (int i = 0; i < kActRows; ++i) {
        const int64_t row = row0 + i * kActTileRows;
        const bool in_range = row < rows_pad && g < gpr, live = row < rows && g < gpr;
        // group absmax on the bf16 pairs (a maximum of magnitudes selects one of its inputs: exact)
        const uint32_t m = 0x7FFF7FFFu;
        const uint32_t mx = pq::max_bf16x2(pq::max_bf16x2(pq::max_bf16x2(lo[i].x & m, lo[i].y & m), pq::max_bf16x2(lo[i].z & m, lo[i].w & m)),
                                           pq::max_bf16x2(pq::max_bf16x2(hi[i].x & m, hi[i].y & m), pq::max_bf16x2(hi[i].z & m, hi[i].w & m)));
        const float amax = fmaxf(__uint_as_float(mx << 16), __uint_as_float(mx & 0xFFFF0000u));
        uint32_t sf8;
        float d, r;
        pq::nvfp4_scale(amax, ts, sf8, d, r);
        const uint32_t c0 = pq::nvfp4_codes_packed(lo[i], r), c1 = pq::nvfp4_codes_packed(hi[i], r);
        // an ordinary store: the GEMM reads the codes next, they should stay in L2 (a streaming store measured
        // 0.2 us more on quantize + GEMM)
        if (live) *reinterpret_cast<uint2 *>(codes + row * (K >> 1) + static_cast<int64_t>(g) * 8) = make_uint2(c0, c1);
        // one scale byte per thread: the lanes of a warp write runs of four adjacent bytes (adjacent in both
        // layouts) in one instruction; padding rows of the tensor-core layout get zeros
        if (!in_range) continue;
        if (SF_LAYOUT == PQ_SF_TCGEN05) sf[pq::sf_tc_offset(row, g, gpr >> 2)] = static_cast<uint8_t>(sf8);
        else if (live) sf[row * gpr + g] = static_cast<uint8_t>(sf8);
    }
}

// ---------------------------------------------------------------- weights
// blockDim (32, 8): lane = 8 adjacent channels, threadIdx.y + blockIdx.y strides over the rows.
__global__ void amax_all_kernel(const uint16_t *__restrict__ W, int64_t rows, int64_t K, int64_t ld,
                                unsigned int *__restrict__ amax_bits) {
    const int64_t oct = static_cast<int64_t>(blockIdx.x) * 32 + threadIdx.x;
    // a maximum of magnitudes selects one of its inputs, so it is taken on the bf16 pairs and in any order:
    // four rows in flight per step
    uint32_t mx = 0;
    if (oct * 8 < K) {
        const int64_t step = static_cast<int64_t>(gridDim.y) * kTileRows;
        for (int64_t row = static_cast<int64_t>(blockIdx.y) * kTileRows + threadIdx.y; row < rows; row += 4 * step) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u)
                v[u] = row + u * step < rows ? __ldg(reinterpret_cast<const uint4 *>(W + (row + u * step) * ld + oct * 8))
                                             : make_uint4(0, 0, 0, 0);
            const uint32_t m = 0x7FFF7FFFu;
#pragma unroll
            for (int u = 0; u < 4; ++u)
                mx = pq::max_bf16x2(mx, pq::max_bf16x2(pq::max_bf16x2(v[u].x & m, v[u].y & m), pq::max_bf16x2(v[u].z & m, v[u].w & m)));
        }
    }
    float a = fmaxf(__uint_as_float(mx << 16), __uint_as_float(mx & 0xFFFF0000u));
    for (int m = 16; m; m >>= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, m));
    // one atomic per block (all of them hit the same word)
    __shared__ float warp_max[kTileRows];
    if (threadIdx.x == 0) warp_max[threadIdx.y] = a;
    __syncthreads();
    if (threadIdx.x == 0 && threadIdx.y == 0) {
#pragma unroll
        for (int w = 1; w < kTileRows; ++w) a = fmaxf(a, warp_max[w]);
        if (a > 0.0f) atomicMax(amax_bits, __float_as_uint(a));
    }
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

// blockDim (32, 8): a warp = 32 adjacent octets (512 bytes) of one row; teams never straddle a
// warp (K % (8 TEAM) == 0 and 32 % TEAM == 0), dead lanes carry zeros through the shuffles.
template <int TEAM>
__global__ void __launch_bounds__(kQuantThreads)
fakequant_int_kernel(const uint16_t *__restrict__ T, int64_t rows, int64_t K, int64_t ld, float Qf,
                     uint16_t *__restrict__ out, int64_t ldo) {
    const int64_t oct = static_cast<int64_t>(blockIdx.x) * 32 + threadIdx.x;
    const int64_t row = row_block_index() * kTileRows + threadIdx.y;
    const bool live = row < rows && oct * 8 < K;
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

namespace {
template <int TILE_ROWS>
pq_status quant_act_launch(const uint16_t *x, int64_t M, int64_t K, int64_t ld, const float *ts_x, uint8_t *codes,
                           uint8_t *sf, int sf_layout, bool wide, cudaStream_t st) {
    const int64_t rows_idx = sf_layout == PQ_SF_TCGEN05 ? pq_ceil_div(M, 128) * 128 : M;
    PQ_REQUIRE(K / 16 <= 32ll * 0x7FFFFFFF && rows_idx / TILE_ROWS < static_cast<int64_t>(kGridYMax) * 65535, PQ_ERR_SHAPE);
    const dim3 grid = tile_grid(pq_ceil_div(K / 16, 32), pq_ceil_div(rows_idx, TILE_ROWS * kActRows));
    const dim3 block(32, TILE_ROWS);
    // The quantizer's blocks should be able to run on an SM beside a GEMM CTA (the batched linear
    // path overlaps the two kernels): ask for the GEMM's shared-memory carve-out, otherwise an SM
    // has to drain before it can switch between the two configurations.
    static PqPerDevice carveout;
    const int dev = pq_device_slot();
    if (dev >= 0) {
        std::lock_guard<std::mutex> guard(carveout.lock);
        if (!carveout.value[dev]) {
            cudaFuncSetAttribute(quant_nvfp4_kernel<PQ_SF_TCGEN05, true, TILE_ROWS>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
            cudaFuncSetAttribute(quant_nvfp4_kernel<PQ_SF_TCGEN05, false, TILE_ROWS>, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
            (void)cudaGetLastError();
            carveout.value[dev] = 1;
        }
    }
    if (sf_layout == PQ_SF_TCGEN05) {
        if (wide) PQ_CUDA_OK(pq::launch_dependent(quant_nvfp4_kernel<PQ_SF_TCGEN05, true, TILE_ROWS>, grid, block, 0, st, x, M, rows_idx, K, ld, ts_x, codes, sf));
        else PQ_CUDA_OK(pq::launch_dependent(quant_nvfp4_kernel<PQ_SF_TCGEN05, false, TILE_ROWS>, grid, block, 0, st, x, M, rows_idx, K, ld, ts_x, codes, sf));
    } else {
        if (wide) PQ_CUDA_OK(pq::launch_dependent(quant_nvfp4_kernel<PQ_SF_LINEAR, true, TILE_ROWS>, grid, block, 0, st, x, M, rows_idx, K, ld, ts_x, codes, sf));
        else PQ_CUDA_OK(pq::launch_dependent(quant_nvfp4_kernel<PQ_SF_LINEAR, false, TILE_ROWS>, grid, block, 0, st, x, M, rows_idx, K, ld, ts_x, codes, sf));
    }
    return pq_launch_status();
}
}  // namespace

// small_blocks != 0: 128-thread blocks, for running beside a GEMM (used by the batched linear path)
pq_status pq_quant_act_nvfp4_shaped(const void *X, int64_t M, int64_t K, int64_t ld, const float *ts_x, uint8_t *codes,
                                    uint8_t *sf, int sf_layout, int small_blocks, void *stream) {
    PQ_REQUIRE(X && ts_x && codes && sf, PQ_ERR_NULL);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || sf_layout == PQ_SF_TCGEN05, PQ_ERR_FORMAT);
    PQ_REQUIRE(M > 0 && K > 0 && K % 16 == 0 && ld >= K, PQ_ERR_SHAPE);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || K % 64 == 0, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(X) && ld % 8 == 0 && pq_aligned16(codes) && pq_aligned16(sf), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint16_t *x = static_cast<const uint16_t *>(X);
    // 256-bit loads need 32-byte aligned groups
    const bool wide = (reinterpret_cast<uintptr_t>(X) & 31u) == 0 && ld % 16 == 0;
    return small_blocks ? quant_act_launch<4>(x, M, K, ld, ts_x, codes, sf, sf_layout, wide, st)
                        : quant_act_launch<kTileRows>(x, M, K, ld, ts_x, codes, sf, sf_layout, wide, st);
}

extern "C" pq_status pq_quant_act_nvfp4(const void *X, int64_t M, int64_t K, int64_t ld,
                                        const float *ts_x, uint8_t *codes, uint8_t *sf, int sf_layout,
                                        void *stream) {
    return pq_quant_act_nvfp4_shaped(X, M, K, ld, ts_x, codes, sf, sf_layout, 0, stream);
}

// Gather by an order (a row of the candidate table, or the one `select` names) and quantize with
// the tensor scale at ts.
static pq_status launch_gather(const uint16_t *w, int64_t N, int64_t K, int64_t ld, const int32_t *perm,
                               const int32_t *perm_select, const float *ts, uint8_t *codes, uint8_t *sf,
                               int sf_layout, cudaStream_t st) {
    const size_t smem = static_cast<size_t>(K) * 2;
    const int grid = static_cast<int>(N < 148 * 8 ? N : 148 * 8);
    if (sf_layout == PQ_SF_TCGEN05) {
        const int64_t rows_pad = pq_ceil_div(N, 128) * 128;
        if (rows_pad > N) sf_zero_pad_kernel<<<64, 256, 0, st>>>(sf, N, rows_pad, K);
        if (allow_smem(quant_nvfp4_gather_kernel<PQ_SF_TCGEN05>, smem) != PQ_OK) return PQ_ERR_CUDA;
        quant_nvfp4_gather_kernel<PQ_SF_TCGEN05><<<grid, kQuantThreads, smem, st>>>(
            w, N, K, ld, perm, perm_select, ts, codes, sf);
    } else {
        if (allow_smem(quant_nvfp4_gather_kernel<PQ_SF_LINEAR>, smem) != PQ_OK) return PQ_ERR_CUDA;
        quant_nvfp4_gather_kernel<PQ_SF_LINEAR><<<grid, kQuantThreads, smem, st>>>(
            w, N, K, ld, perm, perm_select, ts, codes, sf);
    }
    return pq_launch_status();
}

extern "C" pq_status pq_quant_act_nvfp4_perm(const void *X, int64_t M, int64_t K, int64_t ld, const int32_t *perm,
                                             const float *ts_x, uint8_t *codes, uint8_t *sf, int sf_layout,
                                             void *stream) {
    if (!perm) return pq_quant_act_nvfp4(X, M, K, ld, ts_x, codes, sf, sf_layout, stream);
    PQ_REQUIRE(X && ts_x && codes && sf, PQ_ERR_NULL);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || sf_layout == PQ_SF_TCGEN05, PQ_ERR_FORMAT);
    PQ_REQUIRE(M > 0 && K > 0 && K % 16 == 0 && K <= 16384 && ld >= K, PQ_ERR_SHAPE);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || K % 64 == 0, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(X) && ld % 8 == 0 && pq_aligned16(codes) && pq_aligned16(sf), PQ_ERR_ALIGN);
    // rows of up to 6400 channels: four rows per warp share the indices and one gather (the fused producer's
    // kernel without its normalization); wider rows, or an index vector it cannot load 16 bytes at a time: one
    // block per row
    if (pq_gather_quant_grouped_fits(K) && pq_aligned16(perm))
        return pq_gather_quant_grouped(X, M, K, ld, perm, nullptr, ts_x, codes, sf, sf_layout, stream);
    return launch_gather(static_cast<const uint16_t *>(X), M, K, ld, perm, nullptr, ts_x, codes, sf, sf_layout,
                         static_cast<cudaStream_t>(stream));
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
    {
        // column chunks x enough row strides to fill the GPU (8 blocks per SM)
        const int64_t chunks = pq_ceil_div(K / 8, 32);
        const int64_t want_y = pq_ceil_div(grid_for(N * (K / 8), 256, 8), chunks);
        const int64_t max_y = pq_ceil_div(N, kTileRows);
        const int64_t gy = want_y < max_y ? (want_y > 0 ? want_y : 1) : max_y;
        amax_all_kernel<<<dim3(static_cast<unsigned>(chunks), static_cast<unsigned>(gy < kGridYMax ? gy : kGridYMax)),
                          dim3(32, kTileRows), 0, st>>>(w, N, K, ld, amax_bits);
    }
    weight_scale_kernel<<<1, 1, 0, st>>>(amax_bits, ts_w);
    if (!perm) return pq_quant_act_nvfp4(Wt, N, K, ld, ts_w, codes, sf, sf_layout, stream);
    // rows of up to 6400 channels: four rows per warp share the indices and one gather
    if (pq_gather_quant_grouped_fits(K) && pq_aligned16(perm))
        return pq_gather_quant_grouped(Wt, N, K, ld, perm, perm_select, ts_w, codes, sf, sf_layout, stream);
    return launch_gather(w, N, K, ld, perm, perm_select, ts_w, codes, sf, sf_layout, st);
}

extern "C" pq_status pq_fakequant_int(const void *T, int64_t rows, int64_t K, int64_t ld, pq_format fmt,
                                      const int32_t *perm, void *out, int64_t ldo, void *stream) {
    PQ_REQUIRE(T && out, PQ_ERR_NULL);
    PQ_REQUIRE(fmt.kind == 1 && fmt.bits >= 2 && fmt.bits <= 8, PQ_ERR_FORMAT);
    PQ_REQUIRE(fmt.group == 16 || fmt.group == 32 || fmt.group == 64 || fmt.group == 128 || fmt.group == 256, PQ_ERR_FORMAT);
    PQ_REQUIRE(rows > 0 && K > 0 && K % fmt.group == 0 && ld >= K && ldo >= K, PQ_ERR_SHAPE);
    PQ_REQUIRE(!perm || K <= 16384, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(T) && pq_aligned16(out) && ld % 8 == 0 && ldo % 8 == 0, PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint16_t *t = static_cast<const uint16_t *>(T);
    uint16_t *o = static_cast<uint16_t *>(out);
    const float Qf = static_cast<float>((1 << (fmt.bits - 1)) - 1);
    const size_t smem = static_cast<size_t>(K) * 2;
    const int grid_g = static_cast<int>(rows < 148 * 8 ? rows : 148 * 8);
    PQ_REQUIRE(rows / kTileRows < static_cast<int64_t>(kGridYMax) * 65535, PQ_ERR_SHAPE);
    const dim3 grid = tile_grid(pq_ceil_div(K / 8, 32), pq_ceil_div(rows, kTileRows));
#define PQ_FQ_CASE(TEAM)                                                                              \
    if (perm) {                                                                                       \
        if (allow_smem(fakequant_int_gather_kernel<TEAM>, smem) != PQ_OK) return PQ_ERR_CUDA;         \
        fakequant_int_gather_kernel<TEAM><<<grid_g, kQuantThreads, smem, st>>>(t, rows, K, ld, perm, Qf, o, ldo); \
    } else {                                                                                          \
        fakequant_int_kernel<TEAM><<<grid, dim3(32, kTileRows), 0, st>>>(t, rows, K, ld, Qf, o, ldo); \
    }
    switch (fmt.group) {
        case 16: PQ_FQ_CASE(2) break;
        case 32: PQ_FQ_CASE(4) break;
        case 64: PQ_FQ_CASE(8) break;
        case 128: PQ_FQ_CASE(16) break;
        default: PQ_FQ_CASE(32) break;
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
