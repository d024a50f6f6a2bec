// Shared device/host helpers of the CUDA library: argument checks, bf16 unpacking and the
// NVFP4 / integer group arithmetic used by the quantize, fake-quant and error kernels.
//
// Arithmetic contract (bit-exactness with the CPU definition depends on it): no fast-math,
// denormals kept, IEEE division and reciprocal, fused multiply-add only where written.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "../../include/pq.h"

#define PQ_REQUIRE(cond, code) \
    do {                       \
        if (!(cond)) return (code); \
    } while (0)

// Records which CUDA call failed (readable through pq_last_error_detail) -- defined in pq_api.cu.
void pq_note_cuda_error(cudaError_t err, const char *what, int line);

#define PQ_CUDA_OK(expr)                                     \
    do {                                                     \
        const cudaError_t pq_err_ = (expr);                  \
        if (pq_err_ != cudaSuccess) {                        \
            pq_note_cuda_error(pq_err_, #expr, __LINE__);    \
            (void)cudaGetLastError();                        \
            return PQ_ERR_CUDA;                              \
        }                                                    \
    } while (0)

static inline bool pq_aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static inline bool pq_aligned256(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }

static inline pq_status pq_launch_status() {
    const cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) return PQ_OK;
    pq_note_cuda_error(e, "kernel launch", 0);
    return PQ_ERR_CUDA;
}

static inline int64_t pq_ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Kernel attributes (shared-memory opt-in, carve-out) and occupancy answers belong to a device, not
// to the process: a cache of them is indexed by the current device's ordinal and guarded by a lock.
constexpr int kPqMaxDevices = 64;
struct PqPerDevice {
    std::mutex lock;
    int value[kPqMaxDevices] = {};  // 0 = not set up on that device yet
};
// Index of the current device in such a cache, or -1.
static inline int pq_device_slot() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kPqMaxDevices) return -1;
    return dev;
}

// pq_quant_act_nvfp4 with a choice of block shape (library-internal; defined in pq_quant.cu).
pq_status pq_quant_act_nvfp4_shaped(const void *X, int64_t M, int64_t K, int64_t ld, const float *ts_x, uint8_t *codes,
                                    uint8_t *sf, int sf_layout, int small_blocks, void *stream);

// The gather quantizers (pq_quant_act_nvfp4_perm, pq_quant_weight) through the four-rows-per-warp producer
// kernel without a normalization (library-internal; defined in pq_norm.cu).  perm / perm_select as for
// pq_quant_weight; perm 16-byte aligned; arguments already validated by the caller.
bool pq_gather_quant_grouped_fits(int64_t K);
pq_status pq_gather_quant_grouped(const void *X, int64_t M, int64_t K, int64_t ld, const int32_t *perm,
                                  const int32_t *perm_select, const float *ts_x, uint8_t *codes, uint8_t *sf,
                                  int sf_layout, void *stream);

#ifdef __CUDACC__

namespace pq {

// Eight consecutive bf16 values (one 16-byte load) widened to fp32 (exact).
__device__ __forceinline__ void unpack8(const uint4 &v, float (&x)[8]) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
}

__device__ __forceinline__ float bf16_bits_to_f32(uint16_t h) {
    return __uint_as_float(static_cast<uint32_t>(h) << 16);
}

__device__ __forceinline__ float absmax8(const float (&x)[8]) {
    float a = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) a = fmaxf(a, fabsf(x[i]));
    return a;
}

// Maximum over the TEAM consecutive lanes (TEAM = channels per group / 8) a group spans.
template <int TEAM>
__device__ __forceinline__ float team_max(float a) {
#pragma unroll
    for (int m = 1; m < TEAM; m <<= 1) a = fmaxf(a, __shfl_xor_sync(0xFFFFFFFFu, a, m));
    return a;
}

// Balanced adjacent-pair tree over the team's run sums; every lane ends with the same value
// because fp32 addition is commutative.
template <int TEAM>
__device__ __forceinline__ float team_sum(float o) {
#pragma unroll
    for (int m = 1; m < TEAM; m <<= 1) o = __fadd_rn(o, __shfl_xor_sync(0xFFFFFFFFu, o, m));
    return o;
}

// fp32 -> unsigned E4M3 byte, round to nearest even, saturating at 448 (hardware convert).
__device__ __forceinline__ uint32_t f32_to_e4m3(float u) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(0.0f), "f"(u));
    return r & 0xFFu;
}

// E4M3 byte -> fp32 (exact: through the hardware e4m3 -> f16 convert).
__device__ __forceinline__ float e4m3_to_f32(uint32_t b) {
    uint32_t h2;
    asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(static_cast<uint16_t>(b)));
    return __half2float(__ushort_as_half(static_cast<uint16_t>(h2 & 0xFFFFu)));
}

// Eight fp32 -> eight E2M1 nibbles (element i in bits 4i..4i+3), RNE, saturating, sign kept.
__device__ __forceinline__ uint32_t f32x8_to_e2m1(const float (&y)[8]) {
    uint32_t out;
    asm("{\n"
        ".reg .b8 b0, b1, b2, b3;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b0, %2, %1;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b1, %4, %3;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b2, %6, %5;\n"
        "cvt.rn.satfinite.e2m1x2.f32 b3, %8, %7;\n"
        "mov.b32 %0, {b0, b1, b2, b3};\n"
        "}\n"
        : "=r"(out)
        : "f"(y[0]), "f"(y[1]), "f"(y[2]), "f"(y[3]), "f"(y[4]), "f"(y[5]), "f"(y[6]), "f"(y[7]));
    return out;
}

// Eight E2M1 nibbles -> their fp32 values.  Twice the magnitude of code m is the m-th nibble of
// 0xC8643210 (0, 1, 2, 3, 4, 6, 8, 12); the int -> float conversion and the halving are exact.
__device__ __forceinline__ void e2m1x8_to_f32(uint32_t codes, float (&q)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint32_t c = (codes >> (4 * i)) & 0xFu;
        const uint32_t twice = (0xC8643210u >> ((c & 7u) * 4)) & 0xFu;
        const float mag = __fmul_rn(static_cast<float>(twice), 0.5f);
        q[i] = __uint_as_float(__float_as_uint(mag) | ((c & 8u) << 28));
    }
}

// NVFP4 scale of one group from its absmax: E4M3 byte and fp32 decode scale d = sf * ts.
__device__ __forceinline__ void nvfp4_scale(float amax, float ts, uint32_t &sf8, float &d, float &r) {
    const float c = __fmul_rn(6.0f, ts);
    const float u = __fdiv_rn(amax, c);
    sf8 = f32_to_e4m3(u);
    d = __fmul_rn(e4m3_to_f32(sf8), ts);
    r = (d > 0.0f) ? __frcp_rn(d) : 0.0f;
}

// NVFP4 codes of this lane's eight values given the group's reciprocal decode scale.
__device__ __forceinline__ uint32_t nvfp4_codes(const float (&x)[8], float r) {
    float y[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = __fmul_rn(x[i], r);
    return f32x8_to_e2m1(y);
}

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// NVFP4 codes of eight bf16 values (four packed pairs) given the group's reciprocal decode scale: widen,
// multiply in fp32 two at a time (packed f32x2: two IEEE products per instruction), convert.
__device__ __forceinline__ uint32_t nvfp4_codes_packed(const uint4 &v, float r) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    uint64_t r2;
    asm("mov.b64 %0, {%1, %1};" : "=l"(r2) : "f"(r));
    float y[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint64_t x2, p;
        asm("mov.b64 %0, {%1, %2};" : "=l"(x2) : "r"(w[i] << 16), "r"(w[i] & 0xFFFF0000u));
        asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(p) : "l"(x2), "l"(r2));
        asm("mov.b64 {%0, %1}, %2;" : "=f"(y[2 * i]), "=f"(y[2 * i + 1]) : "l"(p));
    }
    return f32x8_to_e2m1(y);
}

// Integer quantizer of Eq. 1-2: s = amax / Q, z = clamp(rint(x * (1/s)), -Q, Q).
__device__ __forceinline__ void int_scale(float amax, float Qf, float &s, float &r) {
    s = __fdiv_rn(amax, Qf);
    r = (s > 0.0f) ? __frcp_rn(s) : 0.0f;
}

__device__ __forceinline__ void int_levels(const float (&x)[8], float r, float Qf, float (&z)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        float q = rintf(__fmul_rn(x[i], r));
        z[i] = fminf(fmaxf(q, -Qf), Qf);
    }
}

// Sum of squared residuals of eight values: delta = fma(-q, d, x); acc = fma(delta, delta, acc).
__device__ __forceinline__ float run_sse(const float (&x)[8], const float (&q)[8], float d) {
    float acc = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float delta = __fmaf_rn(-q[i], d, x[i]);
        acc = __fmaf_rn(delta, delta, acc);
    }
    return acc;
}

// ---- error path on magnitudes.  (x - q d)^2 does not depend on the common sign of x and q, so the
// error kernels quantize |x| and skip the sign handling; every operation below is sign-symmetric
// (round to nearest even), hence the squares equal those of the signed computation bit for bit.

// |x| * r rounded to E2M1, returned as the fp32 values of the codes.  The decode is a byte-table
// lookup: for code c (0..7) the bf16 pattern of its value {0, .5, 1, 1.5, 2, 3, 4, 6} is
// {0x0000, 0x3F00, 0x3F80, 0x3FC0, 0x4000, 0x4040, 0x4080, 0x40C0}; prmt picks the high and low
// bytes with the four codes of a 16-bit half as selectors, a second prmt interleaves them into
// bf16 pairs, and a bf16 widens to fp32 by a shift.
__device__ __forceinline__ void e2m1_levels(uint32_t codes, float (&q)[8]);
__device__ __forceinline__ void nvfp4_levels_abs(const float (&x)[8], float r, float (&q)[8]) {
    float y[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) y[i] = __fmul_rn(fabsf(x[i]), r);
    e2m1_levels(f32x8_to_e2m1(y), q);
}

// Eight E2M1 codes of non-negative values -> their fp32 magnitudes (the byte tables above).
__device__ __forceinline__ void e2m1_levels(uint32_t codes, float (&q)[8]) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const uint32_t sel = h ? codes >> 16 : codes & 0xFFFFu;
        const uint32_t hi = __byte_perm(0x3F3F3F00u, 0x40404040u, sel);
        const uint32_t lo = __byte_perm(0xC0800000u, 0xC0804000u, sel);
        const uint32_t p01 = __byte_perm(lo, hi, 0x5140u), p23 = __byte_perm(lo, hi, 0x7362u);
        q[4 * h + 0] = __uint_as_float(p01 << 16);
        q[4 * h + 1] = __uint_as_float(p01 & 0xFFFF0000u);
        q[4 * h + 2] = __uint_as_float(p23 << 16);
        q[4 * h + 3] = __uint_as_float(p23 & 0xFFFF0000u);
    }
}

// min(rint(|x| * r), Q).  For |y| < 2^22 adding and subtracting 1.5 * 2^23 rounds to the nearest
// integer, ties to even, exactly like rint; beyond that (and for inf) the result is at least Q and
// the clamp takes over; NaN (0 * inf) goes to -Q in the signed definition (fmaxf drops the NaN),
// i.e. to magnitude Q, which fminf(NaN, Q) gives here as well.
__device__ __forceinline__ void int_levels_abs(const float (&x)[8], float r, float Qf, float (&z)[8]) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float y = __fmul_rn(fabsf(x[i]), r);
        const float q = __fadd_rn(__fadd_rn(y, 12582912.0f), -12582912.0f);
        z[i] = fminf(q, Qf);
    }
}

// Sum of squared residuals of eight magnitudes: delta = fma(-q, d, |x|); acc = fma(delta, delta, acc).
__device__ __forceinline__ float run_sse_abs(const float (&x)[8], const float (&q)[8], float d) {
    float acc = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const float delta = __fmaf_rn(-q[i], d, fabsf(x[i]));
        acc = __fmaf_rn(delta, delta, acc);
    }
    return acc;
}

// Byte offset of scale (row, col) in the tensor-core layout; kb4 = number of 4-column blocks.
__device__ __host__ __forceinline__ int64_t sf_tc_offset(int64_t row, int64_t col, int64_t kb4) {
    return ((row >> 7) * kb4 + (col >> 2)) * 512 + (row & 31) * 16 + ((row >> 5) & 3) * 4 + (col & 3);
}

// Programmatic dependent launch: a kernel that calls dependents_may_launch() lets the next
// kernel of the stream (launched with launch_dependent) start its blocks early; that kernel calls
// wait_for_prior_grid() before it touches anything the earlier kernel wrote.  Both are no-ops in
// a plain launch.
__device__ __forceinline__ void dependents_may_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void wait_for_prior_grid() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_dependent(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid, cfg.blockDim = block, cfg.dynamicSmemBytes = smem, cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr, cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Ordered fold of row-block partials into the fp64 totals (the order is part of the arithmetic
// definition).  part[c * n + i] is the partial of row block c for output i, c ascending in rows.
//   PER_SLAB == 1: the partials are fp64 slab sums:  total[i] += part[c][i], c ascending.
//   PER_SLAB == 8: the partials are fp32 chunk sums: every run of 8 consecutive chunks (one slab)
//                  is added in fp64 from zero, then the slab sum is added to total[i].
// WITH_MAX also folds vmax[i] = max(vmax[i], part_max[c][i]).
// The additions are sequential per output but the loads are not: a block owns 16 consecutive
// outputs and stages up to kFoldRoundMax partials per output in (dynamic) shared memory with
// coalesced loads, all in flight at once, then 16 threads add them in order.  Typical sizes take a
// single round.
constexpr int kFoldThreads = 256, kFoldOutputs = 16, kFoldRoundMax = 512;

template <typename PT, bool WITH_MAX>
constexpr size_t fold_smem_bytes(int64_t count) {
    return static_cast<size_t>(count < kFoldRoundMax ? count : kFoldRoundMax) * kFoldOutputs *
           (sizeof(PT) + (WITH_MAX ? sizeof(float) : 0));
}

template <typename PT, int PER_SLAB, bool WITH_MAX>
__global__ void __launch_bounds__(kFoldThreads)
fold_partials(const PT *__restrict__ part, const float *__restrict__ part_max, int64_t count, int64_t n,
              double *__restrict__ total, float *__restrict__ vmax) {
    static_assert(kFoldRoundMax % PER_SLAB == 0, "a round holds whole slabs");
    extern __shared__ __align__(16) unsigned char fold_smem[];
    const int round_rows = static_cast<int>(min(static_cast<int64_t>(kFoldRoundMax), count));
    PT *tile = reinterpret_cast<PT *>(fold_smem);
    float *tile_max = reinterpret_cast<float *>(fold_smem + static_cast<size_t>(round_rows) * kFoldOutputs * sizeof(PT));
    constexpr int kRows = kFoldThreads / kFoldOutputs;  // rows of the round covered by one pass of all threads
    const int o = threadIdx.x % kFoldOutputs, g = threadIdx.x / kFoldOutputs;
    const int64_t i = static_cast<int64_t>(blockIdx.x) * kFoldOutputs + o;
    const bool live = i < n, adder = threadIdx.x < kFoldOutputs;
    double s = 0.0, slab = 0.0;
    float a = 0.0f;
    if (adder && live) {
        s = total[i];
        if (WITH_MAX) a = vmax[i];
    }
    wait_for_prior_grid();
    for (int64_t c0 = 0; c0 < count; c0 += kFoldRoundMax) {
        const int nc = static_cast<int>(min(static_cast<int64_t>(kFoldRoundMax), count - c0));
        __syncthreads();
        for (int c = g; c < nc; c += kRows) {
            tile[c * kFoldOutputs + o] = live ? __ldcs(part + (c0 + c) * n + i) : PT(0);
            if (WITH_MAX) tile_max[c * kFoldOutputs + o] = live ? __ldcs(part_max + (c0 + c) * n + i) : 0.0f;
        }
        __syncthreads();
        if (adder) {
#pragma unroll 8
            for (int c = 0; c < nc; ++c) {
                if (PER_SLAB == 1) {
                    s = __dadd_rn(s, static_cast<double>(tile[c * kFoldOutputs + o]));
                } else {
                    slab = __dadd_rn(slab, static_cast<double>(tile[c * kFoldOutputs + o]));
                    if ((c % PER_SLAB) == PER_SLAB - 1 || c0 + c == count - 1) {
                        s = __dadd_rn(s, slab);
                        slab = 0.0;
                    }
                }
                if (WITH_MAX) a = fmaxf(a, tile_max[c * kFoldOutputs + o]);
            }
        }
    }
    if (adder && live) {
        total[i] = s;
        if (WITH_MAX) vmax[i] = a;
    }
}

// Launch of fold_partials as a programmatic dependent of the kernel that wrote the partials.
template <typename PT, int PER_SLAB, bool WITH_MAX>
cudaError_t launch_fold(const PT *part, const float *part_max, int64_t count, int64_t n, double *total, float *vmax,
                        cudaStream_t st) {
    const size_t smem = fold_smem_bytes<PT, WITH_MAX>(count);
    if (smem > 48 * 1024) {
        const cudaError_t e = cudaFuncSetAttribute(fold_partials<PT, PER_SLAB, WITH_MAX>,
                                                   cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
        if (e != cudaSuccess) return e;
    }
    return launch_dependent(fold_partials<PT, PER_SLAB, WITH_MAX>,
                            dim3(static_cast<unsigned>((n + kFoldOutputs - 1) / kFoldOutputs)), dim3(kFoldThreads), smem, st,
                            part, part_max, count, n, total, vmax);
}

}  // namespace pq
#endif  // __CUDACC__
