// The producer in front of a quantized linear layer, fused: RMSNorm or adaptive LayerNorm (App. C),
// the channel reordering absorbed into it, and the NVFP4 quantizer of the runtime path (Eq. 8)
// attached, so the normalized activations never make a bf16 round trip through HBM.
//
// One warp per token row.  The row is read once with coalesced 16-byte loads (lane l owns the
// octets l, l + 32, ...: the summation order of the row statistics is this walk followed by a
// butterfly over the lanes, and does not depend on the permutation), kept in shared memory in
// fp32, normalized and modulated in place; then each lane takes 16-channel groups of the OUTPUT
// order, gathers their values from shared memory through the permutation and quantizes them like
// the stand-alone quantizer (8-byte code store, scale bytes of four neighbouring groups merged into
// one 32-bit store).  Optionally the reordered bf16 tensor of the unfused kernel is written too.
#include "pq_common.cuh"

namespace {

constexpr int kMaxRowsPerBlock = 8;
constexpr size_t kSmemBudget = 200 * 1024;

__device__ __forceinline__ float lane_butterfly(float p) {
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) p = __fadd_rn(p, __shfl_xor_sync(0xFFFFFFFFu, p, m));
    return p;
}

// Quantize the 16 values (x, y) of output group g of `row` and store codes, scale byte (merged over
// four neighbouring lanes) and, optionally, the bf16 values.  Called by whole warps.
template <int SF_LAYOUT>
__device__ __forceinline__ void quantize_and_store(const float (&x)[8], const float (&y)[8], int64_t row, int g, int gpr,
                                                   int K, bool live, bool have, float ts, uint8_t *__restrict__ codes,
                                                   uint8_t *__restrict__ sf, uint16_t *__restrict__ y_out) {
        const float amax = fmaxf(pq::absmax8(x), pq::absmax8(y));
        uint32_t sf8;
        float d, r;
        pq::nvfp4_scale(amax, ts, sf8, d, r);
        const uint32_t c0 = pq::nvfp4_codes(x, r), c1 = pq::nvfp4_codes(y, r);
        if (live && have) {
            __stcs(reinterpret_cast<uint2 *>(codes + row * (K >> 1) + g * 8), make_uint2(c0, c1));
            if (y_out) {
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    w[e] = __bfloat16_as_ushort(__float2bfloat16_rn(x[2 * e])) |
                           (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(x[2 * e + 1]))) << 16);
                    w[4 + e] = __bfloat16_as_ushort(__float2bfloat16_rn(y[2 * e])) |
                               (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(y[2 * e + 1]))) << 16);
                }
                uint4 *dst = reinterpret_cast<uint4 *>(y_out + row * K + g * 16);
                dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
            }
        }
        // scale bytes of groups g .. g+3 (padding rows write zeros)
        uint32_t word = sf8;
        word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 1) << 8;
        word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 2) << 16;
        word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 3) << 24;
        if (!have) return;
        if (SF_LAYOUT == PQ_SF_TCGEN05) {
            if ((g & 3) == 0) *reinterpret_cast<uint32_t *>(sf + pq::sf_tc_offset(row, g, gpr >> 2)) = word;
        } else if (live) {
            if ((gpr & 3) == 0) {
                if ((g & 3) == 0) *reinterpret_cast<uint32_t *>(sf + row * gpr + g) = word;
            } else {
                sf[row * gpr + g] = static_cast<uint8_t>(sf8);
            }
        }
}

// Shared-memory layout of a row of fp32 values: the two 16-byte halves of octet o live at float4
// index o and octs + o, so that a warp's 16-byte accesses (lane = octet) are contiguous and free of
// bank conflicts.  Channel c = 8 o + e sits at float index 4 ((e >> 2) octs + o) + (e & 3).
__device__ __forceinline__ int swz(int c, int octs) { return (((c >> 2) & 1) * octs + (c >> 3)) * 4 + (c & 3); }

// Rows of up to 8 * 32 * REG_OCTS channels: the lane keeps its octets as packed bf16 in registers,
// so the statistics and the scaling read no memory; only the finished fp32 row goes to shared
// memory, for the gather.
template <int KIND, int SF_LAYOUT, int REG_OCTS>
__global__ void __launch_bounds__(32 * kMaxRowsPerBlock)
norm_quant_reg_kernel(const uint16_t *__restrict__ H, int64_t rows, int64_t rows_pad, int K, int64_t ld,
                      const float *__restrict__ a, const float *__restrict__ b, float eps,
                      const int32_t *__restrict__ perm, const float *__restrict__ ts_ptr,
                      uint8_t *__restrict__ codes, uint8_t *__restrict__ sf, uint16_t *__restrict__ y_out) {
    extern __shared__ __align__(16) float row_s[];  // [warps][K], swizzled
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + warp;
    if (row >= rows_pad) return;  // whole warps only
    const bool live = row < rows;
    float *ys = row_s + static_cast<size_t>(warp) * K;
    const int octs = K >> 3, gpr = K >> 4;
    const float ts = __ldg(ts_ptr);

    if (live) {
        const uint16_t *src = H + row * ld;
        uint4 v[REG_OCTS];
#pragma unroll
        for (int u = 0; u < REG_OCTS; ++u) {
            const int o = lane + 32 * u;
            v[u] = o < octs ? __ldcs(reinterpret_cast<const uint4 *>(src + o * 8)) : make_uint4(0, 0, 0, 0);
        }
        float p = 0.0f;
#pragma unroll
        for (int u = 0; u < REG_OCTS; ++u) {
            if (lane + 32 * u < octs) {
                float x[8];
                pq::unpack8(v[u], x);
#pragma unroll
                for (int e = 0; e < 8; ++e) p = KIND == 0 ? __fmaf_rn(x[e], x[e], p) : __fadd_rn(p, x[e]);
            }
        }
        p = lane_butterfly(p);
        float inv, mu = 0.0f;
        if (KIND == 0) {
            inv = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(p, static_cast<float>(K)), eps)));
        } else {
            mu = __fdiv_rn(p, static_cast<float>(K));
            float q = 0.0f;
#pragma unroll
            for (int u = 0; u < REG_OCTS; ++u) {
                if (lane + 32 * u < octs) {
                    float x[8];
                    pq::unpack8(v[u], x);
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const float d = __fsub_rn(x[e], mu);
                        q = __fmaf_rn(d, d, q);
                    }
                }
            }
            q = lane_butterfly(q);
            inv = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(q, static_cast<float>(K)), eps)));
        }
#pragma unroll
        for (int u = 0; u < REG_OCTS; ++u) {
            const int o = lane + 32 * u;
            if (o < octs) {
                float x[8], y[8];
                pq::unpack8(v[u], x);
                const float4 a0 = __ldg(reinterpret_cast<const float4 *>(a + o * 8)), a1 = __ldg(reinterpret_cast<const float4 *>(a + o * 8) + 1);
                const float w[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                if (KIND == 0) {
#pragma unroll
                    for (int e = 0; e < 8; ++e) y[e] = __fmul_rn(__fmul_rn(x[e], inv), w[e]);
                } else {
                    const float4 b0 = __ldg(reinterpret_cast<const float4 *>(b + o * 8)), b1 = __ldg(reinterpret_cast<const float4 *>(b + o * 8) + 1);
                    const float sh[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        y[e] = __fmaf_rn(__fmul_rn(__fsub_rn(x[e], mu), inv), __fadd_rn(1.0f, w[e]), sh[e]);
                }
                reinterpret_cast<float4 *>(ys)[o] = make_float4(y[0], y[1], y[2], y[3]);
                reinterpret_cast<float4 *>(ys)[octs + o] = make_float4(y[4], y[5], y[6], y[7]);
            }
        }
    }
    __syncwarp();

    for (int g0 = 0; g0 < gpr; g0 += 32) {
        const int g = g0 + lane;
        const bool have = g < gpr;
        float x[8], y[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = 0.0f, y[e] = 0.0f;
        if (live && have) {
            if (perm) {
                const int4 *pi = reinterpret_cast<const int4 *>(perm + g * 16);
                const int4 i0 = __ldg(pi), i1 = __ldg(pi + 1), i2 = __ldg(pi + 2), i3 = __ldg(pi + 3);
                x[0] = ys[swz(i0.x, octs)], x[1] = ys[swz(i0.y, octs)], x[2] = ys[swz(i0.z, octs)], x[3] = ys[swz(i0.w, octs)];
                x[4] = ys[swz(i1.x, octs)], x[5] = ys[swz(i1.y, octs)], x[6] = ys[swz(i1.z, octs)], x[7] = ys[swz(i1.w, octs)];
                y[0] = ys[swz(i2.x, octs)], y[1] = ys[swz(i2.y, octs)], y[2] = ys[swz(i2.z, octs)], y[3] = ys[swz(i2.w, octs)];
                y[4] = ys[swz(i3.x, octs)], y[5] = ys[swz(i3.y, octs)], y[6] = ys[swz(i3.z, octs)], y[7] = ys[swz(i3.w, octs)];
            } else {
                const float4 *v4 = reinterpret_cast<const float4 *>(ys);
                const float4 u0 = v4[2 * g], u1 = v4[octs + 2 * g], u2 = v4[2 * g + 1], u3 = v4[octs + 2 * g + 1];
                x[0] = u0.x, x[1] = u0.y, x[2] = u0.z, x[3] = u0.w, x[4] = u1.x, x[5] = u1.y, x[6] = u1.z, x[7] = u1.w;
                y[0] = u2.x, y[1] = u2.y, y[2] = u2.z, y[3] = u2.w, y[4] = u3.x, y[5] = u3.y, y[6] = u3.z, y[7] = u3.w;
            }
        }
        quantize_and_store<SF_LAYOUT>(x, y, row, g, gpr, K, live, have, ts, codes, sf, y_out);
    }
}

template <int KIND, int SF_LAYOUT>
__global__ void __launch_bounds__(32 * kMaxRowsPerBlock)
norm_quant_kernel(const uint16_t *__restrict__ H, int64_t rows, int64_t rows_pad, int K, int64_t ld,
                  const float *__restrict__ a, const float *__restrict__ b, float eps,
                  const int32_t *__restrict__ perm, const float *__restrict__ ts_ptr, uint8_t *__restrict__ codes,
                  uint8_t *__restrict__ sf, uint16_t *__restrict__ y_out) {
    extern __shared__ __align__(16) float row_s[];  // [warps][K]
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + warp;
    if (row >= rows_pad) return;  // whole warps only
    const bool live = row < rows;
    float *ys = row_s + static_cast<size_t>(warp) * K;
    const int octs = K >> 3, gpr = K >> 4;
    const float ts = __ldg(ts_ptr);

    if (live) {
        // ---- the row, once: fp32 copy in shared memory, first statistic
        const uint16_t *src = H + row * ld;
        float p = 0.0f;
        // four loads in flight per lane and step (the sums still run in ascending octet order)
        for (int o0 = lane; o0 < octs; o0 += 128) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int o = o0 + 32 * u;
                v[u] = o < octs ? __ldcs(reinterpret_cast<const uint4 *>(src + o * 8)) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int o = o0 + 32 * u;
                if (o >= octs) break;
                float x[8];
                pq::unpack8(v[u], x);
                reinterpret_cast<float4 *>(ys + o * 8)[0] = make_float4(x[0], x[1], x[2], x[3]);
                reinterpret_cast<float4 *>(ys + o * 8)[1] = make_float4(x[4], x[5], x[6], x[7]);
#pragma unroll
                for (int e = 0; e < 8; ++e) p = KIND == 0 ? __fmaf_rn(x[e], x[e], p) : __fadd_rn(p, x[e]);
            }
        }
        p = lane_butterfly(p);
        float inv, mu = 0.0f;
        if (KIND == 0) {
            inv = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(p, static_cast<float>(K)), eps)));
        } else {
            mu = __fdiv_rn(p, static_cast<float>(K));
            float q = 0.0f;
            for (int o = lane; o < octs; o += 32) {  // the lane re-reads what it wrote
                float4 *v = reinterpret_cast<float4 *>(ys + o * 8);
                float4 u0 = v[0], u1 = v[1];
                float d[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    d[e] = __fsub_rn(d[e], mu);
                    q = __fmaf_rn(d[e], d[e], q);
                }
                v[0] = make_float4(d[0], d[1], d[2], d[3]);
                v[1] = make_float4(d[4], d[5], d[6], d[7]);
            }
            q = lane_butterfly(q);
            inv = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(q, static_cast<float>(K)), eps)));
        }
        // ---- scale / modulation, in place, original channel order (coalesced parameter loads)
        for (int o = lane; o < octs; o += 32) {
            float4 *v = reinterpret_cast<float4 *>(ys + o * 8);
            const float4 u0 = v[0], u1 = v[1];
            const float4 a0 = __ldg(reinterpret_cast<const float4 *>(a + o * 8)), a1 = __ldg(reinterpret_cast<const float4 *>(a + o * 8) + 1);
            const float x[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
            const float w[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            float y[8];
            if (KIND == 0) {
#pragma unroll
                for (int e = 0; e < 8; ++e) y[e] = __fmul_rn(__fmul_rn(x[e], inv), w[e]);
            } else {
                const float4 b0 = __ldg(reinterpret_cast<const float4 *>(b + o * 8)), b1 = __ldg(reinterpret_cast<const float4 *>(b + o * 8) + 1);
                const float sh[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) y[e] = __fmaf_rn(__fmul_rn(x[e], inv), __fadd_rn(1.0f, w[e]), sh[e]);
            }
            v[0] = make_float4(y[0], y[1], y[2], y[3]);
            v[1] = make_float4(y[4], y[5], y[6], y[7]);
        }
    }
    __syncwarp();

    // ---- output order: gather, quantize, store
    for (int g0 = 0; g0 < gpr; g0 += 32) {
        const int g = g0 + lane;
        const bool have = g < gpr;
        float x[8], y[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) x[e] = 0.0f, y[e] = 0.0f;
        if (live && have) {
            if (perm) {
                const int4 *pi = reinterpret_cast<const int4 *>(perm + g * 16);
                const int4 i0 = __ldg(pi), i1 = __ldg(pi + 1), i2 = __ldg(pi + 2), i3 = __ldg(pi + 3);
                x[0] = ys[i0.x], x[1] = ys[i0.y], x[2] = ys[i0.z], x[3] = ys[i0.w];
                x[4] = ys[i1.x], x[5] = ys[i1.y], x[6] = ys[i1.z], x[7] = ys[i1.w];
                y[0] = ys[i2.x], y[1] = ys[i2.y], y[2] = ys[i2.z], y[3] = ys[i2.w];
                y[4] = ys[i3.x], y[5] = ys[i3.y], y[6] = ys[i3.z], y[7] = ys[i3.w];
            } else {
                const float4 *v = reinterpret_cast<const float4 *>(ys + g * 16);
                const float4 u0 = v[0], u1 = v[1], u2 = v[2], u3 = v[3];
                x[0] = u0.x, x[1] = u0.y, x[2] = u0.z, x[3] = u0.w, x[4] = u1.x, x[5] = u1.y, x[6] = u1.z, x[7] = u1.w;
                y[0] = u2.x, y[1] = u2.y, y[2] = u2.z, y[3] = u2.w, y[4] = u3.x, y[5] = u3.y, y[6] = u3.z, y[7] = u3.w;
            }
        }
        quantize_and_store<SF_LAYOUT>(x, y, row, g, gpr, K, live, have, ts, codes, sf, y_out);
    }
}

template <int KIND, int SF_LAYOUT>
pq_status launch(const uint16_t *H, int64_t M, int64_t rows_pad, int K, int64_t ld, const float *a, const float *b,
                 float eps, const int32_t *perm, const float *ts, uint8_t *codes, uint8_t *sf, uint16_t *y_out,
                 cudaStream_t st) {
    int warps = static_cast<int>(kSmemBudget / (static_cast<size_t>(K) * 4));
    if (warps > kMaxRowsPerBlock) warps = kMaxRowsPerBlock;
    if (warps < 1) return PQ_ERR_SHAPE;
    const size_t smem = static_cast<size_t>(warps) * K * 4;
    if (smem > 48 * 1024)
        PQ_CUDA_OK(cudaFuncSetAttribute(norm_quant_kernel<KIND, SF_LAYOUT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(smem)));
    const int64_t blocks = pq_ceil_div(rows_pad, warps);
    PQ_REQUIRE(blocks < (1ll << 31), PQ_ERR_SHAPE);
    if (K <= 8 * 32 * 16) {  // up to 4096 channels: the row stays in registers as packed bf16
        if (smem > 48 * 1024)
            PQ_CUDA_OK(cudaFuncSetAttribute(norm_quant_reg_kernel<KIND, SF_LAYOUT, 16>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        norm_quant_reg_kernel<KIND, SF_LAYOUT, 16><<<static_cast<unsigned>(blocks), warps * 32, smem, st>>>(
            H, M, rows_pad, K, ld, a, b, eps, perm, ts, codes, sf, y_out);
        return pq_launch_status();
    }
    norm_quant_kernel<KIND, SF_LAYOUT><<<static_cast<unsigned>(blocks), warps * 32, smem, st>>>(
        H, M, rows_pad, K, ld, a, b, eps, perm, ts, codes, sf, y_out);
    return pq_launch_status();
}

}  // namespace

extern "C" pq_status pq_norm_quant_nvfp4(const void *H, int64_t M, int64_t K, int64_t ld, int kind, const float *a,
                                         const float *b, float eps, const int32_t *perm, const float *ts_x,
                                         uint8_t *codes, uint8_t *sf, int sf_layout, void *y_out, void *stream) {
    PQ_REQUIRE(H && a && ts_x && codes && sf, PQ_ERR_NULL);
    PQ_REQUIRE(kind == PQ_NORM_RMS || kind == PQ_NORM_ADALN, PQ_ERR_FORMAT);
    PQ_REQUIRE(kind == PQ_NORM_RMS || b, PQ_ERR_NULL);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || sf_layout == PQ_SF_TCGEN05, PQ_ERR_FORMAT);
    PQ_REQUIRE(M > 0 && K > 0 && K % 16 == 0 && K <= 32768 && ld >= K, PQ_ERR_SHAPE);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || K % 64 == 0, PQ_ERR_SHAPE);
    PQ_REQUIRE(eps >= 0.0f, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(H) && ld % 8 == 0 && pq_aligned16(codes) && pq_aligned16(sf) && pq_aligned16(a) &&
                   (!b || pq_aligned16(b)) && (!perm || pq_aligned16(perm)) && (!y_out || pq_aligned16(y_out)),
               PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint16_t *h = static_cast<const uint16_t *>(H);
    uint16_t *y = static_cast<uint16_t *>(y_out);
    const int64_t rows_pad = sf_layout == PQ_SF_TCGEN05 ? pq_ceil_div(M, 128) * 128 : M;
    const int k = static_cast<int>(K);
    if (kind == PQ_NORM_RMS) {
        return sf_layout == PQ_SF_TCGEN05
                   ? launch<0, PQ_SF_TCGEN05>(h, M, rows_pad, k, ld, a, b, eps, perm, ts_x, codes, sf, y, st)
                   : launch<0, PQ_SF_LINEAR>(h, M, rows_pad, k, ld, a, b, eps, perm, ts_x, codes, sf, y, st);
    }
    return sf_layout == PQ_SF_TCGEN05
               ? launch<1, PQ_SF_TCGEN05>(h, M, rows_pad, k, ld, a, b, eps, perm, ts_x, codes, sf, y, st)
               : launch<1, PQ_SF_LINEAR>(h, M, rows_pad, k, ld, a, b, eps, perm, ts_x, codes, sf, y, st);
}
