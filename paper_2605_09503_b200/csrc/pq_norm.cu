// The producer in front of a quantized linear layer, fused: RMSNorm or adaptive LayerNorm (App. C),
// the channel reordering absorbed into it, and the NVFP4 quantizer of the runtime path (Eq. 8)
// attached, so the normalized activations never make a bf16 round trip through HBM.
//
// A warp owns whole token rows.  A row is read once with coalesced 16-byte loads (lane l owns the
// octets l, l + 32, ...: the summation order of the row statistics is this walk followed by a
// butterfly over the lanes, and does not depend on the permutation) and kept in shared memory as
// bf16; then the lanes walk the OUTPUT order, gather their channels from shared memory through the
// permutation, normalize them with the scale / shift of the output positions (the parameters arrive
// reordered: contiguous 16-byte loads per lane, like the indices) and quantize them like the
// stand-alone quantizer (coalesced code stores; scale bytes of four neighbouring groups merged into
// one 32-bit store).  The normalized values exist only in registers, in fp32.  Optionally the
// reordered bf16 tensor of the unfused kernel is written too.
//
// Three kernels: rows of up to 6400 channels go four per warp (below, second kernel); wider rows one
// per warp, eight positions per lane (first kernel); and without a permutation (channels already in
// output order) rows of up to 4096 channels never leave the registers (third kernel).  KIND 0 is RMSNorm,
// 1 adaptive LayerNorm; the four-row kernel also exists as KIND 2, no normalization at all: the gather
// quantizers of the offline path (a candidate order applied to activations or to the weight) run through it.
#include "pq_common.cuh"

namespace {

constexpr int kMaxRowsPerBlock = 8;
#ifndef PQ_NORM_POS
#define PQ_NORM_POS 8
#endif
constexpr size_t kSmemBudget = 200 * 1024;

__device__ __forceinline__ float lane_butterfly(float p) {
#pragma unroll
    for (int m = 16; m >= 1; m >>= 1) p = __fadd_rn(p, __shfl_xor_sync(0xFFFFFFFFu, p, m));
    return p;
}

template <int KIND, int SF_LAYOUT>
__global__ void __launch_bounds__(32 * kMaxRowsPerBlock)
norm_quant_kernel(const uint16_t *__restrict__ H, int64_t rows, int64_t rows_pad, int K, int64_t ld,
                  const float *__restrict__ a, const float *__restrict__ b, float eps,
                  const int32_t *__restrict__ perm, const float *__restrict__ ts_ptr, uint8_t *__restrict__ codes,
                  uint8_t *__restrict__ sf, uint16_t *__restrict__ y_out) {
    extern __shared__ __align__(16) uint16_t row_s[];  // [warps][K] bf16 bit patterns
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + warp;
    if (row >= rows_pad) return;  // whole warps only
    const bool live = row < rows;
    uint16_t *xs = row_s + static_cast<size_t>(warp) * K;
    const int octs = K >> 3, gpr = K >> 4;
    const float ts = __ldg(ts_ptr);
    float inv = 0.0f, mu = 0.0f;

    if (live) {
        // ---- the row, once: a copy in shared memory (for the gather) and the first statistic;
        // four loads in flight per lane and step, sums in ascending octet order
        const uint16_t *src = H + row * ld;
        float p = 0.0f;
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
                reinterpret_cast<uint4 *>(xs)[o] = v[u];
                float x[8];
                pq::unpack8(v[u], x);
#pragma unroll
                for (int e = 0; e < 8; ++e) p = KIND == 0 ? __fmaf_rn(x[e], x[e], p) : __fadd_rn(p, x[e]);
            }
        }
        p = lane_butterfly(p);
        if (KIND == 0) {
            inv = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(p, static_cast<float>(K)), eps)));
        } else {
            mu = __fdiv_rn(p, static_cast<float>(K));
            float q = 0.0f;
            for (int o = lane; o < octs; o += 32) {  // the lane re-reads what it wrote
                float x[8];
                pq::unpack8(reinterpret_cast<const uint4 *>(xs)[o], x);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float d = __fsub_rn(x[e], mu);
                    q = __fmaf_rn(d, d, q);
                }
            }
            q = lane_butterfly(q);
            inv = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(q, static_cast<float>(K)), eps)));
        }
    }
    __syncwarp();

    // ---- output order, POS = 4 or 8 consecutive positions per lane (a quarter or half of a group;
    // the indices and parameters of a lane are one or two contiguous 16-byte loads): gather,
    // normalize, quantize; the lanes of a group share its absmax by shuffles and each derive the scale.
    constexpr int POS = PQ_NORM_POS, LPG = 16 / POS;  // lanes per group
    const int slots = K / POS;
    for (int q0 = 0; q0 < slots; q0 += 32) {
        const int q = q0 + lane;           // positions POS q .. POS q + POS - 1, group q / LPG
        const bool have = q < slots;
        float out[POS];
#pragma unroll
        for (int j = 0; j < POS; ++j) out[j] = 0.0f;
        if (live && have) {
            float v[POS], w[POS];
#pragma unroll
            for (int h = 0; h < POS / 4; ++h) {
                if (perm) {
                    const int4 idx = __ldg(reinterpret_cast<const int4 *>(perm) + q * (POS / 4) + h);
                    v[4 * h + 0] = pq::bf16_bits_to_f32(xs[idx.x]), v[4 * h + 1] = pq::bf16_bits_to_f32(xs[idx.y]);
                    v[4 * h + 2] = pq::bf16_bits_to_f32(xs[idx.z]), v[4 * h + 3] = pq::bf16_bits_to_f32(xs[idx.w]);
                } else {
                    const uint2 u = reinterpret_cast<const uint2 *>(xs)[q * (POS / 4) + h];
                    v[4 * h + 0] = __uint_as_float(u.x << 16), v[4 * h + 1] = __uint_as_float(u.x & 0xFFFF0000u);
                    v[4 * h + 2] = __uint_as_float(u.y << 16), v[4 * h + 3] = __uint_as_float(u.y & 0xFFFF0000u);
                }
                const float4 a4 = __ldg(reinterpret_cast<const float4 *>(a) + q * (POS / 4) + h);
                w[4 * h + 0] = a4.x, w[4 * h + 1] = a4.y, w[4 * h + 2] = a4.z, w[4 * h + 3] = a4.w;
            }
            if (KIND == 0) {
#pragma unroll
                for (int j = 0; j < POS; ++j) out[j] = __fmul_rn(__fmul_rn(v[j], inv), w[j]);
            } else {
                float sh[POS];
#pragma unroll
                for (int h = 0; h < POS / 4; ++h) {
                    const float4 b4 = __ldg(reinterpret_cast<const float4 *>(b) + q * (POS / 4) + h);
                    sh[4 * h + 0] = b4.x, sh[4 * h + 1] = b4.y, sh[4 * h + 2] = b4.z, sh[4 * h + 3] = b4.w;
                }
#pragma unroll
                for (int j = 0; j < POS; ++j)
                    out[j] = __fmaf_rn(__fmul_rn(__fsub_rn(v[j], mu), inv), __fadd_rn(1.0f, w[j]), sh[j]);
            }
        }
        float amax = 0.0f;
#pragma unroll
        for (int j = 0; j < POS; ++j) amax = fmaxf(amax, fabsf(out[j]));
#pragma unroll
        for (int m = 1; m < LPG; m <<= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, m));
        uint32_t sf8;
        float d, r;
        pq::nvfp4_scale(amax, ts, sf8, d, r);
        uint32_t cw = 0;
#pragma unroll
        for (int h = 0; h < POS / 4; ++h) {
            uint16_t c16;
            asm("{\n"
                ".reg .b8 lo, hi;\n"
                "cvt.rn.satfinite.e2m1x2.f32 lo, %2, %1;\n"
                "cvt.rn.satfinite.e2m1x2.f32 hi, %4, %3;\n"
                "mov.b16 %0, {lo, hi};\n"
                "}\n"
                : "=h"(c16)
                : "f"(__fmul_rn(out[4 * h], r)), "f"(__fmul_rn(out[4 * h + 1], r)), "f"(__fmul_rn(out[4 * h + 2], r)),
                  "f"(__fmul_rn(out[4 * h + 3], r)));
            cw |= static_cast<uint32_t>(c16) << (16 * h);
        }
        if (live && have) {
            uint8_t *cdst = codes + row * (K >> 1) + q * (POS / 2);
            if (POS == 4) *reinterpret_cast<uint16_t *>(cdst) = static_cast<uint16_t>(cw);
            else *reinterpret_cast<uint32_t *>(cdst) = cw;
            if (y_out) {
                uint32_t yw[POS / 2];
#pragma unroll
                for (int j = 0; j < POS / 2; ++j)
                    yw[j] = __bfloat16_as_ushort(__float2bfloat16_rn(out[2 * j])) |
                            (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(out[2 * j + 1]))) << 16);
                if (POS == 4) reinterpret_cast<uint2 *>(y_out + row * K)[q] = make_uint2(yw[0], yw[1]);
                else reinterpret_cast<uint4 *>(y_out + row * K)[q] = make_uint4(yw[0], yw[1], yw[POS / 2 - 2], yw[POS / 2 - 1]);
            }
        }
        // scale bytes: the first lane of each group holds its byte; four neighbouring groups sit LPG
        // lanes apart (padding rows write zeros)
        uint32_t word = sf8;
        word |= __shfl_down_sync(0xFFFFFFFFu, sf8, LPG) << 8;
        word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 2 * LPG) << 16;
        word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 3 * LPG) << 24;
        if (!have || (q % LPG) != 0) continue;
        const int g = q / LPG;
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
}

// ---- several rows per warp ----------------------------------------------------------------------
// The same computation with the rows taken four (or two) at a time by a warp.  Their bf16 values sit
// interleaved per channel in shared memory (8 or 4 bytes per channel), so one shared-memory load
// gathers a channel for all rows of the warp, and the indices and parameters of an output position
// are fetched once for them; a lane takes a whole group (16 output positions), so the scale is derived
// once per group and nothing but the scale bytes crosses lanes.  The 16-byte chunks of an octet are
// XOR-swizzled by bits of the octet index, which makes the transposing stores of the first phase
// conflict-free.  The order of every floating-point operation is that of the one-row kernel.
#ifndef PQ_NORM_ROWS
#define PQ_NORM_ROWS 4
#endif
#ifndef PQ_NORM_WARPS
#define PQ_NORM_WARPS 4
#endif
#ifndef PQ_NORM_SPLIT
#define PQ_NORM_SPLIT 2
#endif
// kGroupWarps row groups per block, kSplit warps per row group: the first reads the rows and takes
// the statistics, then all of them share the walk over the output order
constexpr int kGroupRows = PQ_NORM_ROWS, kGroupWarps = PQ_NORM_WARPS, kSplit = PQ_NORM_SPLIT;
static_assert(kGroupRows == 2 || kGroupRows == 4, "rows per warp");

// 16-byte chunk k of octet o (R = 4: two channels per chunk, four chunks; R = 2: four channels, two chunks)
template <int R>
__device__ __forceinline__ int chunk_of(int o, int k) {
    return R == 4 ? 4 * o + (k ^ ((o >> 1) & 3)) : 2 * o + (k ^ ((o >> 2) & 1));
}
template <int R>
__device__ __forceinline__ int swizzled_channel(int c) {
    return R == 4 ? c ^ (((c >> 4) & 3) << 1) : c ^ (((c >> 5) & 1) << 2);
}
// the rows of one channel: R = 4 in (x, y), R = 2 in x
template <int R>
__device__ __forceinline__ uint2 channel_rows(const uint16_t *xs, int c) {
    if (R == 4) return reinterpret_cast<const uint2 *>(xs)[swizzled_channel<4>(c)];
    return make_uint2(reinterpret_cast<const uint32_t *>(xs)[swizzled_channel<2>(c)], 0u);
}
__device__ __forceinline__ float row_value(const uint2 &g, int r) {
    const uint32_t w = r < 2 ? g.x : g.y;
    return __uint_as_float((r & 1) ? (w & 0xFFFF0000u) : (w << 16));
}

template <int KIND, int SF_LAYOUT>
__global__ void __launch_bounds__(32 * kGroupWarps * kSplit, 2)
norm_quant_grouped_kernel(const uint16_t *__restrict__ H, int64_t rows, int64_t rows_pad, int K, int64_t ld,
                        const float *__restrict__ a, const float *__restrict__ b, float eps,
                        const int32_t *__restrict__ perm, const int32_t *__restrict__ perm_select,
                        const float *__restrict__ ts_ptr, uint8_t *__restrict__ codes, uint8_t *__restrict__ sf,
                        uint16_t *__restrict__ y_out) {
    // perm_select given: perm is a table of candidate orders [., K] and {best, accept} on the device name the
    // row best - 1, or the original order (the offline weight quantizer, whose decision never visits the host)
    if (perm_select) perm = perm_select[1] ? perm + static_cast<int64_t>(perm_select[0] - 1) * K : nullptr;
    extern __shared__ __align__(16) uint16_t row_s[];  // [row groups][K][R rows] bf16 bit patterns
    __shared__ float stat_s[kGroupWarps][2 * kGroupRows];
    constexpr int R = kGroupRows;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int grp_in_block = warp % kGroupWarps, part = warp / kGroupWarps;
    const int64_t row0 = (static_cast<int64_t>(blockIdx.x) * kGroupWarps + grp_in_block) * R;
    const bool present = row0 < rows_pad;  // a row group past the end still joins the barrier
    const int nlive =
        present ? static_cast<int>(min(static_cast<int64_t>(R), max(static_cast<int64_t>(0), rows - row0))) : 0;
    uint16_t *xs = row_s + static_cast<size_t>(grp_in_block) * K * R;
    uint4 *xs4 = reinterpret_cast<uint4 *>(xs);
    const int octs = K >> 3, gpr = K >> 4;
    const float ts = __ldg(ts_ptr);
    float inv[R], mu[R];
#pragma unroll
    for (int r = 0; r < R; ++r) inv[r] = 0.0f, mu[r] = 0.0f;

    if (nlive > 0 && part == 0) {
        // ---- the rows, once: interleaved copy in shared memory and the first statistic; three
        // octets of each row in flight per lane, sums in ascending octet order
        constexpr int U = 3;
        float p[R];
#pragma unroll
        for (int r = 0; r < R; ++r) p[r] = 0.0f;
        for (int o0 = lane; o0 < octs; o0 += 32 * U) {
            uint4 v[U][R];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int o = o0 + 32 * u;
#pragma unroll
                for (int r = 0; r < R; ++r)
                    v[u][r] = (o < octs && r < nlive)
                                  ? __ldcs(reinterpret_cast<const uint4 *>(H + (row0 + r) * ld + o * 8))
                                  : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int o = o0 + 32 * u;
                if (o >= octs) break;
                const uint32_t *w0 = &v[u][0].x, *w1 = &v[u][1].x, *w2 = &v[u][R - 2].x, *w3 = &v[u][R - 1].x;
                if (R == 4) {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        xs4[chunk_of<4>(o, k)] =
                            make_uint4(__byte_perm(w0[k], w1[k], 0x5410), __byte_perm(w2[k], w3[k], 0x5410),
                                       __byte_perm(w0[k], w1[k], 0x7632), __byte_perm(w2[k], w3[k], 0x7632));
                } else {
#pragma unroll
                    for (int k = 0; k < 2; ++k)
                        xs4[chunk_of<2>(o, k)] =
                            make_uint4(__byte_perm(w0[2 * k], w1[2 * k], 0x5410), __byte_perm(w0[2 * k], w1[2 * k], 0x7632),
                                       __byte_perm(w0[2 * k + 1], w1[2 * k + 1], 0x5410),
                                       __byte_perm(w0[2 * k + 1], w1[2 * k + 1], 0x7632));
                }
#pragma unroll
                for (int r = 0; r < R; ++r) {
                    float x[8];
                    pq::unpack8(v[u][r], x);
                    if (KIND != 2) {
#pragma unroll
                        for (int e = 0; e < 8; ++e) p[r] = KIND == 0 ? __fmaf_rn(x[e], x[e], p[r]) : __fadd_rn(p[r], x[e]);
                    }
                }
            }
        }
        if (KIND != 2) {
#pragma unroll
            for (int r = 0; r < R; ++r) p[r] = lane_butterfly(p[r]);
        }
        if (KIND == 2) {
            // no normalization: the values themselves are quantized
        } else if (KIND == 0) {
#pragma unroll
            for (int r = 0; r < R; ++r)
                if (r < nlive) inv[r] = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(p[r], static_cast<float>(K)), eps)));
        } else {
            float q[R];
#pragma unroll
            for (int r = 0; r < R; ++r) mu[r] = __fdiv_rn(p[r], static_cast<float>(K)), q[r] = 0.0f;
            for (int o = lane; o < octs; o += 32) {  // the lane re-reads what it wrote
#pragma unroll
                for (int k = 0; k < R; ++k) {  // R chunks per octet
                    const uint4 c = xs4[chunk_of<R>(o, k)];
                    const uint32_t cw[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
                    for (int i = 0; i < 8 / R; ++i) {  // channels of the chunk, ascending
                        const uint2 ch = R == 4 ? make_uint2(cw[2 * i], cw[2 * i + 1]) : make_uint2(cw[i], 0u);
#pragma unroll
                        for (int r = 0; r < R; ++r) {
                            const float d0 = __fsub_rn(row_value(ch, r), mu[r]);
                            q[r] = __fmaf_rn(d0, d0, q[r]);
                        }
                    }
                }
            }
#pragma unroll
            for (int r = 0; r < R; ++r) {
                q[r] = lane_butterfly(q[r]);
                if (r < nlive) inv[r] = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(q[r], static_cast<float>(K)), eps)));
            }
        }
    }
    if (kSplit > 1) {
        if (part == 0 && lane == 0) {
#pragma unroll
            for (int r = 0; r < R; ++r) stat_s[grp_in_block][r] = inv[r], stat_s[grp_in_block][R + r] = mu[r];
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < R; ++r) inv[r] = stat_s[grp_in_block][r], mu[r] = stat_s[grp_in_block][R + r];
    } else {
        __syncwarp();
    }
    if (!present) return;

    // ---- output order: one whole group (16 consecutive positions) per lane, for all rows of the warp;
    // the indices and parameters are fetched once, the scale is derived once per group and row
    constexpr int POS = 16;
    const bool any_live = nlive > 0;
    for (int q0 = 32 * part; q0 < gpr; q0 += 32 * kSplit) {
        const int q = q0 + lane;  // group
        const bool have = q < gpr;
        uint2 g[POS];
        float w[POS], sh[POS];
#pragma unroll
        for (int j = 0; j < POS; ++j) g[j] = make_uint2(0, 0), w[j] = 0.0f, sh[j] = 0.0f;
        if (have && any_live) {
#pragma unroll
            for (int h = 0; h < POS / 4; ++h) {
                const int j0 = POS * q + 4 * h;
                int4 idx = make_int4(j0, j0 + 1, j0 + 2, j0 + 3);
                if (perm) idx = __ldg(reinterpret_cast<const int4 *>(perm) + (POS / 4) * q + h);
                g[4 * h + 0] = channel_rows<R>(xs, idx.x), g[4 * h + 1] = channel_rows<R>(xs, idx.y);
                g[4 * h + 2] = channel_rows<R>(xs, idx.z), g[4 * h + 3] = channel_rows<R>(xs, idx.w);
                if (KIND != 2) {
                    const float4 a4 = __ldg(reinterpret_cast<const float4 *>(a) + (POS / 4) * q + h);
                    w[4 * h + 0] = a4.x, w[4 * h + 1] = a4.y, w[4 * h + 2] = a4.z, w[4 * h + 3] = a4.w;
                }
                if (KIND == 1) {
                    const float4 b4 = __ldg(reinterpret_cast<const float4 *>(b) + (POS / 4) * q + h);
                    sh[4 * h + 0] = b4.x, sh[4 * h + 1] = b4.y, sh[4 * h + 2] = b4.z, sh[4 * h + 3] = b4.w;
                }
            }
            if (KIND == 1) {
#pragma unroll
                for (int j = 0; j < POS; ++j) w[j] = __fadd_rn(1.0f, w[j]);
            }
        }
#pragma unroll
        for (int r = 0; r < R; ++r) {
            const int64_t row = row0 + r;
            const bool live = r < nlive;  // rows past the end carry inv = mu = 0 and zeros in shared memory
            float out[POS];
            float amax = 0.0f;
#pragma unroll
            for (int j = 0; j < POS; ++j) {
                const float v = row_value(g[j], r);
                out[j] = KIND == 2   ? v
                         : KIND == 0 ? __fmul_rn(__fmul_rn(v, inv[r]), w[j])
                                     : __fmaf_rn(__fmul_rn(__fsub_rn(v, mu[r]), inv[r]), w[j], sh[j]);
                amax = fmaxf(amax, fabsf(out[j]));
            }
            if (!(live && have)) amax = 0.0f;  // nothing of such a row or group is stored but a zero scale byte
            uint32_t sf8;
            float d, rcp;
            pq::nvfp4_scale(amax, ts, sf8, d, rcp);
            if (live && have) {
                float y[8];
                uint2 cw;
#pragma unroll
                for (int j = 0; j < 8; ++j) y[j] = __fmul_rn(out[j], rcp);
                cw.x = pq::f32x8_to_e2m1(y);
#pragma unroll
                for (int j = 0; j < 8; ++j) y[j] = __fmul_rn(out[8 + j], rcp);
                cw.y = pq::f32x8_to_e2m1(y);
                *reinterpret_cast<uint2 *>(codes + row * (K >> 1) + q * 8) = cw;
                if (y_out) {
                    uint32_t yw[POS / 2];
#pragma unroll
                    for (int j = 0; j < POS / 2; ++j)
                        yw[j] = __bfloat16_as_ushort(__float2bfloat16_rn(out[2 * j])) |
                                (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(out[2 * j + 1]))) << 16);
                    uint4 *ydst = reinterpret_cast<uint4 *>(y_out + row * K) + 2 * q;
                    ydst[0] = make_uint4(yw[0], yw[1], yw[2], yw[3]);
                    ydst[1] = make_uint4(yw[4], yw[5], yw[6], yw[7]);
                }
            }
            // scale bytes: four neighbouring groups sit in neighbouring lanes (padding rows write zeros)
            uint32_t word = sf8;
            word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 1) << 8;
            word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 2) << 16;
            word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 3) << 24;
            if (!have || row >= rows_pad) continue;
            if (SF_LAYOUT == PQ_SF_TCGEN05) {
                if ((q & 3) == 0) *reinterpret_cast<uint32_t *>(sf + pq::sf_tc_offset(row, q, gpr >> 2)) = word;
            } else if (live) {
                if ((gpr & 3) == 0) {
                    if ((q & 3) == 0) *reinterpret_cast<uint32_t *>(sf + row * gpr + q) = word;
                } else {
                    sf[row * gpr + q] = static_cast<uint8_t>(sf8);
                }
            }
        }
    }
}

// ---- channels already in output order --------------------------------------------------------------
// When the reordering has been absorbed upstream (the previous linear layer writes its output columns in the
// new order and the norm's parameters are stored reordered, App. C), the producer needs no gather: perm ==
// NULL.  A warp then keeps its row in registers from the load to the codes: lane l owns the octets l, l + 32,
// ... (the walk the statistics are defined on), the two octets of a 16-channel group sit in neighbouring
// lanes (one shuffle for the group's absmax), every lane converts its own eight values and stores four bytes of
// codes (128 contiguous bytes per warp instruction).  No shared memory, nothing but streaming.
constexpr int kDirectMaxOcts = 16;  // octets per lane: rows of up to 4096 channels
constexpr int kDirectThreads = 128;

template <int KIND, int SF_LAYOUT, int NOCT>  // NOCT = octets per lane the registers are sized for
__global__ void __launch_bounds__(kDirectThreads)
norm_quant_ordered_kernel(const uint16_t *__restrict__ H, int64_t rows, int64_t rows_pad, int K, int64_t ld,
                          const float *__restrict__ a, const float *__restrict__ b, float eps,
                          const float *__restrict__ ts_ptr, uint8_t *__restrict__ codes, uint8_t *__restrict__ sf,
                          uint16_t *__restrict__ y_out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row = static_cast<int64_t>(blockIdx.x) * (blockDim.x >> 5) + warp;
    if (row >= rows_pad) return;  // whole warps only
    const bool live = row < rows;
    const int octs = K >> 3, gpr = K >> 4;
    const float ts = __ldg(ts_ptr);
    uint4 raw[NOCT];
#pragma unroll
    for (int u = 0; u < NOCT; ++u) {
        const int o = lane + 32 * u;
        raw[u] = (live && o < octs) ? __ldcs(reinterpret_cast<const uint4 *>(H + row * ld + o * 8)) : make_uint4(0, 0, 0, 0);
    }
    // statistics in the lane walk: this lane's octets in ascending order, then the butterfly over the lanes
    float p = 0.0f;
#pragma unroll
    for (int u = 0; u < NOCT; ++u) {
        if (lane + 32 * u < octs) {
            float x[8];
            pq::unpack8(raw[u], x);
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
        for (int u = 0; u < NOCT; ++u) {
            if (lane + 32 * u < octs) {
                float x[8];
                pq::unpack8(raw[u], x);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float d0 = __fsub_rn(x[e], mu);
                    q = __fmaf_rn(d0, d0, q);
                }
            }
        }
        q = lane_butterfly(q);
        inv = __fdiv_rn(1.0f, __fsqrt_rn(__fadd_rn(__fdiv_rn(q, static_cast<float>(K)), eps)));
    }
    if (!live) inv = 0.0f, mu = 0.0f;
    // normalize, quantize, store: octet o = lane + 32 u, group o / 2 (its other octet is in lane ^ 1)
#pragma unroll
    for (int u = 0; u < NOCT; ++u) {
        const int o = lane + 32 * u;
        if (32 * u >= octs) break;  // uniform over the warp
        const bool have = o < octs;
        float out[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) out[e] = 0.0f;
        if (live && have) {
            float x[8];
            pq::unpack8(raw[u], x);
            const float4 a0 = __ldg(reinterpret_cast<const float4 *>(a) + 2 * o), a1 = __ldg(reinterpret_cast<const float4 *>(a) + 2 * o + 1);
            const float w[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
            if (KIND == 0) {
#pragma unroll
                for (int e = 0; e < 8; ++e) out[e] = __fmul_rn(__fmul_rn(x[e], inv), w[e]);
            } else {
                const float4 b0 = __ldg(reinterpret_cast<const float4 *>(b) + 2 * o), b1 = __ldg(reinterpret_cast<const float4 *>(b) + 2 * o + 1);
                const float sh[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    out[e] = __fmaf_rn(__fmul_rn(__fsub_rn(x[e], mu), inv), __fadd_rn(1.0f, w[e]), sh[e]);
            }
        }
        float amax = pq::absmax8(out);
        amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, 1));
        uint32_t sf8;
        float d, rcp;
        pq::nvfp4_scale(amax, ts, sf8, d, rcp);
        if (live && have) {
            *reinterpret_cast<uint32_t *>(codes + row * (K >> 1) + o * 4) = pq::nvfp4_codes(out, rcp);
            if (y_out) {
                uint32_t yw[4];
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    yw[j] = __bfloat16_as_ushort(__float2bfloat16_rn(out[2 * j])) |
                            (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(out[2 * j + 1]))) << 16);
                reinterpret_cast<uint4 *>(y_out + row * K)[o] = make_uint4(yw[0], yw[1], yw[2], yw[3]);
            }
        }
        // the scale byte of a group: written by the lane that holds its first octet (padding rows write zeros)
        if (!have || (o & 1)) continue;
        const int g = o >> 1;
        if (SF_LAYOUT == PQ_SF_TCGEN05) sf[pq::sf_tc_offset(row, g, gpr >> 2)] = static_cast<uint8_t>(sf8);
        else if (live) sf[row * gpr + g] = static_cast<uint8_t>(sf8);
    }
}

template <int KIND, int SF_LAYOUT>
pq_status launch(const uint16_t *H, int64_t M, int64_t rows_pad, int K, int64_t ld, const float *a, const float *b,
                 float eps, const int32_t *perm, const float *ts, uint8_t *codes, uint8_t *sf, uint16_t *y_out,
                 cudaStream_t st) {
    // no reordering to apply and a row fits a warp's registers: the streaming kernel
    if (!perm && K <= 256 * kDirectMaxOcts) {
        const int64_t blocks = pq_ceil_div(rows_pad, kDirectThreads / 32);
        PQ_REQUIRE(blocks < (1ll << 31), PQ_ERR_SHAPE);
        const unsigned grid = static_cast<unsigned>(blocks);
        const int noct = static_cast<int>(pq_ceil_div(K, 256));
        if (noct <= 4) norm_quant_ordered_kernel<KIND, SF_LAYOUT, 4><<<grid, kDirectThreads, 0, st>>>(H, M, rows_pad, K, ld, a, b, eps, ts, codes, sf, y_out);
        else if (noct <= 8) norm_quant_ordered_kernel<KIND, SF_LAYOUT, 8><<<grid, kDirectThreads, 0, st>>>(H, M, rows_pad, K, ld, a, b, eps, ts, codes, sf, y_out);
        else if (noct <= 12) norm_quant_ordered_kernel<KIND, SF_LAYOUT, 12><<<grid, kDirectThreads, 0, st>>>(H, M, rows_pad, K, ld, a, b, eps, ts, codes, sf, y_out);
        else norm_quant_ordered_kernel<KIND, SF_LAYOUT, 16><<<grid, kDirectThreads, 0, st>>>(H, M, rows_pad, K, ld, a, b, eps, ts, codes, sf, y_out);
        return pq_launch_status();
    }
    // up to 6400 channels: four rows per warp, four warps per block (two blocks per SM at 3072 channels)
    const size_t group_smem = static_cast<size_t>(kGroupWarps) * kGroupRows * K * 2;
    if (group_smem <= kSmemBudget) {
        if (group_smem > 40 * 1024)  // the kernel's static shared memory counts towards the 48 KB default limit
            PQ_CUDA_OK(cudaFuncSetAttribute(norm_quant_grouped_kernel<KIND, SF_LAYOUT>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(group_smem)));
        const int64_t blocks = pq_ceil_div(rows_pad, kGroupWarps * kGroupRows);
        PQ_REQUIRE(blocks < (1ll << 31), PQ_ERR_SHAPE);
        norm_quant_grouped_kernel<KIND, SF_LAYOUT><<<static_cast<unsigned>(blocks), kGroupWarps * kSplit * 32, group_smem, st>>>(
            H, M, rows_pad, K, ld, a, b, eps, perm, nullptr, ts, codes, sf, y_out);
        return pq_launch_status();
    }
    // wider rows: one warp per row, the row as bf16 in shared memory: 8 rows per block up to 12800 channels
    int warps = static_cast<int>(kSmemBudget / (static_cast<size_t>(K) * 2));
    if (warps > kMaxRowsPerBlock) warps = kMaxRowsPerBlock;
    if (warps < 1) return PQ_ERR_SHAPE;
    const size_t smem = static_cast<size_t>(warps) * K * 2;
    if (smem > 48 * 1024)
        PQ_CUDA_OK(cudaFuncSetAttribute(norm_quant_kernel<KIND, SF_LAYOUT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(smem)));
    const int64_t blocks = pq_ceil_div(rows_pad, warps);
    PQ_REQUIRE(blocks < (1ll << 31), PQ_ERR_SHAPE);
    norm_quant_kernel<KIND, SF_LAYOUT><<<static_cast<unsigned>(blocks), warps * 32, smem, st>>>(
        H, M, rows_pad, K, ld, a, b, eps, perm, ts, codes, sf, y_out);
    return pq_launch_status();
}

template <int SF_LAYOUT>
pq_status launch_gather_only(const uint16_t *X, int64_t M, int64_t rows_pad, int K, int64_t ld, const int32_t *perm,
                             const int32_t *perm_select, const float *ts, uint8_t *codes, uint8_t *sf, cudaStream_t st) {
    const size_t group_smem = static_cast<size_t>(kGroupWarps) * kGroupRows * K * 2;
    if (group_smem > 40 * 1024)
        PQ_CUDA_OK(cudaFuncSetAttribute(norm_quant_grouped_kernel<2, SF_LAYOUT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(group_smem)));
    const int64_t blocks = pq_ceil_div(rows_pad, kGroupWarps * kGroupRows);
    PQ_REQUIRE(blocks < (1ll << 31), PQ_ERR_SHAPE);
    norm_quant_grouped_kernel<2, SF_LAYOUT><<<static_cast<unsigned>(blocks), kGroupWarps * kSplit * 32, group_smem, st>>>(
        X, M, rows_pad, K, ld, nullptr, nullptr, 0.0f, perm, perm_select, ts, codes, sf, nullptr);
    return pq_launch_status();
}

}  // namespace

// The gather quantizer of pq_quant_act_nvfp4_perm and pq_quant_weight for rows the four-rows-per-warp kernel can
// hold: that kernel with the normalization left out (the gathered values themselves are quantized).
bool pq_gather_quant_grouped_fits(int64_t K) {
    return K > 0 && static_cast<size_t>(kGroupWarps) * kGroupRows * static_cast<size_t>(K) * 2 <= kSmemBudget;
}
pq_status pq_gather_quant_grouped(const void *X, int64_t M, int64_t K, int64_t ld, const int32_t *perm,
                                  const int32_t *perm_select, const float *ts_x, uint8_t *codes, uint8_t *sf,
                                  int sf_layout, void *stream) {
    const int64_t rows_pad = sf_layout == PQ_SF_TCGEN05 ? pq_ceil_div(M, 128) * 128 : M;
    const uint16_t *x = static_cast<const uint16_t *>(X);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    return sf_layout == PQ_SF_TCGEN05
               ? launch_gather_only<PQ_SF_TCGEN05>(x, M, rows_pad, static_cast<int>(K), ld, perm, perm_select, ts_x, codes, sf, st)
               : launch_gather_only<PQ_SF_LINEAR>(x, M, rows_pad, static_cast<int>(K), ld, perm, perm_select, ts_x, codes, sf, st);
}

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
