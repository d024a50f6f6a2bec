// PermuQuant-H producer (App. D): Hadamard transform of every token row, the channel reordering applied
// when the transformed row is read back (x H P: only the order in which transformed channels are
// consumed changes), and the NVFP4 quantizer of the runtime path (Eq. 8) attached, so the transformed
// activations never make a round trip through HBM.
//
// The transform.  K = m * 2^n with m = 1 or m = 12; y = x (H_m (x) H_{2^n}) / sqrt(K): with channel
// i = a * 2^n + b the matrix entry is H_m[a][a'] * (-1)^popcount(b & b').  H_12 is Paley's matrix for
// q = 11 (I + S, S skew, built from the quadratic character modulo 11).  All arithmetic is IEEE fp32 in
// a fixed order: the 12 segments are combined first (terms added one by one in ascending segment), then
// the butterflies of the fast Walsh-Hadamard transform run inside each segment with strides 1, 2, 4, ...,
// then one multiplication by fl(1 / sqrt(K)).  Within one stride the butterflies are independent, so how
// they are spread over threads does not change a bit of the result.
//
// Work distribution (one thread block = up to 8 rows, each row kept as K fp32 values in shared memory):
//   phase 1  a thread takes one octet position of one row: m 16-byte loads (the same octet of every
//            segment), the segment combination and the strides 1, 2, 4 in registers, on PAIRS of
//            neighbouring channels in packed f32x2 instructions (two IEEE results per issue slot; the
//            stride-1 butterfly of a pair (x, y) is one packed fused multiply-add (x, y) * (1, -1) +
//            (y, x), exact products, one rounding: the same bits as x + y and x - y);
//   phase 2  the remaining strides in one to three passes over shared memory: a thread owns one channel
//            pair position and 2^LOG values of it at the pass's strides (up to 32 packed registers);
//   phase 3  a lane takes one 16-channel group of the OUTPUT order: indices from the permutation,
//            values gathered from shared memory, scaled, quantized like pq_quant_act_nvfp4 (coalesced
//            code stores, four scale bytes merged into a word by shuffles).
// Shared-memory addresses are XOR-swizzled (octet index bits 3-4 with the two bits just above the
// first pass's window) so that the strided accesses of phase 2 spread over all banks.
#include <utility>

#include "pq_common.cuh"

namespace {

constexpr int kMaxRows = 8;         // rows per block (fewer when a row needs more than 24 KB of shared memory)
constexpr int kThreads = 256;
constexpr size_t kSmemBudget = 196 * 1024;

// ---- Paley's Hadamard matrix of order 12 (compile-time)
constexpr int quadratic_character_11(int r) {
    r = ((r % 11) + 11) % 11;
    if (r == 0) return 0;
    for (int t = 1; t < 11; ++t)
        if ((t * t) % 11 == r) return 1;
    return -1;
}
constexpr int paley12(int i, int j) {
    return i == j ? 1 : i == 0 ? 1 : j == 0 ? -1 : quadratic_character_11(i - j);
}
template <int I, int J>
struct Paley12 {
    static constexpr bool plus = paley12(I, J) > 0;
};

// ---- packed fp32 pairs
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
// (x, y) -> (x + y, x - y): (x, y) * (1, -1) + (y, x)
__device__ __forceinline__ uint64_t butterfly_in_pair(uint64_t v) {
    float x, y;
    unpack2(v, x, y);
    return fma2(v, pack2(1.0f, -1.0f), pack2(y, x));
}

// fp32 index of a channel inside its row's shared-memory image
__device__ __forceinline__ int swz(int idx, int sw) { return idx ^ (((idx >> sw) & 3) << 3); }

struct HadParams {
    const uint16_t *X;
    int64_t rows, rows_pad, ld;
    int K, m, n;            // K = m * 2^n
    int log[3];             // bits taken by the passes of phase 2 (0 = no such pass)
    int sw;                 // swizzle source bit
    int rows_per_block;
    float scale;            // fl(1 / sqrt(K))
    const int32_t *perm;
    const float *ts;
    uint8_t *codes, *sf;
    uint16_t *y_out;
};

// ---- phase 1: one octet position of one row
template <int AP, int A>
__device__ __forceinline__ void combine_segments(uint64_t (&acc)[4], const uint64_t (&in)[12][4]) {
    if constexpr (A < 12) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if constexpr (Paley12<A, AP>::plus) acc[e] = add2(acc[e], in[A][e]);
            else acc[e] = sub2(acc[e], in[A][e]);
        }
        combine_segments<AP, A + 1>(acc, in);
    }
}

// strides 1, 2, 4 on the four channel pairs of an octet, then the octet goes to shared memory
__device__ __forceinline__ void finish_octet(uint64_t (&v)[4], float *row_s, int idx, int sw, bool second_half_first) {
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = butterfly_in_pair(v[e]);
    const uint64_t a0 = add2(v[0], v[1]), a1 = sub2(v[0], v[1]), a2 = add2(v[2], v[3]), a3 = sub2(v[2], v[3]);
    const uint64_t b0 = add2(a0, a2), b1 = add2(a1, a3), b2 = sub2(a0, a2), b3 = sub2(a1, a3);
    // two 16-byte stores; every other group of four lanes writes its halves in the opposite order, which
    // keeps the eight lanes of a store wavefront on distinct banks
    ulonglong2 *dst = reinterpret_cast<ulonglong2 *>(row_s + swz(idx, sw));
    const ulonglong2 lo = make_ulonglong2(b0, b1), hi = make_ulonglong2(b2, b3);
    dst[second_half_first ? 1 : 0] = second_half_first ? hi : lo;
    dst[second_half_first ? 0 : 1] = second_half_first ? lo : hi;
}

__device__ __forceinline__ void unpack_pairs(const uint4 &raw, uint64_t (&v)[4]) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = pack2(__uint_as_float(w[e] << 16), __uint_as_float(w[e] & 0xFFFF0000u));
}

template <int AP>
__device__ __forceinline__ void column_12(const uint64_t (&in)[12][4], float *row_s, int seg, int o, int sw, bool flip) {
    uint64_t acc[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] = in[0][e];  // the first row of the matrix is all ones
    combine_segments<AP, 1>(acc, in);
    finish_octet(acc, row_s, AP * seg + o * 8, sw, flip);
}
template <int... APs>
__device__ __forceinline__ void all_columns_12(std::integer_sequence<int, APs...>, const uint64_t (&in)[12][4], float *row_s,
                                               int seg, int o, int sw, bool flip) {
    (column_12<APs>(in, row_s, seg, o, sw, flip), ...);
}

// ---- phase 2: 2^LOG values of one channel-pair position, strides 2^S ... 2^(S+LOG-1)
template <int LOG>
__device__ __forceinline__ void pass_item(float *row_s, int base, int S, int sw, bool last, uint64_t scale2) {
    constexpr int N = 1 << LOG;
    uint64_t v[N];
#pragma unroll
    for (int j = 0; j < N; ++j) v[j] = *reinterpret_cast<const uint64_t *>(row_s + swz(base + (j << S), sw));
#pragma unroll
    for (int l = 0; l < LOG; ++l) {
#pragma unroll
        for (int j = 0; j < N; ++j) {
            if ((j >> l) & 1) continue;
            const uint64_t p = v[j], q = v[j | (1 << l)];
            v[j] = add2(p, q);
            v[j | (1 << l)] = sub2(p, q);
        }
    }
    if (last) {
#pragma unroll
        for (int j = 0; j < N; ++j) v[j] = mul2(v[j], scale2);
    }
#pragma unroll
    for (int j = 0; j < N; ++j) *reinterpret_cast<uint64_t *>(row_s + swz(base + (j << S), sw)) = v[j];
}

// One pass over the rows of the block: items = rows x (K / 2) channel pairs / 2^LOG.
__device__ __forceinline__ void run_pass(float *smem, const HadParams &p, int nrows, int S, int LOG, bool last) {
    const uint64_t scale2 = pack2(p.scale, p.scale);
    const int per_row = (p.K >> 1) >> LOG;  // items per row
    const int low_mask = (1 << (S - 1)) - 1;  // pair-index bits below the window (a pair index is channel >> 1)
    for (int u = threadIdx.x; u < nrows * per_row; u += kThreads) {
        const int r = u / per_row, w = u - r * per_row;
        // w enumerates the pair positions with the window bits removed: low part below the window, the rest above
        const int pair = (w & low_mask) | ((w & ~low_mask) << LOG);
        float *row_s = smem + static_cast<size_t>(r) * p.K;
        const int base = pair << 1;
        switch (LOG) {
            case 1: pass_item<1>(row_s, base, S, p.sw, last, scale2); break;
            case 2: pass_item<2>(row_s, base, S, p.sw, last, scale2); break;
            case 3: pass_item<3>(row_s, base, S, p.sw, last, scale2); break;
            case 4: pass_item<4>(row_s, base, S, p.sw, last, scale2); break;
            default: pass_item<5>(row_s, base, S, p.sw, last, scale2); break;
        }
    }
}

template <int SF_LAYOUT>
__global__ void __launch_bounds__(kThreads, 2) hadamard_quant_kernel(const HadParams p) {
    extern __shared__ __align__(16) float had_smem[];  // [rows_per_block][K]
    const int kRows = p.rows_per_block;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t row0 = static_cast<int64_t>(blockIdx.x) * kRows;
    const int nrows = static_cast<int>(min(static_cast<int64_t>(kRows), max(static_cast<int64_t>(0), p.rows - row0)));
    const int seg = p.K / p.m, octs = seg >> 3;
    pq::wait_for_prior_grid();
    pq::dependents_may_launch();

    // ---- phase 1
    for (int u = threadIdx.x; u < nrows * octs; u += kThreads) {
        const int r = u / octs, o = u - r * octs;
        const uint16_t *src = p.X + (row0 + r) * p.ld + o * 8;
        float *row_s = had_smem + static_cast<size_t>(r) * p.K;
        const bool flip = (o >> 2) & 1;
        if (p.m == 12) {
            uint64_t in[12][4];
#pragma unroll
            for (int a = 0; a < 12; ++a) unpack_pairs(__ldcs(reinterpret_cast<const uint4 *>(src + a * seg)), in[a]);
            all_columns_12(std::make_integer_sequence<int, 12>{}, in, row_s, seg, o, p.sw, flip);
        } else {
            uint64_t v[4];
            unpack_pairs(__ldcs(reinterpret_cast<const uint4 *>(src)), v);
            finish_octet(v, row_s, o * 8, p.sw, flip);
        }
    }
    __syncthreads();
    // ---- phase 2 (the scaling rides on the last pass; without any pass it is applied in phase 3)
    int start = 3;
#pragma unroll 1
    for (int k = 0; k < 3 && p.log[k]; ++k) {
        run_pass(had_smem, p, nrows, start, p.log[k], k == 2 || p.log[k + 1] == 0);
        start += p.log[k];
        __syncthreads();
    }
    const float late_scale = p.log[0] ? 1.0f : p.scale;  // multiplying by one changes nothing

    // ---- phase 3: one row per warp, one output group per lane
    const float ts = p.codes ? __ldg(p.ts) : 1.0f;
    const int gpr = p.K >> 4;
    for (int r = warp; r < kRows; r += kThreads / 32) {
        const int64_t row = row0 + r;
        if (row >= p.rows_pad) break;
        const bool live = row < p.rows;
        const float *row_s = had_smem + static_cast<size_t>(r) * p.K;
        for (int g0 = 0; g0 < gpr; g0 += 32) {
            const int g = g0 + lane;
            const bool have = g < gpr;
            float out[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) out[j] = 0.0f;
            if (live && have) {
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                    const int j0 = 16 * g + 4 * h;
                    int4 idx = make_int4(j0, j0 + 1, j0 + 2, j0 + 3);
                    if (p.perm) idx = __ldg(reinterpret_cast<const int4 *>(p.perm) + 4 * g + h);
                    out[4 * h + 0] = __fmul_rn(row_s[swz(idx.x, p.sw)], late_scale);
                    out[4 * h + 1] = __fmul_rn(row_s[swz(idx.y, p.sw)], late_scale);
                    out[4 * h + 2] = __fmul_rn(row_s[swz(idx.z, p.sw)], late_scale);
                    out[4 * h + 3] = __fmul_rn(row_s[swz(idx.w, p.sw)], late_scale);
                }
                if (p.y_out) {
                    uint32_t yw[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        yw[j] = __bfloat16_as_ushort(__float2bfloat16_rn(out[2 * j])) |
                                (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(out[2 * j + 1]))) << 16);
                    uint4 *ydst = reinterpret_cast<uint4 *>(p.y_out + row * p.K) + 2 * g;
                    ydst[0] = make_uint4(yw[0], yw[1], yw[2], yw[3]);
                    ydst[1] = make_uint4(yw[4], yw[5], yw[6], yw[7]);
                }
            }
            if (!p.codes) continue;
            float amax = 0.0f;
#pragma unroll
            for (int j = 0; j < 16; ++j) amax = fmaxf(amax, fabsf(out[j]));
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
                *reinterpret_cast<uint2 *>(p.codes + row * (p.K >> 1) + g * 8) = cw;
            }
            // scale bytes: four neighbouring groups sit in neighbouring lanes (padding rows write zeros)
            uint32_t word = sf8;
            word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 1) << 8;
            word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 2) << 16;
            word |= __shfl_down_sync(0xFFFFFFFFu, sf8, 3) << 24;
            if (!have) continue;
            if (SF_LAYOUT == PQ_SF_TCGEN05) {
                if ((g & 3) == 0) *reinterpret_cast<uint32_t *>(p.sf + pq::sf_tc_offset(row, g, gpr >> 2)) = word;
            } else if (live) {
                if ((gpr & 3) == 0) {
                    if ((g & 3) == 0) *reinterpret_cast<uint32_t *>(p.sf + row * gpr + g) = word;
                } else {
                    p.sf[row * gpr + g] = static_cast<uint8_t>(sf8);
                }
            }
        }
    }
}

// K = m * 2^n with m in {1, 12} and 2^n >= 8; returns false otherwise.
bool factor_width(int64_t K, int &m, int &n) {
    if (K <= 0) return false;
    int64_t seg;
    if ((K & (K - 1)) == 0) m = 1, seg = K;
    else if (K % 12 == 0 && ((K / 12) & (K / 12 - 1)) == 0) m = 12, seg = K / 12;
    else return false;
    n = 0;
    while ((static_cast<int64_t>(1) << n) < seg) ++n;
    return seg >= 8;
}

}  // namespace

extern "C" pq_status pq_hadamard_quant_nvfp4(const void *X, int64_t M, int64_t K, int64_t ld, const int32_t *perm,
                                             const float *ts_x, uint8_t *codes, uint8_t *sf, int sf_layout, void *y_out,
                                             void *stream) {
    PQ_REQUIRE(X, PQ_ERR_NULL);
    PQ_REQUIRE((codes == nullptr) == (sf == nullptr), PQ_ERR_NULL);
    PQ_REQUIRE(codes || y_out, PQ_ERR_NULL);
    PQ_REQUIRE(!codes || ts_x, PQ_ERR_NULL);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || sf_layout == PQ_SF_TCGEN05, PQ_ERR_FORMAT);
    int m = 0, n = 0;
    PQ_REQUIRE(M > 0 && K >= 16 && K % 16 == 0 && K <= 16384 && ld >= K && factor_width(K, m, n), PQ_ERR_SHAPE);
    PQ_REQUIRE(sf_layout == PQ_SF_LINEAR || !codes || K % 64 == 0, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(X) && ld % 8 == 0 && (!codes || (pq_aligned16(codes) && pq_aligned16(sf))) &&
                   (!perm || pq_aligned16(perm)) && (!y_out || pq_aligned16(y_out)),
               PQ_ERR_ALIGN);
    HadParams p;
    p.X = static_cast<const uint16_t *>(X);
    p.rows = M;
    p.rows_pad = (codes && sf_layout == PQ_SF_TCGEN05) ? pq_ceil_div(M, 128) * 128 : M;
    p.ld = ld;
    p.K = static_cast<int>(K), p.m = m, p.n = n;
    // strides 1, 2, 4 are taken in phase 1; the remaining n - 3 bits in up to three passes of at most 5
    const int rest = n - 3, passes = (rest + 4) / 5;
    PQ_REQUIRE(passes <= 3, PQ_ERR_SHAPE);
    for (int k = 0, left = rest; k < 3; ++k) {
        p.log[k] = k < passes ? (left + (passes - k) - 1) / (passes - k) : 0;
        left -= p.log[k];
    }
    p.sw = p.log[0] ? 3 + p.log[0] : 30;
    p.scale = static_cast<float>(1.0 / sqrt(static_cast<double>(K)));
    p.perm = perm, p.ts = ts_x, p.codes = codes, p.sf = sf, p.y_out = static_cast<uint16_t *>(y_out);
    const size_t row_bytes = static_cast<size_t>(K) * sizeof(float);
    p.rows_per_block = static_cast<int>(kSmemBudget / row_bytes < kMaxRows ? kSmemBudget / row_bytes : kMaxRows);
    const int kRows = p.rows_per_block;
    const size_t smem = static_cast<size_t>(kRows) * row_bytes;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int64_t blocks = pq_ceil_div(p.rows_pad, kRows);
    PQ_REQUIRE(blocks < (1ll << 31), PQ_ERR_SHAPE);
    auto launch = [&](auto kern) -> pq_status {
        if (smem > 48 * 1024)
            PQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        PQ_CUDA_OK(pq::launch_dependent(kern, dim3(static_cast<unsigned>(blocks)), dim3(kThreads), smem, st, p));
        return pq_launch_status();
    };
    return sf_layout == PQ_SF_TCGEN05 ? launch(hadamard_quant_kernel<PQ_SF_TCGEN05>)
                                      : launch(hadamard_quant_kernel<PQ_SF_LINEAR>);
}
