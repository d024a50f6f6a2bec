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
// Work distribution.  A thread block keeps up to 8 rows as K fp32 values each in shared memory and walks
// over batches of rows (persistent grid):
//   phase 1  a thread takes one octet position of one row: m 16-byte loads (the same octet of every
//            segment), the segment combination and the strides 1, 2, 4 in registers, on PAIRS of
//            neighbouring channels in packed f32x2 instructions (two IEEE results per issue slot);
//   phase 2  the remaining strides in one to three passes over shared memory: a thread owns one channel
//            pair position and 2^LOG values of it at the pass's strides (up to 32 packed registers),
//            addressed through eight base pointers and immediate offsets;
//   phase 3  a lane takes one 16-channel group of the OUTPUT order: its 16 read-out positions (the
//            permutation with the shared-memory swizzle applied, as 16-bit byte offsets, prepared once
//            per block) come as two 16-byte loads, the values are gathered from shared memory and
//            quantized like pq_quant_act_nvfp4 (coalesced code stores, four scale bytes merged into a
//            word by shuffles).
// Shared-memory swizzle of a row image (fp32 index i): bits 3-4 are XORed with the two bits just above
// the first pass's window and bit 2 with bit 5.  The first spreads the strided accesses of phase 2 over
// all banks, the second lets the eight lanes of a 16-byte store wavefront of phase 1 hit distinct banks.
#include <algorithm>
#include <utility>

#include "pq_common.cuh"

namespace {

#ifndef PQ_HAD_ROWS
#define PQ_HAD_ROWS 8
#endif
constexpr int kMaxRows = PQ_HAD_ROWS;   // rows per block (fewer when a row needs more than 24 KB of shared memory)
constexpr int kThreads = 32 * kMaxRows;
#ifndef PQ_HAD_BLOCKS
#define PQ_HAD_BLOCKS (512 / (32 * PQ_HAD_ROWS))
#endif
constexpr int kBlocksPerSm = PQ_HAD_BLOCKS;
constexpr size_t kSmemBudget = 192 * 1024;

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
// (x, y) -> (x + y, x - y)
__device__ __forceinline__ uint64_t butterfly_in_pair(uint64_t v) {
    float x, y;
    unpack2(v, x, y);
    return pack2(__fadd_rn(x, y), __fsub_rn(x, y));
}

// fp32 index of a channel inside its row's shared-memory image
__device__ __forceinline__ int swz(int idx, int sw) { return idx ^ (((idx >> sw) & 3) << 3) ^ (((idx >> 5) & 1) << 2); }

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
__device__ __forceinline__ void finish_octet(uint64_t (&v)[4], float *row_s, int idx, int sw) {
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = butterfly_in_pair(v[e]);
    const uint64_t a0 = add2(v[0], v[1]), a1 = sub2(v[0], v[1]), a2 = add2(v[2], v[3]), a3 = sub2(v[2], v[3]);
    const uint64_t b0 = add2(a0, a2), b1 = add2(a1, a3), b2 = sub2(a0, a2), b3 = sub2(a1, a3);
    // two 16-byte stores; the swizzle swaps the halves of every other group of four octets, which keeps
    // the eight lanes of a store wavefront on distinct banks
    const int half = (idx >> 5) & 1;
    ulonglong2 *dst = reinterpret_cast<ulonglong2 *>(row_s + (idx ^ (((idx >> sw) & 3) << 3)));
    dst[half] = make_ulonglong2(b0, b1);
    dst[half ^ 1] = make_ulonglong2(b2, b3);
}

__device__ __forceinline__ void unpack_pairs(const uint4 &raw, uint64_t (&v)[4]) {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) v[e] = pack2(__uint_as_float(w[e] << 16), __uint_as_float(w[e] & 0xFFFF0000u));
}

template <int AP>
__device__ __forceinline__ void column_12(const uint64_t (&in)[12][4], float *row_s, int seg, int o, int sw) {
    uint64_t acc[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] = in[0][e];  // the first row of the matrix is all ones
    combine_segments<AP, 1>(acc, in);
    finish_octet(acc, row_s, AP * seg + o * 8, sw);
}
template <int... APs>
__device__ __forceinline__ void all_columns_12(std::integer_sequence<int, APs...>, const uint64_t (&in)[12][4], float *row_s,
                                               int seg, int o, int sw) {
    (column_12<APs>(in, row_s, seg, o, sw), ...);
}

// ---- phase 2: 2^LOG values of one channel-pair position, strides 2^S ... 2^(S+LOG-1)
// The swizzle reads two bits and bit 5 and writes bits 2-4; of the window's bits only the lowest three can
// be among those, so the address of value j is that of value j % 8 plus an immediate.
template <int LOG>
__device__ __forceinline__ void pass_item(float *row_s, int base, int S, int sw, bool last, uint64_t scale2) {
    constexpr int N = 1 << LOG, NB = N < 8 ? N : 8;
    uint64_t *slot[NB];
#pragma unroll
    for (int m = 0; m < NB; ++m) slot[m] = reinterpret_cast<uint64_t *>(row_s + swz(base + (m << S), sw));
    const int step = 4 << S;  // 64-bit words between value j and value j + 8
    uint64_t v[N];
#pragma unroll
    for (int j = 0; j < N; ++j) v[j] = slot[j % NB][(j / NB) * step];
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
    for (int j = 0; j < N; ++j) slot[j % NB][(j / NB) * step] = v[j];
}

// One pass over the rows of the block: items = rows x (K / 2) channel pairs / 2^LOG.
template <int THREADS>
__device__ __forceinline__ void run_pass(float *smem, const HadParams &p, int nrows, int S, int LOG, bool last) {
    const uint64_t scale2 = pack2(p.scale, p.scale);
    const int per_row = (p.K >> 1) >> LOG;  // items per row
    const int low_mask = (1 << (S - 1)) - 1;  // pair-index bits below the window (a pair index is channel >> 1)
    for (int u = threadIdx.x; u < nrows * per_row; u += THREADS) {
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

// THREADS: 256 (two blocks per SM) while a block holds eight rows; 512 (one block) when rows wider than 6144
// channels leave room for fewer, so that an SM still has 16 warps at work on them
template <int SF_LAYOUT, int THREADS>
__global__ void __launch_bounds__(THREADS, 512 / THREADS) hadamard_quant_kernel(const HadParams p) {
    extern __shared__ __align__(16) float had_smem[];  // [rows_per_block][K] fp32, then K 16-bit read-out offsets
    const int kRows = p.rows_per_block;
    uint16_t *offset_s = reinterpret_cast<uint16_t *>(had_smem + static_cast<size_t>(kRows) * p.K);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int seg = p.K / p.m, octs = seg >> 3;
    const int gpr = p.K >> 4, chunks = (gpr + 31) >> 5;  // output groups per row, in chunks of one per lane
    const int64_t batches = (p.rows_pad + kRows - 1) / kRows;
    pq::wait_for_prior_grid();
    pq::dependents_may_launch();

    // where each output position reads its channel in a row's (swizzled) shared-memory image, as a byte
    // offset: the same for every row, so it is worked out once per block (K <= 16384: 16 bits)
    for (int j = threadIdx.x; j < p.K; j += THREADS)
        offset_s[j] = static_cast<uint16_t>(swz(p.perm ? __ldg(p.perm + j) : j, p.sw) << 2);
    const float ts = p.codes ? __ldg(p.ts) : 1.0f;

    for (int64_t batch = blockIdx.x; batch < batches; batch += gridDim.x) {
        const int64_t row0 = batch * kRows;
        const int nrows = static_cast<int>(min(static_cast<int64_t>(kRows), max(static_cast<int64_t>(0), p.rows - row0)));
        __syncthreads();  // the previous batch has been read out (and the offsets are in place)

        // ---- phase 1
        for (int u = threadIdx.x; u < nrows * octs; u += THREADS) {
            const int r = u / octs, o = u - r * octs;
            const uint16_t *src = p.X + (row0 + r) * p.ld + o * 8;
            float *row_s = had_smem + static_cast<size_t>(r) * p.K;
            if (p.m == 12) {
                uint64_t in[12][4];
#pragma unroll
                for (int a = 0; a < 12; ++a) unpack_pairs(__ldcs(reinterpret_cast<const uint4 *>(src + a * seg)), in[a]);
                all_columns_12(std::make_integer_sequence<int, 12>{}, in, row_s, seg, o, p.sw);
            } else {
                uint64_t v[4];
                unpack_pairs(__ldcs(reinterpret_cast<const uint4 *>(src)), v);
                finish_octet(v, row_s, o * 8, p.sw);
            }
        }
        __syncthreads();
        // ---- phase 2 (the scaling rides on the last pass; without any pass it is applied in phase 3)
        int start = 3;
#pragma unroll 1
        for (int k = 0; k < 3 && p.log[k]; ++k) {
            run_pass<THREADS>(had_smem, p, nrows, start, p.log[k], k == 2 || p.log[k + 1] == 0);
            start += p.log[k];
            __syncthreads();
        }

        // ---- phase 3: a warp takes a chunk of 32 output groups of TWO rows at a time, one group per lane:
        // the read-out offsets are fetched once for both rows and the two quantizer chains interleave
        const int rows_here = static_cast<int>(min(static_cast<int64_t>(kRows), p.rows_pad - row0));
        const int row_pairs = (rows_here + 1) >> 1;
        for (int c = warp; c < row_pairs * chunks; c += THREADS / 32) {
            const int rp = c / chunks, g = (c - rp * chunks) * 32 + lane;
            const bool have = g < gpr;
            uint32_t iw[8];
            if (have) {
                const uint4 i0 = reinterpret_cast<const uint4 *>(offset_s)[2 * g], i1 = reinterpret_cast<const uint4 *>(offset_s)[2 * g + 1];
                iw[0] = i0.x, iw[1] = i0.y, iw[2] = i0.z, iw[3] = i0.w, iw[4] = i1.x, iw[5] = i1.y, iw[6] = i1.z, iw[7] = i1.w;
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) iw[j] = 0;
            }
            float out[2][16];
            bool live[2], present[2];
            int64_t row[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = 2 * rp + h;
                row[h] = row0 + r;
                present[h] = r < rows_here;
                // the second row of the last pair does not exist when the block holds an odd number of rows (three
                // at 16384 channels): that index is the first row of the NEXT batch and lies past this image
                live[h] = present[h] && row[h] < p.rows;
                const char *row_b = reinterpret_cast<const char *>(had_smem + static_cast<size_t>(r) * p.K);
#pragma unroll
                for (int j = 0; j < 16; ++j) out[h][j] = 0.0f;
                if (live[h] && have) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        out[h][2 * j] = *reinterpret_cast<const float *>(row_b + (iw[j] & 0xFFFFu));
                        out[h][2 * j + 1] = *reinterpret_cast<const float *>(row_b + (iw[j] >> 16));
                    }
                    if (!p.log[0]) {  // no pass of phase 2 carried the scaling
#pragma unroll
                        for (int j = 0; j < 16; ++j) out[h][j] = __fmul_rn(out[h][j], p.scale);
                    }
                    if (p.y_out) {
                        uint32_t yw[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            yw[j] = __bfloat16_as_ushort(__float2bfloat16_rn(out[h][2 * j])) |
                                    (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(out[h][2 * j + 1]))) << 16);
                        uint4 *ydst = reinterpret_cast<uint4 *>(p.y_out + row[h] * p.K) + 2 * g;
                        ydst[0] = make_uint4(yw[0], yw[1], yw[2], yw[3]);
                        ydst[1] = make_uint4(yw[4], yw[5], yw[6], yw[7]);
                    }
                }
            }
            if (!p.codes) continue;
            uint32_t sf8[2];
            float rcp[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                float amax = 0.0f, d;
#pragma unroll
                for (int j = 0; j < 16; ++j) amax = fmaxf(amax, fabsf(out[h][j]));
                pq::nvfp4_scale(amax, ts, sf8[h], d, rcp[h]);
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (live[h] && have) {
                    const uint64_t rcp2 = pack2(rcp[h], rcp[h]);
                    float ylo[8], yhi[8];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        unpack2(mul2(pack2(out[h][2 * j], out[h][2 * j + 1]), rcp2), ylo[2 * j], ylo[2 * j + 1]);
                        unpack2(mul2(pack2(out[h][8 + 2 * j], out[h][9 + 2 * j]), rcp2), yhi[2 * j], yhi[2 * j + 1]);
                    }
                    *reinterpret_cast<uint2 *>(p.codes + row[h] * (p.K >> 1) + g * 8) =
                        make_uint2(pq::f32x8_to_e2m1(ylo), pq::f32x8_to_e2m1(yhi));
                }
                // scale bytes: four neighbouring groups sit in neighbouring lanes (padding rows write zeros)
                uint32_t word = sf8[h];
                word |= __shfl_down_sync(0xFFFFFFFFu, sf8[h], 1) << 8;
                word |= __shfl_down_sync(0xFFFFFFFFu, sf8[h], 2) << 16;
                word |= __shfl_down_sync(0xFFFFFFFFu, sf8[h], 3) << 24;
                if (!have || !present[h]) continue;
                if (SF_LAYOUT == PQ_SF_TCGEN05) {
                    if ((g & 3) == 0) *reinterpret_cast<uint32_t *>(p.sf + pq::sf_tc_offset(row[h], g, gpr >> 2)) = word;
                } else if (live[h]) {
                    if ((gpr & 3) == 0) {
                        if ((g & 3) == 0) *reinterpret_cast<uint32_t *>(p.sf + row[h] * gpr + g) = word;
                    } else {
                        p.sf[row[h] * gpr + g] = static_cast<uint8_t>(sf8[h]);
                    }
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
    const size_t smem = static_cast<size_t>(kRows) * row_bytes + static_cast<size_t>(K) * sizeof(uint16_t);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // persistent grid: as many blocks as fit on the device at once, walking over the batches of rows
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const bool wide_block = kRows < kMaxRows;  // fewer rows per block: twice the threads on them, one block per SM
    const int per_sm = static_cast<int>(std::min<size_t>(wide_block ? 1 : kBlocksPerSm, (227 * 1024) / (smem + 1024)));
    const int64_t batches = pq_ceil_div(p.rows_pad, kRows);
    const int64_t blocks = std::min<int64_t>(batches, static_cast<int64_t>(sms) * (per_sm > 0 ? per_sm : 1));
    auto launch = [&](auto kern) -> pq_status {
        if (smem > 48 * 1024)
            PQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        PQ_CUDA_OK(pq::launch_dependent(kern, dim3(static_cast<unsigned>(blocks)), dim3(wide_block ? 2 * kThreads : kThreads),
                                        smem, st, p));
        return pq_launch_status();
    };
    if (wide_block)
        return sf_layout == PQ_SF_TCGEN05 ? launch(hadamard_quant_kernel<PQ_SF_TCGEN05, 2 * kThreads>)
                                          : launch(hadamard_quant_kernel<PQ_SF_LINEAR, 2 * kThreads>);
    return sf_layout == PQ_SF_TCGEN05 ? launch(hadamard_quant_kernel<PQ_SF_TCGEN05, kThreads>)
                                      : launch(hadamard_quant_kernel<PQ_SF_LINEAR, kThreads>);
}
