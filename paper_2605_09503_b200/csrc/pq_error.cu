// Calibration quantization error per candidate order and group column (Eq. 3), the quantity
// the candidate selection (Sec. 3.3) and the acceptance rule (Eq. 10) compare.
//
// The original-order kernel leaves fp64 slab sums [slab][group column] in the workspace, the
// candidate kernel fp32 chunk partials [chunk][order][group column]; a second kernel, launched as a
// programmatic dependent, adds them to the fp64 totals in ascending order (for chunk partials:
// each slab's eight in fp64 from zero first).  No floating-point atomics.
//
//   original order (perms == NULL): a thread owns 16 adjacent channels (two 16-byte loads per
//     row) of one chunk, i.e. a whole NVFP4 group or 1/2 .. 1/8 of an integer group; it loads
//     eight rows at a time and walks them in order; a block covers the eight chunks of a slab.  The pass streams the tensor once from HBM;
//     its cost per element is arithmetic (about ten instructions), so it sits between the HBM and
//     the ALU roof.
//   candidate orders: one block per (chunk, order); the chunk's rows are staged in shared memory four
//     at a time, interleaved per channel, and a thread gathers the 16 channels of its run for four rows
//     with 64-bit loads, then runs the original-order kernel's error routine on them; the tensor is
//     fetched from HBM once per chunk and served from L2 to the other orders' blocks.
#include "pq_common.cuh"

namespace {

constexpr int kErrThreads = 256;

// ---------------------------------------------------------------- original order
constexpr int kDirectThreads = 128;
constexpr int kDirectRows = 4;  // rows in flight per thread (2 x 16 bytes each)

// Decode scale d = sf * ts and its reciprocal for each of the 256 scale bytes (they depend on the
// byte only): built once per block, so a group costs one division, one convert and one 8-byte
// shared-memory load instead of a second convert, a multiply and an IEEE reciprocal.
__device__ __forceinline__ void build_scale_table(float2 *table, float ts) {
    for (int b = threadIdx.x; b < 256; b += blockDim.x) {
        const float d = __fmul_rn(pq::e4m3_to_f32(static_cast<uint32_t>(b)), ts);
        table[b] = make_float2(d, d > 0.0f ? __frcp_rn(d) : 0.0f);
    }
}

// Two fp32 lanes in one 64-bit register and the packed IEEE operations on them: one issue slot
// for two results, each rounded exactly like the scalar instruction.
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
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

__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// Error of one row's 16 channels held by this lane; TEAM16 = group / 16 adjacent lanes share a group.
// c6 = 6 * ts (NVFP4 only).  The lane's two 8-channel runs are carried side by side in packed
// registers: per run the operations and their order are those of the scalar definition (scale the
// magnitude by the reciprocal, round to a level, residual by one fused multiply-add, squares added in
// channel order), two results per instruction.  Magnitudes are taken on the bf16 pairs, which is exact.
template <int KIND, int TEAM16>
__device__ __forceinline__ float row_sse16(const uint4 &lo, const uint4 &hi, float c6, const float2 *table, float Qf) {
    const uint32_t m = 0x7FFF7FFFu;
    const uint4 la = make_uint4(lo.x & m, lo.y & m, lo.z & m, lo.w & m);
    const uint4 ha = make_uint4(hi.x & m, hi.y & m, hi.z & m, hi.w & m);
    float xa[8], xb[8];
    pq::unpack8(la, xa);
    pq::unpack8(ha, xb);
    // absmax of the 16 magnitudes on the bf16 pairs (exact: a maximum selects one of its inputs)
    const uint32_t mx = max_bf16x2(max_bf16x2(max_bf16x2(la.x, la.y), max_bf16x2(la.z, la.w)),
                                   max_bf16x2(max_bf16x2(ha.x, ha.y), max_bf16x2(ha.z, ha.w)));
    float amax = fmaxf(__uint_as_float(mx << 16), __uint_as_float(mx & 0xFFFF0000u));
    amax = pq::team_max<TEAM16>(amax);
    float d, r;
    if (KIND == 0) {
        const float2 dr = table[pq::f32_to_e4m3(__fdiv_rn(amax, c6))];
        d = dr.x, r = dr.y;
    } else {
        pq::int_scale(amax, Qf, d, r);
    }
    const uint64_t r2 = pack2(r, r), nd2 = pack2(-d, -d);
    uint64_t x2[8], q2[8];
    if (KIND == 0) {
        float ya[8], yb[8], qa[8], qb[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            x2[i] = pack2(xa[i], xb[i]);
            unpack2(mul2(x2[i], r2), ya[i], yb[i]);
        }
        pq::e2m1_levels(pq::f32x8_to_e2m1(ya), qa);
        pq::e2m1_levels(pq::f32x8_to_e2m1(yb), qb);
#pragma unroll
        for (int i = 0; i < 8; ++i) q2[i] = pack2(qa[i], qb[i]);
    } else {
        // min(rint(y), Q): adding and subtracting 1.5 * 2^23 rounds like rint for y < 2^22, beyond that the clamp decides
        // (the first addition is written as y * 1 + magic: a packed multiply directly followed by a packed
        // add was seen to come out as one fused operation, which rounds once instead of twice)
        const uint64_t magic = pack2(12582912.0f, 12582912.0f), unmagic = pack2(-12582912.0f, -12582912.0f);
        const uint64_t one2 = pack2(1.0f, 1.0f);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            x2[i] = pack2(xa[i], xb[i]);
            float za, zb;
            unpack2(add2(fma2(mul2(x2[i], r2), one2, magic), unmagic), za, zb);
            q2[i] = pack2(fminf(za, Qf), fminf(zb, Qf));
        }
    }
    uint64_t acc2 = pack2(0.0f, 0.0f);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint64_t delta = fma2(q2[i], nd2, x2[i]);
        acc2 = fma2(delta, delta, acc2);
    }
    float sa, sb;
    unpack2(acc2, sa, sb);
    // runs of 8 channels, then the balanced adjacent-pair tree: its first level is this lane's two runs
    return pq::team_sum<TEAM16>(__fadd_rn(sa, sb));
}

constexpr int kSlabChunks = PQ_SLAB_ROWS / PQ_CHUNK_ROWS;  // 8
constexpr int kDirectRuns = kDirectThreads / kSlabChunks;  // 16 runs of 16 channels per block
static_assert(kDirectRuns == 16, "a warp holds two chunks of 16 runs");

// One block = one 128-row slab x 256 channels: thread (c, j) owns chunk c of the slab and the
// j-th 16-channel run, so a warp reads 2 x 512 contiguous bytes per row step.  The eight chunk
// partials of a group meet in shared memory and one thread adds them in fp64 in chunk order;
// the workspace receives fp64 slab sums [slab][K/g].
template <int KIND, int TEAM16>
__global__ void __launch_bounds__(kDirectThreads, 8)
group_error_direct(const uint16_t *__restrict__ T, int64_t rows, int64_t K, int64_t ld,
                   const float *__restrict__ ts_ptr, float Qf, double *__restrict__ slab_part /*[slabs, K/g]*/) {
    __shared__ float part_s[kSlabChunks][kDirectRuns];
    __shared__ float2 scale_table[KIND == 0 ? 256 : 1];
    pq::dependents_may_launch();
    const int runs = static_cast<int>(K >> 4);  // K % (16 * TEAM16) == 0
    const int c = threadIdx.x / kDirectRuns, j = threadIdx.x % kDirectRuns;
    const int run = blockIdx.y * kDirectRuns + j;
    const int64_t slab = blockIdx.x;
    const int64_t r0 = slab * PQ_SLAB_ROWS + c * PQ_CHUNK_ROWS;
    // 16 % TEAM16 == 0 and runs % TEAM16 == 0: a team is live or dead as a whole, and the
    // shuffles below stay inside its 16-lane half of the warp
    const bool live = run < runs && r0 < rows;
    const int n = live ? static_cast<int>(min(static_cast<int64_t>(PQ_CHUNK_ROWS), rows - r0)) : 0;
    const float ts = (KIND == 0) ? __ldg(ts_ptr) : 1.0f;
    const float c6 = __fmul_rn(6.0f, ts);
    if (KIND == 0) {
        build_scale_table(scale_table, ts);
        __syncthreads();
    }
    const uint16_t *p = T + (live ? r0 * ld + static_cast<int64_t>(run) * 16 : 0);
    float acc = 0.0f;
#pragma unroll 1
    for (int t0 = 0; t0 < PQ_CHUNK_ROWS; t0 += kDirectRows) {
        uint4 lo[kDirectRows], hi[kDirectRows];
        const uint4 zero = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int u = 0; u < kDirectRows; ++u) {
            const bool have = t0 + u < n;
            const uint4 *src = reinterpret_cast<const uint4 *>(p + static_cast<int64_t>(t0 + u) * ld);
            lo[u] = have ? __ldg(src) : zero;
            hi[u] = have ? __ldg(src + 1) : zero;
        }
        // rows past the end are all-zero groups: their error is +0.0 and adding it changes nothing
#pragma unroll
        for (int u = 0; u < kDirectRows; ++u) acc = __fadd_rn(acc, row_sse16<KIND, TEAM16>(lo[u], hi[u], c6, scale_table, Qf));
    }
    part_s[c][j] = acc;
    __syncthreads();
    // chunks past the last row hold +0.0, which leaves the slab sum unchanged
    if (threadIdx.x < kDirectRuns && run < runs && (run % TEAM16) == 0) {
        double sum = 0.0;
#pragma unroll
        for (int k = 0; k < kSlabChunks; ++k) sum = __dadd_rn(sum, static_cast<double>(part_s[k][j]));
        slab_part[slab * (runs / TEAM16) + run / TEAM16] = sum;
    }
}

// ---------------------------------------------------------------- candidate orders
// One block per (chunk of 16 rows, candidate order).  The chunk goes through shared memory four rows at a
// time, interleaved per channel (8 bytes per channel: one 64-bit load gathers a channel for four rows, so a
// random order costs a quarter of the shared-memory wavefronts of a row-by-row gather); the 16-byte pieces of
// an octet are XOR-swizzled by bits of the octet index, which makes the transposing stores conflict-free.  A
// thread owns whole 16-channel runs (GPT of them, blockDim apart), keeps their 16 channel positions packed
// in registers for the whole chunk, and for every row rebuilds the two 16-byte words the original-order
// kernel loads, so the error of a run is computed by the same routine, in row order.
constexpr int kMaxGpt = 4;  // 256 threads x 4 runs x 16 channels = 16384 channels

__device__ __forceinline__ int quad_piece(int o, int k) { return 4 * o + (k ^ ((o >> 1) & 3)); }   // 16-byte piece k of octet o
__device__ __forceinline__ uint32_t quad_channel(uint32_t c) { return c ^ (((c >> 4) & 3u) << 1); }  // 8-byte slot of channel c

// one run per thread (up to 4096 channels): held to 64 registers, five 192-thread blocks per SM instead of four
template <int KIND, int TEAM16, int GPT>
__global__ void __launch_bounds__(kErrThreads, GPT == 1 ? 4 : 1)
group_error_gather(const uint16_t *__restrict__ T, int64_t rows, int64_t K, int64_t ld,
                   const float *__restrict__ ts_ptr, float Qf, const int32_t *__restrict__ perms, int P,
                   float *__restrict__ part /*[chunks, P, K/g]*/) {
    extern __shared__ __align__(16) uint16_t quad_s[];  // [K][4 rows]
    __shared__ float2 scale_table[KIND == 0 ? 256 : 1];
    pq::dependents_may_launch();
    const int64_t chunk = blockIdx.x;
    const int p = blockIdx.y;
    const int32_t *perm = perms + static_cast<int64_t>(p) * K;
    const int octs = static_cast<int>(K >> 3), runs = static_cast<int>(K >> 4);
    const int64_t r0 = chunk * PQ_CHUNK_ROWS;
    const float ts = (KIND == 0) ? __ldg(ts_ptr) : 1.0f;
    const float c6 = __fmul_rn(6.0f, ts);
    if (KIND == 0) build_scale_table(scale_table, ts);  // the first barrier below publishes it

    // positions of this thread's channels in the interleaved image, two per register
    uint32_t ch[GPT][8];
    float acc[GPT];
#pragma unroll
    for (int t = 0; t < GPT; ++t) {
        acc[t] = 0.0f;
        const int q = threadIdx.x + t * blockDim.x;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            uint32_t lo = 0, hi = 0;
            if (q < runs) {
                lo = quad_channel(static_cast<uint32_t>(perm[q * 16 + 2 * w]));
                hi = quad_channel(static_cast<uint32_t>(perm[q * 16 + 2 * w + 1]));
            }
            ch[t][w] = lo | (hi << 16);
        }
    }

    uint4 *quad4 = reinterpret_cast<uint4 *>(quad_s);
    const uint2 *quad2 = reinterpret_cast<const uint2 *>(quad_s);
#pragma unroll 1
    for (int quad = 0; quad < PQ_CHUNK_ROWS / 4; ++quad) {
        const int64_t row = r0 + 4 * quad;
        __syncthreads();  // the previous four rows have been used
        for (int o = threadIdx.x; o < octs; o += blockDim.x) {
            uint4 v[4];
#pragma unroll
            for (int r = 0; r < 4; ++r)  // rows past the end are zeros: their error is +0.0 and adding it changes nothing
                v[r] = row + r < rows ? __ldg(reinterpret_cast<const uint4 *>(T + (row + r) * ld) + o) : make_uint4(0, 0, 0, 0);
            const uint32_t *w0 = &v[0].x, *w1 = &v[1].x, *w2 = &v[2].x, *w3 = &v[3].x;
#pragma unroll
            for (int k = 0; k < 4; ++k)
                quad4[quad_piece(o, k)] = make_uint4(__byte_perm(w0[k], w1[k], 0x5410), __byte_perm(w2[k], w3[k], 0x5410),
                                                     __byte_perm(w0[k], w1[k], 0x7632), __byte_perm(w2[k], w3[k], 0x7632));
        }
        __syncthreads();
#pragma unroll
        for (int t = 0; t < GPT; ++t) {
            if (t * static_cast<int>(blockDim.x) >= runs) break;  // uniform over the block
            uint2 g[16];
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                g[2 * w] = quad2[ch[t][w] & 0xFFFFu];
                g[2 * w + 1] = quad2[ch[t][w] >> 16];
            }
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                uint32_t pr[8];
#pragma unroll
                for (int w = 0; w < 8; ++w) {
                    const uint32_t a = r < 2 ? g[2 * w].x : g[2 * w].y, b = r < 2 ? g[2 * w + 1].x : g[2 * w + 1].y;
                    pr[w] = __byte_perm(a, b, (r & 1) ? 0x7632 : 0x5410);
                }
                acc[t] = __fadd_rn(acc[t], row_sse16<KIND, TEAM16>(make_uint4(pr[0], pr[1], pr[2], pr[3]),
                                                                   make_uint4(pr[4], pr[5], pr[6], pr[7]), c6, scale_table, Qf));
            }
        }
    }
    const int64_t Kg = runs / TEAM16;
#pragma unroll
    for (int t = 0; t < GPT; ++t) {
        const int q = threadIdx.x + t * blockDim.x;
        if (q < runs && (q % TEAM16) == 0) part[(chunk * P + p) * Kg + q / TEAM16] = acc[t];
    }
}

template <typename PT, int PER_SLAB>
pq_status fold(const void *part, int64_t count, int64_t n, double *err, cudaStream_t st) {
    PQ_CUDA_OK((pq::launch_fold<PT, PER_SLAB, false>(static_cast<const PT *>(part), nullptr, count, n, err, nullptr, st)));
    return pq_launch_status();
}

template <int KIND, int TEAM>  // TEAM = group / 8
pq_status launch(const uint16_t *T, int64_t rows, int64_t K, int64_t ld, const float *ts, float Qf,
                 const int32_t *perms, int P, void *ws, double *err, cudaStream_t st) {
    const int64_t chunks = pq_ceil_div(rows, PQ_CHUNK_ROWS), slabs = pq_ceil_div(rows, PQ_SLAB_ROWS);
    const int64_t Kg = K / (8 * TEAM);
    if (!perms) {
        dim3 grid(static_cast<unsigned>(slabs), static_cast<unsigned>(pq_ceil_div(K / 16, kDirectRuns)));
        group_error_direct<KIND, TEAM / 2><<<grid, kDirectThreads, 0, st>>>(T, rows, K, ld, ts, Qf, static_cast<double *>(ws));
        if (pq_launch_status() != PQ_OK) return PQ_ERR_CUDA;
        return fold<double, 1>(ws, slabs, Kg, err, st);
    }
    const int runs = static_cast<int>(K >> 4);
    const int threads = runs >= kErrThreads ? kErrThreads : ((runs + 31) / 32) * 32;
    const int gpt = static_cast<int>(pq_ceil_div(runs, threads));
    if (gpt > kMaxGpt) return PQ_ERR_SHAPE;
    const size_t smem = static_cast<size_t>(K) * 8;  // four rows, interleaved per channel
    dim3 grid(static_cast<unsigned>(chunks), static_cast<unsigned>(P));
    auto run = [&](auto kern) -> pq_status {
        if (smem > 40 * 1024)  // the kernel's static shared memory counts towards the 48 KB default limit
            PQ_CUDA_OK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
        kern<<<grid, threads, smem, st>>>(T, rows, K, ld, ts, Qf, perms, P, static_cast<float *>(ws));
        return PQ_OK;
    };
    constexpr int TEAM16 = TEAM / 2;
    const pq_status rl = gpt == 1   ? run(group_error_gather<KIND, TEAM16, 1>)
                         : gpt == 2 ? run(group_error_gather<KIND, TEAM16, 2>)
                                    : run(group_error_gather<KIND, TEAM16, 4>);
    if (rl != PQ_OK) return rl;
    if (pq_launch_status() != PQ_OK) return PQ_ERR_CUDA;
    return fold<float, kSlabChunks>(ws, chunks, static_cast<int64_t>(P) * Kg, err, st);
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
        PQ_REQUIRE(group == 16 || group == 32 || group == 64 || group == 128 || group == 256, PQ_ERR_FORMAT);
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
    const float Qf = fmt.kind == 1 ? static_cast<float>((1 << (fmt.bits - 1)) - 1) : 0.0f;
    if (fmt.kind == 0) return launch<0, 2>(t, rows, K, ld, ts, Qf, perms, P, ws, err, st);
    switch (group) {
        case 16: return launch<1, 2>(t, rows, K, ld, ts, Qf, perms, P, ws, err, st);
        case 32: return launch<1, 4>(t, rows, K, ld, ts, Qf, perms, P, ws, err, st);
        case 64: return launch<1, 8>(t, rows, K, ld, ts, Qf, perms, P, ws, err, st);
        case 128: return launch<1, 16>(t, rows, K, ld, ts, Qf, perms, P, ws, err, st);
        default: return launch<1, 32>(t, rows, K, ld, ts, Qf, perms, P, ws, err, st);   // 256: a whole warp per group
    }
}
