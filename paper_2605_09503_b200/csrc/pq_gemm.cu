// W4A4 NVFP4 block-scaled GEMM (right-hand side of Eq. 8) on the sm_100a tensor cores.
//
//   Y[m,n] = bf16( ts_x*ts_w * sum_k (qx[m,k]*sfx[m,k/16]) * (qw[n,k]*sfw[n,k/16]) )
//
// Design (one CTA per SM, persistent over output tiles of 128 x 192):
//   warp 0      producer: TMA loads of the packed E2M1 operand tiles (128-byte swizzle) and bulk
//               copies of the scale-factor blocks into a 4-stage shared-memory ring;
//   warp 1      issues tcgen05.mma.kind::mxf4nvf4.block_scale (K = 64 per instruction, 4 per stage)
//               into one of two 128 x 192 fp32 accumulators in tensor memory;
//   warps 2..5  epilogue: tcgen05.ld the finished accumulator, scale by ts_x*ts_w, round to bf16,
//               store -- overlapping the next tile's main loop through the second accumulator;
//   warps 6..9  scale-factor stagers: read the stage's scale blocks from shared memory and write
//               them into one of two scale slots in tensor memory with tcgen05.st (one warp per
//               lane quadrant).  Measured on B200: a tcgen05.cp of one 512-byte block costs about
//               80 cycles of the tensor pipe and twelve are needed per stage, more than the stage's
//               four MMAs (384 cycles); the register path costs the pipe nothing.
// K is consumed 256 channels (128 bytes of codes per row) per stage.  192 divides every FLUX
// output width (3072, 9216, 12288) and leaves room in the 512 tensor-memory columns for two
// accumulators plus the scale factors.
//
// Scale factors live in global memory in 512-byte blocks of 128 rows x 4 groups (see pq.h); a
// block occupies 4 tensor-memory columns (row r of the block -> lane r%32, column r/32, the same
// in all four lane quadrants), which is the layout the MMA reads: lane l of every stager warp
// loads the 16 bytes at offset 16 l of the block and stores them as 4 columns of its quadrant.  A 192-wide tile that starts in the middle of a 128-row block (n0 % 128 == 64) loads
// the two blocks it touches and offsets the B scale address by two columns.
//
// Every wait on an mbarrier is bounded.  If one expires the CTA records PQ_ERR_TIMEOUT in the
// status word, raises a shared abort flag that every role polls, drains its outstanding loads
// (bounded), frees its tensor memory and returns.
#include <cuda.h>

#include "pq_common.cuh"

namespace {

constexpr int BM = 128, BN = 192, BK = 256;
constexpr int kStages = 4;
constexpr int kABytes = BM * BK / 2;       // 16384
constexpr int kBBytes = BN * BK / 2;       // 24576
constexpr int kSfBlock = 512;              // 128 rows x 4 groups
constexpr int kSfaBytes = 4 * kSfBlock;    // 4 K-blocks of one 128-row block
constexpr int kSfbBytes = 2 * kSfaBytes;   // two 128-row blocks
constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;  // 47104 = 46 * 1024
constexpr int kThreads = 320;
constexpr int kTmemCols = 512;
constexpr uint32_t kAccStride = 256;  // accumulator b starts at column b * 256
// two scale slots in the columns the accumulators leave free: 16 columns of A scales, 32 of B scales
__device__ __forceinline__ uint32_t sf_slot_col(uint32_t t) { return t ? 448u : 192u; }
constexpr uint32_t kSfbOfs = 16;
constexpr long long kWaitCycles = 4000000000ll;  // about two seconds of SM clock per wait
constexpr size_t kSmemBytes = kStages * kStageBytes + 1024 /*alignment slack*/ + 256 /*barriers*/;
constexpr int kNumBars = 2 * kStages + 6;  // full[S] empty[S] acc_full[2] acc_empty[2] sf_full[2]

struct GemmParams {
    const uint8_t *sfx, *sfw;
    const float *ts_x, *ts_w;
    uint16_t *Y;
    int64_t ldy;
    int M, N, K;
    int m_tiles, n_tiles, k_tiles, kb_total, kb4;
    int n_rowblocks;
    int *status;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: polls until the phase completes, the abort flag goes up, or kWaitCycles SM
// clock cycles have passed (then it raises the flag and records the timeout).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, int *status) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    for (uint32_t spins = 1;; ++spins) {
        if (mbar_try(bar, parity)) return true;
        if ((spins & 63u) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > kWaitCycles) break;
        }
    }
    *abort_flag = 1;
    atomicExch(status, static_cast<int>(PQ_ERR_TIMEOUT));
    return false;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_st4(uint32_t taddr, const uint4 &v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};" ::"r"(taddr), "r"(v.x), "r"(v.y),
                 "r"(v.z), "r"(v.w)
                 : "memory");
}
__device__ __forceinline__ void tc_st8(uint32_t taddr, const uint4 &a, const uint4 &b) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr),
                 "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w)
                 : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t sfa,
                                       uint32_t sfb, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
        : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand tile with 128-byte swizzle: rows of
// 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t operand_desc(uint32_t smem_addr) {
    return static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) |
           (2ull << 61);
}
// Instruction descriptor: E2M1 x E2M1, UE4M3 scales, both K-major, M = 128, N = BN, K = 64.
constexpr uint32_t kIdesc = (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) | (0u << 23) |
                            (static_cast<uint32_t>(BM >> 4) << 24);

// ---------------------------------------------------------------- kernel
__global__ void __launch_bounds__(kThreads, 1)
gemm_w4a4_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *base_ptr = smem_raw + (base - raw);
    const uint32_t bars = base + kStages * kStageBytes;
    uint8_t *bars_ptr = base_ptr + kStages * kStageBytes;
    // barrier block: full[S] | empty[S] | acc_full[2] | acc_empty[2] | sf_full[2] | tmem base | abort flag
    auto full_bar = [&](int s) { return bars + 8u * s; };
    auto empty_bar = [&](int s) { return bars + 8u * (kStages + s); };
    auto acc_full_bar = [&](int b) { return bars + 8u * (2 * kStages + b); };
    auto acc_empty_bar = [&](int b) { return bars + 8u * (2 * kStages + 2 + b); };
    auto sf_full_bar = [&](int t) { return bars + 8u * (2 * kStages + 4 + t); };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars_ptr + 8 * kNumBars);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars_ptr + 8 * kNumBars + 8);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar(s), 1);
            mbar_init(empty_bar(s), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(acc_full_bar(b), 1);
            mbar_init(acc_empty_bar(b), 4);
            mbar_init(sf_full_bar(b), 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int total_tiles = p.m_tiles * p.n_tiles;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                const int m_blk = tile % p.m_tiles, n_blk = tile / p.m_tiles;
                const int m0 = m_blk * BM, n0 = n_blk * BN;
                const int nb0 = n0 >> 7;
                const int rb0 = min(nb0, p.n_rowblocks - 1), rb1 = min(nb0 + 1, p.n_rowblocks - 1);
                for (int kt = 0; kt < p.k_tiles; ++kt, ++it) {
                    const int s = it % kStages;
                    const uint32_t par = (it / kStages) & 1u;
                    if (!mbar_wait(empty_bar(s), par ^ 1u, abort_flag, p.status)) {
                        ok = false;
                        break;
                    }

                    const int kb_valid = min(4, p.kb_total - kt * 4);
                    const uint32_t sf_bytes = static_cast<uint32_t>(kb_valid) * kSfBlock;
                    const uint32_t stage = base + s * kStageBytes;
                    mbar_expect_tx(full_bar(s), kABytes + kBBytes + 3u * sf_bytes);
                    tma_load_2d(stage, &map_a, kt * (BK / 2), m0, full_bar(s));
                    tma_load_2d(stage + kABytes, &map_b, kt * (BK / 2), n0, full_bar(s));
                    const int64_t kofs = static_cast<int64_t>(kt) * 4 * kSfBlock;
                    bulk_load(stage + kABytes + kBBytes,
                              p.sfx + static_cast<int64_t>(m_blk) * p.kb4 * kSfBlock + kofs, sf_bytes, full_bar(s));
                    bulk_load(stage + kABytes + kBBytes + kSfaBytes,
                              p.sfw + static_cast<int64_t>(rb0) * p.kb4 * kSfBlock + kofs, sf_bytes, full_bar(s));
                    bulk_load(stage + kABytes + kBBytes + kSfaBytes + kSfaBytes,
                              p.sfw + static_cast<int64_t>(rb1) * p.kb4 * kSfBlock + kofs, sf_bytes, full_bar(s));
                }
            }
            if (!ok) {
                // drain: give every load already issued a bounded chance to land before leaving
                const uint32_t issued = it;
                const uint32_t first = issued > kStages ? issued - kStages : 0;
                for (uint32_t j = first; j < issued; ++j)
                    for (uint32_t i = 0; i < 4096 && !mbar_try(full_bar(j % kStages), (j / kStages) & 1u); ++i) {}
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        // The whole warp walks the loop (uniform control flow, so descriptors live in uniform
        // registers); lane 0 issues the tensor-core instructions.
        uint32_t it = 0, tcount = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tcount) {
            const int n_blk = tile / p.m_tiles;
            const uint32_t sfb_shift = ((n_blk * BN) & 127) ? 2u : 0u;
            const uint32_t b = tcount & 1u, accpar = (tcount >> 1) & 1u;
            if (!mbar_wait(acc_empty_bar(b), accpar ^ 1u, abort_flag, p.status)) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + b * kAccStride;
            for (int kt = 0; kt < p.k_tiles; ++kt, ++it) {
                const int s = it % kStages;
                const uint32_t par = (it / kStages) & 1u;
                const uint32_t t = it & 1u;
                if (!mbar_wait(full_bar(s), par, abort_flag, p.status) ||
                    !mbar_wait(sf_full_bar(t), (it >> 1) & 1u, abort_flag, p.status)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const int kb_valid = min(4, p.kb_total - kt * 4);
                const uint32_t stage = base + s * kStageBytes;
                const uint64_t da = operand_desc(stage), db = operand_desc(stage + kABytes);
                const uint32_t sfa_t = tmem_base + sf_slot_col(t), sfb_t = sfa_t + kSfbOfs + sfb_shift;
                if (lane == 0) {
                    if (kb_valid == 4) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            tc_mma(d_tmem, da + 2 * kk, db + 2 * kk, kIdesc, sfa_t + 4 * kk, sfb_t + 8 * kk,
                                   (kt | kk) ? 1u : 0u);
                    } else {
                        for (int kk = 0; kk < kb_valid; ++kk)
                            tc_mma(d_tmem, da + 2 * kk, db + 2 * kk, kIdesc, sfa_t + 4 * kk, sfb_t + 8 * kk,
                                   (kt | kk) ? 1u : 0u);
                    }
                    tc_commit(empty_bar(s));
                }
                __syncwarp();
            }
            if (ok && lane == 0) tc_commit(acc_full_bar(b));
            __syncwarp();
        }
    } else if (warp >= 6) {
        // ------------------------------------------------------------ scale-factor stagers
        const uint32_t q = warp & 3;  // tensor-memory lane quadrant this warp may write
        const uint32_t lane_ofs = (q * 32u) << 16;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
            for (int kt = 0; kt < p.k_tiles; ++kt, ++it) {
                const int s = it % kStages;
                const uint32_t t = it & 1u;
                // the stage's scale blocks have landed, and the MMAs that read this slot two
                // iterations ago have completed (their commit released that iteration's stage)
                if (!mbar_wait(full_bar(s), (it / kStages) & 1u, abort_flag, p.status) ||
                    (it >= 2 && !mbar_wait(empty_bar((it - 2) % kStages), ((it - 2) / kStages) & 1u, abort_flag,
                                           p.status))) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                const int kb_valid = min(4, p.kb_total - kt * 4);
                const uint32_t sf_s = base + s * kStageBytes + kABytes + kBBytes + lane * 16u;
                const uint32_t sf_t = tmem_base + lane_ofs + sf_slot_col(t);
                for (int kk = 0; kk < kb_valid; ++kk) {
                    const uint4 a = lds128(sf_s + kk * kSfBlock);
                    const uint4 b0 = lds128(sf_s + kSfaBytes + kk * kSfBlock);
                    const uint4 b1 = lds128(sf_s + 2 * kSfaBytes + kk * kSfBlock);
                    tc_st4(sf_t + 4 * kk, a);
                    tc_st8(sf_t + kSfbOfs + 8 * kk, b0, b1);
                }
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(sf_full_bar(t));
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        const int q = warp & 3;  // tensor-memory lane quadrant this warp may read
        const float alpha = __fmul_rn(__ldg(p.ts_x), __ldg(p.ts_w));
        uint32_t tcount = 0;
        for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++tcount) {
            const int m_blk = tile % p.m_tiles, n_blk = tile / p.m_tiles;
            const int m0 = m_blk * BM, n0 = n_blk * BN;
            const uint32_t b = tcount & 1u, accpar = (tcount >> 1) & 1u;
            const bool got = mbar_wait(acc_full_bar(b), accpar, abort_flag, p.status);
            if (!__all_sync(0xFFFFFFFFu, got)) break;
            tc_fence_after();

            const int row = m0 + q * 32 + lane;
            uint16_t *yrow = p.Y + static_cast<int64_t>(row) * p.ldy;
#pragma unroll 1
            for (int c = 0; c < BN / 32; ++c) {
                uint32_t v[32];
                tc_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + b * kAccStride + c * 32, v);
                tc_wait_ld();
                const int col0 = n0 + c * 32;
                if (row < p.M) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (col0 + j * 8 + 8 <= p.N) {
                            uint32_t w[4];
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const float lo = __fmul_rn(__uint_as_float(v[j * 8 + 2 * i]), alpha);
                                const float hi = __fmul_rn(__uint_as_float(v[j * 8 + 2 * i + 1]), alpha);
                                w[i] = static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(lo))) |
                                       (static_cast<uint32_t>(__bfloat16_as_ushort(__float2bfloat16_rn(hi))) << 16);
                            }
                            *reinterpret_cast<uint4 *>(yrow + col0 + j * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acc_empty_bar(b));
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();

    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// Packed E2M1 codes [rows, K/2] bytes, row-major: a byte tensor with 128-byte-swizzled boxes
// of 128 bytes (256 channels) x box_rows rows.  Out-of-range rows / columns read as zero.
struct MapKey {
    const uint8_t *ptr;
    int64_t rows, K;
    int box_rows;
};
struct MapSlot {
    MapKey key;
    CUtensorMap map;
    bool used;
};
// Encoding a tensor map costs several microseconds of host time; a layer calls the GEMM with
// the same operand buffers over and over, so the last few encodings are kept.
bool make_codes_map(CUtensorMap *map, const uint8_t *ptr, int64_t rows, int64_t K, int box_rows) {
    static thread_local MapSlot cache[8];
    static thread_local int next = 0;
    for (MapSlot &c : cache)
        if (c.used && c.key.ptr == ptr && c.key.rows == rows && c.key.K == K && c.key.box_rows == box_rows) {
            *map = c.map;
            return true;
        }
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(K / 2), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(K / 2)};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(BK / 2), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    if (enc(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t *>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    MapSlot &slot = cache[next];
    next = (next + 1) % 8;
    slot.key = MapKey{ptr, rows, K, box_rows};
    slot.map = *map;
    slot.used = true;
    return true;
}

}  // namespace

extern "C" pq_status pq_gemm_w4a4(const uint8_t *xq, const uint8_t *sfx, const float *ts_x, const uint8_t *wq,
                                  const uint8_t *sfw, const float *ts_w, int64_t M, int64_t N, int64_t K, void *Y,
                                  int64_t ldy, void *ws, size_t ws_bytes, void *stream) {
    PQ_REQUIRE(xq && sfx && ts_x && wq && sfw && ts_w && Y, PQ_ERR_NULL);
    PQ_REQUIRE(M > 0 && N > 0 && K >= 64 && K % 64 == 0 && N % 8 == 0 && ldy >= N, PQ_ERR_SHAPE);
    PQ_REQUIRE(M < (1ll << 31) - 256 && N < (1ll << 31) - 256 && K < (1ll << 31), PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(xq) && pq_aligned16(sfx) && pq_aligned16(wq) && pq_aligned16(sfw) && pq_aligned16(Y) &&
                   ldy % 8 == 0,
               PQ_ERR_ALIGN);
    PQ_REQUIRE(ws && ws_bytes >= pq_workspace_bytes(PQ_OP_GEMM, M, K, N, 0), PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    CUtensorMap map_a, map_b;
    if (!make_codes_map(&map_a, xq, M, K, BM) || !make_codes_map(&map_b, wq, N, K, BN)) return PQ_ERR_CUDA;

    static bool attr_set = false;
    if (!attr_set) {
        PQ_CUDA_OK(cudaFuncSetAttribute(gemm_w4a4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(kSmemBytes)));
        attr_set = true;
    }
    static int sms = 0;
    if (sms == 0) {
        int dev = 0;
        PQ_CUDA_OK(cudaGetDevice(&dev));
        PQ_CUDA_OK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    }

    GemmParams p;
    p.sfx = sfx, p.sfw = sfw, p.ts_x = ts_x, p.ts_w = ts_w;
    p.Y = static_cast<uint16_t *>(Y);
    p.ldy = ldy;
    p.M = static_cast<int>(M), p.N = static_cast<int>(N), p.K = static_cast<int>(K);
    p.m_tiles = static_cast<int>(pq_ceil_div(M, BM));
    p.n_tiles = static_cast<int>(pq_ceil_div(N, BN));
    p.k_tiles = static_cast<int>(pq_ceil_div(K, BK));
    p.kb_total = static_cast<int>(K / 64);
    p.kb4 = p.kb_total;
    p.n_rowblocks = static_cast<int>(pq_ceil_div(N, 128));
    p.status = static_cast<int *>(ws);
    const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
    const int grid = static_cast<int>(tiles < sms ? tiles : sms);
    gemm_w4a4_kernel<<<grid, kThreads, kSmemBytes, st>>>(map_a, map_b, p);
    return pq_launch_status();
}

extern "C" pq_status pq_linear_w4a4(const void *X, int64_t M, int64_t K, int64_t ld, const float *ts_x, uint8_t *xq,
                                    uint8_t *sfx, const uint8_t *wq, const uint8_t *sfw, const float *ts_w, int64_t N,
                                    void *Y, int64_t ldy, void *ws, size_t ws_bytes, void *stream) {
    const pq_status rc = pq_quant_act_nvfp4(X, M, K, ld, ts_x, xq, sfx, PQ_SF_TCGEN05, stream);
    if (rc != PQ_OK) return rc;
    return pq_gemm_w4a4(xq, sfx, ts_x, wq, sfw, ts_w, M, N, K, Y, ldy, ws, ws_bytes, stream);
}

extern "C" pq_status pq_linear_w4a4_host(const void *X_host, int64_t M, int64_t K, const float *ts_x, void *X_dev,
                                         uint8_t *xq, uint8_t *sfx, const uint8_t *wq, const uint8_t *sfw,
                                         const float *ts_w, int64_t N, void *Y_dev, void *Y_host, void *ws,
                                         size_t ws_bytes, void *stream) {
    PQ_REQUIRE(X_host && X_dev && Y_dev && Y_host, PQ_ERR_NULL);
    PQ_REQUIRE(M > 0 && K > 0 && N > 0, PQ_ERR_SHAPE);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PQ_CUDA_OK(cudaMemcpyAsync(X_dev, X_host, static_cast<size_t>(M) * K * 2, cudaMemcpyHostToDevice, st));
    const pq_status rc = pq_linear_w4a4(X_dev, M, K, K, ts_x, xq, sfx, wq, sfw, ts_w, N, Y_dev, N, ws, ws_bytes, stream);
    if (rc != PQ_OK) return rc;
    PQ_CUDA_OK(cudaMemcpyAsync(Y_host, Y_dev, static_cast<size_t>(M) * N * 2, cudaMemcpyDeviceToHost, st));
    return PQ_OK;
}

extern "C" pq_status pq_device_status(const void *ws, void *stream) {
    PQ_REQUIRE(ws, PQ_ERR_NULL);
    int word = 0;
    if (cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) {
        (void)cudaGetLastError();
        return PQ_ERR_CUDA;
    }
    PQ_CUDA_OK(cudaMemcpy(&word, ws, sizeof(int), cudaMemcpyDeviceToHost));
    return word == 0 ? PQ_OK : static_cast<pq_status>(word);
}
