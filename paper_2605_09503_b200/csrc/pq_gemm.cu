// W4A4 NVFP4 block-scaled GEMM (right-hand side of Eq. 8) on the sm_100a tensor cores.
//
//   Y[m,n] = bf16( ts_x*ts_w * sum_k (qx[m,k]*sfx[m,k/16]) * (qw[n,k]*sfw[n,k/16]) )
//
// Design.  Thread-block clusters of two CTAs (one per SM) work as a pair on output tiles of
// 256 x 256, persistent over the tile list: tcgen05.mma.cta_group::2 lets each CTA hold 128 rows
// of the accumulator while the B operand is split between the two shared memories, so a CTA
// fetches 128 rows of X codes and 128 rows of W codes per 256-channel K step (38 KB with the
// scales, for 512 cycles of MMA).  What bounds the main loop is the rate at which the SMs can take
// operands in from L2 (about 70 bytes per clock each when all of them pull), so the tile is as
// large as tensor memory allows.  Roles of the 18 warps of a CTA:
//   warp 0       producer: TMA loads of the packed E2M1 operand tiles (128-byte swizzle) and bulk
//                copies of the scale-factor blocks into a 5-stage shared-memory ring.  Operand
//                loads of both CTAs signal the pair leader's barrier (cp.async.bulk.tensor with
//                .cta_group::2).
//   warp 1       (leader CTA) issues tcgen05.mma.kind::mxf4nvf4.block_scale, K = 64 per instruction,
//                4 per stage, into the 256-column fp32 accumulator in tensor memory.
//   warps 2..9   epilogue (lane quadrant x column half): tcgen05.ld the finished accumulator (own
//                CTA's 128 rows) 16 columns at a time, scale by ts_x*ts_w, round to bf16 and keep the
//                32 x 128 piece as 64 packed registers; hand the accumulator back; then stage 32 x 64
//                boxes in swizzled shared memory and write them with TMA stores (full 128-byte
//                lines) while the next tile's main loop runs.
//   warps 10..17 scale-factor stagers: read the stage's scale blocks from shared memory and write
//                them into one of two scale slots in tensor memory with tcgen05.st (one warp per
//                lane quadrant; two sets of four warps take alternate K iterations).
// 256 divides every FLUX output width (3072, 9216, 12288).  The 512 tensor-memory columns hold one
// 256-column accumulator plus two scale slots (2 x 48); the epilogue warps pull the accumulator
// into registers as packed bf16 within a few hundred cycles and store it from there.
//
// Measurements on B200 behind these choices:
//   - a tcgen05.cp of one 512-byte scale block occupies the tensor pipe for about 80 cycles and
//     twelve are needed per stage, more than the stage's four MMAs (384 cycles); the register path
//     (ld.shared + tcgen05.st, 7 to 16 cycles per store) costs the pipe nothing;
//   - TMA and tcgen05 instructions take their operands from uniform registers.  Issued from a
//     divergent single-lane loop (`if (lane == 0) for (...)`) every operand is moved there one by
//     one and an MMA costs about 190 cycles of issue time instead of 96; the producer and the MMA
//     issuer therefore run their loops with the whole warp and single out one lane with
//     elect.sync only around those instructions;
//   - a remote mbarrier arrive with cluster-scope release semantics costs 500 to 2500 cycles;
//     what the arrivals here publish has already completed (tcgen05.wait) when they are issued,
//     so the default semantics are used.
//
// Scale factors live in global memory in 512-byte blocks of 128 rows x 4 groups (see pq.h); a
// block occupies 4 tensor-memory columns (row r of the block -> lane r%32, column r/32, the same
// in all four lane quadrants), which is the layout the MMA reads: lane l of every stager warp
// loads the 16 bytes at offset 16 l of the block and stores them as columns of its quadrant.
// The 256 B-scale rows of a tile are two whole blocks: 8 columns per K block.
//
// Cross-CTA signalling uses plain remote mbarrier arrives and, for the completion of a stage's
// MMAs and of a tile's accumulator, one tcgen05.commit per CTA (issued by the pair leader's MMA
// warp onto each CTA's own copy of the barrier).  Every wait on an mbarrier is bounded.  If one
// expires the CTA records PQ_ERR_TIMEOUT in the status word, raises a shared abort flag that every role polls,
// and falls through to the common teardown (cluster barrier, tensor-memory release).
#include <cuda.h>

#include <mutex>

#include "pq_common.cuh"

namespace {

constexpr int BM = 256, BM_CTA = 128, BK = 256;
constexpr int kABytes = BM_CTA * BK / 2;   // 16384
constexpr int kSfBlock = 512;              // 128 rows x 4 groups
constexpr int kSfaBytes = 4 * kSfBlock;    // 4 K-blocks of one 128-row block
constexpr int kTmemCols = 512;
constexpr long long kWaitCycles = 4000000000ll;  // default limit of a wait: about two seconds of SM clock

constexpr int BN = 256, BN_CTA = BN / 2;
constexpr int kStages = 5;
constexpr int kBBytes = BN_CTA * BK / 2;   // 16384
constexpr int kSfbBytes = 2 * kSfaBytes;   // the two 128-row blocks of the tile's 256 B rows
constexpr int kStageBytes = kABytes + kBBytes + kSfaBytes + kSfbBytes;  // 38912 = 38 * 1024
constexpr int kEpiWarps = 8;               // lane quadrant x column half of the accumulator
constexpr int kBoxCols = 64;               // output staging box: 32 rows x 64 bf16, one TMA store
constexpr int kEpiBox = 32 * kBoxCols * 2;
constexpr int kEpiBytes = kEpiWarps * kEpiBox;      // one staging box per epilogue warp: 32 KB
constexpr int kStagerSets = 2;             // sets of four stager warps taking alternate K iterations
constexpr int kFirstStager = 2 + kEpiWarps;
constexpr int kThreads = 32 * (kFirstStager + 4 * kStagerSets);   // producer, MMA issuer, 8 epilogue and 8 stager warps
// One 256-column accumulator, then the scale slots.  A slot holds the scales of one stage: per 64-channel
// K block 4 columns of A scales (128 rows) and 8 columns of B scales (256 rows).  Slot it % kSfSlots
// serves iteration it; it is rewritten only after the MMAs of iteration it - kSfSlots have completed
// (their commit releases that iteration's stage).
//
// Why the slot count is tied to the stage count.  Every wait here is a PARITY wait: it tells "phase n
// of this barrier has completed" from "it has not" only if the barrier cannot still be in phase n - 1,
// i.e. only if the waiter already knows that phase n - 1 has completed.  A role that waits on every
// phase of a barrier in turn (producer on stage_free, MMA issuer on stage_full and acc_empty, each
// epilogue warp on acc_full) knows it from its own previous wait.  The stagers do not: the stage
// count is odd and the two stager sets take alternate iterations, so the previous phase of
// sf_ready(s), iteration it - kStages, was waited for by the OTHER set.  What a set knows when it
// reaches iteration `it` is what its own iteration it - kStagerSets waited for: the MMAs of
// it - kStagerSets - kSfSlots have completed.  Those of it - kStages (hence that iteration's scale
// copies, which its stagers had to see before its MMAs could be issued) are then known complete only if
//     it - kStagerSets - kSfSlots >= it - kStages,   i.e.  kSfSlots + kStagerSets <= kStages.
// With 4 slots, 2 sets and 5 stages the condition fails: when the scale copies of it - kStages were
// still in flight the wait for phase n returned true one phase early, the warp read the previous
// occupant's scale bytes from shared memory and stored them to tensor memory -- one lane quadrant of
// one CTA, all columns, wrong by the ratio of two scale factors -- about once in 450 launches of the
// 4608 x 3072 x 9216 product.  2 and 3 slots, and 4 slots with the stagers held to three stages
// ahead, satisfy the condition and never failed.  The stagers also wait for the release of iteration
// it - kStages (stage_free, which the producer waited for before it refilled the stage) in front of
// the sf_ready wait, so that wait is sound whatever the slot count; the assertions keep the original
// condition as well.
constexpr int kSfSlots = 2;
constexpr uint32_t kSfSlotCol0 = BN, kSfbColsPerKb = 8, kSfbOfs = 16;
constexpr uint32_t kSfSlotCols = 4 * (4 + kSfbColsPerKb);   // 48
static_assert(kSfSlotCol0 + kSfSlots * kSfSlotCols <= 512, "tensor memory columns");
static_assert(kSfSlots + kStagerSets <= kStages, "a stager set must know that the previous phase of sf_ready has completed");
static_assert(kSfSlots <= 2 * kStages - 2, "the stagers' parity waits on stage_free must be unambiguous");
// barriers: stage_full[S] sf_ready[S] stage_free[S] acc_full acc_empty
constexpr int kNumBars = 3 * kStages + 2;
constexpr size_t kSmemBytes = kStages * kStageBytes + kEpiBytes + 1024 /*alignment slack*/ + 8 * kNumBars + 64;
static_assert(kSmemBytes <= 227 * 1024, "shared memory per CTA");

struct GemmParams {
    const uint8_t *sfx, *sfw;
    const float *ts_x, *ts_w;
    int M, N, K;
    int m_tiles, n_tiles, k_tiles, kb_total, kb4;
    int m_rowblocks, n_rowblocks;
    long long wait_cycles;  // limit of every mbarrier wait, in SM clock cycles
    int *status;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// Address of the same shared-memory location in CTA `rank` of the cluster.
__device__ __forceinline__ uint32_t mapa(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
// One lane of a converged warp; the branch on it stays friendly to uniform registers.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred = 0;
    asm volatile(
        "{\n"
        ".reg .b32 rx;\n"
        ".reg .pred px;\n"
        "elect.sync rx|px, %1;\n"
        "@px mov.s32 %0, 1;\n"
        "}\n"
        : "+r"(pred)
        : "r"(0xFFFFFFFFu));
    return pred != 0;
}
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
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
// Arrive on the copy of a barrier in CTA `rank` of the pair.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar, uint32_t rank) {
    asm volatile(
        "{\n"
        ".reg .b32 remote;\n"
        "mapa.shared::cluster.u32 remote, %0, %1;\n"
        "mbarrier.arrive.shared::cluster.b64 _, [remote];\n"
        "}\n" ::"r"(bar), "r"(rank)
        : "memory");
}
// Arrive on the pair leader's copy of a barrier.
__device__ __forceinline__ void mbar_arrive_leader(uint32_t bar, uint32_t rank) {
    if (rank == 0) mbar_arrive(bar);
    else mbar_arrive_remote(bar, 0);
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
// Bounded wait: polls until the phase completes, the abort flag goes up, or `limit` SM clock cycles
// have passed (then it raises the flag and records the timeout).
struct WaitCtx {
    volatile int *abort_flag;
    int *status;
    long long limit;
};
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const WaitCtx w) {
    const long long t0 = clock64();
    for (uint32_t spins = 1;; ++spins) {
        if (mbar_try(bar, parity)) return true;
        if ((spins & 63u) == 0) {
            if (*w.abort_flag) return false;
            if (clock64() - t0 > w.limit) break;
        }
    }
    *w.abort_flag = 1;
    atomicExch(w.status, static_cast<int>(PQ_ERR_TIMEOUT));
    return false;
}
// Wait of a single thread (or of lanes that vote on the result themselves).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtx w) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, w);
}
// Wait of a converged warp: every lane returns the same answer and the warp is converged again
// afterwards, so .sync.aligned instructions (elect, tcgen05.st / ld) may follow on either outcome.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, const WaitCtx w) {
    bool ok = mbar_try(bar, parity);
    if (__all_sync(0xFFFFFFFFu, ok)) return true;
    ok = ok || mbar_wait_slow(bar, parity, w);
    return __all_sync(0xFFFFFFFFu, ok);
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
// Operand tile load of a CTA pair: data lands in this CTA's shared memory, the byte count is
// credited to the barrier at `bar_cluster` (the pair leader's).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *map, int x, int y,
                                                 uint32_t bar_cluster) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar_cluster)
        : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void tma_store_2d(const CUtensorMap *map, int x, int y, uint32_t src) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                 ::"l"(map), "r"(x), "r"(y), "r"(src)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Arrive on `bar` (cluster-window address: this CTA's or the peer's) once every tcgen05 operation
// issued so far by this thread has completed in both CTAs of the pair.
__device__ __forceinline__ void tc_commit_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_pair(uint32_t d_tmem, uint64_t da, uint64_t db, uint32_t idesc, uint32_t sfa,
                                            uint32_t sfb, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::mxf4nvf4.block_scale.block16 [%0], %1, %2, %3, [%5], [%6], p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(sfa), "r"(sfb)
        : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
// The registers of a tcgen05.ld hold its result only after tcgen05.wait::ld.  The wait names them as
// in/out operands: whatever reads them afterwards then depends on the wait and cannot be scheduled in
// front of it (arithmetic on the loaded values has no other tie to the wait instruction; without it a
// tile was occasionally packed from registers the load had not written yet).
__device__ __forceinline__ void tc_wait_ld(uint32_t (&v)[16]) {
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(v[0]), "+r"(v[1]), "+r"(v[2]), "+r"(v[3]), "+r"(v[4]), "+r"(v[5]), "+r"(v[6]), "+r"(v[7]),
                   "+r"(v[8]), "+r"(v[9]), "+r"(v[10]), "+r"(v[11]), "+r"(v[12]), "+r"(v[13]), "+r"(v[14]), "+r"(v[15])
                 :
                 : "memory");
}
__device__ __forceinline__ void tc_st4(uint32_t taddr, const uint4 &v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};" ::"r"(taddr), "r"(v.x), "r"(v.y),
                 "r"(v.z), "r"(v.w)
                 : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// Shared-memory matrix descriptor of a K-major operand tile with 128-byte swizzle: rows of
// 128 bytes, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t operand_desc(uint32_t smem_addr) {
    return static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) |
           (2ull << 61);
}
// Instruction descriptor: E2M1 x E2M1, UE4M3 scales, both K-major, M = 256 (pair), N = BN, K = 64.
constexpr uint32_t kIdesc = (1u << 7) | (1u << 10) | (static_cast<uint32_t>(BN >> 3) << 17) | (0u << 23) |
                            (static_cast<uint32_t>(BM >> 4) << 24);


// Two accumulator values times alpha, each rounded to bf16 (nearest even), packed low | high.
#ifndef PQ_GEMM_EPI_PACKED
#define PQ_GEMM_EPI_PACKED 1
#endif
__device__ __forceinline__ uint32_t pack_bf16(uint32_t lo_bits, uint32_t hi_bits, float alpha) {
    uint32_t r;
#if PQ_GEMM_EPI_PACKED
    // one packed multiply (two IEEE products per issue slot), then the two-way convert
    asm("{\n"
        ".reg .b64 v, a;\n"
        ".reg .f32 lo, hi;\n"
        "mov.b64 v, {%1, %2};\n"
        "mov.b64 a, {%3, %3};\n"
        "mul.rn.f32x2 v, v, a;\n"
        "mov.b64 {lo, hi}, v;\n"
        "cvt.rn.bf16x2.f32 %0, hi, lo;\n"
        "}\n"
        : "=r"(r)
        : "r"(lo_bits), "r"(hi_bits), "f"(alpha));
#else
    const float lo = __fmul_rn(__uint_as_float(lo_bits), alpha);
    const float hi = __fmul_rn(__uint_as_float(hi_bits), alpha);
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
#endif
    return r;
}

// ---------------------------------------------------------------- kernel
// Register budget: the register file is split over the four SM sub-partitions (16384 registers
// each) and two of them receive five of this CTA's 18 warps: 5 x 32 x 96 = 15360 fits, 104 would not.
// The 1024 registers left there take one warp of a 32-register kernel, so 128-thread blocks of
// other kernels can still run on the SM beside the GEMM.
constexpr int kMaxRegs = 96;
__global__ void __cluster_dims__(2, 1, 1) __maxnreg__(kMaxRegs)
gemm_w4a4_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_y, const GemmParams p) {
    constexpr int kNB = BN / 128;  // 128-row scale blocks of B per tile
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;  // identical in both CTAs of the pair
    uint8_t *base_ptr = smem_raw + (base - raw);
    const uint32_t epi = base + kStages * kStageBytes;
    const uint32_t bars = epi + kEpiBytes;
    uint8_t *bars_ptr = base_ptr + kStages * kStageBytes + kEpiBytes;
    // stage_full: operand bytes of both CTAs have landed (1 arrival + transaction bytes) and the
    // stage's scales are in tensor memory in both CTAs (8 stager-warp arrivals); leader's copy only
    auto stage_full_bar = [&](int s) { return bars + 8u * s; };
    auto sf_ready_bar = [&](int s) { return bars + 8u * (kStages + s); };     // scale blocks landed (own CTA)
    auto stage_free_bar = [&](int s) { return bars + 8u * (2 * kStages + s); };  // the stage's MMAs have run
    const uint32_t acc_full_bar = bars + 8u * (3 * kStages);       // one copy per CTA, both signalled by the issuer
    const uint32_t acc_empty_bar = bars + 8u * (3 * kStages + 1);  // leader's copy only
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars_ptr + 8 * kNumBars);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars_ptr + 8 * kNumBars + 8);
    const WaitCtx wctx{abort_flag, p.status, p.wait_cycles};
    auto sf_slot_col = [](uint32_t t) { return kSfSlotCol0 + t * kSfSlotCols; };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();  // 0 = pair leader
    const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(stage_full_bar(s), 9);  // producer + 4 stager warps in each CTA
            mbar_init(sf_ready_bar(s), 1);
            mbar_init(stage_free_bar(s), 1);
        }
        mbar_init(acc_full_bar, 1);
        mbar_init(acc_empty_bar, 2 * kEpiWarps);  // the epilogue warps of both CTAs
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        prefetch_tensormap(&map_a);
        prefetch_tensormap(&map_b);
        prefetch_tensormap(&map_y);
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();  // both CTAs' barriers are initialised before anyone signals across
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // When launched as a programmatic dependent of the activation quantizer, everything above ran
    // while that kernel was finishing; its output (and any earlier work in the stream) is complete
    // and visible from here on.  A no-op for an ordinary launch.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // ... and a kernel launched as this one's programmatic dependent may start its own set-up as
    // soon as this kernel's CTAs leave their SMs.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    const int total_tiles = p.m_tiles * p.n_tiles;

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        uint32_t it = 0;
        bool ok = true;
        for (int tile = pair; tile < total_tiles && ok; tile += num_pairs) {
            const int m_blk = tile % p.m_tiles, n_blk = tile / p.m_tiles;
            const int m0 = m_blk * BM + static_cast<int>(rank) * BM_CTA;
            const int n0 = n_blk * BN;
            const int ra = min(m0 >> 7, p.m_rowblocks - 1);
            const int nb0 = n0 >> 7;
            const uint8_t *sfa_src = p.sfx + static_cast<int64_t>(ra) * p.kb4 * kSfBlock;
            const uint8_t *sfb_src[kNB];
#pragma unroll
            for (int j = 0; j < kNB; ++j)
                sfb_src[j] = p.sfw + static_cast<int64_t>(min(nb0 + j, p.n_rowblocks - 1)) * p.kb4 * kSfBlock;
            for (int kt = 0; kt < p.k_tiles; ++kt, ++it) {
                const int s = it % kStages;
                const uint32_t par = (it / kStages) & 1u;
                ok = mbar_wait_warp(stage_free_bar(s), par ^ 1u, wctx);
                if (!ok) break;
                const int kb_valid = min(4, p.kb_total - kt * 4);
                const uint32_t sf_bytes = static_cast<uint32_t>(kb_valid) * kSfBlock;
                const uint32_t stage = base + s * kStageBytes;
                const uint32_t sf_stage = stage + kABytes + kBBytes;
                const uint32_t full_leader = mapa(stage_full_bar(s), 0);
                const int64_t kofs = static_cast<int64_t>(kt) * 4 * kSfBlock;
                if (elect_one()) {
                    if (rank == 0) mbar_expect_tx(stage_full_bar(s), 2u * (kABytes + kBBytes));
                    mbar_expect_tx(sf_ready_bar(s), (1u + kNB) * sf_bytes);
                    bulk_load(sf_stage, sfa_src + kofs, sf_bytes, sf_ready_bar(s));
#pragma unroll
                    for (int j = 0; j < kNB; ++j)
                        bulk_load(sf_stage + (1 + j) * kSfaBytes, sfb_src[j] + kofs, sf_bytes, sf_ready_bar(s));
                    tma_load_2d_pair(stage, &map_a, kt * (BK / 2), m0, full_leader);
                    tma_load_2d_pair(stage + kABytes, &map_b, kt * (BK / 2), n0 + static_cast<int>(rank) * BN_CTA,
                                     full_leader);
                }
                __syncwarp();
            }
        }
        if (!ok && lane == 0) {
            // give the scale copies already issued a bounded chance to land before leaving
            const uint32_t first = it > kStages ? it - kStages : 0;
            for (uint32_t j = first; j < it; ++j)
                for (uint32_t i = 0; i < 4096 && !mbar_try(sf_ready_bar(j % kStages), (j / kStages) & 1u); ++i) {}
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (pair leader)
        if (rank == 0) {
            // Ring positions are kept incrementally: operand stage s with phase ph, scale slot t.
            const uint32_t peer = mapa(bars, 1) - bars;  // cluster-window offset of the peer's shared memory
            uint32_t s = 0, ph = 0, t = 0, tcount = 0;
            bool ok = true;
            for (int tile = pair; tile < total_tiles && ok; tile += num_pairs, ++tcount) {
                // the accumulator is free once the epilogue has read the previous tile out of it
                ok = mbar_wait_warp(acc_empty_bar, (tcount & 1u) ^ 1u, wctx);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base;
                uint32_t acc = 0;
                for (int kt = 0; kt < p.k_tiles; ++kt) {
                    ok = mbar_wait_warp(stage_full_bar(s), ph, wctx);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t stage = base + s * kStageBytes;
                    const uint64_t da = operand_desc(stage), db = operand_desc(stage + kABytes);
                    const uint32_t sfa_t = tmem_base + sf_slot_col(t), sfb_t = sfa_t + kSfbOfs;
                    const int kb_valid = min(4, p.kb_total - kt * 4);
                    if (elect_one()) {
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk) {
                            if (kk < kb_valid) {
                                const uint32_t accumulate = acc | static_cast<uint32_t>(kk);
                                tc_mma_pair(d_tmem, da + 2 * kk, db + 2 * kk, kIdesc, sfa_t + 4 * kk,
                                            sfb_t + kSfbColsPerKb * kk, accumulate);
                            }
                        }
                        // the stage (and its scale slot) is free in both CTAs once these MMAs have run
                        tc_commit_pair(stage_free_bar(s));
                        tc_commit_pair(stage_free_bar(s) + peer);
                        if (kt == p.k_tiles - 1) {  // ... and with them the tile's accumulator is complete
                            tc_commit_pair(acc_full_bar);
                            tc_commit_pair(acc_full_bar + peer);
                        }
                    }
                    __syncwarp();
                    acc = 1u;
                    s = (s + 1 == kStages) ? 0u : s + 1;
                    ph ^= (s == 0) ? 1u : 0u;
                    t = (t + 1 == kSfSlots) ? 0u : t + 1;
                }
            }
        }
    } else if (warp >= kFirstStager) {
        // ------------------------------------------------------------ scale-factor stagers
        // Two sets of four warps (one warp per tensor-memory lane quadrant) take alternate K
        // iterations, so a set has two stages' worth of MMA time for one stage of scales.
        const uint32_t q = warp & 3;  // tensor-memory lane quadrant this warp may write
        const uint32_t set = static_cast<uint32_t>(warp - kFirstStager) >> 2;
        const uint32_t lane_ofs = (q * 32u) << 16;
        uint32_t it = 0;
        bool ok = true;
        for (int tile = pair; tile < total_tiles && ok; tile += num_pairs) {
            for (int kt = 0; kt < p.k_tiles; ++kt, ++it) {
                if ((it % kStagerSets) != set) continue;
                const int s = it % kStages;
                const uint32_t t = it % kSfSlots;
                // The stage's previous occupant has been released (which makes the parity wait that
                // follows unambiguous: see kSfSlots), then: this iteration's scale blocks have landed.
                if (it >= kStages) ok = mbar_wait_warp(stage_free_bar(s), ((it - kStages) / kStages) & 1u, wctx);
                ok = ok && mbar_wait_warp(sf_ready_bar(s), (it / kStages) & 1u, wctx);
                if (!ok) break;
                const int kb_valid = min(4, p.kb_total - kt * 4);
                const uint32_t sf_s = base + s * kStageBytes + kABytes + kBBytes + lane * 16u;
                const uint32_t sf_t = tmem_base + lane_ofs + sf_slot_col(t);
                // the shared-memory reads do not depend on the slot: start them before waiting for it
                uint4 sa[4], sb[kNB][4];
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    if (kk < kb_valid) {
                        sa[kk] = lds128(sf_s + kk * kSfBlock);
#pragma unroll
                        for (int j = 0; j < kNB; ++j) sb[j][kk] = lds128(sf_s + (1 + j) * kSfaBytes + kk * kSfBlock);
                    }
                }
                // the MMAs that read this slot kSfSlots iterations ago have completed (their commit
                // released that iteration's stage)
                if (it >= kSfSlots)
                    ok = mbar_wait_warp(stage_free_bar((it - kSfSlots) % kStages), ((it - kSfSlots) / kStages) & 1u, wctx);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    if (kk < kb_valid) {
                        tc_st4(sf_t + 4 * kk, sa[kk]);
#pragma unroll
                        for (int j = 0; j < kNB; ++j)
                            tc_st4(sf_t + kSfbOfs + kSfbColsPerKb * kk + 4 * j, sb[j][kk]);
                    }
                }
                tc_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_leader(stage_full_bar(s), rank);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue
        // Eight warps: lane quadrant q x column half h.  A warp reads its 32 rows x 128 columns out of
        // tensor memory, scales and rounds them to bf16 and keeps them packed in 64 registers; the
        // accumulator goes back to the MMA issuer after those loads (a few hundred cycles), and the
        // two 64-column boxes leave through one staging box and TMA stores behind the next tile's
        // main loop.
        constexpr int kBoxes = 128 / kBoxCols, kChunks = kBoxCols / 8;  // boxes per warp, 16-byte chunks per box row
        const int q = warp & 3;                // tensor-memory lane quadrant this warp may read
        const int h = (warp - 2) >> 2;         // 128-column part
        const float alpha = __fmul_rn(__ldg(p.ts_x), __ldg(p.ts_w));
        const uint32_t buf = epi + static_cast<uint32_t>(warp - 2) * kEpiBox;
        // 128-byte swizzle of the staging box (what the store's tensor map expects): chunk ^ (row & 7)
        const uint32_t row_ofs = static_cast<uint32_t>(lane) * (kBoxCols * 2), sw = static_cast<uint32_t>(lane & 7);
        uint32_t tcount = 0;
        for (int tile = pair; tile < total_tiles; tile += num_pairs, ++tcount) {
            const int m_blk = tile % p.m_tiles, n_blk = tile / p.m_tiles;
            const int m0 = m_blk * BM + static_cast<int>(rank) * BM_CTA + q * 32, n0 = n_blk * BN + h * 128;
            const bool got = mbar_wait(acc_full_bar, tcount & 1u, wctx);
            if (!__all_sync(0xFFFFFFFFu, got)) break;
            tc_fence_after();
            const uint32_t acc = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + h * 128;
            uint32_t pk[64];  // pk[8 c + i] = columns 16 c + 2 i, 16 c + 2 i + 1 of this lane's row
            // two loads in flight: chunk c + 1 is on its way while chunk c is scaled and packed
            uint32_t va[16], vb[16];
            tc_ld16(acc, va);
#pragma unroll
            for (int c = 0; c < 8; c += 2) {
                tc_wait_ld(va);
                tc_ld16(acc + (c + 1) * 16, vb);
#pragma unroll
                for (int i = 0; i < 8; ++i) pk[8 * c + i] = pack_bf16(va[2 * i], va[2 * i + 1], alpha);
                tc_wait_ld(vb);
                if (c + 2 < 8) tc_ld16(acc + (c + 2) * 16, va);
#pragma unroll
                for (int i = 0; i < 8; ++i) pk[8 * (c + 1) + i] = pack_bf16(vb[2 * i], vb[2 * i + 1], alpha);
            }
            // this warp's part of the accumulator has been read: hand it back to the MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_leader(acc_empty_bar, rank);
#pragma unroll
            for (int c = 0; c < kBoxes; ++c) {
                // the store that read the box before (previous box or previous tile) must be done with it
                if (lane == 0) bulk_wait_read<0>();
                __syncwarp();
#pragma unroll
                for (int i = 0; i < kChunks; ++i)
                    sts128(buf + row_ofs + ((static_cast<uint32_t>(i) ^ sw) << 4), pk[4 * kChunks * c + 4 * i],
                           pk[4 * kChunks * c + 4 * i + 1], pk[4 * kChunks * c + 4 * i + 2], pk[4 * kChunks * c + 4 * i + 3]);
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (m0 < p.M && n0 + c * kBoxCols < p.N) tma_store_2d(&map_y, n0 + c * kBoxCols, m0, buf);
                    bulk_commit();
                }
            }
        }
        if (lane == 0) bulk_wait_all();  // shared memory must outlive the stores that read it
        __syncwarp();
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    cluster_sync();  // the peer may still signal this CTA's barriers or read its operands until here
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

// One warp waits, with the kernel's own bounded wait, on a barrier that nobody arrives at: the way
// the expiry path (status word, abort flag, orderly return) is exercised without a fault or a hang.
__global__ void __launch_bounds__(32) wait_expiry_kernel(int *status, long long limit, int *observed) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_word;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_word = 0;
    }
    __syncwarp();
    const WaitCtx w{&abort_word, status, limit};
    const bool ok = mbar_wait_warp(smem_u32(&bar), 0u, w);
    // every lane has the same answer and the warp is converged: what the roles of the GEMM rely on
    if (threadIdx.x == 0) {
        observed[0] = ok ? 1 : 0;
        observed[1] = abort_word;
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

// A row-major 2-D tensor [rows, row_bytes / elem] cut into 128-byte-swizzled boxes of 128 bytes x
// box_rows rows.  Loads read out-of-range rows / columns as zero, stores skip them.
struct MapKey {
    const void *ptr;
    int64_t rows, row_bytes, pitch;
    int box_rows, elem;
};
struct MapSlot {
    MapKey key;
    CUtensorMap map;
    bool used;
};
// Encoding a tensor map costs several microseconds of host time; a layer calls the GEMM with
// the same buffers over and over, so the last few encodings are kept.
bool make_map(CUtensorMap *map, const void *ptr, int64_t rows, int64_t row_bytes, int64_t pitch, int box_rows,
              int elem) {
    constexpr int kSlots = 16;
    static thread_local MapSlot cache[kSlots];
    static thread_local int next = 0;
    for (MapSlot &c : cache)
        if (c.used && c.key.ptr == ptr && c.key.rows == rows && c.key.row_bytes == row_bytes && c.key.pitch == pitch &&
            c.key.box_rows == box_rows && c.key.elem == elem) {
            *map = c.map;
            return true;
        }
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(row_bytes / elem), static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(pitch)};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / elem), static_cast<cuuint32_t>(box_rows)};
    const cuuint32_t estr[2] = {1, 1};
    const CUtensorMapDataType dt = elem == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
    if (enc(map, dt, 2, const_cast<void *>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    MapSlot &slot = cache[next];
    next = (next + 1) % kSlots;
    slot.key = MapKey{ptr, rows, row_bytes, pitch, box_rows, elem};
    slot.map = *map;
    slot.used = true;
    return true;
}

// Number of CTA pairs that can be resident at once on the current device (a cluster must fit inside
// one GPC), after opting the kernel in to its dynamic shared memory there.  Both are per device.
int resident_pairs() {
    static PqPerDevice cache;
    const int dev = pq_device_slot();
    if (dev < 0) return 0;
    std::lock_guard<std::mutex> guard(cache.lock);
    if (cache.value[dev]) return cache.value[dev];
    if (cudaFuncSetAttribute(gemm_w4a4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             static_cast<int>(kSmemBytes)) != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kSmemBytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_w4a4_kernel, &cfg) != cudaSuccess || n <= 0) {
        (void)cudaGetLastError();
        return 0;
    }
    cache.value[dev] = n;
    return n;
}

pq_status gemm_launch(const uint8_t *xq, const uint8_t *sfx, const float *ts_x, const uint8_t *wq, const uint8_t *sfw,
                      const float *ts_w, int64_t M, int64_t N, int64_t K, void *Y, int64_t ldy, void *ws,
                      size_t ws_bytes, void *stream) {
    PQ_REQUIRE(xq && sfx && ts_x && wq && sfw && ts_w && Y, PQ_ERR_NULL);
    PQ_REQUIRE(M > 0 && N > 0 && K >= 64 && K % 64 == 0 && N % 8 == 0 && ldy >= N, PQ_ERR_SHAPE);
    PQ_REQUIRE(M < (1ll << 31) - 256 && N < (1ll << 31) - 256 && K < (1ll << 31), PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(xq) && pq_aligned16(sfx) && pq_aligned16(wq) && pq_aligned16(sfw) && pq_aligned16(Y) &&
                   ldy % 8 == 0,
               PQ_ERR_ALIGN);
    PQ_REQUIRE(ws && ws_bytes >= pq_workspace_bytes(PQ_OP_GEMM, M, K, N, 0), PQ_ERR_WORKSPACE);
    PQ_REQUIRE(pq_aligned256(ws), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    CUtensorMap map_a, map_b, map_y;
    if (!make_map(&map_a, xq, M, K / 2, K / 2, BM_CTA, 1) || !make_map(&map_b, wq, N, K / 2, K / 2, BN_CTA, 1) ||
        !make_map(&map_y, Y, M, N * 2, ldy * 2, 32, 2))
        return PQ_ERR_CUDA;

    const int pairs_max = resident_pairs();
    if (pairs_max <= 0) return PQ_ERR_CUDA;

    GemmParams p;
    p.sfx = sfx, p.sfw = sfw, p.ts_x = ts_x, p.ts_w = ts_w;
    p.M = static_cast<int>(M), p.N = static_cast<int>(N), p.K = static_cast<int>(K);
    p.m_tiles = static_cast<int>(pq_ceil_div(M, BM));
    p.n_tiles = static_cast<int>(pq_ceil_div(N, BN));
    p.k_tiles = static_cast<int>(pq_ceil_div(K, BK));
    p.kb_total = static_cast<int>(K / 64);
    p.kb4 = p.kb_total;
    p.m_rowblocks = static_cast<int>(pq_ceil_div(M, 128));
    p.n_rowblocks = static_cast<int>(pq_ceil_div(N, 128));
    p.wait_cycles = kWaitCycles;
    p.status = static_cast<int *>(ws);
    const int64_t tiles = static_cast<int64_t>(p.m_tiles) * p.n_tiles;
    const int pairs = static_cast<int>(tiles < pairs_max ? tiles : pairs_max);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = st;
    // Programmatic dependent launch: the kernel may start (barrier set-up, tensor-memory allocation,
    // tensor-map prefetch) while the kernel in front of it in the stream drains (the quantizer, or
    // the previous GEMM of a chain of layers); it waits for that kernel to complete with
    // griddepcontrol.wait before touching global memory, so stream order is what the caller sees.
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    PQ_CUDA_OK(cudaLaunchKernelEx(&cfg, gemm_w4a4_kernel, map_a, map_b, map_y, p));
    return PQ_OK;
}
}  // namespace

extern "C" pq_status pq_gemm_w4a4(const uint8_t *xq, const uint8_t *sfx, const float *ts_x, const uint8_t *wq,
                                  const uint8_t *sfw, const float *ts_w, int64_t M, int64_t N, int64_t K, void *Y,
                                  int64_t ldy, void *ws, size_t ws_bytes, void *stream) {
    return gemm_launch(xq, sfx, ts_x, wq, sfw, ts_w, M, N, K, Y, ldy, ws, ws_bytes, stream);
}

extern "C" pq_status pq_linear_w4a4(const void *X, int64_t M, int64_t K, int64_t ld, const float *ts_x, uint8_t *xq,
                                    uint8_t *sfx, const uint8_t *wq, const uint8_t *sfw, const float *ts_w, int64_t N,
                                    void *Y, int64_t ldy, void *ws, size_t ws_bytes, void *stream) {
    const pq_status rc = pq_quant_act_nvfp4(X, M, K, ld, ts_x, xq, sfx, PQ_SF_TCGEN05, stream);
    if (rc != PQ_OK) return rc;
    return gemm_launch(xq, sfx, ts_x, wq, sfw, ts_w, M, N, K, Y, ldy, ws, ws_bytes, stream);
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

// ---------------------------------------------------------------- batches through one layer
namespace {
constexpr int kMaxSets = 8, kMaxPipeDevices = 64;

// Two internal streams and the events that order them, created once per device (host objects,
// no device memory).
struct Pipe {
    cudaStream_t q = nullptr, g = nullptr, up = nullptr, down = nullptr;
    cudaEvent_t fork = nullptr, join_q = nullptr, join_g = nullptr, join_up = nullptr, join_down = nullptr;
    cudaEvent_t q_done[kMaxSets] = {}, g_done[kMaxSets] = {}, up_done[kMaxSets] = {}, down_done[kMaxSets] = {};
    bool ready = false;
};

Pipe *pipe_for_current_device() {
    static std::mutex lock;
    static Pipe pipes[kMaxPipeDevices];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxPipeDevices) return nullptr;
    std::lock_guard<std::mutex> guard(lock);
    Pipe &p = pipes[dev];
    if (!p.ready) {
        bool ok = cudaStreamCreateWithFlags(&p.q, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&p.g, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&p.up, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&p.down, cudaStreamNonBlocking) == cudaSuccess;
        auto make = [&](cudaEvent_t *e) { ok = ok && cudaEventCreateWithFlags(e, cudaEventDisableTiming) == cudaSuccess; };
        make(&p.fork), make(&p.join_q), make(&p.join_g), make(&p.join_up), make(&p.join_down);
        for (int i = 0; i < kMaxSets; ++i)
            make(&p.q_done[i]), make(&p.g_done[i]), make(&p.up_done[i]), make(&p.down_done[i]);
        if (!ok) {
            (void)cudaGetLastError();
            return nullptr;
        }
        p.ready = true;
    }
    return &p;
}
}  // namespace

extern "C" pq_status pq_linear_w4a4_batched(int n, const void *const *X, int64_t M, int64_t K, int64_t ld,
                                            const float *ts_x, uint8_t *const *xq, uint8_t *const *sfx, int n_sets,
                                            const uint8_t *wq, const uint8_t *sfw, const float *ts_w, int64_t N,
                                            void *const *Y, int64_t ldy, void *ws, size_t ws_bytes, void *stream) {
    PQ_REQUIRE(X && xq && sfx && Y, PQ_ERR_NULL);
    PQ_REQUIRE(n >= 1 && n_sets >= 2 && n_sets <= kMaxSets, PQ_ERR_SHAPE);
    for (int i = 0; i < n; ++i) PQ_REQUIRE(X[i] && Y[i], PQ_ERR_NULL);
    for (int s = 0; s < n_sets; ++s) PQ_REQUIRE(xq[s] && sfx[s], PQ_ERR_NULL);
    Pipe *pipe = pipe_for_current_device();
    if (!pipe) return PQ_ERR_CUDA;
    cudaStream_t user = static_cast<cudaStream_t>(stream);
    // fork: both internal streams start after everything already in the caller's stream
    PQ_CUDA_OK(cudaEventRecord(pipe->fork, user));
    PQ_CUDA_OK(cudaStreamWaitEvent(pipe->q, pipe->fork, 0));
    PQ_CUDA_OK(cudaStreamWaitEvent(pipe->g, pipe->fork, 0));
    pq_status rc = PQ_OK;
    // The GEMMs go out in pairs: both quantizer events are awaited in front of the pair, so the
    // second GEMM directly follows the first in its stream and may be its programmatic dependent
    // (its set-up overlaps the first one's last tiles).
    for (int i0 = 0; i0 < n && rc == PQ_OK; i0 += 2) {
        const int i1 = (i0 + 2 < n) ? i0 + 2 : n;
        for (int i = i0; i < i1 && rc == PQ_OK; ++i) {
            const int s = i % n_sets;
            // the GEMM that last read this set of intermediates has to be done with it
            if (i >= n_sets && cudaStreamWaitEvent(pipe->q, pipe->g_done[s], 0) != cudaSuccess) rc = PQ_ERR_CUDA;
            // 128-thread blocks: they fit on an SM beside the GEMM's CTA
            if (rc == PQ_OK) rc = pq_quant_act_nvfp4_shaped(X[i], M, K, ld, ts_x, xq[s], sfx[s], PQ_SF_TCGEN05, 1, pipe->q);
            if (rc == PQ_OK && cudaEventRecord(pipe->q_done[s], pipe->q) != cudaSuccess) rc = PQ_ERR_CUDA;
            if (rc == PQ_OK && cudaStreamWaitEvent(pipe->g, pipe->q_done[s], 0) != cudaSuccess) rc = PQ_ERR_CUDA;
        }
        for (int i = i0; i < i1 && rc == PQ_OK; ++i) {
            const int s = i % n_sets;
            rc = gemm_launch(xq[s], sfx[s], ts_x, wq, sfw, ts_w, M, N, K, Y[i], ldy, ws, ws_bytes, pipe->g);
            if (rc == PQ_OK && cudaEventRecord(pipe->g_done[s], pipe->g) != cudaSuccess) rc = PQ_ERR_CUDA;
        }
    }
    // join (also after an error, so that a stream capture in progress stays well-formed)
    bool joined = cudaEventRecord(pipe->join_q, pipe->q) == cudaSuccess &&
                  cudaEventRecord(pipe->join_g, pipe->g) == cudaSuccess &&
                  cudaStreamWaitEvent(user, pipe->join_q, 0) == cudaSuccess &&
                  cudaStreamWaitEvent(user, pipe->join_g, 0) == cudaSuccess;
    if (!joined) {
        (void)cudaGetLastError();
        return rc == PQ_OK ? PQ_ERR_CUDA : rc;
    }
    return rc;
}

extern "C" pq_status pq_linear_w4a4_host_batched(int n, const void *const *X_host, int64_t M, int64_t K,
                                                 const float *ts_x, void *const *X_dev, void *const *Y_dev, int n_sets,
                                                 uint8_t *xq, uint8_t *sfx, const uint8_t *wq, const uint8_t *sfw,
                                                 const float *ts_w, int64_t N, void *const *Y_host, void *ws,
                                                 size_t ws_bytes, void *stream) {
    PQ_REQUIRE(X_host && X_dev && Y_dev && Y_host, PQ_ERR_NULL);
    PQ_REQUIRE(n >= 1 && n_sets >= 2 && n_sets <= kMaxSets && M > 0 && K > 0 && N > 0, PQ_ERR_SHAPE);
    for (int i = 0; i < n; ++i) PQ_REQUIRE(X_host[i] && Y_host[i], PQ_ERR_NULL);
    for (int s = 0; s < n_sets; ++s) PQ_REQUIRE(X_dev[s] && Y_dev[s], PQ_ERR_NULL);
    Pipe *pipe = pipe_for_current_device();
    if (!pipe) return PQ_ERR_CUDA;
    cudaStream_t user = static_cast<cudaStream_t>(stream), up = pipe->up, run = pipe->g, down = pipe->down;
    const size_t x_bytes = static_cast<size_t>(M) * K * 2, y_bytes = static_cast<size_t>(M) * N * 2;
    PQ_CUDA_OK(cudaEventRecord(pipe->fork, user));
    PQ_CUDA_OK(cudaStreamWaitEvent(up, pipe->fork, 0));
    PQ_CUDA_OK(cudaStreamWaitEvent(run, pipe->fork, 0));
    PQ_CUDA_OK(cudaStreamWaitEvent(down, pipe->fork, 0));
    pq_status rc = PQ_OK;
    auto cuda_ok = [&](cudaError_t e) {
        if (e != cudaSuccess && rc == PQ_OK) rc = PQ_ERR_CUDA;
        return rc == PQ_OK;
    };
    for (int i = 0; i < n && rc == PQ_OK; ++i) {
        const int s = i % n_sets;
        // upload: the staging buffer is free once the quantizer of its previous batch has read it
        if (i >= n_sets && !cuda_ok(cudaStreamWaitEvent(up, pipe->q_done[s], 0))) break;
        if (!cuda_ok(cudaMemcpyAsync(X_dev[s], X_host[i], x_bytes, cudaMemcpyHostToDevice, up))) break;
        if (!cuda_ok(cudaEventRecord(pipe->up_done[s], up))) break;
        // compute: needs the upload, and the output buffer's previous download to have finished
        if (!cuda_ok(cudaStreamWaitEvent(run, pipe->up_done[s], 0))) break;
        if (i >= n_sets && !cuda_ok(cudaStreamWaitEvent(run, pipe->down_done[s], 0))) break;
        rc = pq_quant_act_nvfp4(X_dev[s], M, K, K, ts_x, xq, sfx, PQ_SF_TCGEN05, run);
        if (rc != PQ_OK || !cuda_ok(cudaEventRecord(pipe->q_done[s], run))) break;
        rc = gemm_launch(xq, sfx, ts_x, wq, sfw, ts_w, M, N, K, Y_dev[s], N, ws, ws_bytes, run);
        if (rc != PQ_OK || !cuda_ok(cudaEventRecord(pipe->g_done[s], run))) break;
        // download
        if (!cuda_ok(cudaStreamWaitEvent(down, pipe->g_done[s], 0))) break;
        if (!cuda_ok(cudaMemcpyAsync(Y_host[i], Y_dev[s], y_bytes, cudaMemcpyDeviceToHost, down))) break;
        if (!cuda_ok(cudaEventRecord(pipe->down_done[s], down))) break;
    }
    const bool joined = cudaEventRecord(pipe->join_up, up) == cudaSuccess &&
                        cudaEventRecord(pipe->join_g, run) == cudaSuccess &&
                        cudaEventRecord(pipe->join_down, down) == cudaSuccess &&
                        cudaStreamWaitEvent(user, pipe->join_up, 0) == cudaSuccess &&
                        cudaStreamWaitEvent(user, pipe->join_g, 0) == cudaSuccess &&
                        cudaStreamWaitEvent(user, pipe->join_down, 0) == cudaSuccess;
    if (!joined) {
        (void)cudaGetLastError();
        return rc == PQ_OK ? PQ_ERR_CUDA : rc;
    }
    return rc;
}

extern "C" pq_status pq_selftest_wait_expiry(void *ws, size_t ws_bytes, long long limit_cycles, int *observed,
                                             void *stream) {
    PQ_REQUIRE(ws && observed, PQ_ERR_NULL);
    PQ_REQUIRE(ws_bytes >= sizeof(int), PQ_ERR_WORKSPACE);
    PQ_REQUIRE(limit_cycles > 0 && limit_cycles <= 100000000ll, PQ_ERR_SHAPE);
    wait_expiry_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<int *>(ws), limit_cycles, observed);
    return pq_launch_status();
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
