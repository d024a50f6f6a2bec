// Machine probes: how fast one SM takes data in from L2 (bulk copies into shared memory) and how
// fast it writes to L2 / HBM (coalesced 16-byte stores), as a function of how many SMs do so at
// once.  The paper has no counterpart; the two rates bound the GEMM's tile shape (operand bytes per
// MMA cycle on the way in, output bytes per tile on the way out) and are quoted beside its roofline.
#include "pq_common.cuh"

namespace {

constexpr int kChunk = 32768, kStages = 6;       // 6 x 32 KB in flight per SM
constexpr long long kWaitCycles = 2000000000ll;  // bound of every wait below (about a second)

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ bool try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

// One thread per CTA streams `iters` chunks of 32 KB from an L2-resident region into a ring of
// shared-memory buffers with cp.async.bulk; cycles[0] receives the longest CTA's cycle count.
__global__ void __launch_bounds__(32, 1)
ingest_probe(const uint8_t *__restrict__ src, size_t region, int iters, int sm_select, unsigned long long *cycles,
             int *status) {
    extern __shared__ __align__(1024) uint8_t ring[];
    __shared__ uint64_t bars[kStages];
    const uint32_t b0 = smem_addr(bars);
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(b0 + 8 * i), "r"(1));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    // sm_select 1: only SMs with an even id work (one SM of every pair of neighbours);
    // sm_select 2: only SMs whose id / 2 is even (both SMs of every other pair)
    uint32_t smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    if ((sm_select == 1 && (smid & 1u)) || (sm_select == 2 && ((smid >> 1) & 1u))) return;
    const uint32_t dst = smem_addr(ring);
    size_t ofs = (static_cast<size_t>(blockIdx.x) * 1048576u) % region;
    if (ofs + kChunk > region) ofs = 0;
    const long long t0 = clock64();
    bool ok = true;
    for (int i = 0; i < iters + kStages && ok; ++i) {
        const int s = i % kStages;
        if (i >= kStages) {  // the copy issued kStages iterations ago
            const uint32_t parity = ((i / kStages) - 1) & 1;
            const long long w0 = clock64();
            while (!try_wait(b0 + 8 * s, parity)) {
                if (clock64() - w0 > kWaitCycles) {
                    ok = false;
                    break;
                }
            }
        }
        if (i < iters && ok) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(b0 + 8 * s), "r"(kChunk) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(dst + s * kChunk), "l"(src + ofs), "r"(kChunk), "r"(b0 + 8 * s) : "memory");
            ofs += kChunk;
            if (ofs + kChunk > region) ofs = 0;
        }
    }
    const long long t1 = clock64();
    // On a timeout copies may still be in flight into this CTA's shared memory: give them the same
    // bounded time before the CTA (and its shared memory) goes away.
    if (!ok) {
        atomicExch(status, PQ_ERR_TIMEOUT);
        const long long w0 = clock64();
        while (clock64() - w0 < kWaitCycles / 4) {
        }
    }
    atomicMax(cycles, static_cast<unsigned long long>(t1 - t0));
}

// Four warps per CTA write `iters` x 2 KB to the CTA's own region, 512 contiguous bytes per warp
// instruction; cycles[0] receives the longest CTA's cycle count (stores are fire-and-forget: the
// count is the time to hand them to the memory system, which throttles once its queues are full).
__global__ void __launch_bounds__(128, 1)
store_probe(uint4 *__restrict__ out, int iters, size_t per_cta, unsigned long long *cycles) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    char *base = reinterpret_cast<char *>(out) + blockIdx.x * per_cta;
    const uint4 v = make_uint4(lane, warp, blockIdx.x, 7);
    __syncthreads();
    const long long t0 = clock64();
    for (int i = 0; i < iters; ++i)
        *reinterpret_cast<uint4 *>(base + static_cast<size_t>(i * 4 + warp) * 512 + lane * 16) = v;
    const long long t1 = clock64();
    __syncthreads();
    if (threadIdx.x == 0) atomicMax(cycles, static_cast<unsigned long long>(t1 - t0));
}

// Do copies from a neighbour's shared memory compete with the stream from L2?  CTA pairs
// (clusters of two): in both CTAs thread 0 pulls from L2 as in ingest_probe (ring of 4 x 32 KB);
// with forward != 0 thread 32 of rank 0 also pushes 32 KB blocks of its own shared memory into a
// two-buffer ring of rank 1 (cp.async.bulk shared -> shared::cluster), rank 1 hands the buffers
// back.  cycles[0] = slowest L2 stream, cycles[1] = slowest forwarding loop (fwd_iters blocks).
constexpr int kPullStages = 4, kFwdStages = 2;

__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity) {
    const long long w0 = clock64();
    while (!try_wait(bar, parity))
        if (clock64() - w0 > kWaitCycles) return false;
    return true;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(64, 1)
forward_probe(const uint8_t *__restrict__ src, size_t region, int iters, int fwd_iters, unsigned long long *cycles,
              int *status) {
    extern __shared__ __align__(1024) uint8_t smem[];  // [pull ring 4 x 32 KB][forward source 32 KB][forward ring 2 x 32 KB]
    __shared__ uint64_t pull_bar[kPullStages], fwd_full[kFwdStages], fwd_free[kFwdStages];
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
    const uint32_t pb = smem_addr(pull_bar), ff = smem_addr(fwd_full), fe = smem_addr(fwd_free);
    if (threadIdx.x == 0) {
        for (int i = 0; i < kPullStages; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(pb + 8 * i), "r"(1));
        for (int i = 0; i < kFwdStages; ++i) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(ff + 8 * i), "r"(1));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(fe + 8 * i), "r"(1));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    bool ok = true;
    if (threadIdx.x == 0) {
        // ---- the stream from L2, both CTAs
        const uint32_t dst = smem_addr(smem);
        size_t ofs = (static_cast<size_t>(blockIdx.x) * 1048576u) % region;
        if (ofs + kChunk > region) ofs = 0;
        const long long t0 = clock64();
        for (int i = 0; i < iters + kPullStages && ok; ++i) {
            const int s = i % kPullStages;
            if (i >= kPullStages) ok = bounded_wait(pb + 8 * s, ((i / kPullStages) - 1) & 1);
            if (i < iters && ok) {
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(pb + 8 * s), "r"(kChunk) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(dst + s * kChunk), "l"(src + ofs), "r"(kChunk), "r"(pb + 8 * s) : "memory");
                ofs += kChunk;
                if (ofs + kChunk > region) ofs = 0;
            }
        }
        atomicMax(cycles, static_cast<unsigned long long>(clock64() - t0));
    } else if (threadIdx.x == 32 && fwd_iters > 0) {
        // ---- shared memory of rank 0 -> shared memory of rank 1
        const uint32_t fwd_src = smem_addr(smem) + kPullStages * kChunk, fwd_ring = fwd_src + kChunk;
        const long long t0 = clock64();
        if (rank == 0) {
            for (int i = 0; i < fwd_iters && ok; ++i) {
                const int s = i % kFwdStages;
                if (i >= kFwdStages) ok = bounded_wait(fe + 8 * s, ((i / kFwdStages) - 1) & 1);  // rank 1 gave it back
                if (ok)
                    asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(map_to_rank(fwd_ring + s * kChunk, 1)), "r"(fwd_src), "r"(kChunk),
                                   "r"(map_to_rank(ff + 8 * s, 1)) : "memory");
            }
            // every block has been handed back before this CTA's source may go away
            for (int i = (fwd_iters > kFwdStages ? fwd_iters - kFwdStages : 0); i < fwd_iters && ok; ++i)
                ok = bounded_wait(fe + 8 * (i % kFwdStages), (i / kFwdStages) & 1);
        } else {
            for (int i = 0; i < fwd_iters && ok; ++i) {
                const int s = i % kFwdStages;
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(ff + 8 * s), "r"(kChunk) : "memory");
                ok = bounded_wait(ff + 8 * s, (i / kFwdStages) & 1);
                if (ok) asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(map_to_rank(fe + 8 * s, 0)) : "memory");
            }
        }
        atomicMax(cycles + 1, static_cast<unsigned long long>(clock64() - t0));
    }
    if (!ok) {
        atomicExch(status, PQ_ERR_TIMEOUT);
        const long long w0 = clock64();  // copies may still be in flight into this pair's shared memory
        while (clock64() - w0 < kWaitCycles / 4) {
        }
    }
    __syncthreads();
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

}  // namespace

extern "C" pq_status pq_probe_sm_ingest(const void *src, size_t region_bytes, int ctas, int iters, int sm_select,
                                        unsigned long long *cycles, int *status, void *stream) {
    PQ_REQUIRE(src && cycles && status, PQ_ERR_NULL);
    PQ_REQUIRE(ctas >= 1 && ctas <= 65535 && iters >= 1 && iters <= (1 << 20), PQ_ERR_SHAPE);
    PQ_REQUIRE(sm_select >= 0 && sm_select <= 2, PQ_ERR_SHAPE);
    PQ_REQUIRE(region_bytes >= 2 * static_cast<size_t>(kChunk) && region_bytes % kChunk == 0, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(src), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    static bool attr_set = false;
    if (!attr_set) {
        PQ_CUDA_OK(cudaFuncSetAttribute(ingest_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, kChunk * kStages));
        attr_set = true;
    }
    PQ_CUDA_OK(cudaMemsetAsync(cycles, 0, sizeof(unsigned long long), st));
    PQ_CUDA_OK(cudaMemsetAsync(status, 0, sizeof(int), st));
    ingest_probe<<<ctas, 32, kChunk * kStages, st>>>(static_cast<const uint8_t *>(src), region_bytes, iters, sm_select, cycles,
                                                      status);
    return pq_launch_status();
}

extern "C" pq_status pq_probe_sm_store(void *dst, size_t dst_bytes, int ctas, int iters, unsigned long long *cycles,
                                       void *stream) {
    PQ_REQUIRE(dst && cycles, PQ_ERR_NULL);
    PQ_REQUIRE(ctas >= 1 && ctas <= 65535 && iters >= 1 && iters <= (1 << 20), PQ_ERR_SHAPE);
    const size_t per_cta = static_cast<size_t>(iters) * 2048;
    PQ_REQUIRE(dst_bytes >= per_cta * static_cast<size_t>(ctas), PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(dst), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PQ_CUDA_OK(cudaMemsetAsync(cycles, 0, sizeof(unsigned long long), st));
    store_probe<<<ctas, 128, 0, st>>>(static_cast<uint4 *>(dst), iters, per_cta, cycles);
    return pq_launch_status();
}

extern "C" pq_status pq_probe_sm_forward(const void *src, size_t region_bytes, int ctas, int iters, int fwd_iters,
                                         unsigned long long *cycles, int *status, void *stream) {
    PQ_REQUIRE(src && cycles && status, PQ_ERR_NULL);
    PQ_REQUIRE(ctas >= 2 && ctas % 2 == 0 && ctas <= 65534 && iters >= 1 && iters <= (1 << 20) && fwd_iters >= 0 &&
                   fwd_iters <= (1 << 20),
               PQ_ERR_SHAPE);
    PQ_REQUIRE(region_bytes >= 2 * static_cast<size_t>(kChunk) && region_bytes % kChunk == 0, PQ_ERR_SHAPE);
    PQ_REQUIRE(pq_aligned16(src), PQ_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    constexpr int kSmem = (kPullStages + 1 + kFwdStages) * kChunk;
    static bool attr_set = false;
    if (!attr_set) {
        PQ_CUDA_OK(cudaFuncSetAttribute(forward_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmem));
        attr_set = true;
    }
    PQ_CUDA_OK(cudaMemsetAsync(cycles, 0, 2 * sizeof(unsigned long long), st));
    PQ_CUDA_OK(cudaMemsetAsync(status, 0, sizeof(int), st));
    forward_probe<<<ctas, 64, kSmem, st>>>(static_cast<const uint8_t *>(src), region_bytes, iters, fwd_iters, cycles, status);
    return pq_launch_status();
}
