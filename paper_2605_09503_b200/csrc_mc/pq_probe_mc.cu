// Machine probe, single-GPU only: per-SM ingest rate when the CTAs of a cluster receive the same
// bytes through one bulk copy with cluster multicast (one read of L2 feeding several SMs).  The
// source is always this GPU's own memory.  Built into libpq_mc.so, which the rest of the package
// does not need.
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/pq.h"

namespace {

constexpr int kChunk = 32768, kStages = 6;
constexpr long long kWaitCycles = 2000000000ll;

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ bool try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity) {
    const long long w0 = clock64();
    while (!try_wait(bar, parity))
        if (clock64() - w0 > kWaitCycles) return false;
    return true;
}
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\nbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Rank 0 of every cluster copies iters x 32 KB from an L2-resident region into the ring of every
// CTA of its cluster (one multicast copy per chunk); every CTA waits for its copies in order.
// handshake != 0: a stage is reused only after every CTA has reported it consumed (what a real
// pipeline does; the round trip then limits the rate).  handshake == 0: rank 0 reuses a stage as
// soon as its own copy of the data has landed -- the copies land in all CTAs together and nothing
// reads the data, so this measures the transport alone; a CTA that fell a whole ring behind would
// stall its barrier and end the probe with PQ_ERR_TIMEOUT.  cycles[0] = the slowest CTA's cycles.
__global__ void __launch_bounds__(32, 1)
ingest_multicast_probe(const uint8_t *__restrict__ src, size_t region, int iters, int handshake,
                       unsigned long long *cycles, int *status) {
    extern __shared__ __align__(1024) uint8_t ring[];
    __shared__ uint64_t full[kStages], empty[kStages];
    const uint32_t rank = cluster_rank(), csize = cluster_size();
    const uint32_t full0 = smem_addr(full), empty0 = smem_addr(empty);
    if (threadIdx.x == 0) {
        for (int i = 0; i < kStages; ++i) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(full0 + 8 * i), "r"(1));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty0 + 8 * i), "r"(csize));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    cluster_barrier();  // every CTA's barriers exist before anyone signals across
    bool ok = true;
    long long t0 = 0, t1 = 0;
    if (threadIdx.x == 0) {
        const uint32_t dst = smem_addr(ring);
        const uint16_t mask = static_cast<uint16_t>((1u << csize) - 1u);
        size_t ofs = (static_cast<size_t>(blockIdx.x / csize) * 1048576u) % region;
        if (ofs + kChunk > region) ofs = 0;
        t0 = clock64();
        // this CTA expects every stage's bytes; rank 0 also issues the copies, kStages ahead
        for (int i = 0; i < iters + kStages && ok; ++i) {
            const int s = i % kStages;
            if (i >= kStages) {
                const int j = i - kStages;  // the chunk that used stage s before
                ok = bounded_wait(full0 + 8 * s, (j / kStages) & 1);
                if (!ok) break;
                // stage s of this CTA is consumed: tell rank 0
                if (handshake)
                    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(map_to_rank(empty0 + 8 * s, 0)) : "memory");
            }
            if (i < iters) {
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full0 + 8 * s), "r"(kChunk) : "memory");
                if (rank == 0) {
                    if (handshake && i >= kStages) {
                        ok = bounded_wait(empty0 + 8 * s, ((i / kStages) - 1) & 1);  // all CTAs done with the stage
                        if (!ok) break;
                    }
                    asm volatile(
                        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.multicast::cluster [%0], [%1], %2, [%3], %4;"
                        ::"r"(dst + s * kChunk), "l"(src + ofs), "r"(kChunk), "r"(full0 + 8 * s), "h"(mask) : "memory");
                    ofs += kChunk;
                    if (ofs + kChunk > region) ofs = 0;
                }
            }
        }
        t1 = clock64();
        if (!ok) {
            atomicExch(status, PQ_ERR_TIMEOUT);
            const long long w0 = clock64();  // copies may still be landing in this cluster's rings
            while (clock64() - w0 < kWaitCycles / 4) {
            }
        }
        atomicMax(cycles, static_cast<unsigned long long>(t1 - t0));
    }
    __syncwarp();
    cluster_barrier();  // nobody leaves while a peer may still signal its barriers or fill its ring
}

}  // namespace

extern "C" pq_status pq_probe_sm_ingest_multicast(const void *src, size_t region_bytes, int ctas, int cluster, int iters,
                                                  int handshake, unsigned long long *cycles, int *status, void *stream) {
    if (!src || !cycles || !status) return PQ_ERR_NULL;
    if (cluster < 1 || cluster > 8 || (cluster & (cluster - 1)) || ctas < cluster || ctas % cluster || ctas > 65535 ||
        iters < 1 || iters > (1 << 20))
        return PQ_ERR_SHAPE;
    if (region_bytes < 2 * static_cast<size_t>(kChunk) || region_bytes % kChunk) return PQ_ERR_SHAPE;
    if (reinterpret_cast<uintptr_t>(src) & 15u) return PQ_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaFuncSetAttribute(ingest_multicast_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, kChunk * kStages) != cudaSuccess ||
        cudaMemsetAsync(cycles, 0, sizeof(unsigned long long), st) != cudaSuccess ||
        cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) {
        (void)cudaGetLastError();
        return PQ_ERR_CUDA;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(ctas), cfg.blockDim = dim3(32), cfg.dynamicSmemBytes = kChunk * kStages, cfg.stream = st;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = cluster, attr.val.clusterDim.y = 1, attr.val.clusterDim.z = 1;
    cfg.attrs = &attr, cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, ingest_multicast_probe, static_cast<const uint8_t *>(src), region_bytes, iters,
                           handshake, cycles, status) != cudaSuccess) {
        (void)cudaGetLastError();
        return PQ_ERR_CUDA;
    }
    return PQ_OK;
}
