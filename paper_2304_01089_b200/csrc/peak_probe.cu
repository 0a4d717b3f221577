// rptq_probe_int8_peak: a measurement aid, not part of the method. It issues the GEMM kernel's own
// tensor-core instruction (tcgen05.mma kind::i8, CTA pairs, M 256 x N 256 x K 32, unsigned x signed
// 8-bit into int32 tensor-memory accumulators) back to back on operands that already sit in shared
// memory, with no loads, unpacking or epilogue: the rate it reaches is the ceiling the cluster GEMM
// is compared with.
//
// The first warp of the first CTA of every pair issues batches of 32 instructions (eight passes over
// the four K steps of a 128-byte-wide operand tile, alternating between two accumulators) and
// commits each batch to one of two barriers; it waits for batch k before issuing batch k + 2, so at
// most 64 instructions are queued and the pipe never drains. Every wait is bounded.
#include <cuda_runtime.h>
#include <stdint.h>

#include "rptq.h"

namespace rptq {
namespace probe {

constexpr int THREADS = 128;
constexpr int BATCH = 32;
constexpr long long WAIT_BUDGET_CYCLES = 2000000000ll;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
#pragma unroll 1
    while (true) {
#pragma unroll 1
        for (int i = 0; i < 256; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > WAIT_BUDGET_CYCLES) return false;
    }
}
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                         // leading byte offset (ignored for swizzled K-major tiles)
    d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset: 8-row groups are 1024 bytes apart
    d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                         // 128-byte swizzle
    return d;
}

__global__ void __launch_bounds__(THREADS, 1)
int8_peak_kernel(int n_batches, int* failed)
{
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (base - smem_u32(smem_raw));
    // operand tiles: 128 rows x 128 bytes each (A: this CTA's token rows, B: this CTA's half of the 256 weight rows)
    uint32_t* tiles = reinterpret_cast<uint32_t*>(smem);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + 2 * 16384);
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2);
    const int tid = threadIdx.x, warp = tid >> 5;
    uint32_t rank;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));

    for (int i = tid; i < 2 * 16384 / 4; i += THREADS) tiles[i] = 0x01010101u * (uint32_t)((i * 7 + 3) & 7);
    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars)) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(bars + 1)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(s_tmem)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // the tiles were written with ordinary stores
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *s_tmem;

    if (warp == 0 && rank == 0) {
        // The whole warp runs the loop in converged control flow; elect.sync picks the issuing lane.
        // D = s32, A = unsigned 8-bit, B = signed 8-bit, both K-major, M = 256 over the pair, N = 256
        const uint32_t idesc = (2u << 4) | (0u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((256u >> 4) << 24);
        const uint64_t a_desc = smem_desc_sw128(base), b_desc = smem_desc_sw128(base + 16384);
        bool ok = true;
        for (int b = 0; b < n_batches && ok; ++b) {
            if (b >= 2) ok = __any_sync(0xffffffffu, mbar_wait(smem_u32(bars + (b & 1)), (uint32_t)((b >> 1) - 1) & 1u));
            if (!ok) break;
#pragma unroll 1
            for (int i = 0; i < BATCH; i += 4) {
                const uint32_t d = tmem + ((i >> 2) & 1) * 256;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    asm volatile(
                        "{\n\t.reg .pred p, q;\n\t"
                        "elect.sync _|q, 0xffffffff;\n\t"
                        "setp.ne.b32 p, %4, 0;\n\t"
                        "@q tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                        ::"r"(d), "l"(a_desc + 2 * j), "l"(b_desc + 2 * j), "r"(idesc), "r"(b | i | j) : "memory");
            }
            asm volatile(
                "{\n\t.reg .pred q;\n\t"
                "elect.sync _|q, 0xffffffff;\n\t"
                "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
                ::"r"(smem_u32(bars + (b & 1))) : "memory");
        }
        // the last two batches
        for (int b = n_batches > 2 ? n_batches - 2 : 0; b < n_batches && ok; ++b)
            ok = __any_sync(0xffffffffu, mbar_wait(smem_u32(bars + (b & 1)), (uint32_t)(b >> 1) & 1u));
        if (!ok && tid == 0) atomicExch(failed, 1);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
}

}  // namespace probe
}  // namespace rptq

extern "C" int rptq_probe_int8_peak(int n_batches, int* failed_dev, double* ops_out, void* stream)
{
    using namespace rptq::probe;
    if (n_batches < 1 || n_batches > (1 << 20) || !failed_dev || !ops_out) return RPTQ_ERR_INVALID_ARG;
    int dev = -1, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    const int smem = 2 * 16384 + 64 + 1024;
    if (cudaFuncSetAttribute(int8_peak_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return RPTQ_ERR_CUDA;
    const int pairs = n_sm / 2;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(2 * pairs));
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, int8_peak_kernel, n_batches, failed_dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    *ops_out = 2.0 * 256.0 * 256.0 * 32.0 * (double)BATCH * (double)n_batches * (double)pairs;
    return RPTQ_OK;
}
