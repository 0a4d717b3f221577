// rptq_ln_reorder_quant: LayerNorm with the channel reorder fused in (Sec. 4.2), followed by the
// per-cluster quantiser (Eq. 1 applied per cluster, Appendix) and packed stores.
//
// The paper scatters on write ("the write address is additionally offset based on the reorder
// index"). Packed sub-byte codes need whole words written at once, so here the row is normalised
// into shared memory in channel order and every thread gathers the 32 channels of one output
// unit (32 consecutive padded positions, always inside one cluster), quantises them with that
// cluster's parameters held in registers, and stores 12/16/32 contiguous bytes.
//
// Memory-bound by design. A block is persistent over rows; rows arrive through a ring of
// shared-memory slots filled by the copy engine several rows ahead; the shared-memory addresses
// of a thread's 32 source channels and its unit's parameters stay in registers across rows; the
// LayerNorm arithmetic uses the packed two-wide fp32 instructions of sm_100.
#include <cuda_fp16.h>

#include <mutex>
#include <vector>

#include "pack.cuh"
#include "rptq_internal.h"

namespace rptq {

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Two-wide fp32 arithmetic (one instruction for two lanes of a register pair).
__device__ __forceinline__ float2 add2(float2 a, float2 b)
{
    float2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(reinterpret_cast<uint64_t&>(d))
        : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)));
    return d;
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b)
{
    float2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(reinterpret_cast<uint64_t&>(d))
        : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)));
    return d;
}
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c)
{
    float2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(reinterpret_cast<uint64_t&>(d))
        : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)), "l"(reinterpret_cast<uint64_t&>(c)));
    return d;
}

__device__ __forceinline__ float lds_f32(uint32_t addr)
{
    float v;
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}

__device__ __forceinline__ void bar_sync(int id, int count) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ void bar_arrive(int id, int count) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(count) : "memory"); }
__device__ __forceinline__ uint4 lds_v4(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}
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

// The block is split into two groups of warps that work on consecutive rows at the same time:
//   LN warps      (TL threads)  take a row from a shared-memory ring that the copy engine fills
//                               several rows ahead (one contiguous cp.async.bulk per row: at 18-24 KB
//                               a row, one row in flight per SM would leave HBM idle most of the
//                               time), reduce mean and variance, and normalise the row into one of
//                               two shared-memory buffers in channel order
//   gather warps  (TG threads)  each thread owns one output unit (32 consecutive padded positions,
//                               always inside one cluster): it reads its 32 source channels from the
//                               buffer, quantises with the cluster's parameters and stores 12/16/32
//                               contiguous bytes
// so the reductions of row i+1 overlap the gather of row i. Named barriers hand the buffers over.
// The only wait on the copy engine is bounded: if it runs out the row is processed as it is, the
// status word is set, and every thread still reaches every barrier.
// DBG adds the optional fp32 output of the reordered LayerNorm values (off the fast path).
// GB32: gains and biases are kept as fp32 in shared memory (when they fit), else as fp16.
enum { BAR_LN = 1, BAR_FULL0 = 2, BAR_EMPTY0 = 4 };
constexpr long long kLnWaitBudgetCycles = 4000000000ll;

struct LnParams {
    const __half* x; int64_t ldx; const __half* gamma; const __half* beta; float eps;
    int M, C, n_units, TL, depth;
    const uint16_t* src_tab; const UnitInfo* unit_tab;
    uint8_t* codes; int64_t row_bytes; float* y_dbg; int* status;
};

// MAXT bounds the block size (512: up to 128 registers per thread; 1024: 64).
template <int NCH, int BITS, bool DBG, int MAXT, bool GB32>
__global__ void __launch_bounds__(MAXT)
ln_reorder_quant_kernel(const LnParams p)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const int T = blockDim.x, TL = p.TL, TG = T - TL, C = p.C;
    const int tid = threadIdx.x;
    const int n_chunks = C >> 3;
    const int ybuf_stride = (C + 4 + 3) & ~3;           // C floats in split-half order + the pad slot
    float* ybuf0 = reinterpret_cast<float*>(smem_raw);
    uint8_t* gb = smem_raw + 2 * ybuf_stride * 4;        // gains, then biases (fp32 or fp16)
    uint8_t* ring = gb + (GB32 ? 8 : 4) * C;             // `depth` raw rows of 2 C bytes
    float* red = reinterpret_cast<float*>(ring + (size_t)p.depth * 2 * C);   // [2][2][32]
    uint64_t* bars = reinterpret_cast<uint64_t*>(red + 128);                 // [depth] row landed
    const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);
    const uint32_t bar_s = (uint32_t)__cvta_generic_to_shared(bars);
    const int n_rows = (p.M - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // rows of this block

    if (tid == 0) {
        // pad positions read this slot: -inf quantises to code 0 whatever the parameters
        ybuf0[C] = -INFINITY; ybuf0[ybuf_stride + C] = -INFINITY;
        for (int d = 0; d < p.depth; ++d) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_s + 8 * d) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int ch = tid; ch < n_chunks; ch += T) {
        const uint4 gv = __ldg(reinterpret_cast<const uint4*>(p.gamma + ch * 8));
        const uint4 bv = __ldg(reinterpret_cast<const uint4*>(p.beta + ch * 8));
        if constexpr (GB32) {
            // four regions of one float4 per chunk (gains 0-3, gains 4-7, biases 0-3, biases 4-7) so
            // that the LayerNorm warps' vector reads are contiguous across lanes
            float* g = reinterpret_cast<float*>(gb);
            const __half2* gh = reinterpret_cast<const __half2*>(&gv);
            const __half2* bh = reinterpret_cast<const __half2*>(&bv);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                *reinterpret_cast<float2*>(g + ((e >> 1) * n_chunks + ch) * 4 + 2 * (e & 1)) = __half22float2(gh[e]);
                *reinterpret_cast<float2*>(g + ((2 + (e >> 1)) * n_chunks + ch) * 4 + 2 * (e & 1)) = __half22float2(bh[e]);
            }
        } else {
            reinterpret_cast<uint4*>(gb)[ch] = gv;
            reinterpret_cast<uint4*>(gb)[n_chunks + ch] = bv;
        }
    }
    __syncthreads();

    if (tid < TL) {
        // ------------------------------------------------------------ LayerNorm warps
        const int lane = tid & 31, warp = tid >> 5, nwarps = TL >> 5;
        const float inv_C = 1.0f / (float)C;
        const uint32_t row_bytes_in = 2u * (uint32_t)C;
        // One thread keeps the ring full. Slots, parities and source pointers advance by increments:
        // this is a single thread of dependent instructions on every row's critical path.
        const int64_t row_step = (int64_t)gridDim.x * p.ldx;
        const __half* next_src = p.x + (int64_t)blockIdx.x * p.ldx;
        int next_row = 0, next_slot = 0;
        auto issue_row = [&]() {             // row `next_row` of this block into ring slot `next_slot`
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_s + 8 * next_slot), "r"(row_bytes_in) : "memory");
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                         ::"r"(ring_s + next_slot * row_bytes_in), "l"(next_src), "r"(row_bytes_in), "r"(bar_s + 8 * next_slot) : "memory");
            next_src += row_step;
            ++next_row;
            if (++next_slot == p.depth) next_slot = 0;
        };
        if (tid == 0)
            while (next_row < p.depth - 1 && next_row < n_rows) issue_row();
        int slot = 0;
        uint32_t parity = 0;
        for (int i = 0; i < n_rows; ++i) {
            const int b = i & 1;
            // Refill the slot of row i-1: every LayerNorm thread read it before that row's first barrier.
            if (tid == 0 && next_row < n_rows) issue_row();
            if (!mbar_try_wait(bar_s + 8 * slot, parity)) {
                const long long t0 = clock64();
                while (!mbar_try_wait(bar_s + 8 * slot, parity)) {
                    if (clock64() - t0 > kLnWaitBudgetCycles) { if (p.status) atomicExch(p.status, RPTQ_ERR_DEVICE_TIMEOUT); break; }
                }
            }
            const uint32_t row_s = ring_s + slot * row_bytes_in;
            if (++slot == p.depth) { slot = 0; parity ^= 1u; }
            float2 xf[NCH][4];
#pragma unroll
            for (int k = 0; k < NCH; ++k) {
                const int ch = tid + k * TL;
                const uint4 raw = ch < n_chunks ? lds_v4(row_s + ch * 16) : make_uint4(0, 0, 0, 0);
                const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
                for (int e = 0; e < 4; ++e) xf[k][e] = __half22float2(h[e]);
            }
            float* redm = red + b * 64;
            // mean
            float2 s2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int k = 0; k < NCH; ++k)
#pragma unroll
                for (int e = 0; e < 4; ++e) s2 = add2(s2, xf[k][e]);
            const float s = warp_sum(s2.x + s2.y);
            if (lane == 0) redm[warp] = s;
            bar_sync(BAR_LN, TL);
            float tot = 0.f;
            for (int w = 0; w < nwarps; ++w) tot += redm[w];
            const float mu = tot * inv_C;
            // variance, two-pass on the registers
            const float2 neg_mu = make_float2(-mu, -mu);
            float2 q2 = make_float2(0.f, 0.f);
#pragma unroll
            for (int k = 0; k < NCH; ++k) {
                const bool live = (tid + k * TL) < n_chunks;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    xf[k][e] = live ? add2(xf[k][e], neg_mu) : make_float2(0.f, 0.f);
                    q2 = fma2(xf[k][e], xf[k][e], q2);
                }
            }
            const float sq = warp_sum(q2.x + q2.y);
            if (lane == 0) redm[32 + warp] = sq;
            bar_sync(BAR_LN, TL);
            float tq = 0.f;
            for (int w = 0; w < nwarps; ++w) tq += redm[32 + w];
            const float rstd = 1.0f / sqrtf(tq * inv_C + p.eps);
            const float2 rstd2 = make_float2(rstd, rstd);
            // the gather of row i-2 must have finished with this buffer
            if (i >= 2) bar_sync(BAR_EMPTY0 + b, T);
            float* ybuf = ybuf0 + b * ybuf_stride;
#pragma unroll
            for (int k = 0; k < NCH; ++k) {
                const int ch = tid + k * TL;
                if (ch < n_chunks) {
                    float2 g[4], bt[4];
                    if constexpr (GB32) {
                        const float4* g4 = reinterpret_cast<const float4*>(gb) + ch;
                        const float4 ga = g4[0], gc = g4[n_chunks], ba = g4[2 * n_chunks], bc = g4[3 * n_chunks];
                        g[0] = make_float2(ga.x, ga.y); g[1] = make_float2(ga.z, ga.w); g[2] = make_float2(gc.x, gc.y); g[3] = make_float2(gc.z, gc.w);
                        bt[0] = make_float2(ba.x, ba.y); bt[1] = make_float2(ba.z, ba.w); bt[2] = make_float2(bc.x, bc.y); bt[3] = make_float2(bc.z, bc.w);
                    } else {
                        const uint4 gv = reinterpret_cast<const uint4*>(gb)[ch], bv = reinterpret_cast<const uint4*>(gb)[n_chunks + ch];
                        const __half2* gh = reinterpret_cast<const __half2*>(&gv);
                        const __half2* bh = reinterpret_cast<const __half2*>(&bv);
#pragma unroll
                        for (int e = 0; e < 4; ++e) { g[e] = __half22float2(gh[e]); bt[e] = __half22float2(bh[e]); }
                    }
                    float2 y[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) y[e] = fma2(mul2(xf[k][e], rstd2), g[e], bt[e]);
                    *reinterpret_cast<float4*>(ybuf + ch * 4) = make_float4(y[0].x, y[0].y, y[1].x, y[1].y);
                    *reinterpret_cast<float4*>(ybuf + (C >> 1) + ch * 4) = make_float4(y[2].x, y[2].y, y[3].x, y[3].y);
                }
            }
            __threadfence_block();
            bar_arrive(BAR_FULL0 + b, T);
        }
    } else {
        // ------------------------------------------------------------ gather warps
        const int gt = tid - TL;
        const uint32_t ybuf_s = (uint32_t)__cvta_generic_to_shared(ybuf0);
        const bool one_unit = p.n_units <= TG;             // the fast case: my unit's table stays in registers
        uint32_t src_addr[32];
        UnitInfo ui = {1.0f, 0, 0, 0};
        auto load_unit = [&](int u) {
            const uint4* sp = reinterpret_cast<const uint4*>(p.src_tab + u * 32);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 v = __ldg(sp + i);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    src_addr[8 * i + 2 * j] = ybuf_s + 4u * (w[j] & 0xFFFFu);
                    src_addr[8 * i + 2 * j + 1] = ybuf_s + 4u * (w[j] >> 16);
                }
            }
            const uint4 t4 = __ldg(reinterpret_cast<const uint4*>(p.unit_tab + u));
            ui.inv_s = __uint_as_float(t4.x); ui.zc = (int)t4.y; ui.j0 = (int)t4.z; ui.nvalid = (int)t4.w;
        };
        if (one_unit && gt < p.n_units) load_unit(gt);
        const int qmax = (1 << BITS) - 1;
        int m = blockIdx.x;
        for (int i = 0; i < n_rows; ++i, m += gridDim.x) {
            const int b = i & 1;
            const uint32_t boff = (uint32_t)(b * ybuf_stride) * 4u;
            bar_sync(BAR_FULL0 + b, T);
            uint8_t* out_row = p.codes + (int64_t)m * p.row_bytes;
            for (int u = gt; u < p.n_units; u += TG) {
                if (!one_unit) load_unit(u);
                uint32_t q[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    const float yv = lds_f32(src_addr[e] + boff);
                    q[e] = quant_code(yv, ui.inv_s, ui.zc, qmax);
                    if constexpr (DBG) {
                        if (e < ui.nvalid) p.y_dbg[(int64_t)m * C + ui.j0 + e] = yv;
                    }
                }
                uint32_t w[BITS];
                pack32<BITS>(q, w);
                if constexpr (BITS == 8) {
                    uint4* dst = reinterpret_cast<uint4*>(out_row + u * 32);
                    dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                    dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                } else if constexpr (BITS == 4) {
                    *reinterpret_cast<uint4*>(out_row + u * 16) = make_uint4(w[0], w[1], w[2], w[3]);
                } else {
                    uint32_t* dst = reinterpret_cast<uint32_t*>(out_row + u * 12);
                    dst[0] = w[0]; dst[1] = w[1]; dst[2] = w[2];
                }
            }
            if (i + 2 < n_rows) bar_arrive(BAR_EMPTY0 + b, T);
        }
    }
}

using KernelFn = void (*)(const LnParams);

template <int BITS, bool DBG, int MAXT, bool GB32>
static KernelFn pick_kernel(int nch)
{
    switch (nch) {
        case 1: return ln_reorder_quant_kernel<1, BITS, DBG, MAXT, GB32>;
        case 2: return ln_reorder_quant_kernel<2, BITS, DBG, MAXT, GB32>;
        case 3: return ln_reorder_quant_kernel<3, BITS, DBG, MAXT, GB32>;
        case 4: return ln_reorder_quant_kernel<4, BITS, DBG, MAXT, GB32>;
        case 5: case 6: return ln_reorder_quant_kernel<6, BITS, DBG, MAXT, GB32>;
        default: return ln_reorder_quant_kernel<8, BITS, DBG, MAXT, GB32>;
    }
}
template <bool DBG, int MAXT, bool GB32>
static KernelFn pick_kernel_bits(int bits, int nch)
{
    return bits == 3 ? pick_kernel<3, DBG, MAXT, GB32>(nch) : bits == 4 ? pick_kernel<4, DBG, MAXT, GB32>(nch) : pick_kernel<8, DBG, MAXT, GB32>(nch);
}
template <bool DBG>
static KernelFn pick_kernel_all(int bits, int nch, bool big, bool gb32)
{
    if (big) return gb32 ? pick_kernel_bits<DBG, 1024, true>(bits, nch) : pick_kernel_bits<DBG, 1024, false>(bits, nch);
    return gb32 ? pick_kernel_bits<DBG, 512, true>(bits, nch) : pick_kernel_bits<DBG, 512, false>(bits, nch);
}

// Launch shape of one kernel instance on one device, computed on first use (the attribute and
// occupancy queries cost more host time than a small launch).
struct LaunchPlan { const void* fn; int device, T; size_t smem; int blocks; };
static std::mutex g_plan_mutex;
static std::vector<LaunchPlan> g_plans;

static int planned_blocks(const void* fn, int device, int T, size_t smem, int* blocks)
{
    std::lock_guard<std::mutex> lock(g_plan_mutex);
    for (const LaunchPlan& pl : g_plans)
        if (pl.fn == fn && pl.device == device && pl.T == T && pl.smem == smem) { *blocks = pl.blocks; return RPTQ_OK; }
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return RPTQ_ERR_CUDA;
    int n_sm = 0, per_sm = 0;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, T, smem) != cudaSuccess || per_sm < 1) return RPTQ_ERR_CUDA;
    g_plans.push_back({fn, device, T, smem, n_sm * per_sm});
    *blocks = n_sm * per_sm;
    return RPTQ_OK;
}

}  // namespace rptq

using namespace rptq;

extern "C" int rptq_ln_reorder_quant(const rptq_layout_t* L, const void* x, int64_t ldx, const void* gamma,
                                     const void* beta, float eps, int M, void* codes, float* y_dbg, void* stream)
{
    if (!L || !x || !gamma || !beta || !codes) return RPTQ_ERR_INVALID_ARG;
    if (M < 0 || ldx < L->C || (ldx % 8) != 0 || !(eps >= 0.0f)) return RPTQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(gamma) || !aligned16(beta) || !aligned16(codes) || !aligned16(y_dbg))
        return RPTQ_ERR_INVALID_ARG;
    if (M == 0) return RPTQ_OK;
    int dev = -1;
    if (L->device < 0 || cudaGetDevice(&dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (dev != L->device) return RPTQ_ERR_INVALID_ARG;

    // Shared memory: two normalised rows (8 C bytes), gains and biases (8 C as fp32, else 4 C as
    // fp16), and a ring of raw rows (2 C each), at least 2 and at most 6 deep.
    const int C = L->C;
    const size_t fixed = (size_t)2 * ((C + 4 + 3) & ~3) * 4 + 512 + 64;
    const size_t limit = 227 * 1024;
    bool gb32 = fixed + (size_t)8 * C + (size_t)4 * 2 * C <= limit;
    const size_t gb_bytes = (size_t)(gb32 ? 8 : 4) * C;
    if (fixed + gb_bytes + (size_t)2 * 2 * C > limit) return RPTQ_ERR_UNSUPPORTED;
    int depth = (int)((limit - fixed - gb_bytes) / ((size_t)2 * C));
    depth = depth > 6 ? 6 : depth;
    const size_t smem = fixed + gb_bytes + (size_t)depth * 2 * C;

    // Gather threads: one per output unit up to 512 (beyond that each thread loops over units).
    // LayerNorm threads: a thread holds NCH chunks of 8 channels in registers. Blocks of up to 512
    // threads may use 128 registers per thread (NCH <= 6); larger blocks only 64 (NCH <= 3 wanted).
    const int n_chunks = C / 8;
    const int TG = L->n_units >= 512 ? 512 : (L->n_units + 31) / 32 * 32;
    int TL = 64;
    while (TL + TG + 32 <= 512 && (n_chunks + TL - 1) / TL > 3) TL += 32;
    const bool big = (n_chunks + TL - 1) / TL > 6;
    if (big) {
        TL = 64;
        while (TL + TG + 32 <= 1024 && (n_chunks + TL - 1) / TL > 3) TL += 32;
    }
    const int nch = (n_chunks + TL - 1) / TL;
    if (nch > 8) return RPTQ_ERR_UNSUPPORTED;
    const int T = TL + TG;

    KernelFn fn = y_dbg ? pick_kernel_all<true>(L->bits, nch, big, gb32) : pick_kernel_all<false>(L->bits, nch, big, gb32);
    int blocks = 0;
    const int rc = planned_blocks(reinterpret_cast<const void*>(fn), dev, T, smem, &blocks);
    if (rc != RPTQ_OK) return rc;
    LnParams p{};
    p.x = static_cast<const __half*>(x); p.ldx = ldx; p.gamma = static_cast<const __half*>(gamma);
    p.beta = static_cast<const __half*>(beta); p.eps = eps; p.M = M; p.C = C; p.n_units = L->n_units; p.TL = TL;
    p.depth = depth; p.src_tab = L->d_src; p.unit_tab = L->d_unit; p.codes = static_cast<uint8_t*>(codes);
    p.row_bytes = L->row_bytes; p.y_dbg = y_dbg; p.status = device_status_word();
    fn<<<M < blocks ? M : blocks, T, smem, static_cast<cudaStream_t>(stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}
