// rptq_ln_reorder_quant: LayerNorm with the channel reorder fused in (Sec. 4.2), followed by the
// per-cluster quantiser (Eq. 1 applied per cluster, Appendix) and packed stores.
//
// The paper scatters on write ("the write address is additionally offset based on the reorder
// index"). Packed sub-byte codes need whole words written at once, so here the row is normalised
// into shared memory in channel order and every thread gathers the 32 channels of one output
// unit (32 consecutive padded positions, always inside one cluster), quantises them with that
// cluster's parameters held in registers, and stores 12/16/32 contiguous bytes.
//
// Memory-bound: one fp16 row in, one packed row out. A block is persistent over rows; the
// per-unit source indices and the LayerNorm gain/bias of the thread's channels stay in
// registers across rows, and the next row's loads are issued before the current row is reduced.
#include <cuda_fp16.h>

#include "rptq_internal.h"

namespace rptq {

constexpr float kMagic = 12582912.0f;   // 1.5 * 2^23: adding it rounds |t| < 2^22 to an integer, half to even

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Shared-memory address (in floats) of channel c of the normalised row. The two 16-byte halves of
// each 8-channel chunk live in separate regions so that both vector stores of a warp are
// contiguous across lanes. The host-built source table already holds these addresses.
// (rptq::ybuf_addr in rptq_internal.h)

// Quantise one value: t = y * inv_s rounded once to an integer (the fused multiply-add with the
// magic constant performs the product exactly and rounds the sum half to even), then + z and clamp.
__device__ __forceinline__ int quant_code(float y, float inv_s, int zc, int qmax)
{
    const float v = __fmaf_rn(y, inv_s, kMagic);
    int q = __float_as_int(v) + zc;
    return min(max(q, 0), qmax);
}

template <int NCH, int BITS>
__global__ void __launch_bounds__(512)
ln_reorder_quant_kernel(const __half* __restrict__ x, int64_t ldx, const __half* __restrict__ gamma,
                        const __half* __restrict__ beta, float eps, int M, int C, int n_units,
                        const uint16_t* __restrict__ src_tab, const UnitInfo* __restrict__ unit_tab,
                        uint8_t* __restrict__ codes, int64_t row_bytes, float* __restrict__ y_dbg)
{
    extern __shared__ __align__(16) float smem[];
    const int T = blockDim.x;
    const int tid = threadIdx.x;
    const int lane = tid & 31, warp = tid >> 5, nwarps = T >> 5;
    const int n_chunks = C >> 3;
    const int ybuf_stride = (C + 4 + 3) & ~3;          // C floats + the pad sentinel, 16-byte multiple
    float* ybuf0 = smem;
    float* red = smem + 2 * ybuf_stride;                // [2 rows in flight][2 reductions][32]

    // pad positions read this slot: -inf quantises to code 0 whatever the parameters
    if (tid == 0) { ybuf0[C] = -INFINITY; ybuf0[ybuf_stride + C] = -INFINITY; }

    // per-thread constants: gain/bias of my channels, source indices and parameters of my unit(s)
    __half2 gb[NCH][8];
#pragma unroll
    for (int k = 0; k < NCH; ++k) {
        const int ch = tid + k * T;
        if (ch < n_chunks) {
            const uint4 gv = *reinterpret_cast<const uint4*>(gamma + ch * 8);
            const uint4 bv = *reinterpret_cast<const uint4*>(beta + ch * 8);
            const __half* gh = reinterpret_cast<const __half*>(&gv);
            const __half* bh = reinterpret_cast<const __half*>(&bv);
#pragma unroll
            for (int e = 0; e < 8; ++e) gb[k][e] = __halves2half2(gh[e], bh[e]);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) gb[k][e] = __halves2half2(__float2half(0.f), __float2half(0.f));
        }
    }
    const bool one_unit = n_units <= T;                 // the fast case: my unit's table stays in registers
    uint32_t srcp[16];
    UnitInfo ui = {1.0f, 0, 0, 0};
    if (one_unit && tid < n_units) {
        const uint4* sp = reinterpret_cast<const uint4*>(src_tab + tid * 32);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const uint4 v = sp[i];
            srcp[4 * i + 0] = v.x; srcp[4 * i + 1] = v.y; srcp[4 * i + 2] = v.z; srcp[4 * i + 3] = v.w;
        }
        ui = unit_tab[tid];
    }
    const int qmax = (1 << BITS) - 1;
    const float inv_C = 1.0f / (float)C;

    uint4 raw[NCH];
    int m = blockIdx.x;
    if (m < M) {
#pragma unroll
        for (int k = 0; k < NCH; ++k) {
            const int ch = tid + k * T;
            raw[k] = (ch < n_chunks) ? __ldg(reinterpret_cast<const uint4*>(x + (int64_t)m * ldx + ch * 8)) : make_uint4(0, 0, 0, 0);
        }
    }
    int par = 0;
    for (; m < M; m += gridDim.x, par ^= 1) {
        float xf[NCH][8];
#pragma unroll
        for (int k = 0; k < NCH; ++k) {
            const __half2* h = reinterpret_cast<const __half2*>(&raw[k]);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 f = __half22float2(h[e]);
                xf[k][2 * e] = f.x; xf[k][2 * e + 1] = f.y;
            }
        }
        const int m_next = m + gridDim.x;
        if (m_next < M) {
#pragma unroll
            for (int k = 0; k < NCH; ++k) {
                const int ch = tid + k * T;
                if (ch < n_chunks) raw[k] = __ldg(reinterpret_cast<const uint4*>(x + (int64_t)m_next * ldx + ch * 8));
            }
        }
        float* redm = red + par * 64;
        // mean
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < NCH; ++k)
#pragma unroll
            for (int e = 0; e < 8; ++e) s += xf[k][e];
        s = warp_sum(s);
        if (lane == 0) redm[warp] = s;
        __syncthreads();
        float tot = 0.f;
        for (int w = 0; w < nwarps; ++w) tot += redm[w];
        const float mu = tot * inv_C;
        // variance, two-pass on the registers
        float sq = 0.f;
#pragma unroll
        for (int k = 0; k < NCH; ++k) {
            const bool live = (tid + k * T) < n_chunks;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                xf[k][e] = live ? xf[k][e] - mu : 0.f;
                sq = __fmaf_rn(xf[k][e], xf[k][e], sq);
            }
        }
        sq = warp_sum(sq);
        if (lane == 0) redm[32 + warp] = sq;
        __syncthreads();
        float tq = 0.f;
        for (int w = 0; w < nwarps; ++w) tq += redm[32 + w];
        const float rstd = 1.0f / sqrtf(tq * inv_C + eps);
        // normalise + affine into shared memory, channel order (split halves)
        float* ybuf = ybuf0 + par * ybuf_stride;
#pragma unroll
        for (int k = 0; k < NCH; ++k) {
            const int ch = tid + k * T;
            if (ch < n_chunks) {
                float yv[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float2 g_b = __half22float2(gb[k][e]);
                    yv[e] = __fmaf_rn(xf[k][e] * rstd, g_b.x, g_b.y);
                }
                *reinterpret_cast<float4*>(ybuf + ch * 4) = make_float4(yv[0], yv[1], yv[2], yv[3]);
                *reinterpret_cast<float4*>(ybuf + (C >> 1) + ch * 4) = make_float4(yv[4], yv[5], yv[6], yv[7]);
            }
        }
        __syncthreads();
        // gather + quantise + pack
        uint8_t* out_row = codes + (int64_t)m * row_bytes;
        for (int u = tid; u < n_units; u += T) {
            if (!one_unit) {
                const uint4* sp = reinterpret_cast<const uint4*>(src_tab + u * 32);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 v = __ldg(sp + i);
                    srcp[4 * i + 0] = v.x; srcp[4 * i + 1] = v.y; srcp[4 * i + 2] = v.z; srcp[4 * i + 3] = v.w;
                }
                const uint4 t4 = __ldg(reinterpret_cast<const uint4*>(unit_tab + u));
                ui.inv_s = __uint_as_float(t4.x); ui.zc = (int)t4.y; ui.j0 = (int)t4.z; ui.nvalid = (int)t4.w;
            }
            uint32_t w[BITS == 3 ? 4 : BITS];
#pragma unroll
            for (int i = 0; i < (BITS == 3 ? 4 : BITS); ++i) w[i] = 0u;
#pragma unroll
            for (int e = 0; e < 32; ++e) {
                const uint32_t sidx = (srcp[e >> 1] >> (16 * (e & 1))) & 0xFFFFu;
                const float yv = ybuf[sidx];
                const uint32_t q = (uint32_t)quant_code(yv, ui.inv_s, ui.zc, qmax);
                if (y_dbg != nullptr && e < ui.nvalid) y_dbg[(int64_t)m * C + ui.j0 + e] = yv;
                if constexpr (BITS == 8) {
                    w[e >> 2] |= q << (8 * (e & 3));
                } else {
                    const int t = e & 7;
                    w[e >> 3] |= q << (8 * (t & 3) + 4 * (t >> 2));   // for BITS == 3, w[3] collects codes 24..31
                }
            }
            if constexpr (BITS == 8) {
                uint4* dst = reinterpret_cast<uint4*>(out_row + u * 32);
                dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
            } else if constexpr (BITS == 4) {
                *reinterpret_cast<uint4*>(out_row + u * 16) = make_uint4(w[0], w[1], w[2], w[3]);
            } else {
                uint32_t* dst = reinterpret_cast<uint32_t*>(out_row + u * 12);
#pragma unroll
                for (int j = 0; j < 3; ++j) dst[j] = w[j] | (((w[3] >> j) & 0x11111111u) << 3);
            }
        }
        // no barrier here: the next row writes the other half of the double buffers, and the two
        // barriers of that row order this row's gather before anything overwrites its buffers
    }
}

using KernelFn = void (*)(const __half*, int64_t, const __half*, const __half*, float, int, int, int,
                          const uint16_t*, const UnitInfo*, uint8_t*, int64_t, float*);

template <int BITS>
static KernelFn pick_kernel(int nch)
{
    switch (nch) {
        case 1: return ln_reorder_quant_kernel<1, BITS>;
        case 2: return ln_reorder_quant_kernel<2, BITS>;
        case 3: return ln_reorder_quant_kernel<3, BITS>;
        case 4: return ln_reorder_quant_kernel<4, BITS>;
        case 5: case 6: return ln_reorder_quant_kernel<6, BITS>;
        case 7: case 8: return ln_reorder_quant_kernel<8, BITS>;
        default: return ln_reorder_quant_kernel<16, BITS>;
    }
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
    if (L->C > 16384) return RPTQ_ERR_UNSUPPORTED;      // the normalised row must fit in shared memory twice
    if (M == 0) return RPTQ_OK;

    int dev = -1;
    if (L->device < 0 || cudaGetDevice(&dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (dev != L->device) return RPTQ_ERR_INVALID_ARG;

    const int n_chunks = L->C / 8;
    int T = 512;
    for (int cand : {128, 256, 384, 512})
        if (L->n_units <= cand) { T = cand; break; }
    // small rows: do not leave most of a wide block without a chunk to normalise
    while (T > 128 && n_chunks <= (T - 128) && L->n_units <= T - 128) T -= 128;
    int nch = (n_chunks + T - 1) / T;
    while (nch > 16 && T < 512) { T += 128; nch = (n_chunks + T - 1) / T; }
    if (nch > 16) return RPTQ_ERR_UNSUPPORTED;

    KernelFn fn = L->bits == 3 ? pick_kernel<3>(nch) : L->bits == 4 ? pick_kernel<4>(nch) : pick_kernel<8>(nch);
    const int ybuf_stride = (L->C + 4 + 3) & ~3;
    const size_t smem = (size_t)(2 * ybuf_stride + 128) * sizeof(float);
    if (cudaFuncSetAttribute(reinterpret_cast<const void*>(fn), cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return RPTQ_ERR_CUDA;
    int n_sm = 0, per_sm = 0;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, reinterpret_cast<const void*>(fn), T, smem) != cudaSuccess || per_sm < 1)
        return RPTQ_ERR_CUDA;
    const int grid = M < n_sm * per_sm ? M : n_sm * per_sm;
    fn<<<grid, T, smem, static_cast<cudaStream_t>(stream)>>>(
        static_cast<const __half*>(x), ldx, static_cast<const __half*>(gamma), static_cast<const __half*>(beta),
        eps, M, L->C, L->n_units, L->d_src, L->d_unit, static_cast<uint8_t*>(codes), L->row_bytes, y_dbg);
    return cudaGetLastError() == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}
