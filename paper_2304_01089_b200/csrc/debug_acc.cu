// rptq_cluster_gemm_debug_acc: raw per-cluster integer accumulators of an output window
// (Appendix, second method: X~_q,c W~_q,c before de-quantisation), computed with plain integer
// dot-product instructions. A slow, independent-of-the-tensor-core cross-check and inspection aid.
#include "rptq_internal.h"
#include "unpack.cuh"

namespace rptq {

// four unsigned bytes times four signed bytes, accumulated
__device__ __forceinline__ int dp4a_u8_s8(uint32_t a, uint32_t b, int c)
{
    int d;
    asm("dp4a.u32.s32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}

template <int BITS>
__global__ void debug_acc_kernel(const uint8_t* __restrict__ a_codes, int64_t a_row_bytes,
                                 const uint8_t* __restrict__ w_codes, int n_kb,
                                 const int32_t* __restrict__ unit_cluster, int n_units, int m0, int m1, int n0, int n1,
                                 int32_t* __restrict__ acc)
{
    const int n = n0 + blockIdx.x * blockDim.x + threadIdx.x;
    const int m = m0 + blockIdx.y;
    const int c = blockIdx.z;
    if (n >= n1 || m >= m1) return;
    const uint32_t* arow = reinterpret_cast<const uint32_t*>(a_codes + (int64_t)m * a_row_bytes);
    int sum = 0;
    for (int s = 0; s < n_units; ++s) {
        if (unit_cluster[s] != c) continue;      // a cluster's steps need not be adjacent
        uint32_t ap[BITS], wp[4], a8[8], w8[8];
#pragma unroll
        for (int i = 0; i < BITS; ++i) ap[i] = arow[s * BITS + i];
#pragma unroll
        for (int i = 0; i < 4; ++i) wp[i] = reinterpret_cast<const uint32_t*>(w_codes + weight_tile_offset(n, s >> 2, n_kb) + (s & 3) * 16)[i];
        unpack_act32<BITS>(ap, a8);
        unpack_w32_x16(wp, w8);
#pragma unroll
        for (int i = 0; i < 8; ++i) sum = dp4a_u8_s8(a8[i], w8[i], sum);
    }
    acc[((int64_t)c * (m1 - m0) + (m - m0)) * (n1 - n0) + (n - n0)] = sum >> 4;   // operands were 16 * w
}

}  // namespace rptq

using namespace rptq;

extern "C" int rptq_cluster_gemm_debug_acc(const rptq_layout_t* Lin, const void* a_codes, int M, const void* w_codes,
                                           int N, int m0, int m1, int n0, int n1, int32_t* acc, void* stream)
{
    if (!Lin || !a_codes || !w_codes || !acc) return RPTQ_ERR_INVALID_ARG;
    if (m0 < 0 || m1 > M || m0 > m1 || n0 < 0 || n1 > N || n0 > n1) return RPTQ_ERR_INVALID_ARG;
    if (!aligned16(a_codes) || !aligned16(w_codes)) return RPTQ_ERR_INVALID_ARG;
    int dev = -1;
    if (Lin->device < 0 || cudaGetDevice(&dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (dev != Lin->device) return RPTQ_ERR_INVALID_ARG;
    if (m0 == m1 || n0 == n1) return RPTQ_OK;
    if (m1 - m0 > 65535 || Lin->g > 65535) return RPTQ_ERR_UNSUPPORTED;
    if (!Lin->d_unit_cluster) return RPTQ_ERR_CUDA;
    dim3 block(128), grid((n1 - n0 + 127) / 128, m1 - m0, Lin->g);
    auto st = static_cast<cudaStream_t>(stream);
    const auto* a = static_cast<const uint8_t*>(a_codes);
    const auto* w = static_cast<const uint8_t*>(w_codes);
    const int wrb = Lin->K_pad / 128;      // K blocks per row of the tile-major weight buffer
    if (Lin->bits == 3) debug_acc_kernel<3><<<grid, block, 0, st>>>(a, Lin->row_bytes, w, wrb, Lin->d_unit_cluster, Lin->n_units, m0, m1, n0, n1, acc);
    else if (Lin->bits == 4) debug_acc_kernel<4><<<grid, block, 0, st>>>(a, Lin->row_bytes, w, wrb, Lin->d_unit_cluster, Lin->n_units, m0, m1, n0, n1, acc);
    else debug_acc_kernel<8><<<grid, block, 0, st>>>(a, Lin->row_bytes, w, wrb, Lin->d_unit_cluster, Lin->n_units, m0, m1, n0, n1, acc);
    return cudaGetLastError() == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}
