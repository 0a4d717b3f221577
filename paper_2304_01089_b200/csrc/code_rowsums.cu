// rptq_code_rowsums: per token and cluster, the sum of the activation codes over the cluster's
// positions, xsum[m][c] = sum_{k in S^c} X_q[m][k] -- the factor of the weight zero point in the
// second computation method of the Appendix (the term z^W_i sum_k X_q). One block per token row:
// every thread unpacks units of 32 codes, adds their bytes with dp4a and adds the unit's sum to
// its cluster's entry in shared memory. Pad positions hold code 0 and add nothing.
#include "rptq_internal.h"
#include "unpack.cuh"

namespace rptq {

template <int BITS>
__global__ void __launch_bounds__(128)
code_rowsums_kernel(const uint8_t* __restrict__ codes, int64_t row_bytes, int n_units,
                    const int32_t* __restrict__ unit_cluster, int g, int32_t* __restrict__ xsum)
{
    extern __shared__ int32_t s_sum[];
    for (int c = threadIdx.x; c < g; c += blockDim.x) s_sum[c] = 0;
    __syncthreads();
    const uint32_t* row = reinterpret_cast<const uint32_t*>(codes + (int64_t)blockIdx.x * row_bytes);
    for (int u = threadIdx.x; u < n_units; u += blockDim.x) {
        const int c = __ldg(unit_cluster + u);
        if (c < 0) continue;
        uint32_t p[BITS], o[8];
#pragma unroll
        for (int i = 0; i < BITS; ++i) p[i] = __ldg(row + u * BITS + i);
        unpack_act32<BITS>(p, o);
        int s = 0;
#pragma unroll
        for (int i = 0; i < 8; ++i) s = (int)__dp4a(o[i], 0x01010101u, (unsigned)s);
        atomicAdd(&s_sum[c], s);
    }
    __syncthreads();
    for (int c = threadIdx.x; c < g; c += blockDim.x) xsum[(int64_t)blockIdx.x * g + c] = s_sum[c];
}

}  // namespace rptq

extern "C" int rptq_code_rowsums(const rptq_layout_t* L, const void* codes, int M, int32_t* xsum, void* stream)
{
    using namespace rptq;
    if (!L || !codes || !xsum || M < 0) return RPTQ_ERR_INVALID_ARG;
    if (!aligned16(codes) || !aligned16(xsum)) return RPTQ_ERR_INVALID_ARG;
    if (L->g > 8192) return RPTQ_ERR_UNSUPPORTED;
    if (M == 0) return RPTQ_OK;
    int dev = -1;
    if (L->device < 0 || cudaGetDevice(&dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (dev != L->device) return RPTQ_ERR_INVALID_ARG;
    auto st = static_cast<cudaStream_t>(stream);
    const size_t smem = sizeof(int32_t) * (size_t)L->g;
    const uint8_t* c = static_cast<const uint8_t*>(codes);
    if (L->bits == 3) code_rowsums_kernel<3><<<M, 128, smem, st>>>(c, L->row_bytes, L->n_units, L->d_unit_cluster, L->g, xsum);
    else if (L->bits == 4) code_rowsums_kernel<4><<<M, 128, smem, st>>>(c, L->row_bytes, L->n_units, L->d_unit_cluster, L->g, xsum);
    else code_rowsums_kernel<8><<<M, 128, smem, st>>>(c, L->row_bytes, L->n_units, L->d_unit_cluster, L->g, xsum);
    return cudaGetLastError() == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}
