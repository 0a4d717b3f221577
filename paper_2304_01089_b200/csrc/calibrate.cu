// Calibration on the device (Sec. 4.1): the per-channel ranges of Eq. 3 over the calibration tokens
// at a LayerNorm site, and the K-Means clustering of the channels on their (min, max) points.
// Off the hot path; written for exactness of the decisions, not for speed.
#include <cuda_fp16.h>

#include <cmath>

#include "rptq_internal.h"

namespace rptq {
namespace calib {

// ---------------------------------------------------------------- Eq. 3 at a LayerNorm output
__global__ void minmax_init_kernel(float* x_min, float* x_max, int C)
{
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c < C) { x_min[c] = INFINITY; x_max[c] = -INFINITY; }
}

__device__ __forceinline__ void atomic_min_float(float* addr, float v)
{
    // IEEE order equals integer order for non-negative floats and reversed unsigned order for negative ones
    if (v >= 0.f) atomicMin(reinterpret_cast<int*>(addr), __float_as_int(v));
    else atomicMax(reinterpret_cast<unsigned int*>(addr), __float_as_uint(v));
}
__device__ __forceinline__ void atomic_max_float(float* addr, float v)
{
    if (v >= 0.f) atomicMax(reinterpret_cast<int*>(addr), __float_as_int(v));
    else atomicMin(reinterpret_cast<unsigned int*>(addr), __float_as_uint(v));
}

__device__ __forceinline__ float block_sum(float v, float* red)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();                       // red may still be read from the previous call
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += red[w];
    return t;
}

// One block walks token rows blockIdx.x, blockIdx.x + gridDim.x, ...: LayerNorm in fp32 (the
// arithmetic of the quantising kernel: mean, centred variance, y = ((x rstd - mean rstd) gain + bias)),
// running minimum and maximum of every channel in shared memory (each thread owns its channels),
// merged into the global arrays with ordered-integer atomics at the end.
__global__ void __launch_bounds__(256)
ln_minmax_kernel(const __half* __restrict__ x, int64_t ldx, const __half* __restrict__ gamma, const __half* __restrict__ beta,
                 float eps, int T, int C, float* __restrict__ x_min, float* __restrict__ x_max)
{
    extern __shared__ float sm[];
    float* s_min = sm;
    float* s_max = sm + C;
    float* red = sm + 2 * C;                                   // 8 floats
    __half* s_row = reinterpret_cast<__half*>(sm + 2 * C + 8);
    for (int c = threadIdx.x; c < C; c += blockDim.x) { s_min[c] = INFINITY; s_max[c] = -INFINITY; }
    const float inv_C = 1.0f / (float)C;
    for (int t = blockIdx.x; t < T; t += gridDim.x) {
        const __half* row = x + (int64_t)t * ldx;
        __syncthreads();                                       // the previous row is no longer read
        float s = 0.f;
        for (int c = threadIdx.x; c < C; c += blockDim.x) { const __half h = row[c]; s_row[c] = h; s += __half2float(h); }
        const float mu = block_sum(s, red) * inv_C;
        float q = 0.f;
        for (int c = threadIdx.x; c < C; c += blockDim.x) { const float d = __half2float(s_row[c]) - mu; q = __fmaf_rn(d, d, q); }
        const float var = block_sum(q, red) * inv_C;
        const float rstd = 1.0f / sqrtf(var + eps), nm = -mu * rstd;
        for (int c = threadIdx.x; c < C; c += blockDim.x) {
            const float y = __fmaf_rn(__fmaf_rn(__half2float(s_row[c]), rstd, nm), __half2float(gamma[c]), __half2float(beta[c]));
            s_min[c] = fminf(s_min[c], y);
            s_max[c] = fmaxf(s_max[c], y);
        }
    }
    for (int c = threadIdx.x; c < C; c += blockDim.x) {
        if (s_min[c] <= s_max[c]) { atomic_min_float(x_min + c, s_min[c]); atomic_max_float(x_max + c, s_max[c]); }
    }
}

// ---------------------------------------------------------------- K-Means (Sec. 4.1)
// One block. Every decision is taken in the order and arithmetic of a plain sequential program
// (fp64, no fused multiply-add, running sums in point order), so a CPU implementation of the same
// steps gives the same labels: k-means++ seeding driven by the caller's uniform draws, then Lloyd
// iterations with squared Euclidean distance, ties to the lowest centre, an empty centre re-seeded at
// the point farthest from its own centre. Distances are computed by all threads; the running sums
// that pick a seed, the inertia and the re-seeding run in one thread; centre c is updated by thread c.
__device__ __forceinline__ double dist2(const double* __restrict__ p, const double* __restrict__ c, int dim)
{
    double d = 0.0;
    for (int a = 0; a < dim; ++a) {
        const double t = __dsub_rn(p[a], c[a]);
        d = __dadd_rn(d, __dmul_rn(t, t));
    }
    return d;
}

__global__ void __launch_bounds__(1024)
kmeans_kernel(const double* __restrict__ pts, int n, int dim, int g, const double* __restrict__ u, int iters,
              int32_t* __restrict__ labels, double* __restrict__ centres, double* __restrict__ inertia,
              double* __restrict__ d2, int32_t* __restrict__ count)
{
    __shared__ int s_pick;
    const int tid = threadIdx.x, nt = blockDim.x;
    // seeding
    if (tid == 0) {
        int first = (int)floor(u[0] * n);
        if (first >= n) first = n - 1;
        for (int a = 0; a < dim; ++a) centres[a] = pts[(size_t)first * dim + a];
    }
    for (int i = tid; i < n; i += nt) d2[i] = INFINITY;
    __syncthreads();
    for (int k = 1; k < g; ++k) {
        for (int i = tid; i < n; i += nt) {
            const double d = dist2(pts + (size_t)i * dim, centres + (size_t)(k - 1) * dim, dim);
            if (d < d2[i]) d2[i] = d;
        }
        __syncthreads();
        if (tid == 0) {
            double total = 0.0;
            for (int i = 0; i < n; ++i) total = __dadd_rn(total, d2[i]);
            const double target = __dmul_rn(u[k], total);
            double run = 0.0;
            int pick = n - 1;
            for (int i = 0; i < n; ++i) {
                run = __dadd_rn(run, d2[i]);
                if (run > target) { pick = i; break; }
            }
            s_pick = pick;
        }
        __syncthreads();
        if (tid < dim) centres[(size_t)k * dim + tid] = pts[(size_t)s_pick * dim + tid];
        __syncthreads();
    }
    for (int it = 0; it < iters; ++it) {
        // assignment
        for (int i = tid; i < n; i += nt) {
            double best = INFINITY;
            int bk = 0;
            for (int k = 0; k < g; ++k) {
                const double d = dist2(pts + (size_t)i * dim, centres + (size_t)k * dim, dim);
                if (d < best) { best = d; bk = k; }
            }
            labels[i] = bk;
            d2[i] = best;
        }
        for (int k = tid; k < g; k += nt) count[k] = 0;
        __syncthreads();
        if (tid == 0) {
            double total = 0.0;
            for (int i = 0; i < n; ++i) { total = __dadd_rn(total, d2[i]); count[labels[i]]++; }
            if (inertia) inertia[it] = total;
            // re-seed empty centres at the farthest point, one at a time
            for (int k = 0; k < g; ++k) {
                if (count[k] != 0) continue;
                int far = -1;
                double fd = -1.0;
                for (int i = 0; i < n; ++i)
                    if (count[labels[i]] > 1 && d2[i] > fd) { fd = d2[i]; far = i; }
                if (far < 0) continue;              // fewer distinct points than centres
                count[labels[far]]--;
                labels[far] = k;
                count[k] = 1;
                d2[far] = 0.0;
            }
        }
        __syncthreads();
        // update: centre k is the mean of its points, summed in point order
        for (int k = tid; k < g; k += nt) {
            if (count[k] == 0) continue;
            for (int a = 0; a < dim; ++a) {
                double sum = 0.0;
                for (int i = 0; i < n; ++i)
                    if (labels[i] == k) sum = __dadd_rn(sum, pts[(size_t)i * dim + a]);
                centres[(size_t)k * dim + a] = __ddiv_rn(sum, (double)count[k]);
            }
        }
        __syncthreads();
    }
}

}  // namespace calib
}  // namespace rptq

using namespace rptq;

extern "C" int rptq_ln_channel_minmax(const void* x, int64_t ldx, const void* gamma, const void* beta, float eps,
                                      int T, int C, float* x_min, float* x_max, void* stream)
{
    if (!x || !gamma || !beta || !x_min || !x_max) return RPTQ_ERR_INVALID_ARG;
    if (T < 0 || C <= 0 || ldx < C || !(eps >= 0.0f)) return RPTQ_ERR_INVALID_ARG;
    if (C > 16384) return RPTQ_ERR_UNSUPPORTED;          // the running ranges of a block live in shared memory
    auto st = static_cast<cudaStream_t>(stream);
    calib::minmax_init_kernel<<<(C + 255) / 256, 256, 0, st>>>(x_min, x_max, C);
    if (cudaGetLastError() != cudaSuccess) return RPTQ_ERR_CUDA;
    if (T == 0) return RPTQ_OK;
    int dev = -1, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    const size_t smem = sizeof(float) * (2 * (size_t)C + 8) + sizeof(__half) * (size_t)C;
    if (cudaFuncSetAttribute(calib::ln_minmax_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return RPTQ_ERR_CUDA;
    const int blocks = T < n_sm ? T : n_sm;
    calib::ln_minmax_kernel<<<blocks, 256, smem, st>>>(static_cast<const __half*>(x), ldx, static_cast<const __half*>(gamma),
                                                      static_cast<const __half*>(beta), eps, T, C, x_min, x_max);
    return cudaGetLastError() == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}

extern "C" int64_t rptq_kmeans_workspace_bytes(int n, int g)
{
    if (n <= 0 || g <= 0) return RPTQ_ERR_INVALID_ARG;
    return (int64_t)sizeof(double) * n + (int64_t)sizeof(int32_t) * ((g + 1) / 2 * 2);
}

extern "C" int rptq_kmeans(const double* pts, int n, int dim, int g, const double* u, int iters, int32_t* labels,
                           double* centres, double* inertia, void* workspace, void* stream)
{
    if (!pts || !u || !labels || !centres || !workspace) return RPTQ_ERR_INVALID_ARG;
    if (n <= 0 || g <= 0 || iters < 0 || dim < 1 || dim > 8) return RPTQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(workspace) & 7u) != 0) return RPTQ_ERR_INVALID_ARG;
    double* d2 = static_cast<double*>(workspace);
    int32_t* count = reinterpret_cast<int32_t*>(d2 + n);
    calib::kmeans_kernel<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(pts, n, dim, g, u, iters, labels, centres, inertia, d2, count);
    return cudaGetLastError() == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}
