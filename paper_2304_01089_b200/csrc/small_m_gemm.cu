// The cluster GEMM for at most 16 tokens (decoding): Appendix, second computation method, with the
// same arithmetic as the tcgen05 kernel of cluster_gemm.cu -- exact integer sums per cluster, the
// same fp32 fused multiply-adds in the same order afterwards -- so a token's result does not depend
// on which of the two kernels computed it.
//
// With so few tokens the product is bound by reading the packed weights once (N * K_pad / 2 bytes);
// the 128 x 256 tensor-memory tile of the large kernel would be almost empty and its unpacking of
// the weights to bytes in shared memory costs more than the reading. Here:
//   - a block owns 256 output channels (two 128-row weight tiles). A producer warp streams their
//     8 KiB tiles, K block after K block, into an eight-stage shared-memory ring with cp.async.bulk
//     (ordinary loads keep too few bytes in flight per SM to fill the memory pipe with a read-only
//     stream);
//   - the tokens' codes sit in shared memory as 4-bit nibbles in the packed format of the 4-bit
//     codes (16 x K_pad / 2 bytes), written once per block;
//   - each of the 16 consumer warps owns 16 channels (weight rows) for the whole contraction and
//     multiplies with mma.sync m16n8k32: the weight rows are the instruction's M dimension (signed
//     8-bit operands = 16 w, as in the large kernel, three logic instructions per operand pair), the
//     tokens its N dimension (unsigned 8-bit), so the per-channel constants of the epilogue are
//     per-thread scalars. Lane (g, t) reads the 16 bytes of unit t of rows g and g + 8 of the K
//     block; instruction j of the block's four takes word j of every lane, i.e. positions 8j..8j+7
//     of all four units.
//   - an instruction therefore mixes the block's four units. Where they belong to one cluster (most
//     blocks) that is the cluster's sum; where a block holds several clusters, it is multiplied once
//     per cluster with the other clusters' lanes zeroed ("passes", prepared per K block when the
//     kernel starts, in the order in which the clusters end).
#include <cuda_fp16.h>

#include "rptq_internal.h"
#include "unpack.cuh"

namespace rptq {
namespace smallm {

constexpr int CONSUMER_WARPS = 16;
constexpr int THREADS = 32 * (CONSUMER_WARPS + 1);
constexpr int STAGES = 8;
constexpr int STAGE_BYTES = 16384;          // two 8 KiB weight tiles: K block kb of both 128-row tiles
constexpr long long WAIT_BUDGET_CYCLES = 4000000000ll;   // about two seconds

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool mbar_try_wait_for(uint32_t bar, uint32_t parity, uint32_t ns)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
// Bounded wait: false when the budget ran out or another wait of the block already gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    if (mbar_try_wait_for(bar, parity, 0u)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait_for(bar, parity, 2000u)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > WAIT_BUDGET_CYCLES) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ void mma_s8u8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.u8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// One pass of a K block: which of its four units take part (bits 0..3), the accumulator (bit 4), whether the
// cluster ends in this block (bit 5), and the cluster's s_c / 16.
struct Pass { uint32_t ctrl; float sc; };
constexpr uint32_t PASS_BUF = 16u, PASS_LAST = 32u;

template <int BITS, int NT>
__global__ void __launch_bounds__(THREADS, 1)
small_m_kernel(const SmallMParams p)
{
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 127u) & ~127u;
    uint8_t* smem = smem_raw + (base - smem_u32(smem_raw));
    // ring | token codes (nibbles) | passes | barriers
    const int a_pitch = p.K_pad / 2 + (((p.K_pad / 2) & 127) ? 0 : 64);      // odd multiple of 64: two token rows fill the 32 banks
    uint8_t* ring = smem;
    uint8_t* act = ring + STAGES * STAGE_BYTES;
    Pass* passes = reinterpret_cast<Pass*>(act + 8 * NT * a_pitch);          // [n_kb][4]
    uint64_t* bars = reinterpret_cast<uint64_t*>(passes + 4 * p.n_kb);       // full[STAGES], empty[STAGES]
    __shared__ int s_abort_flag;
    volatile int* s_abort = &s_abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g8 = lane >> 2, t4 = lane & 3;
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + STAGES);

    if (tid == 0) {
        s_abort_flag = 0;
        for (int s = 0; s < STAGES; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(full0 + 8 * s) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(empty0 + 8 * s), "r"(CONSUMER_WARPS) : "memory");
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int tileA = 2 * (int)blockIdx.x;
    const bool haveB = tileA + 1 < p.n_wtiles;

    float R[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt)
#pragma unroll
        for (int e = 0; e < 4; ++e) R[nt][e] = 0.f;

    if (warp == CONSUMER_WARPS) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            const uint8_t* srcA = p.w + (int64_t)tileA * p.n_kb * 8192;
            const uint8_t* srcB = srcA + (int64_t)p.n_kb * 8192;
            const uint32_t bytes = haveB ? STAGE_BYTES : STAGE_BYTES / 2;
            int issued = 0;
            for (int kb = 0; kb < p.n_kb; ++kb) {
                const int s = kb % STAGES;
                if (kb >= STAGES && !mbar_wait(empty0 + 8 * s, (uint32_t)(kb / STAGES - 1) & 1u, s_abort)) break;
                if (*s_abort) break;
                const uint32_t dst = smem_u32(ring + s * STAGE_BYTES), bar = full0 + 8 * s;
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(dst), "l"(srcA + (int64_t)kb * 8192), "r"(8192), "r"(bar) : "memory");
                if (haveB)
                    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                                 ::"r"(dst + 8192), "l"(srcB + (int64_t)kb * 8192), "r"(8192), "r"(bar) : "memory");
                issued = kb + 1;
            }
            // After a give-up the consumers no longer wait for the copies still in flight: they must have
            // landed before the block's shared memory goes away (bounded like every other wait).
            if (*s_abort) {
                const long long t0 = clock64();
                for (int kb = issued > STAGES ? issued - STAGES : 0; kb < issued; ++kb)
                    while (!mbar_try_wait_for(full0 + 8 * (kb % STAGES), (uint32_t)(kb / STAGES) & 1u, 2000u) && clock64() - t0 <= WAIT_BUDGET_CYCLES) {}
            }
        }
    } else {
        // ------------------------------------------------------------ consumers
        // (the producer is already streaming weights while the consumers prepare their tables)
        // the tokens' codes as nibbles: word i of a unit holds positions 8i..8i+3 in the low and 8i+4..8i+7
        // in the high nibbles of its bytes (the packed format of 4-bit codes); rows >= M are zero
        for (int it = tid; it < 8 * NT * p.n_units; it += 32 * CONSUMER_WARPS) {
            const int r = it / p.n_units, u = it - r * p.n_units;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (r < p.M) {
                const uint8_t* row = p.a + (int64_t)r * p.a_row_bytes;
                if constexpr (BITS == 4) {
                    v = __ldg(reinterpret_cast<const uint4*>(row) + u);
                } else {
                    const uint32_t* w = reinterpret_cast<const uint32_t*>(row) + u * 3;
                    const uint32_t q[3] = {__ldg(w), __ldg(w + 1), __ldg(w + 2)};
                    uint32_t o[8];
                    unpack_act32<3>(q, o);
                    v = make_uint4(o[0] | (o[1] << 4), o[2] | (o[3] << 4), o[4] | (o[5] << 4), o[6] | (o[7] << 4));
                }
            }
            *reinterpret_cast<uint4*>(act + r * a_pitch + 16 * u) = v;
        }
        // the passes of every K block
        for (int kb = tid; kb < p.n_kb; kb += 32 * CONSUMER_WARPS) {
            int cl[4]; uint32_t ctrl[4]; float sc[4]; int lastpos[4]; int n = 0;
            for (int ul = 0; ul < 4; ++ul) {
                const int u = 4 * kb + ul;
                const int fl = __ldg(p.step_flags + u);
                if (fl & STEP_SKIP) continue;
                const int c = __ldg(p.unit_cluster + u);
                int k = 0;
                while (k < n && cl[k] != c) ++k;
                if (k == n) { cl[n] = c; ctrl[n] = (fl & STEP_BUF) ? PASS_BUF : 0u; sc[n] = __ldg(&p.unit_sz[u].x) * 0.0625f; lastpos[n] = 9; ++n; }
                ctrl[k] |= 1u << ul;
                if (fl & STEP_LAST) { ctrl[k] |= PASS_LAST; lastpos[k] = ul; }
            }
            for (int i = 1; i < n; ++i)                      // clusters that end here first, in the order they end
                for (int j = i; j > 0 && lastpos[j] < lastpos[j - 1]; --j) {
                    const int tc = cl[j]; cl[j] = cl[j - 1]; cl[j - 1] = tc;
                    const uint32_t tt = ctrl[j]; ctrl[j] = ctrl[j - 1]; ctrl[j - 1] = tt;
                    const float ts = sc[j]; sc[j] = sc[j - 1]; sc[j - 1] = ts;
                    const int tl = lastpos[j]; lastpos[j] = lastpos[j - 1]; lastpos[j - 1] = tl;
                }
            for (int i = 0; i < 4; ++i) passes[4 * kb + i] = Pass{i < n ? ctrl[i] : 0u, i < n ? sc[i] : 0.f};
        }
        asm volatile("bar.sync 1, %0;" ::"n"(32 * CONSUMER_WARPS) : "memory");
        const int tile_sel = warp >> 3;                       // which of the block's two tiles
        const bool active = tile_sel == 0 || haveB;
        const uint8_t* wrow = ring + tile_sel * 8192 + (16 * (warp & 7) + g8) * 64 + 16 * t4;
        const uint8_t* arow = act + g8 * a_pitch + 16 * t4;
        int acc0[2][NT][4], acc1[2][NT][4];                   // [instruction parity][token tile]: two accumulators per buffer
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) { acc0[h][nt][e] = 0; acc1[h][nt][e] = 0; }

        for (int kb = 0; kb < p.n_kb; ++kb) {
            const int s = kb % STAGES;
            if (!mbar_wait(full0 + 8 * s, (uint32_t)(kb / STAGES) & 1u, s_abort)) break;
            uint4 X0 = make_uint4(0, 0, 0, 0), X1 = X0;
            if (active) {
                X0 = *reinterpret_cast<const uint4*>(wrow + s * STAGE_BYTES);
                X1 = *reinterpret_cast<const uint4*>(wrow + s * STAGE_BYTES + 512);
            }
            uint4 B[NT];
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) B[nt] = *reinterpret_cast<const uint4*>(arow + 8 * nt * a_pitch + 64 * kb);
            const uint4 ps01 = *reinterpret_cast<const uint4*>(passes + 4 * kb);
            const uint4 ps23 = *reinterpret_cast<const uint4*>(passes + 4 * kb + 2);
            __syncwarp();
            if (lane == 0) mbar_arrive(empty0 + 8 * s);       // the stage's bytes are in registers
            const uint32_t xw0[4] = {X0.x, X0.y, X0.z, X0.w}, xw1[4] = {X1.x, X1.y, X1.z, X1.w};
            const uint32_t ctrls[4] = {ps01.x, ps01.z, ps23.x, ps23.z};
            const float scs[4] = {__uint_as_float(ps01.y), __uint_as_float(ps01.w), __uint_as_float(ps23.y), __uint_as_float(ps23.w)};
            uint32_t bw[NT][4][2];                            // the tokens' bytes for instruction j: positions 8j..8j+3, 8j+4..8j+7
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                const uint32_t w[4] = {B[nt].x, B[nt].y, B[nt].z, B[nt].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) { bw[nt][j][0] = w[j] & 0x0F0F0F0Fu; bw[nt][j][1] = (w[j] >> 4) & 0x0F0F0F0Fu; }
            }
#pragma unroll
            for (int ps = 0; ps < 4; ++ps) {
                const uint32_t ctrl = ctrls[ps];
                if ((ctrl & 15u) == 0u) break;
                const uint32_t keep = 0u - ((ctrl >> t4) & 1u);            // all ones where my unit belongs to the pass's cluster
                const uint32_t m_lo = 0xF0F0F0F0u & keep;
                uint32_t aw[4][4];                                         // the four instructions' weight operands
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    aw[j][0] = (xw0[j] << 4) & m_lo; aw[j][2] = xw0[j] & m_lo;
                    aw[j][1] = (xw1[j] << 4) & m_lo; aw[j][3] = xw1[j] & m_lo;
                }
                const float sc = scs[ps];
                auto run = [&](int (&acc)[2][NT][4]) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
                            mma_s8u8(acc[j & 1][nt], aw[j][0], aw[j][1], aw[j][2], aw[j][3], bw[nt][j][0], bw[nt][j][1]);
                    if (ctrl & PASS_LAST) {
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                R[nt][e] = __fmaf_rn(sc, (float)(acc[0][nt][e] + acc[1][nt][e]), R[nt][e]);
                                acc[0][nt][e] = 0; acc[1][nt][e] = 0;
                            }
                    }
                };
                if (ctrl & PASS_BUF) run(acc1); else run(acc0);
            }
        }

        // -------------------------------------------------------- epilogue: y = s_w (R - corr) + bias
        const int n0 = (tileA + tile_sel) * 128 + 16 * (warp & 7);
        if (active && n0 < p.N && !*s_abort) {
            float corr = 0.f, sw = 0.f, bs = 0.f;      // lanes 0..15 each take one of the warp's channels
            const int nl = n0 + (lane & 15);
            if (lane < 16 && nl < p.N) {
                if (p.corr) corr = __ldg(p.corr + nl);
                else for (int c = 0; c < p.g; ++c) corr = __fmaf_rn(__ldg(p.cl_sz + c), (float)__ldg(p.wsum + (int64_t)c * p.ld_w + nl), corr);
                sw = __ldg(p.s_w + nl);
                bs = p.bias ? __ldg(p.bias + nl) : 0.f;
            }
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {             // rows g (accumulator entries 0, 1) and g + 8 (entries 2, 3)
                const int src = g8 + 8 * hh, n = n0 + src;
                const float c = __shfl_sync(0xffffffffu, corr, src), s = __shfl_sync(0xffffffffu, sw, src), b = __shfl_sync(0xffffffffu, bs, src);
                if (n >= p.N) continue;
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const int m = 8 * nt + 2 * t4 + e;
                        if (m >= p.M) continue;
                        float v = __fmaf_rn(s, R[nt][2 * hh + e] - c, b);
                        if (p.act == RPTQ_ACT_RELU) v = fmaxf(v, 0.f);
                        if (p.y_dtype == RPTQ_OUT_F32) static_cast<float*>(p.y)[(int64_t)m * p.ldy + n] = v;
                        else static_cast<__half*>(p.y)[(int64_t)m * p.ldy + n] = __float2half_rn(v);
                    }
            }
        }
    }
    __syncthreads();
    if (tid == 0 && *s_abort && p.status) atomicExch(p.status, RPTQ_ERR_DEVICE_TIMEOUT);
}

static int smem_bytes(int nt, int K_pad)
{
    const int a_pitch = K_pad / 2 + (((K_pad / 2) & 127) ? 0 : 64);
    return 128 + STAGES * STAGE_BYTES + 8 * nt * a_pitch + (K_pad / 128) * 4 * (int)sizeof(Pass) + 2 * STAGES * 8;
}

template <int BITS, int NT>
static int launch_one(const SmallMParams& p, cudaStream_t st)
{
    const int smem = smem_bytes(NT, p.K_pad);
    if (cudaFuncSetAttribute(small_m_kernel<BITS, NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return RPTQ_ERR_CUDA;
    const int blocks = (p.n_wtiles + 1) / 2;
    small_m_kernel<BITS, NT><<<blocks, THREADS, smem, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}

bool fits(int M, int bits, int K_pad)
{
    return M <= 16 && (bits == 3 || bits == 4) && smem_bytes(M <= 8 ? 1 : 2, K_pad) <= 226 * 1024;
}

int launch(const SmallMParams& p, int bits, cudaStream_t st)
{
    if (p.M <= 8) return bits == 3 ? launch_one<3, 1>(p, st) : launch_one<4, 1>(p, st);
    return bits == 3 ? launch_one<3, 2>(p, st) : launch_one<4, 2>(p, st);
}

}  // namespace smallm
}  // namespace rptq
