// rptq_ln_reorder_quant: LayerNorm with the channel reorder fused in (Sec. 4.2), followed by the
// per-cluster quantiser (Eq. 1 applied per cluster, Appendix) and packed stores.
//
// The paper scatters on write (Sec. 4.2: LayerNorm's write address carries the reorder index).
// Packed sub-byte codes need whole words written at once, so here every thread gathers the
// 32 channels of one output unit (32 consecutive padded positions, always inside one cluster)
// straight from the raw fp16 row in shared memory, normalises them with the row's statistics and
// its own channels' gains and biases (held in registers across rows), quantises them with the
// cluster's parameters and stores 12/16/32 contiguous bytes.
//
// The quantiser decision (Eq. 1: round(x / s) + z, clamped) costs one fused multiply-add and half a
// saturating pack instruction per element. The LayerNorm output is carried scaled by 2^-100 (gains
// and biases are scaled once per launch; exact), the reciprocal step by 2^-49, the zero point by
// 2^-149: t = fma(y 2^-100, 2^-49 / s, z 2^-149) is then a multiple of the smallest subnormal, the
// sum is rounded once, half to even, at exactly the integer grid of y / s + z, and the bit pattern
// of t IS the integer rne(y / s) + z for every result in [0, 2^24) -- larger results keep their
// order, negative ones have the sign bit set, so the saturating pack clamps every finite input to
// the right end. Adding z before the rounding moves exact ties only when z is odd; units with an odd
// zero point therefore compute the mirrored code qmax - q = clamp(rne(-y / s) + (qmax - z)) (the offset
// is even again) and flip the packed bits afterwards.
//
// Memory-bound by design. A block is persistent over rows. Rows arrive through a ring of
// shared-memory slots that the copy engine fills many rows ahead; a few warps compute each row's
// mean and variance (one warp per row, no block-wide barrier); the gather warps follow. The
// hand-offs are mbarriers per ring slot: landed -> statistics ready -> slot free.
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
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c)
{
    float2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(reinterpret_cast<uint64_t&>(d))
        : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)), "l"(reinterpret_cast<uint64_t&>(c)));
    return d;
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
// The same test, but the warp may stay suspended in the instruction for up to `ns` nanoseconds
// while the phase has not completed (it wakes up when it does).
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
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
constexpr long long kLnWaitBudgetCycles = 4000000000ll;   // about two seconds at the SM clock

// Bounded wait. A warp that has to wait sleeps inside the barrier instruction (a few microseconds
// at a time) instead of polling: the waiting roles would otherwise take a fifth of the block's
// issue slots. When the budget runs out the status word is set, every later wait in the block
// returns at once, and the caller carries on with whatever the slot holds: the loops have fixed
// trip counts, so the kernel still ends.
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status,
                                          long long budget = kLnWaitBudgetCycles)
{
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
#pragma unroll 1
    while (true) {
        if (mbar_try_wait_for(bar, parity, 4000u)) return;
        if (*abort_flag) return;
        if (clock64() - t0 > budget) {
            *abort_flag = 1;
            if (status) atomicExch(status, RPTQ_ERR_DEVICE_TIMEOUT);
            return;
        }
    }
}

// Parameters of the self-test variant only (rptq_selftest_ln_timeout sets them before its launch). They live here
// and not in LnParams: two more fields there cost the 3-bit kernel spills in its gather loop.
__constant__ long long c_selftest_wait_budget;     // cycles a wait may take before the block gives up
__constant__ uint32_t c_selftest_tx_extra;         // bytes a row's barrier expects beyond what its copy delivers

struct LnParams {
    const __half* x; int64_t ldx; const __half* gamma; const __half* beta; float eps;
    int M, C, n_units, n_stats_warps, depth, n_groups;
    const uint16_t* ch_tab;      // [K_pad] channel read for each padded position (pads: any channel, masked later)
    const int32_t* jidx_tab;     // [K_pad] reordered index of each padded position, -1 at pads (debug output)
    const UnitInfo* unit_tab;
    uint8_t* codes; int64_t row_bytes; float* y_dbg; int* status;
};

// Warp roles:
//   warp 0                 lane 0 keeps the ring full: one contiguous cp.async.bulk per row (at 18-24 KB
//                          a row, a few rows in flight per SM would leave HBM idle most of the time)
//   warps 1 .. S           statistics: a warp takes every S-th row, forms the sum and the sum of squares on
//                          the tensor cores (a centred second pass only for rows whose mean is far from
//                          zero) and publishes (rstd, -mean * rstd)
//   the other warps        gather: each thread owns one output unit. Its 32 source offsets, gains and
//                          biases stay in registers across rows; per row it reads its 32 raw fp16
//                          values, forms y = ((x * rstd - mean * rstd) * gain + bias) in fp32 (three
//                          fused multiply-adds per element, the last one being the quantiser decision),
//                          packs and stores 12/16/32 contiguous bytes
// Per ring slot three mbarriers hand the row over: landed (copy engine) -> ready (statistics) ->
// free (all gather warps), which lets the producer refill it.
// DBG adds the optional fp32 output of the reordered LayerNorm values (off the fast path).
// SELFTEST: the wait budget and the extra expected bytes come from constant memory (rptq_selftest_ln_timeout);
// otherwise they are compile-time constants.
template <int BITS, bool DBG, bool SELFTEST = false>
__global__ void __launch_bounds__(512)
ln_reorder_quant_kernel(const LnParams p)
{
    const long long wait_budget = SELFTEST ? c_selftest_wait_budget : kLnWaitBudgetCycles;
    const uint32_t tx_extra = SELFTEST ? c_selftest_tx_extra : 0u;
    extern __shared__ __align__(128) uint8_t smem_raw[];
    const int T = blockDim.x, C = p.C, D = p.depth, S = p.n_stats_warps;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t row_bytes_in = 2u * (uint32_t)C;
    const uint32_t pitch = row_bytes_in + 16u;            // 16 spare bytes keep successive slots 4 banks apart
    uint8_t* ring = smem_raw;
    float2* stats = reinterpret_cast<float2*>(ring + (size_t)D * pitch);
    uint8_t* zero16 = ring + (size_t)D * pitch + ((8 * (size_t)D + 15) & ~(size_t)15);   // 16 zero bytes, 16-byte aligned
    uint64_t* bars = reinterpret_cast<uint64_t*>(zero16 + 16);               // landed[D], ready[D], free[D], tables
    volatile int* s_abort = reinterpret_cast<volatile int*>(bars + 3 * D + 1);
    const uint32_t ring_s = (uint32_t)__cvta_generic_to_shared(ring);
    const uint32_t bar_s = (uint32_t)__cvta_generic_to_shared(bars);
    // The gather threads form n_groups groups of TG threads; group j takes rows j, j + n_groups, ...
    // (narrow layouts leave room for several groups, and a short row is mostly hand-over latency)
    const int G = p.n_groups, TG = (T - 32 * (1 + S)) / G, n_gather_warps = TG >> 5;
    const int n_rows = (p.M - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;   // rows of this block

    if (tid == 0) {
        for (int d = 0; d < D; ++d) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_s + 8 * d) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_s + 8 * (D + d)) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar_s + 8 * (2 * D + d)), "r"(n_gather_warps) : "memory");
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar_s + 8 * (3 * D)), "r"(G * n_gather_warps) : "memory");
        *s_abort = 0;
        *reinterpret_cast<uint4*>(zero16) = make_uint4(0u, 0u, 0u, 0u);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // Gains and biases pass through the last two ring slots (coalesced loads) so that the gather
    // threads can pick their own channels' values from shared memory; scattered 2-byte global loads
    // for 64 values per thread would cost more than a few hundred rows of the kernel proper. The
    // producer fills the other slots meanwhile and waits for the `tables` barrier before it reaches
    // these two.
    uint8_t* stage_g = ring + (size_t)(D - 2) * pitch;
    uint8_t* stage_b = ring + (size_t)(D - 1) * pitch;
    {
        uint4* g_s = reinterpret_cast<uint4*>(stage_g);
        uint4* b_s = reinterpret_cast<uint4*>(stage_b);
        for (int ch = tid; ch < (C >> 3); ch += T) {
            g_s[ch] = __ldg(reinterpret_cast<const uint4*>(p.gamma) + ch);
            b_s[ch] = __ldg(reinterpret_cast<const uint4*>(p.beta) + ch);
        }
    }
    __syncthreads();
    const __half* gamma_s = reinterpret_cast<const __half*>(stage_g);
    const __half* beta_s = reinterpret_cast<const __half*>(stage_b);
    const bool tables_in_regs = p.n_units <= TG;       // else the gather threads reload tables per unit, from global memory

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        if (lane == 0) {
            const int64_t row_step = (int64_t)gridDim.x * p.ldx;
            const __half* src = p.x + (int64_t)blockIdx.x * p.ldx;
            int d = 0, n_issued = 0;
            uint32_t par = 1;                // parity to wait for on free[d]: passes at once the first time round
            for (int k = 0; k < n_rows; ++k) {
                // the gather threads have taken their gains and biases out of the last two slots
                if (k == D - 2) mbar_wait(bar_s + 8 * (3 * D), 0u, s_abort, p.status, wait_budget);
                mbar_wait(bar_s + 8 * (2 * D + d), par, s_abort, p.status, wait_budget);
                if (*s_abort) break;         // a wait ran out somewhere in the block: issue nothing more
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_s + 8 * d), "r"(row_bytes_in + tx_extra) : "memory");
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(ring_s + d * pitch), "l"(src), "r"(row_bytes_in), "r"(bar_s + 8 * d) : "memory");
                src += row_step;
                ++n_issued;
                if (++d == D) { d = 0; par ^= 1u; }
            }
            // Every copy has landed before the block's shared memory goes away. Normally the statistics
            // warps have waited for each of them; after a give-up they no longer wait, so this lane
            // does, for the copies that may still be in flight (a bounded number of polls each).
            if (*s_abort) {
                for (int i = n_issued > D ? n_issued - D : 0; i < n_issued; ++i) {
                    const uint32_t b = bar_s + 8 * (i % D), ph = (uint32_t)(i / D) & 1u;
                    if constexpr (SELFTEST) {
                        const long long t0 = clock64();
                        while (!mbar_try_wait_for(b, ph, 4000u) && clock64() - t0 <= wait_budget) {}
                    } else {
                        for (int t = 0; t < (1 << 22) && !mbar_try_wait(b, ph); ++t) __nanosleep(64);
                    }
                }
            }
        }
    } else if (warp <= S) {
        // ------------------------------------------------------------ statistics warps
        // Sum and sum of squares of the row on the tensor cores (mma.sync m16n8k16, fp16 inputs, fp32
        // accumulators): 32 chunks of 8 values are one 16 x 16 operand A, whatever their arrangement;
        // A times a matrix of ones accumulates the sum, and A times its own upper (lower) eight rows as
        // the other operand puts the sums of squares of those rows on a diagonal. One shared-memory
        // instruction and three tensor instructions per 256 values replace some forty conversions
        // and additions per lane. fp16 products are exact in fp32; the variance is
        // sum(x^2) / C - mean^2, whose relative error grows with (mean / std)^2, so rows whose mean
        // is more than two standard deviations from zero take a second, centred pass (below).
        const int n_chunks = C >> 3;
        const float inv_C = 1.0f / (float)C;
        const uint32_t zero_s = (uint32_t)__cvta_generic_to_shared(zero16);
        for (int k = warp - 1; k < n_rows; k += S) {
            const int d = k % D;
            mbar_wait(bar_s + 8 * d, (uint32_t)(k / D) & 1u, s_abort, p.status, wait_budget);
            const uint32_t row_s = ring_s + (uint32_t)d * pitch;
            float cs[4] = {0.f, 0.f, 0.f, 0.f}, qa[4] = {0.f, 0.f, 0.f, 0.f}, qb[4] = {0.f, 0.f, 0.f, 0.f};
            const uint32_t ones = 0x3C003C00u;       // two fp16 ones
            auto tile = [&](uint32_t addr) {
                uint32_t a0, a1, a2, a3;
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                             : "=r"(a0), "=r"(a1), "=r"(a2), "=r"(a3) : "r"(addr));
                asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                             : "+f"(cs[0]), "+f"(cs[1]), "+f"(cs[2]), "+f"(cs[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(ones), "r"(ones));
                asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                             : "+f"(qa[0]), "+f"(qa[1]), "+f"(qa[2]), "+f"(qa[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(a0), "r"(a2));
                asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                             : "+f"(qb[0]), "+f"(qb[1]), "+f"(qb[2]), "+f"(qb[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(a1), "r"(a3));
            };
            // whole groups of 32 chunks (512 bytes per step), then the ragged end with zeros for the missing chunks
            const int n_full = n_chunks >> 5;
            uint32_t addr = row_s + 16u * (uint32_t)lane;
#pragma unroll 4
            for (int i = 0; i < n_full; ++i, addr += 512u) tile(addr);
            if (n_chunks & 31) tile((n_full << 5) + lane < n_chunks ? addr : zero_s);
            // accumulator fragment: c0, c1 = row lane / 4, columns 2 (lane % 4) + {0, 1}; c2, c3 = row lane / 4 + 8
            const int r = lane >> 2, cq = (lane & 3) * 2;
            const float my_sum = (lane & 3) == 0 ? cs[0] + cs[2] : 0.f;                 // column 0 of all 16 rows
            const float my_sq = (cq == r ? qa[0] : 0.f) + (cq + 1 == r ? qa[1] : 0.f)     // rows 0-7: D[i][i]
                              + (cq == r ? qb[2] : 0.f) + (cq + 1 == r ? qb[3] : 0.f);    // rows 8-15: D[8 + j][j]
            const float mu = warp_sum(my_sum) * inv_C;
            float var = fmaxf(warp_sum(my_sq) * inv_C - mu * mu, 0.f);
            if (mu * mu > 4.0f * var) {
                // The row's mean is more than two standard deviations from zero: sum(x^2)/C - mean^2
                // cancels too much (relative error ~ 1e-6 (1 + mean^2/var)). Take the centred sum of
                // squares instead, on the CUDA cores; rows of LayerNorm inputs rarely come here.
                const uint4* row = reinterpret_cast<const uint4*>(ring + (size_t)d * pitch);
                const float2 neg_mu = make_float2(-mu, -mu);
                float2 q2 = make_float2(0.f, 0.f), q2b = make_float2(0.f, 0.f);
#pragma unroll 2
                for (int ch = lane; ch < n_chunks; ch += 32) {
                    const uint4 raw = row[ch];
                    const __half2* h = reinterpret_cast<const __half2*>(&raw);
                    const float2 a = add2(__half22float2(h[0]), neg_mu), b = add2(__half22float2(h[1]), neg_mu);
                    const float2 c = add2(__half22float2(h[2]), neg_mu), e = add2(__half22float2(h[3]), neg_mu);
                    q2 = fma2(a, a, q2); q2b = fma2(b, b, q2b);
                    q2 = fma2(c, c, q2); q2b = fma2(e, e, q2b);
                }
                var = warp_sum((q2.x + q2.y) + (q2b.x + q2b.y)) * inv_C;
            }
            const float rstd = 1.0f / sqrtf(var + p.eps);
            if (lane == 0) {
                stats[d] = make_float2(rstd, -mu * rstd);
                mbar_arrive(bar_s + 8 * (D + d));            // release: the statistics are visible to whoever sees the phase
            }
        }
    } else {
        // ------------------------------------------------------------ gather warps
        const int grp = (tid - 32 * (1 + S)) / TG, gt = (tid - 32 * (1 + S)) - grp * TG;
        const bool one_unit = tables_in_regs;              // the fast case: my unit's tables stay in registers
        uint32_t off[32];                                  // shared-memory address of each source channel in ring slot 0
        float2 g2[16], b2[16];                             // gains and biases of source channels 2 i, 2 i + 1, times 2^-100
        float2 inv_s2 = make_float2(0.f, 0.f), z2 = make_float2(0.f, 0.f);   // +-2^-49 / s_c and the (even) offset times 2^-149, twice
        uint32_t flip = 0u;                                // all ones when the unit computes the mirrored code
        // packed words with all bits set at the unit's real positions (8-bit codes: the count of real
        // positions is enough, a byte mask per word is made on the spot for the few units that have pads)
        uint32_t keep[BITS == 8 ? 1 : BITS];
        constexpr int qmax = (1 << BITS) - 1;
        constexpr float k2m100 = 7.888609052210118e-31f;    // 2^-100
        constexpr float k2m49 = 1.7763568394002505e-15f;    // 2^-49
        auto load_unit = [&](int u, const __half* gamma, const __half* beta) {
            const uint4* sp = reinterpret_cast<const uint4*>(p.ch_tab + u * 32);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint4 v = __ldg(sp + i);
                const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t c0 = w[j] & 0xFFFFu, c1 = w[j] >> 16;
                    off[8 * i + 2 * j] = ring_s + 2u * c0;
                    off[8 * i + 2 * j + 1] = ring_s + 2u * c1;
                    g2[4 * i + j] = make_float2(__half2float(gamma[c0]) * k2m100, __half2float(gamma[c1]) * k2m100);
                    b2[4 * i + j] = make_float2(__half2float(beta[c0]) * k2m100, __half2float(beta[c1]) * k2m100);
                }
            }
            const uint4 t4 = __ldg(reinterpret_cast<const uint4*>(p.unit_tab + u));
            const int z = (int)t4.y + 0x4B400000, nvalid = (int)t4.w;
            const bool odd = (z & 1) != 0;
            const int z_even = odd ? qmax - z : z;
            const float inv_s_sc = (odd ? -__uint_as_float(t4.x) : __uint_as_float(t4.x)) * k2m49;
            // z_even * 2^-149: the subnormal whose fraction field is |z_even|
            const float z_sc = __uint_as_float(z_even >= 0 ? (uint32_t)z_even : (0x80000000u | (uint32_t)(-z_even)));
            inv_s2 = make_float2(inv_s_sc, inv_s_sc);
            z2 = make_float2(z_sc, z_sc);
            flip = odd ? 0xFFFFFFFFu : 0u;
            // pad positions read some real channel (the layout picks one that costs no bank conflict); their codes are masked to 0
            if constexpr (BITS == 8) {
                keep[0] = (uint32_t)nvalid;
            } else {
                uint32_t full[32];
#pragma unroll
                for (int e = 0; e < 32; ++e) full[e] = e < nvalid ? (uint32_t)qmax : 0u;
                pack32<BITS>(full, keep);
            }
        };
        if (one_unit && gt < p.n_units) load_unit(gt, gamma_s, beta_s);
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_s + 8 * (3 * D));
        // Every gather thread walks all of the block's rows with counters that do not depend on the
        // thread (slot, parity, whose turn it is), so the slot's base address is the same value in
        // every thread of the kernel's view; a group only works on its own rows.
        int d = 0, turn = 0;
        uint32_t par = 0;
        for (int k = 0; k < n_rows; ++k) {
            if (turn == grp) {
                mbar_wait(bar_s + 8 * (D + d), par, s_abort, p.status, wait_budget);
                const float2 st = stats[d];
                const float2 rs2 = make_float2(st.x, st.x), nm2 = make_float2(st.y, st.y);
                const uint32_t slot = (uint32_t)d * pitch;
                const int m = (int)blockIdx.x + k * (int)gridDim.x;
                uint8_t* out_row = p.codes + (int64_t)m * p.row_bytes;
                for (int u = gt; u < p.n_units; u += TG) {
                    if (!one_unit) load_unit(u, p.gamma, p.beta);
                    int q[32];                   // rne(y / s) + z (or its mirror), not yet clamped
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        uint16_t h0, h1;
                        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h0) : "r"(off[2 * i] + slot));
                        asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h1) : "r"(off[2 * i + 1] + slot));
                        const float2 xh = fma2(make_float2(__half2float(__ushort_as_half(h0)), __half2float(__ushort_as_half(h1))), rs2, nm2);
                        const float2 y = fma2(xh, g2[i], b2[i]);             // LayerNorm outputs times 2^-100
                        const float2 t = fma2(y, inv_s2, z2);                // the integers themselves (see the head of the file)
                        q[2 * i] = __float_as_int(t.x);
                        q[2 * i + 1] = __float_as_int(t.y);
                        if constexpr (DBG) {
                            const int ja = __ldg(p.jidx_tab + u * 32 + 2 * i), jb = __ldg(p.jidx_tab + u * 32 + 2 * i + 1);
                            if (ja >= 0) p.y_dbg[(int64_t)m * C + ja] = y.x * 1.2676506002282294e30f;   // times 2^100, exact
                            if (jb >= 0) p.y_dbg[(int64_t)m * C + jb] = y.y * 1.2676506002282294e30f;
                        }
                    }
                    uint32_t w[BITS];
                    pack32_sat<BITS>(q, w, flip);      // clamps to [0, 2^BITS - 1], packs, flips mirrored units
                    if constexpr (BITS == 8) {
                        if (keep[0] < 32u) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                const int nb = (int)keep[0] - 4 * i;          // real bytes in word i
                                w[i] &= nb >= 4 ? 0xFFFFFFFFu : nb <= 0 ? 0u : (1u << (8 * nb)) - 1u;
                            }
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < BITS; ++i) w[i] &= keep[i];
                    }
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
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_s + 8 * (2 * D + d));     // this warp has read everything it needs from the slot
            }
            if (++d == D) { d = 0; par ^= 1u; }
            if (++turn == G) turn = 0;
        }
    }
}

using KernelFn = void (*)(const LnParams);

template <bool DBG>
static KernelFn pick_kernel(int bits)
{
    return bits == 3 ? ln_reorder_quant_kernel<3, DBG> : bits == 4 ? ln_reorder_quant_kernel<4, DBG> : ln_reorder_quant_kernel<8, DBG>;
}
static KernelFn pick_selftest_kernel(int bits)
{
    return bits == 3 ? ln_reorder_quant_kernel<3, false, true> : bits == 4 ? ln_reorder_quant_kernel<4, false, true>
                                                                           : ln_reorder_quant_kernel<8, false, true>;
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
    // the attribute belongs to the kernel, not to this plan: always the largest size any plan may ask
    // for, or a later, smaller plan would take the room away from an earlier one that is cached
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024) != cudaSuccess) return RPTQ_ERR_CUDA;
    int n_sm = 0, per_sm = 0;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, T, smem) != cudaSuccess || per_sm < 1) return RPTQ_ERR_CUDA;
    g_plans.push_back({fn, device, T, smem, n_sm * per_sm});
    *blocks = n_sm * per_sm;
    return RPTQ_OK;
}

}  // namespace rptq

using namespace rptq;

static int launch_ln(const rptq_layout_t* L, const void* x, int64_t ldx, const void* gamma, const void* beta, float eps,
                     int M, void* codes, float* y_dbg, void* stream, long long wait_budget, uint32_t tx_extra)
{
    if (!L || !x || !gamma || !beta || !codes) return RPTQ_ERR_INVALID_ARG;
    if (M < 0 || ldx < L->C || (ldx % 8) != 0 || !(eps >= 0.0f)) return RPTQ_ERR_INVALID_ARG;
    if (!aligned16(x) || !aligned16(gamma) || !aligned16(beta) || !aligned16(codes) || !aligned16(y_dbg))
        return RPTQ_ERR_INVALID_ARG;
    if (M == 0) return RPTQ_OK;
    int dev = -1;
    if (L->device < 0 || cudaGetDevice(&dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (dev != L->device) return RPTQ_ERR_INVALID_ARG;

    // Shared memory: a ring of raw rows (2 C + 16 bytes each), as deep as fits up to
    // 16 rows, with two floats and three barriers per slot.
    const int C = L->C;
    const size_t pitch = (size_t)2 * C + 16;
    const size_t limit = 227 * 1024;
    int depth = (int)((limit - 64) / (pitch + 32));
    if (depth < 2) return RPTQ_ERR_UNSUPPORTED;
    depth = depth > 16 ? 16 : depth;
    const size_t smem = (size_t)depth * (pitch + 32) + 64;     // slots, then per slot 8 bytes of statistics and 3 barriers, 16 zero bytes, a flag

    // One gather thread per output unit where that fits beside four or five statistics warps in a
    // block of 512 threads (128 registers each), in up to four groups that take alternate rows when
    // the layout is narrow; wider layouts get two statistics warps (one beyond 416 units), and beyond 448
    // units each gather thread loops over several units and reloads its tables.
    const int want = (L->n_units + 31) / 32 * 32;
    int TG, S, groups = 1;
    if (want <= 320) { TG = want; S = 5; groups = 320 / TG; groups = groups > 4 ? 4 : groups; }
    else if (want <= 352) { TG = want; S = 4; }
    else if (want <= 416) { TG = want; S = 2; }
    else if (want <= 448) { TG = want; S = 1; }        // one statistics warp keeps up with 14 gather warps on these long rows
    else { TG = 416; S = 2; }
    if (groups > depth) groups = depth;
    const int T = 32 * (1 + S) + groups * TG;

    const bool selftest = tx_extra != 0u || wait_budget != kLnWaitBudgetCycles;
    KernelFn fn = selftest ? pick_selftest_kernel(L->bits) : y_dbg ? pick_kernel<true>(L->bits) : pick_kernel<false>(L->bits);
    int blocks = 0;
    const int rc = planned_blocks(reinterpret_cast<const void*>(fn), dev, T, smem, &blocks);
    if (rc != RPTQ_OK) return rc;
    LnParams p{};
    p.x = static_cast<const __half*>(x); p.ldx = ldx; p.gamma = static_cast<const __half*>(gamma);
    p.beta = static_cast<const __half*>(beta); p.eps = eps; p.M = M; p.C = C; p.n_units = L->n_units;
    p.n_stats_warps = S; p.depth = depth; p.n_groups = groups; p.ch_tab = L->d_src; p.jidx_tab = L->d_jidx; p.unit_tab = L->d_unit;
    p.codes = static_cast<uint8_t*>(codes); p.row_bytes = L->row_bytes; p.y_dbg = y_dbg; p.status = device_status_word();
    if (selftest) {
        if (cudaMemcpyToSymbol(c_selftest_wait_budget, &wait_budget, sizeof(wait_budget)) != cudaSuccess ||
            cudaMemcpyToSymbol(c_selftest_tx_extra, &tx_extra, sizeof(tx_extra)) != cudaSuccess) return RPTQ_ERR_CUDA;
    }
    fn<<<M < blocks ? M : blocks, T, smem, static_cast<cudaStream_t>(stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}

extern "C" int rptq_ln_reorder_quant(const rptq_layout_t* L, const void* x, int64_t ldx, const void* gamma,
                                     const void* beta, float eps, int M, void* codes, float* y_dbg, void* stream)
{
    return launch_ln(L, x, ldx, gamma, beta, eps, M, codes, y_dbg, stream, kLnWaitBudgetCycles, 0u);
}

// Self-test of the give-up path: the same launch, but every row's barrier is told to expect 16 bytes
// more than the row's copy delivers, so it never completes, and a wait may take 10 M cycles (~5 ms)
// only. The statistics warps' waits run out, the block records RPTQ_ERR_DEVICE_TIMEOUT, every later
// wait returns at once, the loops (fixed trip counts) run out and the kernel returns; nothing
// faults and nothing spins without a limit. The codes it writes are undefined.
extern "C" int rptq_selftest_ln_timeout(const rptq_layout_t* L, const void* x, int64_t ldx, const void* gamma,
                                        const void* beta, float eps, int M, void* codes, void* stream)
{
    return launch_ln(L, x, ldx, gamma, beta, eps, M, codes, nullptr, stream, 10000000ll, 16u);
}
