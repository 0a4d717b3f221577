// rptq_cluster_gemm: cluster-segmented integer GEMM (Appendix, second computation method).
//
//   acc_c[m][n] = sum_{k in segment c} X_q[m][k] * W_q[n][k]        int32, tcgen05.mma kind::i8
//   y[m][n]     = s_w[n] * sum_c s_c * (acc_c[m][n] - z_c * Wsum_c[n])  (+ bias) (ReLU) (re-quantise)
//
// Two variants of one kernel template. NCTA = 1: one persistent CTA per SM works on 128 (tokens) x
// 256 (output channels) tiles. NCTA = 2: the two CTAs of a cluster (an SM pair) share a 256 x 256
// tile through tcgen05.mma.cta_group::2 -- each CTA stages and unpacks its own 128 token rows and
// its own 128 of the 256 weight rows, which halves the weight unpacking and the shared-memory
// traffic per MMA; the first CTA of the pair issues the MMAs for both and its commits arrive on
// both CTAs' barriers; every CTA drains its own 128 accumulator lanes. No load is multicast.
// Warp roles (per CTA):
//   warp 0      bulk-copy producer: one contiguous 8 KiB cp.async.bulk per 128 weight rows per K
//               block (the packed weights are stored tile-major for this) into a ring of stages
//   warps 4-7   unpack: packed codes -> 8-bit operands, written in the K-major 128-byte-swizzled
//               layout that the tensor core reads (weights become 16 * w, see unpack.cuh). The
//               activation codes of a K block are 48/64/128 bytes per token row, too narrow for the
//               copy engine to move at speed (measured: ~10 clk per row), so each unpack thread
//               fetches the words of its own items with cp.async into a private ring of
//               shared-memory slots, several K blocks ahead. 8-bit codes need no unpacking: with
//               CTA pairs they are copied straight into the operand stage (template flag A8)
//   warp 1      MMA issuer (the whole warp in converged control flow, one elected lane issues):
//               four tcgen05.mma (K = 32 each) per K block; each cluster accumulates
//               into one of two 256-column TMEM buffers (the layout's step flags say which) and
//               is committed at its last step. A cluster's steps need not be adjacent: in the
//               interleaved unit order a small cluster's step sits between those of a large one,
//               which keeps its buffer, so the small cluster's drain runs under the large
//               cluster's remaining products
//   warps 8-15  epilogue: drain a finished cluster's accumulator (tcgen05.ld), add s_c * acc into
//               fp32 running sums held in registers while the next cluster's MMAs run; after the
//               last cluster apply the zero-point correction, s_w, bias, activation, and store
// Every wait is bounded: a wait that runs out sets RPTQ_ERR_DEVICE_TIMEOUT in the status word and
// all roles drain and return.
#include <cuda_fp16.h>

#include <mutex>

#include "pack.cuh"
#include "rptq_internal.h"
#include "unpack.cuh"

namespace rptq {
namespace gemm {

constexpr int TILE_M = 128, TILE_N = 256, KBLK = 128;   // TILE_M is per CTA
constexpr int THREADS = 512;
constexpr int UNPACK_WARP0 = 4, N_UNPACK_WARPS = 4;
constexpr int EPI_WARP0 = 8, N_EPI_WARPS = 8;
// registers per thread after the in-kernel re-partition (the block is launched with 128 each): the
// producer / MMA-issuer group, the unpack group, the two epilogue groups (128 running sums per thread)
constexpr int REGS_WG0 = 40, REGS_UNPACK = 88, REGS_EPI = 192;
static_assert(128 * (REGS_WG0 + REGS_UNPACK + 2 * REGS_EPI) <= 128 * THREADS, "register pool");
constexpr int A8_BYTES = TILE_M * KBLK;                  // 16 KiB of 8-bit activation operands per stage
constexpr int WTILE_BYTES = 8192;                        // one packed weight tile: 128 rows x 64 bytes
constexpr long long WAIT_BUDGET_CYCLES = 4000000000ll;   // about two seconds at the SM clock

__host__ __device__ constexpr int w_rows(int ncta) { return TILE_N / ncta; }           // weight rows staged per CTA
// packed weight stages; the single-CTA variant (at most 128 tokens) is a weight stream and takes what shared memory is left
__host__ __device__ constexpr int n_p_stages(int ncta, int bits) { return ncta == 2 ? 4 : (bits == 3 ? 5 : 4); }
__host__ __device__ constexpr int n_u_stages(int ncta, bool a8) { return ncta == 2 ? (a8 ? 5 : 4) : 2; }   // operand stages
// ring of packed activation K blocks fetched ahead by the unpack threads: one slot per token row
// per K block; the pitch is an odd number of 16-byte units so that the threads' vector reads of
// their own slots do not collide in the banks
__host__ __device__ constexpr int a_slot_pitch(int bits) { return bits == 3 ? 48 : 16 * bits + 16; }
__host__ __device__ constexpr int n_a_stages(int bits) { return bits == 8 ? 2 : 4; }

struct SmemLayout {
    int u_stage, p_stage, a_stage, off_p, off_a, off_flags, off_seg_scale, off_seg_buf, off_cl_sz, off_tab, off_bar, total;
};
__host__ __device__ constexpr SmemLayout smem_layout(int ncta, int bits, bool a8)
{
    SmemLayout s{};
    s.u_stage = A8_BYTES + w_rows(ncta) * KBLK;
    s.p_stage = w_rows(ncta) * KBLK / 2;
    s.a_stage = a8 ? 0 : TILE_M * a_slot_pitch(bits);      // 8-bit activations go straight to the operand stage
    s.off_p = n_u_stages(ncta, a8) * s.u_stage;
    s.off_a = s.off_p + n_p_stages(ncta, bits) * s.p_stage;
    s.off_flags = s.off_a + n_a_stages(bits) * s.a_stage;
    s.off_seg_scale = s.off_flags + 2048;
    s.off_seg_buf = s.off_seg_scale + kMaxGemmSegments * 4;
    s.off_cl_sz = s.off_seg_buf + kMaxGemmSegments;
    s.off_tab = s.off_cl_sz + kMaxGemmSegments * 4;
    s.off_bar = s.off_tab + 2 * 3 * TILE_N * 4;
    s.total = s.off_bar + 256;
    return s;
}

struct Params {
    int M, N, n_kb, n_seg, g;
    int tiles_m, n_tiles;
    const uint8_t* a_codes;      // [M][a_row_bytes]
    int64_t a_row_bytes;
    const uint8_t* w_codes;      // tile-major: n_wtiles * n_kb tiles of 8 KiB
    int n_wtiles;
    const uint8_t* step_flags;
    const float* seg_scale;      // [n_seg] in the order the clusters' last steps come
    const uint8_t* seg_buf;      // [n_seg] accumulator of each, same order
    const float* cl_sz;
    const float* corr;           // optional [N]: sum_c s_c z_c Wsum_c[n] computed beforehand, else NULL
    const float* s_w;
    const int32_t* wsum;
    int64_t ld_w;
    // per-cluster asymmetric weight parameters (template flag ASYM): [g][ld_w] tables of s^W_c[n] and
    // z^W_c[n], the cluster of every entry of seg_scale, n_c, and the activation code sums [M][g]
    const float* sw_c;
    const int32_t* zw_c;
    const int32_t* seg_cluster;
    const float* cl_n;
    const int32_t* xsum;
    // first computation method (template mode MODE_DEQ): per unit of 32 positions {s_c, (float) z_c}
    const float2* unit_sz;
    const float* bias;
    int act, y_dtype;
    void* y;
    int64_t ldy;
    const UnitInfo* out_unit;
    int out_bits;
    int64_t out_row_bytes;
    int* status;
};

// ---------------------------------------------------------------- PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t bar, uint32_t rank)
{
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.shared::cluster.b64 _, [ra];\n\t}"
        ::"r"(bar), "r"(rank) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// Bounded wait. Returns false when the budget ran out or another role already gave up. The common
// case (the phase has already completed, or completes within a few polls) touches no timer; the
// budget is counted on the SM's cycle counter, read once per batch of polls.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, bool heed_abort = true)
{
    auto poll = [&]() { return mbar_try_wait(bar, parity); };
    if (poll()) return true;
    if (poll()) return true;
    const long long t0 = clock64();
#pragma unroll 1
    while (true) {
#pragma unroll 1
        for (int i = 0; i < 1024; ++i)
            if (poll()) return true;
        if (heed_abort && *abort_flag) return false;
        if (clock64() - t0 > WAIT_BUDGET_CYCLES) { *abort_flag = 1; return false; }
    }
}
// The same wait for a whole warp that must stay converged (the MMA-issuing warp): the lanes vote on
// every poll, so all of them leave the loop in the same iteration whatever each one saw.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag)
{
    if (__any_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
    const long long t0 = clock64();
#pragma unroll 1
    while (true) {
#pragma unroll 1
        for (int i = 0; i < 1024; ++i)
            if (__any_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
        const bool give_up = *abort_flag != 0 || clock64() - t0 > WAIT_BUDGET_CYCLES;
        if (__any_sync(0xffffffffu, give_up)) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// One contiguous global -> shared copy by the copy engine; completion is counted on `bar`.
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// Asynchronous 16-byte global -> shared copy issued by an ordinary thread; `valid` false writes
// zeros and reads nothing.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, bool valid)
{
    const uint32_t n = valid ? 16u : 0u;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// The two tensor-core instructions below are executed by the WHOLE issuing warp in converged
// control flow; elect.sync picks the one lane that issues. Measured on an operand-resident loop: a
// tcgen05.mma issued from a branch that a single lane took costs the issuing thread ~120 clocks,
// one issued this way ~85, against 134 clocks of tensor-pipe time per instruction.
template <int NCTA>
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    if constexpr (NCTA == 1) {
        asm volatile(
            "{\n\t.reg .pred q;\n\t"
            "elect.sync _|q, 0xffffffff;\n\t"
            "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
            ::"r"(bar) : "memory");
    } else {
        // arrives on the barrier at this offset in both CTAs of the pair
        const uint16_t mask = 3;
        asm volatile(
            "{\n\t.reg .pred q;\n\t"
            "elect.sync _|q, 0xffffffff;\n\t"
            "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
            ::"r"(bar), "h"(mask) : "memory");
    }
}
template <int NCTA>
__device__ __forceinline__ void tc_mma_i8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    if constexpr (NCTA == 1) {
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "elect.sync _|q, 0xffffffff;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "@q tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "elect.sync _|q, 0xffffffff;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "@q tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    }
}
// bf16 x bf16 -> fp32, same operand layout and issue pattern as tc_mma_i8 (K = 16 elements = 32 bytes)
template <int NCTA>
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    if constexpr (NCTA == 1) {
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "elect.sync _|q, 0xffffffff;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "elect.sync _|q, 0xffffffff;\n\t"
            "setp.ne.b32 p, %4, 0;\n\t"
            "@q tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
            ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
    }
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// K-major operand tile with 128-byte rows and the 128-byte swizzle: 8-row groups are 1024 bytes
// apart (stride byte offset), the leading byte offset is unused for swizzled K-major layouts.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);        // start address, 16-byte units
    d |= (uint64_t)1 << 16;                         // leading byte offset (ignored)
    d |= (uint64_t)(1024 >> 4) << 32;               // stride byte offset
    d |= (uint64_t)1 << 46;                         // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                         // 128-byte swizzle
    return d;
}
// kind::i8, D = s32, A = unsigned 8-bit (activation codes), B = signed 8-bit (weights), both
// K-major, M = 128 per CTA, N = 256.
__host__ __device__ constexpr uint32_t instr_desc(int ncta)
{
    return (2u << 4) | (0u << 7) | (1u << 10) | ((uint32_t)(TILE_N >> 3) << 17) | ((uint32_t)((TILE_M * ncta) >> 4) << 24);
}

// kind::f16 with bfloat16 operands: D = fp32, A and B bfloat16, both K-major
__host__ __device__ constexpr uint32_t instr_desc_bf16(int ncta)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(TILE_N >> 3) << 17) | ((uint32_t)((TILE_M * ncta) >> 4) << 24);
}
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
// two fp32 values rounded to bfloat16 (nearest even): lo in bits 0-15, hi in bits 16-31
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
// Byte i of w as the float 2^23 + byte: the byte is dropped into the low mantissa bits of 0x4B000000.
template <int I>
__device__ __forceinline__ float byte_as_magic(uint32_t w)
{
    return __uint_as_float(__byte_perm(w, 0x4B000000u, 0x7650u | (uint32_t)I));
}
// Four 8-bit values of one word -> four bfloat16 (two words): v = (byte - c1) * s with c1 = 2^23 + z.
// byte - c1 is exact, the product is rounded once to fp32 and once more to bfloat16.
__device__ __forceinline__ void bytes_to_bf16(uint32_t w, float2 neg_c1, float2 s2, bool scale, uint32_t& out_lo, uint32_t& out_hi)
{
    float2 a = add2(make_float2(byte_as_magic<0>(w), byte_as_magic<1>(w)), neg_c1);
    float2 b = add2(make_float2(byte_as_magic<2>(w), byte_as_magic<3>(w)), neg_c1);
    if (scale) { a = mul2(a, s2); b = mul2(b, s2); }
    out_lo = pack_bf16(a.x, a.y);
    out_hi = pack_bf16(b.x, b.y);
}

// packed fp32 pairs: one instruction, two independent IEEE results
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c)
{
    float2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(reinterpret_cast<uint64_t&>(d))
        : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)), "l"(reinterpret_cast<uint64_t&>(c)));
    return d;
}

__device__ __forceinline__ void sts128(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d)
{
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
    return v;
}

// ASYM: the weights carry one scale and one zero point per (cluster, output channel) (Appendix,
// W~_q,i = Q_k(W~_i, s^W_i, z^W_i)). The stored nibble is the code minus 8, so the integer products
// are acc' = sum X_q (W_q - 8) and the second method's four terms become
//   Y_q,c = acc'_c - (z^W_c[n] - 8) * sum_k X_q[m][k] - z^X_c * Wsum_c[n] + n_c z^X_c z^W_c[n] :
// the first two are applied per element while a cluster's accumulator is drained, the last two are a
// constant of the output column.
// MODE_DEQ: the first computation method of the Appendix (de-quantise, then one floating-point product):
// the unpack warps write X^ = s_c (X_q - z_c) as bfloat16 and the weight codes as bfloat16 integers
// (16 w, exact), the MMAs are kind::f16 into ONE fp32 accumulator per tile -- no per-cluster
// accumulators, no drains at cluster boundaries -- and s_w[n] multiplies the finished sum. A bfloat16
// operand row of 128 bytes holds 64 positions, so a K block of 128 positions is two operand stages.
enum { MODE_INT = 0, MODE_ASYM = 1, MODE_DEQ = 2 };
template <int BITS, int NCTA, bool A8, int MODE>
__global__ void __launch_bounds__(THREADS, 1)
cluster_gemm_kernel(const Params p)
{
    constexpr bool ASYM = MODE == MODE_ASYM, DEQ = MODE == MODE_DEQ;
    static_assert(!(DEQ && A8), "the de-quantising variant unpacks every bit width");
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    constexpr SmemLayout SL = smem_layout(NCTA, BITS, A8);
    constexpr int W_ROWS = w_rows(NCTA);                 // weight rows this CTA stages and unpacks
    constexpr int N_P = n_p_stages(NCTA, BITS), N_U = n_u_stages(NCTA, A8);
    constexpr uint32_t kInstrDesc = DEQ ? instr_desc_bf16(NCTA) : instr_desc(NCTA);
    // dynamic shared memory is only guaranteed 16-byte alignment: round up to the swizzle span
    // (the offset is the same in both CTAs of a pair, as cta_group::2 descriptors require)
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem = smem_raw + (smem_base - smem_u32(smem_raw));

    uint8_t* s_flags = smem + SL.off_flags;
    float* s_seg_scale = reinterpret_cast<float*>(smem + SL.off_seg_scale);
    uint8_t* s_seg_buf = smem + SL.off_seg_buf;
    float* s_cl_sz = reinterpret_cast<float*>(smem + SL.off_cl_sz);
    float* s_tab = reinterpret_cast<float*>(smem + SL.off_tab);           // [2][3][TILE_N]
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + SL.off_bar);
    // barrier indices
    constexpr int B_PFULL = 0, B_PEMPTY = B_PFULL + N_P, B_UFULL = B_PEMPTY + N_P, B_UEMPTY = B_UFULL + N_U,
                  B_ACCFULL = B_UEMPTY + N_U, B_ACCEMPTY = B_ACCFULL + 2, B_TAB = B_ACCEMPTY + 2, B_DRAIN = B_TAB + 2,
                  N_BARS = B_DRAIN + 1;
    static_assert(N_BARS * 8 + 16 <= 256, "barrier block too small");
    uint32_t* s_tmem_ptr = reinterpret_cast<uint32_t*>(bars + N_BARS);
    volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem_ptr + 1);
    const uint32_t bar0 = smem_u32(bars);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n_steps = p.n_kb * 4;
    const uint32_t cta_rank = NCTA == 2 ? cluster_ctarank() : 0u;       // rank 0 issues the MMAs
    const int pair_id = (int)blockIdx.x / NCTA, n_pairs = (int)gridDim.x / NCTA;
    // arrive on a barrier that lives in the issuing CTA of the pair
    auto arrive_leader = [&](uint32_t b) { if constexpr (NCTA == 1) mbar_arrive(b); else mbar_arrive_remote(b, 0); };

    if (tid == 0) {
        for (int i = 0; i < N_P; ++i) { mbar_init(bar(B_PFULL + i), 1); mbar_init(bar(B_PEMPTY + i), N_UNPACK_WARPS); }
        for (int i = 0; i < N_U; ++i) { mbar_init(bar(B_UFULL + i), N_UNPACK_WARPS * NCTA); mbar_init(bar(B_UEMPTY + i), 1); }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(B_ACCFULL + i), 1); mbar_init(bar(B_ACCEMPTY + i), N_EPI_WARPS * NCTA); mbar_init(bar(B_TAB + i), N_EPI_WARPS);
        }
        mbar_init(bar(B_DRAIN), 1);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < n_steps; i += THREADS) s_flags[i] = p.step_flags[i];
    for (int i = tid; i < p.n_seg; i += THREADS) { s_seg_scale[i] = p.seg_scale[i] * 0.0625f; s_seg_buf[i] = p.seg_buf[i]; }   // operands were 16 * w
    for (int i = tid; i < p.g; i += THREADS) s_cl_sz[i] = p.cl_sz[i];
    if (warp == 1) {
        if constexpr (NCTA == 1) {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(s_tmem_ptr)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        } else {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(s_tmem_ptr)) : "memory");
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
        }
    }
    tc_fence_before();
    __syncthreads();
    if constexpr (NCTA == 2) cluster_sync_all();       // the peer's barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem_base = *s_tmem_ptr;

    // The register file is re-partitioned by warpgroup (the epilogue holds 128 running sums per
    // thread); each setmaxnreg is executed by the four warps of its group at one place.
    if (warp < UNPACK_WARP0) {
      asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_WG0));
      if (warp == 0) {
        // ------------------------------------------------------------ bulk-copy producer
        if (lane == 0) {
            uint32_t n_issued = 0;
            bool ok = true;
            for (int t = pair_id; t < p.n_tiles && ok; t += n_pairs) {
                // 128-row weight tiles this CTA stages; tiles past the end of the buffer are skipped
                // (their columns are never stored)
                const int wt0 = ((t / p.tiles_m) * TILE_N + (int)cta_rank * W_ROWS) >> 7;
                int n_valid = p.n_wtiles - wt0;
                n_valid = n_valid < 0 ? 0 : (n_valid > W_ROWS / 128 ? W_ROWS / 128 : n_valid);
                for (int kb = 0; kb < p.n_kb; ++kb, ++n_issued) {
                    const int s = n_issued % N_P;
                    const uint32_t ph = (n_issued / N_P) & 1;
                    if (!mbar_wait(bar(B_PEMPTY + s), ph ^ 1, s_abort)) { ok = false; break; }
                    const uint32_t dst = smem_base + SL.off_p + s * SL.p_stage;
                    mbar_arrive_expect_tx(bar(B_PFULL + s), (uint32_t)(n_valid * WTILE_BYTES));
                    for (int j = 0; j < n_valid; ++j)
                        bulk_load(dst + j * WTILE_BYTES, p.w_codes + ((int64_t)(wt0 + j) * p.n_kb + kb) * WTILE_BYTES,
                                  (uint32_t)WTILE_BYTES, bar(B_PFULL + s));
                }
            }
            if (!ok) {
                // let copies that were already issued land before the CTA's shared memory goes away
                const uint32_t lo = n_issued > N_P ? n_issued - N_P : 0;
                for (uint32_t i = lo; i < n_issued; ++i) mbar_wait(bar(B_PFULL + i % N_P), (i / N_P) & 1, s_abort, false);
            }
        }
      } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer (first CTA of a pair only)
        if (cta_rank == 0) {
            // The whole warp runs this loop in converged control flow (every value in it is the same
            // in all lanes); one elected lane issues. It is a single stream of dependent
            // instructions, so the loop is kept short:
            // stage descriptors are built once, a K block's four step flags come as one word, and a
            // block that lies inside one cluster issues its four MMAs without any test.
            // (the loop runs over all K blocks of all of this pair's tiles with one counter: the
            // lane has few registers)
            uint32_t par = 0;                // bit b: parity of how many clusters accumulator b has held
            bool ok = true;
            const uint64_t a_desc0 = smem_desc_sw128(smem_base);
            const uint32_t* flags4 = reinterpret_cast<const uint32_t*>(s_flags);
            uint32_t f4 = flags4[0];
            const uint32_t total_kb = (uint32_t)(((p.n_tiles - pair_id + n_pairs - 1) / n_pairs) * p.n_kb);
            int kb = 0;
            if constexpr (DEQ) {
                // One accumulator per tile, the two buffers alternate from tile to tile; every operand
                // stage is half a K block (64 positions, four MMAs of K = 16).
                const uint32_t steps_per_tile = 2u * (uint32_t)p.n_kb, total_steps = 2u * total_kb;
                uint32_t in_tile = 0, b = 0;
                for (uint32_t n = 0; n < total_steps; ++n) {
                    const int st = n % N_U;
                    if (in_tile == 0) {
                        if (!mbar_wait_warp(bar(B_ACCEMPTY + b), ((par >> b) & 1u) ^ 1u, s_abort)) { ok = false; break; }
                        tc_fence_after();
                    }
                    if (!mbar_wait_warp(bar(B_UFULL + st), (n / N_U) & 1, s_abort)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t ad = a_desc0 + (uint64_t)(st * (SL.u_stage >> 4)), wd = ad + (uint64_t)(A8_BYTES >> 4);
                    const uint32_t d_tmem = tmem_base + b * TILE_N;
                    tc_mma_bf16<NCTA>(d_tmem, ad, wd, kInstrDesc, in_tile);
                    tc_mma_bf16<NCTA>(d_tmem, ad + 2, wd + 2, kInstrDesc, 1u);
                    tc_mma_bf16<NCTA>(d_tmem, ad + 4, wd + 4, kInstrDesc, 1u);
                    tc_mma_bf16<NCTA>(d_tmem, ad + 6, wd + 6, kInstrDesc, 1u);
                    tc_commit<NCTA>(bar(B_UEMPTY + st));
                    if (++in_tile == steps_per_tile) {
                        tc_commit<NCTA>(bar(B_ACCFULL + b));
                        par ^= 1u << b;
                        b ^= 1u;
                        in_tile = 0;
                    }
                }
            } else
            for (uint32_t n_kb_done = 0; n_kb_done < total_kb; ++n_kb_done) {
                    const int s = n_kb_done % N_U;
                    kb = kb + 1 == p.n_kb ? 0 : kb + 1;
                    const uint32_t f4_next = flags4[kb];                              // read while waiting
                    if (!mbar_wait_warp(bar(B_UFULL + s), (n_kb_done / N_U) & 1, s_abort)) { ok = false; break; }
                    tc_fence_after();
                    // the start-address field counts 16-byte units: one stage further, 32 bytes per step;
                    // the weight operand follows the activation operand in the stage
                    const uint64_t ad = a_desc0 + (uint64_t)(s * (SL.u_stage >> 4)), wd = ad + (uint64_t)(A8_BYTES >> 4);
                    if (f4 == 0u || f4 == 0x01010101u * STEP_BUF) {
                        // four steps inside one cluster
                        const uint32_t d_tmem = tmem_base + (f4 ? TILE_N : 0);
                        tc_mma_i8<NCTA>(d_tmem, ad, wd, kInstrDesc, 1u);
                        tc_mma_i8<NCTA>(d_tmem, ad + 2, wd + 2, kInstrDesc, 1u);
                        tc_mma_i8<NCTA>(d_tmem, ad + 4, wd + 4, kInstrDesc, 1u);
                        tc_mma_i8<NCTA>(d_tmem, ad + 6, wd + 6, kInstrDesc, 1u);
                    } else {
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint32_t f = (f4 >> (8 * j)) & 0xFFu;
                            const uint32_t b = (f / STEP_BUF) & 1u;
                            const uint32_t d_tmem = tmem_base + b * TILE_N;
                            if ((f & (STEP_FIRST | STEP_LAST | STEP_SKIP)) == 0) {       // inside a cluster
                                tc_mma_i8<NCTA>(d_tmem, ad + 2 * j, wd + 2 * j, kInstrDesc, 1u);
                                continue;
                            }
                            if (f & STEP_SKIP) continue;
                            if (f & STEP_FIRST) {
                                // the accumulator's previous cluster has been drained
                                if (!mbar_wait_warp(bar(B_ACCEMPTY + b), ((par >> b) & 1u) ^ 1u, s_abort)) { ok = false; break; }
                                tc_fence_after();
                            }
                            tc_mma_i8<NCTA>(d_tmem, ad + 2 * j, wd + 2 * j, kInstrDesc, (f & STEP_FIRST) ? 0u : 1u);
                            if (f & STEP_LAST) {
                                tc_commit<NCTA>(bar(B_ACCFULL + b));
                                par ^= 1u << b;
                            }
                        }
                        if (!ok) break;
                    }
                    tc_commit<NCTA>(bar(B_UEMPTY + s));      // the stage may be overwritten once these MMAs have read it
                    f4 = f4_next;
            }
            if (!ok) {
                tc_commit<NCTA>(bar(B_DRAIN));
                mbar_wait(bar(B_DRAIN), 0, s_abort, false);
            }
        }
      }   // warps 2 and 3 only fill the first warpgroup
    } else if (warp < EPI_WARP0) {
        // ------------------------------------------------------------ unpack warps
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS_UNPACK));
        const int ut = tid - UNPACK_WARP0 * 32;      // 0..127
        uint32_t n_done = 0;
        const int total_kb = ((p.n_tiles - pair_id + n_pairs - 1) / n_pairs) * p.n_kb;
        // Weight item i of this thread is row (ut >> 2) + 32 i, unit ut & 3, so its two chunk positions in
        // the swizzled row (16-byte chunk j of row r lives at position j ^ (r & 7)) are the same for every i.
        const int row0 = ut >> 2, unit = ut & 3, sw = row0 & 7;
        const uint32_t off0 = row0 * 128 + (((2 * unit) ^ sw) << 4), off1 = row0 * 128 + (((2 * unit + 1) ^ sw) << 4);
        constexpr int W_ITEMS = W_ROWS * 4 / 128;    // weight items per thread
        const uint32_t a_off = ut * 128, a_sw = ut & 7;          // my operand row and its swizzle
        int t_f = pair_id, kb_f = 0, n_fetched = 0;             // next K block to fetch
        const uint8_t* a_src = p.a_codes;
        if constexpr (A8) {
            // The codes are bytes already: a K block of a token row is 128 contiguous bytes. Eight
            // lanes copy the eight 16-byte chunks of one row (one cache line per row, so a warp-wide
            // cp.async touches 4 lines, not 32) straight into that row's swizzled place in the
            // operand stage; a warp covers its 32 rows in eight such instructions, PF K blocks
            // ahead of the weights. The stage is waited for (its previous MMAs have read it) first.
            constexpr int PF = N_U - 2;
            bool ok = true;
            const int wrow = (warp - UNPACK_WARP0) * 32 + (lane >> 3), ch = lane & 7;   // rows wrow + 4 i, chunk ch
            const uint32_t d_even = (uint32_t)wrow * 128 + ((ch ^ (lane >> 3)) << 4);
            const uint32_t d_odd = (uint32_t)wrow * 128 + ((ch ^ ((lane >> 3) + 4)) << 4);
            const int64_t step4 = 4 * p.a_row_bytes;
            int n_rows_ok = 0;                               // how many of my 8 rows exist
            auto a8_tile = [&]() {
                const int row = (t_f % p.tiles_m) * (TILE_M * NCTA) + (int)cta_rank * TILE_M + wrow;
                const int left = p.M - row;
                n_rows_ok = left <= 0 ? 0 : (left + 3) >> 2;
                a_src = p.a_codes + (int64_t)(left > 0 ? row : 0) * p.a_row_bytes + 16 * ch;
            };
            a8_tile();
            auto fetch_next = [&]() {
                if (n_fetched < total_kb && ok) {
                    const int s2 = n_fetched % N_U;
                    if (!mbar_wait(bar(B_UEMPTY + s2), ((n_fetched / N_U) & 1) ^ 1, s_abort)) { ok = false; }
                    else {
                        tc_fence_after();
                        const uint32_t dst = smem_base + s2 * SL.u_stage;
#pragma unroll
                        for (int i = 0; i < 8; ++i) {
                            const bool v = i < n_rows_ok;
                            cp_async16(dst + ((i & 1) ? d_odd : d_even) + i * 512, v ? a_src + i * step4 : p.a_codes, v);
                        }
                        a_src += KBLK;
                        if (++kb_f == p.n_kb) { kb_f = 0; t_f += n_pairs; a8_tile(); }
                    }
                }
                ++n_fetched;
                cp_async_commit();                           // one group per K block, empty past the end
            };
#pragma unroll 1
            for (int i = 0; i < PF; ++i) fetch_next();
            for (int it = 0; it < total_kb && ok; ++it, ++n_done) {
                const int sp = n_done % N_P, su = n_done % N_U;
                fetch_next();
                if (!ok) break;
                if (!mbar_wait(bar(B_PFULL + sp), (n_done / N_P) & 1, s_abort)) break;
                const uint32_t pw = smem_base + SL.off_p + sp * SL.p_stage;
                const uint32_t w_tile = smem_base + su * SL.u_stage + A8_BYTES;
                uint32_t pw_w[W_ITEMS][4];
#pragma unroll
                for (int i = 0; i < W_ITEMS; ++i) {
                    const uint4 v = lds128(pw + (ut + i * 128) * 16);
                    pw_w[i][0] = v.x; pw_w[i][1] = v.y; pw_w[i][2] = v.z; pw_w[i][3] = v.w;
                }
#pragma unroll
                for (int i = 0; i < W_ITEMS; ++i) {
                    uint32_t o[8];
                    unpack_w32_x16(pw_w[i], o);
                    sts128(w_tile + off0 + i * 4096, o[0], o[1], o[2], o[3]);
                    sts128(w_tile + off1 + i * 4096, o[4], o[5], o[6], o[7]);
                }
                cp_async_wait<PF>();                         // my copies of K block `it` have landed
                fence_proxy_async();          // make the generic-proxy writes visible to the tensor core
                __syncwarp();                 // ... and every lane's copies and stores of this warp
                if (lane == 0) { arrive_leader(bar(B_UFULL + su)); mbar_arrive(bar(B_PEMPTY + sp)); }
            }
            cp_async_wait<0>();
        } else {
        // Activation codes: this thread owns token row `ut` of the tile and unpacks it. A K block of a
        // row is 16 BITS contiguous bytes; the rows' K blocks are fetched N_A - 1 K blocks ahead with
        // 16-byte cp.async into one shared-memory slot per row. The 32 BITS chunks of a warp's 32 rows
        // are spread over the lanes in memory order (lane l of copy i takes chunk 32 i + l: row
        // (32 i + l) / BITS of the warp, part (32 i + l) % BITS), so that one warp-wide copy touches
        // 32 / BITS rows, not 32: the load path looks up one cache line per row touched, and with one
        // row per lane those look-ups, not the bytes, set the pace. A row's chunks are copied by
        // lanes of the row owner's own warp, so a __syncwarp after the wait is all the hand-over needs.
        constexpr int N_A = n_a_stages(BITS), PITCH = a_slot_pitch(BITS);
        const uint32_t a_ring0 = smem_base + SL.off_a;
        const uint32_t a_ring = a_ring0 + ut * PITCH;
        uint32_t d_off[BITS], s_off[BITS];               // where my chunks go in a ring stage / come from in the tile's rows
        int r_of[BITS];                                  // their rows within the tile
#pragma unroll
        for (int i = 0; i < BITS; ++i) {
            const int c = 32 * i + lane;
            r_of[i] = (ut & ~31) + c / BITS;
            d_off[i] = (uint32_t)r_of[i] * PITCH + 16u * (uint32_t)(c % BITS);
            s_off[i] = (uint32_t)r_of[i] * (uint32_t)p.a_row_bytes + 16u * (uint32_t)(c % BITS);
        }
        int rows_left = 0;                               // rows of the tile being fetched that exist
        auto fetch_tile_row = [&]() {
            const int row0 = (t_f % p.tiles_m) * (TILE_M * NCTA) + (int)cta_rank * TILE_M;
            rows_left = p.M - row0;
            a_src = p.a_codes + (int64_t)(rows_left > 0 ? row0 : 0) * p.a_row_bytes;
        };
        fetch_tile_row();
        auto fetch_next = [&]() {
            if (n_fetched < total_kb) {
                const uint32_t dst = a_ring0 + (n_fetched % N_A) * SL.a_stage;
#pragma unroll
                for (int i = 0; i < BITS; ++i) {
                    const bool v = r_of[i] < rows_left;
                    cp_async16(dst + d_off[i], v ? a_src + s_off[i] : p.a_codes, v);
                }
                a_src += 16 * BITS;
                if (++kb_f == p.n_kb) { kb_f = 0; t_f += n_pairs; fetch_tile_row(); }
            }
            ++n_fetched;
            cp_async_commit();                           // one group per K block, empty past the end
        };
#pragma unroll 1
        for (int i = 0; i < N_A - 1; ++i) fetch_next();
        for (int it = 0; it < total_kb; ++it, ++n_done) {
            const int sp = n_done % N_P, su = n_done % N_U;
            fetch_next();
            cp_async_wait<N_A - 1>();                    // my copies of K block `it` have landed
            __syncwarp();                                // ... and those of the lanes that copied my row
            uint32_t pa_w[4][BITS];                      // [unit][word]: unit u of the row is words BITS u ..
            {
                const uint32_t slot = a_ring + (it % N_A) * SL.a_stage;
                uint32_t raw[4 * BITS];
#pragma unroll
                for (int j = 0; j < BITS; ++j) {
                    const uint4 v = lds128(slot + 16 * j);
                    raw[4 * j] = v.x; raw[4 * j + 1] = v.y; raw[4 * j + 2] = v.z; raw[4 * j + 3] = v.w;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int j = 0; j < BITS; ++j) pa_w[u][j] = raw[BITS * u + j];
            }
            if (!mbar_wait(bar(B_PFULL + sp), (n_done / N_P) & 1, s_abort)) break;
            if constexpr (DEQ) {
                // Two operand stages per K block, 64 positions each. My token row: units 2 h and 2 h + 1,
                // de-quantised to bfloat16 with the unit's (s_c, z_c). Weights: for half h this thread
                // converts unit 2 h + (ut & 1) of rows (ut >> 1) + 64 i.
                const uint32_t pw = smem_base + SL.off_p + sp * SL.p_stage;
                const int kb_now = it % p.n_kb;
                bool ok = true;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t n_step = 2u * n_done + (uint32_t)h;
                    const int st = n_step % N_U;
                    if (!mbar_wait(bar(B_UEMPTY + st), ((n_step / N_U) & 1) ^ 1, s_abort)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a_tile = smem_base + st * SL.u_stage, w_tile = a_tile + A8_BYTES;
#pragma unroll
                    for (int uu = 0; uu < 2; ++uu) {
                        const int u = 2 * h + uu;
                        const float2 sz = __ldg(p.unit_sz + 4 * kb_now + u);
                        const float c1 = -(8388608.0f + sz.y);
                        const float2 neg_c1 = make_float2(c1, c1), s2 = make_float2(sz.x, sz.x);
                        uint32_t o[8];
                        unpack_act32<BITS>(pa_w[u], o);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t b0, b1, b2, b3;
                            bytes_to_bf16(o[2 * c], neg_c1, s2, true, b0, b1);
                            bytes_to_bf16(o[2 * c + 1], neg_c1, s2, true, b2, b3);
                            sts128(a_tile + a_off + (((4 * uu + c) ^ a_sw) << 4), b0, b1, b2, b3);
                        }
                    }
                    const float cw = -(8388608.0f + 128.0f);
                    const float2 neg_cw = make_float2(cw, cw);
#pragma unroll
                    for (int i = 0; i < W_ROWS / 64; ++i) {
                        const int r = (ut >> 1) + 64 * i;
                        const uint4 v = lds128(pw + r * 64 + (2 * h + (ut & 1)) * 16);
                        const uint32_t pk[4] = {v.x, v.y, v.z, v.w};
                        uint32_t o[8];
                        unpack_w32_x16(pk, o);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            uint32_t b0, b1, b2, b3;       // 16 w as bfloat16: the byte, sign bit flipped, minus 128
                            bytes_to_bf16(o[2 * c] ^ 0x80808080u, neg_cw, neg_cw, false, b0, b1);
                            bytes_to_bf16(o[2 * c + 1] ^ 0x80808080u, neg_cw, neg_cw, false, b2, b3);
                            sts128(w_tile + r * 128 + (((4 * (ut & 1) + c) ^ (r & 7)) << 4), b0, b1, b2, b3);
                        }
                    }
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) arrive_leader(bar(B_UFULL + st));
                }
                if (!ok) break;
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_PEMPTY + sp));
                continue;
            }
            if (!mbar_wait(bar(B_UEMPTY + su), ((n_done / N_U) & 1) ^ 1, s_abort)) break;
            tc_fence_after();
            const uint32_t pw = smem_base + SL.off_p + sp * SL.p_stage;
            const uint32_t a_tile = smem_base + su * SL.u_stage, w_tile = a_tile + A8_BYTES;
            // all packed weight words of my items first (independent loads), then unpack and store
            uint32_t pw_w[W_ITEMS][4];
#pragma unroll
            for (int i = 0; i < W_ITEMS; ++i) {
                const uint4 v = lds128(pw + (ut + i * 128) * 16);
                pw_w[i][0] = v.x; pw_w[i][1] = v.y; pw_w[i][2] = v.z; pw_w[i][3] = v.w;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                uint32_t o[8];
                unpack_act32<BITS>(pa_w[u], o);
                sts128(a_tile + a_off + (((2 * u) ^ a_sw) << 4), o[0], o[1], o[2], o[3]);
                sts128(a_tile + a_off + (((2 * u + 1) ^ a_sw) << 4), o[4], o[5], o[6], o[7]);
            }
#pragma unroll
            for (int i = 0; i < W_ITEMS; ++i) {
                uint32_t o[8];
                unpack_w32_x16(pw_w[i], o);
                sts128(w_tile + off0 + i * 4096, o[0], o[1], o[2], o[3]);
                sts128(w_tile + off1 + i * 4096, o[4], o[5], o[6], o[7]);
            }
            fence_proxy_async();          // make the generic-proxy stores visible to the tensor core
            __syncwarp();
            if (lane == 0) { arrive_leader(bar(B_UFULL + su)); mbar_arrive(bar(B_PEMPTY + sp)); }
        }
        cp_async_wait<0>();
        }
    } else {
        // ------------------------------------------------------------ epilogue warps
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS_EPI));
        const int ew = warp - EPI_WARP0;
        const int q = ew & 3, h = ew >> 2;           // TMEM lane quarter (= warp % 4), column half
        const int et = ew * 32 + lane;               // 0..255: the column whose tile constants I prepare
        uint32_t n_tile_done = 0;
        uint32_t par = 0;                    // bit b: parity of how many clusters of accumulator b I have drained
        bool ok = true;
        float2 R[64];                                // running sums of columns 2 i, 2 i + 1
        for (int t = pair_id; t < p.n_tiles && ok; t += n_pairs, ++n_tile_done) {
            const int m0 = (t % p.tiles_m) * (TILE_M * NCTA) + (int)cta_rank * TILE_M, n0 = (t / p.tiles_m) * TILE_N;
            float* tab = s_tab + (n_tile_done & 1) * 3 * TILE_N;
            // a warp whose 32 accumulator lanes all lie beyond the last token row keeps the barriers'
            // protocol but reads and accumulates nothing (few-token calls: most of the tile is empty)
            const bool live = m0 + 32 * q < p.M;
            {   // per-tile column constants: zero-point correction sum_c s_c z_c Wsum_c[n], s_w[n], bias[n]
                const int n = n0 + et;
                float corr = 0.f, sw = 0.f, bs = 0.f;
                if (n < p.N) {
                    if constexpr (ASYM) {
                        // sum_c s^X_c z^X_c s^W_c[n] (Wsum_c[n] - n_c z^W_c[n]); the column's scale is applied per cluster
                        for (int c = 0; c < p.g; ++c) {
                            const int64_t i = (int64_t)c * p.ld_w + n;
                            const float t = (float)__ldg(p.wsum + i) - __ldg(p.cl_n + c) * (float)__ldg(p.zw_c + i);
                            corr = __fmaf_rn(s_cl_sz[c] * __ldg(p.sw_c + i), t, corr);
                        }
                        sw = 1.0f;
                    } else if constexpr (DEQ) {
                        sw = __ldg(p.s_w + n) * 0.0625f;             // the weight operands were 16 w; zero points are in X^
                    } else {
                        if (p.corr) corr = __ldg(p.corr + n);
                        else for (int c = 0; c < p.g; ++c) corr = __fmaf_rn(s_cl_sz[c], (float)__ldg(p.wsum + (int64_t)c * p.ld_w + n), corr);
                        sw = __ldg(p.s_w + n);
                    }
                    bs = p.bias ? __ldg(p.bias + n) : 0.f;
                }
                tab[et] = corr; tab[TILE_N + et] = sw; tab[2 * TILE_N + et] = bs;
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_TAB + (n_tile_done & 1)));
            }
#pragma unroll
            for (int i = 0; i < 64; ++i) R[i] = make_float2(0.f, 0.f);
            for (int sgi = 0; sgi < (DEQ ? 1 : p.n_seg); ++sgi) {
                const uint32_t buf = DEQ ? (n_tile_done & 1u) : (uint32_t)s_seg_buf[sgi];
                if (!mbar_wait(bar(B_ACCFULL + buf), (par >> buf) & 1u, s_abort)) { ok = false; break; }
                par ^= 1u << buf;
                tc_fence_after();
                const float sc = s_seg_scale[sgi];
                const float2 sc2 = make_float2(sc, sc);
                const uint32_t taddr = tmem_base + ((uint32_t)(32 * q) << 16) + buf * TILE_N + h * 128;
                if (live) {
                uint32_t va[16], vb[16];
                tc_ld16(taddr, va);
                // ASYM: this cluster's row of the weight tables and my token's code sum
                int64_t tab_row = 0;
                float xs = 0.f, sx = 0.f;
                if constexpr (ASYM) {
                    const int cid = __ldg(p.seg_cluster + sgi);
                    const int m_row = m0 + 32 * q + lane;
                    tab_row = (int64_t)cid * p.ld_w + n0 + h * 128;
                    xs = m_row < p.M ? (float)__ldg(p.xsum + (int64_t)m_row * p.g + cid) : 0.f;
                    sx = sc * 16.0f;                 // s^X_c itself (s_seg_scale carries the 1/16 of the operands)
                }
                // R += s_c * acc, two columns per packed fused multiply-add
                auto accumulate = [&](const uint32_t (&v)[16], int c0) {
                    if constexpr (ASYM) {
                        // R += s^X_c s^W_c[n] (acc' - (z^W_c[n] - 8) xsum): 16 columns, the tables four at a time
                        const int col = 2 * c0;                      // first of these columns within my 128
#pragma unroll
                        for (int i4 = 0; i4 < 4; ++i4) {
                            float sw4[4] = {0.f, 0.f, 0.f, 0.f};
                            int zw4[4] = {8, 8, 8, 8};
                            if (n0 + h * 128 + col + 4 * i4 + 4 <= p.ld_w) {
                                const float4 a = __ldg(reinterpret_cast<const float4*>(p.sw_c + tab_row + col + 4 * i4));
                                const int4 b = __ldg(reinterpret_cast<const int4*>(p.zw_c + tab_row + col + 4 * i4));
                                sw4[0] = a.x; sw4[1] = a.y; sw4[2] = a.z; sw4[3] = a.w;
                                zw4[0] = b.x; zw4[1] = b.y; zw4[2] = b.z; zw4[3] = b.w;
                            }
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int i = 4 * i4 + e;
                                const float t = __fmaf_rn((float)(int)v[i], 0.0625f, -(float)(zw4[e] - 8) * xs);
                                float& r = (i & 1) ? R[c0 + (i >> 1)].y : R[c0 + (i >> 1)].x;
                                r = __fmaf_rn(sx * sw4[e], t, r);
                            }
                        }
                    } else if constexpr (DEQ) {
#pragma unroll
                        for (int i = 0; i < 8; ++i) R[c0 + i] = make_float2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));   // the fp32 sums themselves
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            R[c0 + i] = fma2(sc2, make_float2((float)(int)v[2 * i], (float)(int)v[2 * i + 1]), R[c0 + i]);
                    }
                };
#pragma unroll
                for (int ch = 0; ch < 8; ch += 2) {
                    tc_wait_ld();
                    tc_ld16(taddr + (ch + 1) * 16, vb);
                    accumulate(va, ch * 8);
                    tc_wait_ld();
                    if (ch + 2 < 8) tc_ld16(taddr + (ch + 2) * 16, va);
                    accumulate(vb, (ch + 1) * 8);
                }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) arrive_leader(bar(B_ACCEMPTY + buf));
            }
            if (!ok) break;
            if (!mbar_wait(bar(B_TAB + (n_tile_done & 1)), (n_tile_done >> 1) & 1, s_abort)) { ok = false; break; }
            // y = s_w * (R - corr) + bias, activation, store
            const int m = m0 + 32 * q + lane;
            const int nb = n0 + h * 128;
            const float* t_corr = tab + h * 128;
            const float* t_sw = tab + TILE_N + h * 128;
            const float* t_bs = tab + 2 * TILE_N + h * 128;
            auto Rf = [&](int i) -> float& { return (i & 1) ? R[i >> 1].y : R[i >> 1].x; };
            if (live) {
#pragma unroll
                for (int i = 0; i < 128; ++i) {
                    float v = __fmaf_rn(t_sw[i], Rf(i) - t_corr[i], t_bs[i]);
                    if (p.act == RPTQ_ACT_RELU) v = fmaxf(v, 0.f);
                    Rf(i) = v;
                }
            }
            if (m < p.M) {
                if (p.y_dtype == RPTQ_OUT_F32) {
                    float* dst = static_cast<float*>(p.y) + (int64_t)m * p.ldy + nb;
                    if (nb + 128 <= p.N) {
#pragma unroll
                        for (int i = 0; i < 128; i += 4) *reinterpret_cast<float4*>(dst + i) = make_float4(Rf(i), Rf(i + 1), Rf(i + 2), Rf(i + 3));
                    } else {
#pragma unroll
                        for (int i = 0; i < 128; ++i) if (nb + i < p.N) dst[i] = Rf(i);
                    }
                } else if (p.y_dtype == RPTQ_OUT_F16) {
                    __half* dst = static_cast<__half*>(p.y) + (int64_t)m * p.ldy + nb;
                    if (nb + 128 <= p.N) {
#pragma unroll
                        for (int i = 0; i < 128; i += 8) {
                            __half2 h0 = __floats2half2_rn(Rf(i), Rf(i + 1)), h1 = __floats2half2_rn(Rf(i + 2), Rf(i + 3));
                            __half2 h2 = __floats2half2_rn(Rf(i + 4), Rf(i + 5)), h3 = __floats2half2_rn(Rf(i + 6), Rf(i + 7));
                            uint4 v;
                            v.x = *reinterpret_cast<uint32_t*>(&h0); v.y = *reinterpret_cast<uint32_t*>(&h1);
                            v.z = *reinterpret_cast<uint32_t*>(&h2); v.w = *reinterpret_cast<uint32_t*>(&h3);
                            *reinterpret_cast<uint4*>(dst + i) = v;
                        }
                    } else {
#pragma unroll
                        for (int i = 0; i < 128; ++i) if (nb + i < p.N) dst[i] = __float2half_rn(Rf(i));
                    }
                } else {
                    // re-quantise for the next site: column n is padded position n of the output layout
                    uint8_t* row = static_cast<uint8_t*>(p.y) + (int64_t)m * p.out_row_bytes;
                    const int qmax = (1 << p.out_bits) - 1;
#pragma unroll
                    for (int uu = 0; uu < 4; ++uu) {
                        const int unit = (nb >> 5) + uu;
                        if (nb + 32 * uu >= p.N) break;
                        const uint4 t4 = __ldg(reinterpret_cast<const uint4*>(p.out_unit + unit));
                        const float inv_s = __uint_as_float(t4.x);
                        const int zc = (int)t4.y, nvalid = (int)t4.w;
                        uint32_t qv[32];
#pragma unroll
                        for (int e = 0; e < 32; ++e) qv[e] = e < nvalid ? quant_code(Rf(32 * uu + e), inv_s, zc, qmax) : 0u;
                        if (p.out_bits == 4) {
                            uint32_t w[4]; pack32<4>(qv, w);
                            *reinterpret_cast<uint4*>(row + unit * 16) = make_uint4(w[0], w[1], w[2], w[3]);
                        } else if (p.out_bits == 3) {
                            uint32_t w[3]; pack32<3>(qv, w);
                            uint32_t* d = reinterpret_cast<uint32_t*>(row + unit * 12);
                            d[0] = w[0]; d[1] = w[1]; d[2] = w[2];
                        } else {
                            uint32_t w[8]; pack32<8>(qv, w);
                            uint4* d = reinterpret_cast<uint4*>(row + unit * 32);
                            d[0] = make_uint4(w[0], w[1], w[2], w[3]); d[1] = make_uint4(w[4], w[5], w[6], w[7]);
                        }
                    }
                }
            }
        }
    }

    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if constexpr (NCTA == 2) cluster_sync_all();       // the peer no longer arrives here nor reads this CTA's memory
    tc_fence_after();
    if (warp == 1) {
        if constexpr (NCTA == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
        else asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
    }
    if (tid == 0 && *s_abort && p.status) atomicExch(p.status, RPTQ_ERR_DEVICE_TIMEOUT);
}

// ---------------------------------------------------------------- host side
template <int BITS, int NCTA, bool A8, int MODE>
static int launch(const Params& p, int n_sm, cudaStream_t st)
{
    constexpr SmemLayout SL = smem_layout(NCTA, BITS, A8);
    const int smem = SL.total + 1024;     // slack for the in-kernel 1024-byte alignment
    const void* fn = reinterpret_cast<const void*>(cluster_gemm_kernel<BITS, NCTA, A8, MODE>);
    cudaFuncAttributes attr;
    if (cudaFuncGetAttributes(&attr, fn) != cudaSuccess) return RPTQ_ERR_CUDA;
    // the register re-partition inside the kernel (setmaxnreg) assumes this pool; refuse to launch otherwise
    if (attr.numRegs * THREADS < 128 * (REGS_WG0 + REGS_UNPACK + 2 * REGS_EPI)) return RPTQ_ERR_UNSUPPORTED;
    if (cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return RPTQ_ERR_CUDA;
    const int slots = n_sm / NCTA;
    const int groups = p.n_tiles < slots ? p.n_tiles : slots;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)(groups * NCTA));
    cfg.blockDim = dim3(THREADS);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = NCTA; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, cluster_gemm_kernel<BITS, NCTA, A8, MODE>, p) == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}

}  // namespace gemm
}  // namespace rptq

using namespace rptq;

// Argument checks shared by the entry points. Returns RPTQ_OK when a launch should follow.
static int check_gemm_args(const rptq_layout_t* Lin, const void* a_codes, int M, const void* w_codes,
                           const float* s_w, const int32_t* wsum, int64_t ld_w, const void* bias, int N,
                           int act, const rptq_layout_t* Lout, void* y, int y_dtype, int64_t ldy, int* dev_out)
{
    if (!Lin || !a_codes || !w_codes || !s_w || !wsum || !y) return RPTQ_ERR_INVALID_ARG;
    if (M < 0 || N <= 0 || ld_w < N) return RPTQ_ERR_INVALID_ARG;
    if (act != RPTQ_ACT_NONE && act != RPTQ_ACT_RELU) return RPTQ_ERR_INVALID_ARG;
    if (!aligned16(a_codes) || !aligned16(w_codes) || !aligned16(y) || !aligned16(s_w) || !aligned16(wsum) || !aligned16(bias))
        return RPTQ_ERR_INVALID_ARG;
    if (y_dtype == RPTQ_OUT_F32) {
        if (Lout || ldy < N || (ldy * 4) % 16) return RPTQ_ERR_INVALID_ARG;
    } else if (y_dtype == RPTQ_OUT_F16) {
        if (Lout || ldy < N || (ldy * 2) % 16) return RPTQ_ERR_INVALID_ARG;
    } else if (y_dtype == RPTQ_OUT_CODES) {
        if (!Lout || Lout->K_pad != N) return RPTQ_ERR_INVALID_ARG;
    } else {
        return RPTQ_ERR_INVALID_ARG;
    }
    if (Lin->g > kMaxGemmSegments || Lin->n_units > 2048) return RPTQ_ERR_UNSUPPORTED;
    int dev = -1;
    if (Lin->device < 0 || cudaGetDevice(&dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (dev != Lin->device || (Lout && Lout->device != dev)) return RPTQ_ERR_INVALID_ARG;
    *dev_out = dev;
    return RPTQ_OK;
}

// Fills the launch parameters and launches the variant that fits M. `status` and `corr` may be NULL.
static int launch_gemm(const rptq_layout_t* Lin, const void* a_codes, int M, const void* w_codes,
                       const float* s_w, const int32_t* wsum, int64_t ld_w, const void* bias, int N,
                       int act, const rptq_layout_t* Lout, void* y, int y_dtype, int64_t ldy, void* stream,
                       int dev, int* status, const float* corr,
                       const float* sw_c = nullptr, const int32_t* zw_c = nullptr, const int32_t* xsum = nullptr, bool deq = false)
{
    gemm::Params p{};
    p.M = M; p.N = N; p.n_kb = Lin->K_pad / gemm::KBLK; p.n_seg = Lin->n_seg; p.g = Lin->g;
    // CTA pairs share a 256-row tile; one token tile or less gains nothing from pairing
    const int ncta = M > gemm::TILE_M ? 2 : 1;
    p.tiles_m = (M + gemm::TILE_M * ncta - 1) / (gemm::TILE_M * ncta);
    p.n_tiles = p.tiles_m * ((N + gemm::TILE_N - 1) / gemm::TILE_N);
    p.a_codes = static_cast<const uint8_t*>(a_codes); p.a_row_bytes = Lin->row_bytes;
    p.w_codes = static_cast<const uint8_t*>(w_codes); p.n_wtiles = (int)((ld_w + 127) / 128);
    p.step_flags = Lin->d_step_flags; p.seg_scale = Lin->d_seg_scale; p.seg_buf = Lin->d_seg_buf; p.cl_sz = Lin->d_cl_sz;
    p.s_w = s_w; p.wsum = wsum; p.ld_w = ld_w; p.bias = static_cast<const float*>(bias);
    p.act = act; p.y_dtype = y_dtype; p.y = y; p.ldy = ldy;
    p.out_unit = Lout ? Lout->d_unit : nullptr;
    p.out_bits = Lout ? Lout->bits : 0;
    p.out_row_bytes = Lout ? Lout->row_bytes : 0;
    p.status = status;
    p.corr = corr;
    p.sw_c = sw_c; p.zw_c = zw_c; p.xsum = xsum; p.seg_cluster = Lin->d_seg_cluster; p.cl_n = Lin->d_cl_n;

    int n_sm = 0;
    if (cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    auto st = static_cast<cudaStream_t>(stream);
    // a few tokens (decoding): the kernel that streams the weights through mma.sync with the channels as its M dimension
    if (!deq && !sw_c && y_dtype != RPTQ_OUT_CODES && smallm::fits(M, Lin->bits, Lin->K_pad)) {
        SmallMParams q{};
        q.a = p.a_codes; q.a_row_bytes = p.a_row_bytes; q.M = M; q.K_pad = Lin->K_pad; q.n_units = Lin->n_units; q.n_kb = p.n_kb;
        q.w = p.w_codes; q.n_wtiles = p.n_wtiles;
        q.step_flags = Lin->d_step_flags; q.unit_cluster = Lin->d_unit_cluster; q.unit_sz = Lin->d_unit_sz; q.cl_sz = Lin->d_cl_sz; q.g = Lin->g;
        q.corr = corr; q.s_w = s_w; q.wsum = wsum; q.ld_w = ld_w; q.bias = p.bias;
        q.N = N; q.act = act; q.y_dtype = y_dtype; q.y = y; q.ldy = ldy; q.status = status;
        return smallm::launch(q, Lin->bits, st);
    }
    if (deq) {
        p.unit_sz = Lin->d_unit_sz;
        if (ncta == 2) {
            if (Lin->bits == 3) return gemm::launch<3, 2, false, gemm::MODE_DEQ>(p, n_sm, st);
            if (Lin->bits == 4) return gemm::launch<4, 2, false, gemm::MODE_DEQ>(p, n_sm, st);
            return gemm::launch<8, 2, false, gemm::MODE_DEQ>(p, n_sm, st);
        }
        if (Lin->bits == 3) return gemm::launch<3, 1, false, gemm::MODE_DEQ>(p, n_sm, st);
        if (Lin->bits == 4) return gemm::launch<4, 1, false, gemm::MODE_DEQ>(p, n_sm, st);
        return gemm::launch<8, 1, false, gemm::MODE_DEQ>(p, n_sm, st);
    }
    if (sw_c) {
        if (ncta == 2) {
            if (Lin->bits == 3) return gemm::launch<3, 2, false, gemm::MODE_ASYM>(p, n_sm, st);
            if (Lin->bits == 4) return gemm::launch<4, 2, false, gemm::MODE_ASYM>(p, n_sm, st);
            return gemm::launch<8, 2, true, gemm::MODE_ASYM>(p, n_sm, st);
        }
        if (Lin->bits == 3) return gemm::launch<3, 1, false, gemm::MODE_ASYM>(p, n_sm, st);
        if (Lin->bits == 4) return gemm::launch<4, 1, false, gemm::MODE_ASYM>(p, n_sm, st);
        return gemm::launch<8, 1, false, gemm::MODE_ASYM>(p, n_sm, st);
    }
    if (ncta == 2) {
        if (Lin->bits == 3) return gemm::launch<3, 2, false, gemm::MODE_INT>(p, n_sm, st);
        if (Lin->bits == 4) return gemm::launch<4, 2, false, gemm::MODE_INT>(p, n_sm, st);
        return gemm::launch<8, 2, true, gemm::MODE_INT>(p, n_sm, st);      // 8-bit codes need no unpacking
    }
    if (Lin->bits == 3) return gemm::launch<3, 1, false, gemm::MODE_INT>(p, n_sm, st);
    if (Lin->bits == 4) return gemm::launch<4, 1, false, gemm::MODE_INT>(p, n_sm, st);
    return gemm::launch<8, 1, false, gemm::MODE_INT>(p, n_sm, st);
}

extern "C" int rptq_cluster_gemm_clustered(const rptq_layout_t* Lin, const void* a_codes, int M, const int32_t* xsum,
                                           const void* w_codes, const float* s_w, const int32_t* z_w, const int32_t* wsum,
                                           int64_t ld_w, const void* bias, int N, int act, const rptq_layout_t* Lout,
                                           void* y, int y_dtype, int64_t ldy, void* stream)
{
    int dev = -1;
    const int rc = check_gemm_args(Lin, a_codes, M, w_codes, s_w, wsum, ld_w, bias, N, act, Lout, y, y_dtype, ldy, &dev);
    if (rc != RPTQ_OK) return rc;
    if (!z_w || !xsum || !aligned16(z_w) || !aligned16(xsum)) return RPTQ_ERR_INVALID_ARG;
    if (ld_w % 4 != 0) return RPTQ_ERR_UNSUPPORTED;       // the tables are read four columns at a time
    if (M == 0) return RPTQ_OK;
    int* status = device_status_word();
    if (!status) return RPTQ_ERR_ALLOC;
    return launch_gemm(Lin, a_codes, M, w_codes, nullptr, wsum, ld_w, bias, N, act, Lout, y, y_dtype, ldy, stream, dev, status,
                       nullptr, s_w, z_w, xsum);
}

extern "C" int rptq_cluster_gemm(const rptq_layout_t* Lin, const void* a_codes, int M, const void* w_codes,
                                 const float* s_w, const int32_t* wsum, int64_t ld_w, const void* bias, int N,
                                 int act, const rptq_layout_t* Lout, void* y, int y_dtype, int64_t ldy, void* stream)
{
    int dev = -1;
    const int rc = check_gemm_args(Lin, a_codes, M, w_codes, s_w, wsum, ld_w, bias, N, act, Lout, y, y_dtype, ldy, &dev);
    if (rc != RPTQ_OK) return rc;
    if (M == 0) return RPTQ_OK;
    int* status = device_status_word();
    if (!status) return RPTQ_ERR_ALLOC;
    return launch_gemm(Lin, a_codes, M, w_codes, s_w, wsum, ld_w, bias, N, act, Lout, y, y_dtype, ldy, stream, dev, status, nullptr);
}

extern "C" int rptq_dequant_gemm(const rptq_layout_t* Lin, const void* a_codes, int M, const void* w_codes,
                                 const float* s_w, int64_t ld_w, const void* bias, int N, int act,
                                 void* y, int y_dtype, int64_t ldy, void* stream)
{
    int dev = -1;
    if (y_dtype != RPTQ_OUT_F32 && y_dtype != RPTQ_OUT_F16) return RPTQ_ERR_INVALID_ARG;
    // (the integer tables of the second method are not needed: any aligned non-null pointer passes the shared checks)
    const int rc = check_gemm_args(Lin, a_codes, M, w_codes, s_w, reinterpret_cast<const int32_t*>(s_w), ld_w, bias, N, act,
                                   nullptr, y, y_dtype, ldy, &dev);
    if (rc != RPTQ_OK) return rc;
    if (M == 0) return RPTQ_OK;
    int* status = device_status_word();
    if (!status) return RPTQ_ERR_ALLOC;
    return launch_gemm(Lin, a_codes, M, w_codes, s_w, nullptr, ld_w, bias, N, act, nullptr, y, y_dtype, ldy, stream, dev, status,
                       nullptr, nullptr, nullptr, nullptr, true);
}

// ---------------------------------------------------------------- entry point that allocates nothing
namespace rptq {
namespace gemm {

// Scratch of rptq_cluster_gemm_noalloc: one zero-point correction per output column, resident in
// every device that loads the library (256 KiB) until the process exits.
static __device__ __align__(256) float g_noalloc_corr[RPTQ_NOALLOC_MAX_N];

// corr[n] = sum_c s_c z_c Wsum_c[n], the same fused multiply-adds, in the same order, as the GEMM
// epilogue performs when it is given no table.
__global__ void noalloc_corr_kernel(const float* __restrict__ cl_sz, const int32_t* __restrict__ wsum, int64_t ld_w,
                                    int g, int N, float* __restrict__ corr)
{
    const int n = blockIdx.x * blockDim.x + threadIdx.x;
    if (n >= N) return;
    float acc = 0.f;
    for (int c = 0; c < g; ++c) acc = __fmaf_rn(__ldg(cl_sz + c), (float)__ldg(wsum + (int64_t)c * ld_w + n), acc);
    corr[n] = acc;
}

// Device address of the scratch array, looked up once per device. In host code the array's name
// is only a handle for the runtime; the address a kernel can use comes from cudaGetSymbolAddress
// with that device current.
static int noalloc_scratch(int dev, float** out)
{
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static float* ptrs[kMaxDevices] = {};
    if (dev < 0 || dev >= kMaxDevices) return RPTQ_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_corr) != cudaSuccess || !p) return RPTQ_ERR_CUDA;
        ptrs[dev] = static_cast<float*>(p);
    }
    *out = ptrs[dev];
    return RPTQ_OK;
}

}  // namespace gemm
}  // namespace rptq

extern "C" int rptq_cluster_gemm_noalloc(const rptq_layout_t* Lin, const void* a_codes, int M, const void* w_codes,
                                         const float* s_w, const int32_t* wsum, int64_t ld_w, const void* bias, int N,
                                         int act, const rptq_layout_t* Lout, void* y, int y_dtype, int64_t ldy, void* stream)
{
    int dev = -1;
    int rc = check_gemm_args(Lin, a_codes, M, w_codes, s_w, wsum, ld_w, bias, N, act, Lout, y, y_dtype, ldy, &dev);
    if (rc != RPTQ_OK) return rc;
    if (N > RPTQ_NOALLOC_MAX_N) return RPTQ_ERR_UNSUPPORTED;    // more output columns than the resident table holds
    if (M == 0) return RPTQ_OK;
    float* corr = nullptr;
    rc = gemm::noalloc_scratch(dev, &corr);
    if (rc != RPTQ_OK) return rc;
    auto st = static_cast<cudaStream_t>(stream);
    // Every column the GEMM will read is rewritten here first, so nothing of the previous call's
    // contents survives where it matters and nothing needs to start at zero.
    gemm::noalloc_corr_kernel<<<(N + 255) / 256, 256, 0, st>>>(Lin->d_cl_sz, wsum, ld_w, Lin->g, N, corr);
    if (cudaGetLastError() != cudaSuccess) return RPTQ_ERR_CUDA;
    return launch_gemm(Lin, a_codes, M, w_codes, s_w, wsum, ld_w, bias, N, act, Lout, y, y_dtype, ldy, stream, dev, nullptr, corr);
}
