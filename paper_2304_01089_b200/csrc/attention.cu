// rptq_attention: self-attention on quantised Q, K and V (Sec. 4.2: Q and K share one reorder index;
// Sec. 5.1: the reorders of the attention sites are per head with their own clusters, the softmax
// output is quantised at 8 bits).
//
// One block of four warps handles one head and 64 queries; a warp owns 16 query rows. Codes are
// unpacked to bytes in shared memory and multiplied with mma.sync m16n8k32 (unsigned 8-bit operands,
// int32 sums): one instruction is one unit of 32 head positions of a 16 x 8 block of scores, so a
// cluster's sum is the sum of its units' instructions, scaled once by s^Q_c s^K_c when the cluster
// ends. Of the four terms of (Q_q - z^Q)(K_q - z^K) the two that depend only on the query row shift a
// whole row of scores and cancel in the softmax; the term -z^Q_c sum_p K_q[j][p] is added per key.
//
// The softmax output is quantised from the finished probabilities, so the row maximum and the row sum
// must be known first: pass 1 computes them over all visible keys, pass 2 recomputes the scores,
// forms P_q = min(rne(P / s_P), 255) and multiplies the codes with the V codes, again in integers
// (P_q's zero point is required to be 0). The scores' 16 x 8 accumulator blocks give each thread two
// adjacent keys of a row; four of them (from two blocks) form one operand word of the second product,
// so the keys of a tile enter that product in a permuted order, and the V tile is transposed into
// shared memory in the same order. Pass 2 holds the sums of up to eight V units (a whole head) in
// registers. The packed codes of the next key tile are copied into a staging buffer (cp.async) while
// the current tile is multiplied.
#include <cuda_fp16.h>

#include "rptq_internal.h"
#include "unpack.cuh"

namespace rptq {
namespace attn {

constexpr int BM = 64, BN = 64, THREADS = 128;
constexpr int MAX_UNITS = 8;                 // units of 32 positions per head
constexpr int QK_PITCH_MAX = 32 * MAX_UNITS + 16;
constexpr int V_CHUNK_UNITS = 8;
constexpr int VT_PITCH = BN + 16;
constexpr float NEG_BIG = -1.0e30f;

struct Params {
    const uint8_t *q, *k, *v;
    int64_t q_row_bytes, k_row_bytes, v_row_bytes;
    int bits_q, bits_k, bits_v;
    int Tq, Tk, H, gh_qk, gh_v, causal;     // Tq queries and Tk keys per sequence; blockIdx.z is the sequence
    int n_used_qk, n_used_v;                 // units that belong to a cluster
    const int32_t *unit_cluster_qk, *unit_cluster_v;
    const float2 *unit_sz_q, *unit_sz_k, *unit_sz_v;
    const uint16_t* src_v;                   // channel at each padded position of V's layout
    const int32_t* jidx_v;                   // -1 at pad positions
    float inv_sP, s_P, qk_scale_log2e;
    __half* out;
    int64_t ldo;
    uint8_t* p_dbg;
    int raw_pitch;                           // bytes per key row of the staging buffers for packed codes
};

__device__ __forceinline__ void load_unit(const uint8_t* row, int unit, int bits, uint32_t (&o)[8])
{
    if (bits == 4) {
        const uint4 t = __ldg(reinterpret_cast<const uint4*>(row) + unit);
        const uint32_t p[4] = {t.x, t.y, t.z, t.w};
        unpack_act32<4>(p, o);
    } else if (bits == 3) {
        const uint32_t* w = reinterpret_cast<const uint32_t*>(row) + unit * 3;
        const uint32_t p[3] = {__ldg(w), __ldg(w + 1), __ldg(w + 2)};
        unpack_act32<3>(p, o);
    } else {
        const uint4* w = reinterpret_cast<const uint4*>(row) + unit * 2;
        const uint4 a = __ldg(w), b = __ldg(w + 1);
        o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
    }
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// The same from a staged copy of the packed row in shared memory (`row` points at the head's first unit;
// 4-byte aligned for 3-bit codes, 16-byte aligned otherwise).
__device__ __forceinline__ void load_unit_smem(const uint8_t* row, int unit, int bits, uint32_t (&o)[8])
{
    if (bits == 4) {
        const uint4 t = *(reinterpret_cast<const uint4*>(row) + unit);
        const uint32_t p[4] = {t.x, t.y, t.z, t.w};
        unpack_act32<4>(p, o);
    } else if (bits == 3) {
        const uint32_t* w = reinterpret_cast<const uint32_t*>(row) + unit * 3;
        const uint32_t p[3] = {w[0], w[1], w[2]};
        unpack_act32<3>(p, o);
    } else {
        const uint4* w = reinterpret_cast<const uint4*>(row) + unit * 2;
        const uint4 a = w[0], b = w[1];
        o[0] = a.x; o[1] = a.y; o[2] = a.z; o[3] = a.w; o[4] = b.x; o[5] = b.y; o[6] = b.z; o[7] = b.w;
    }
}
// 16 bytes global -> shared without passing through registers; src_bytes = 0 writes zeros
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_u8(int (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// first unit whose cluster is >= c among the first n units (their clusters do not decrease)
__device__ __forceinline__ int first_unit_of(const int32_t* unit_cluster, int n, int c)
{
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(unit_cluster + mid) < c) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// Key of the tile that sits in slot s (0..63) of the second product's contraction: slots 4t..4t+3 of a
// 16-slot half hold keys 2t, 2t+1, 8+2t, 8+2t+1 of the half's 16 keys.
__device__ __forceinline__ int key_of_slot(int s)
{
    const int b = s & 3, t = (s >> 2) & 3;
    return (s & ~15) + 8 * (b >> 1) + 2 * t + (b & 1);
}

__global__ void __launch_bounds__(THREADS)
attention_kernel(const Params p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    __shared__ int s_rng[4];
    __shared__ float s_coef[MAX_UNITS], s_czq[MAX_UNITS], s_col[BN];
    __shared__ uint8_t s_last[MAX_UNITS];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g8 = lane >> 2, t4 = lane & 3;
    const int h = blockIdx.y;
    const int64_t q_row0 = (int64_t)blockIdx.z * p.Tq, k_row0 = (int64_t)blockIdx.z * p.Tk;      // this sequence's first rows
    const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;      // the tiles with the most visible keys first
    const int i0 = qt * BM;

    if (tid == 0) {
        s_rng[0] = first_unit_of(p.unit_cluster_qk, p.n_used_qk, h * p.gh_qk);
        s_rng[1] = first_unit_of(p.unit_cluster_qk, p.n_used_qk, (h + 1) * p.gh_qk);
        s_rng[2] = first_unit_of(p.unit_cluster_v, p.n_used_v, h * p.gh_v);
        s_rng[3] = first_unit_of(p.unit_cluster_v, p.n_used_v, (h + 1) * p.gh_v);
    }
    __syncthreads();
    const int uq0 = s_rng[0], nuq = s_rng[1] - s_rng[0], uv0 = s_rng[2], nuv = s_rng[3] - s_rng[2];
    const int pitch = 32 * nuq + 16;
    uint8_t* Qs = smem;
    uint8_t* Ks = Qs + BM * QK_PITCH_MAX;
    uint8_t* Vt = Ks + BN * QK_PITCH_MAX;
    uint8_t* rawK = Vt + 32 * V_CHUNK_UNITS * VT_PITCH;         // [2][BN][raw_pitch] packed K codes of a tile, as they lie in memory
    uint8_t* rawV = rawK + 2 * BN * p.raw_pitch;
    // a head's packed codes are a contiguous piece of a row; the staged window starts at the 16-byte boundary below it
    const int bytesK = 4 * p.bits_k, bytesV = 4 * p.bits_v;
    const int winK = (bytesK * uq0) & ~15, offK = bytesK * uq0 - winK, nK16 = (offK + bytesK * nuq + 15) >> 4;
    const int winV = (bytesV * uv0) & ~15, offV = bytesV * uv0 - winV, nV16 = (offV + bytesV * nuv + 15) >> 4;

    if (tid < nuq) {
        const float2 q = __ldg(p.unit_sz_q + uq0 + tid), k = __ldg(p.unit_sz_k + uq0 + tid);
        const float c = q.x * k.x * p.qk_scale_log2e;
        s_coef[tid] = c;
        s_czq[tid] = -c * q.y;
        s_last[tid] = (tid == nuq - 1) || (__ldg(p.unit_cluster_qk + uq0 + tid + 1) != __ldg(p.unit_cluster_qk + uq0 + tid));
    }
    // the queries' codes, as bytes
    for (int it = tid; it < BM * nuq; it += THREADS) {
        const int r = it / nuq, u = it - r * nuq;
        uint32_t o[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (i0 + r < p.Tq) load_unit(p.q + (q_row0 + i0 + r) * p.q_row_bytes, uq0 + u, p.bits_q, o);
        uint4* d = reinterpret_cast<uint4*>(Qs + r * pitch + 32 * u);
        d[0] = make_uint4(o[0], o[1], o[2], o[3]);
        d[1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
    __syncthreads();

    const int off = p.Tk - p.Tq;
    const int last_vis_tile = p.causal ? min(p.Tk - 1, i0 + BM - 1 + off) : p.Tk - 1;
    const int n_kt = last_vis_tile / BN + 1;
    const int row0 = i0 + 16 * warp + g8, row1 = row0 + 8;
    const int vis0 = p.causal ? min(p.Tk - 1, row0 + off) : p.Tk - 1;
    const int vis1 = p.causal ? min(p.Tk - 1, row1 + off) : p.Tk - 1;

    // Start the copies of key tile kt (and its V tile) into staging buffer kt & 1; rows past the last key are zero-filled.
    auto stage_tile = [&](int kt, bool with_v) {
        const int buf = kt & 1;
        for (int it = tid; it < BN * nK16; it += THREADS) {
            const int r = it / nK16, c = it - r * nK16, j = kt * BN + r;
            cp_async16(smem_u32(rawK + (buf * BN + r) * p.raw_pitch + 16 * c),
                       p.k + (k_row0 + min(j, p.Tk - 1)) * p.k_row_bytes + winK + 16 * c, j < p.Tk ? 16 : 0);
        }
        if (with_v)
            for (int it = tid; it < BN * nV16; it += THREADS) {
                const int r = it / nV16, c = it - r * nV16, j = kt * BN + r;
                cp_async16(smem_u32(rawV + (buf * BN + r) * p.raw_pitch + 16 * c),
                           p.v + (k_row0 + min(j, p.Tk - 1)) * p.v_row_bytes + winV + 16 * c, j < p.Tk ? 16 : 0);
            }
        cp_async_commit();
    };
    // Tile kt has been staged and a block-wide barrier passed since: unpack it to bytes
    auto load_k_tile = [&](int kt) {
        const uint8_t* raw = rawK + (kt & 1) * BN * p.raw_pitch + offK;
        for (int it = tid; it < BN * nuq; it += THREADS) {
            const int r = it / nuq, u = it - r * nuq;
            uint32_t o[8];
            load_unit_smem(raw + r * p.raw_pitch, u, p.bits_k, o);
            uint4* d = reinterpret_cast<uint4*>(Ks + r * pitch + 32 * u);
            d[0] = make_uint4(o[0], o[1], o[2], o[3]);
            d[1] = make_uint4(o[4], o[5], o[6], o[7]);
        }
        __syncthreads();
        if (tid < BN) {                      // the per-key term  - sum_c s^Q s^K z^Q_c sum_p K_q
            float c = 0.f;
            for (int u = 0; u < nuq; ++u) {
                const uint4* w = reinterpret_cast<const uint4*>(Ks + tid * pitch + 32 * u);
                const uint4 a = w[0], b = w[1];
                unsigned s = 0;
                s = __dp4a(a.x, 0x01010101u, s); s = __dp4a(a.y, 0x01010101u, s);
                s = __dp4a(a.z, 0x01010101u, s); s = __dp4a(a.w, 0x01010101u, s);
                s = __dp4a(b.x, 0x01010101u, s); s = __dp4a(b.y, 0x01010101u, s);
                s = __dp4a(b.z, 0x01010101u, s); s = __dp4a(b.w, 0x01010101u, s);
                c = __fmaf_rn(s_czq[u], (float)s, c);
            }
            s_col[tid] = c;
        }
        __syncthreads();
    };

    // scores of my 16 rows against the 64 keys of the tile, times log2(e), hidden keys at NEG_BIG
    auto scores = [&](int kt, float (&S)[8][4]) {
        int acc[8][4];
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) { S[n][e] = 0.f; acc[n][e] = 0; }
        const uint32_t q_addr = smem_u32(Qs + (16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1)) * pitch + 16 * (lane >> 4));
        const uint32_t k_addr = smem_u32(Ks + ((lane & 7) + 8 * (lane >> 4)) * pitch + 16 * ((lane >> 3) & 1));
        for (int u = 0; u < nuq; ++u) {
            uint32_t a[4];
            ldsm4(q_addr + 32 * u, a);
#pragma unroll
            for (int n = 0; n < 8; n += 2) {
                uint32_t b[4];
                ldsm4(k_addr + 8 * n * pitch + 32 * u, b);
                mma_u8(acc[n], a, b[0], b[1]);
                mma_u8(acc[n + 1], a, b[2], b[3]);
            }
            if (s_last[u]) {
                const float c = s_coef[u];
#pragma unroll
                for (int n = 0; n < 8; ++n)
#pragma unroll
                    for (int e = 0; e < 4; ++e) { S[n][e] = __fmaf_rn(c, (float)acc[n][e], S[n][e]); acc[n][e] = 0; }
            }
        }
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int j = kt * BN + 8 * n + 2 * t4 + (e & 1);
                const float v = S[n][e] + s_col[8 * n + 2 * t4 + (e & 1)];
                S[n][e] = j <= ((e & 2) ? vis1 : vis0) ? v : NEG_BIG;
            }
    };

    // ---------------------------------------------------------------- pass 1: row maximum and row sum
    float m0 = NEG_BIG, m1 = NEG_BIG, l0 = 0.f, l1 = 0.f;
    stage_tile(0, false);
    for (int kt = 0; kt < n_kt; ++kt) {
        if (kt + 1 < n_kt) { stage_tile(kt + 1, false); cp_async_wait<1>(); } else cp_async_wait<0>();
        __syncthreads();                     // everyone's copies of tile kt have landed
        load_k_tile(kt);
        float S[8][4];
        scores(kt, S);
        float x0 = NEG_BIG, x1 = NEG_BIG;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            x0 = fmaxf(x0, fmaxf(S[n][0], S[n][1]));
            x1 = fmaxf(x1, fmaxf(S[n][2], S[n][3]));
        }
        x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, 1)); x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, 2));
        x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, 1)); x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, 2));
        const float n0 = fmaxf(m0, x0), n1 = fmaxf(m1, x1);
        float a0 = 0.f, a1 = 0.f;
#pragma unroll
        for (int n = 0; n < 8; ++n) {
            a0 += ex2(S[n][0] - n0) + ex2(S[n][1] - n0);
            a1 += ex2(S[n][2] - n1) + ex2(S[n][3] - n1);
        }
        l0 = l0 * ex2(m0 - n0) + a0;
        l1 = l1 * ex2(m1 - n1) + a1;
        m0 = n0; m1 = n1;
        __syncthreads();                     // every warp is done with this tile
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float f0 = p.inv_sP / l0, f1 = p.inv_sP / l1;      // code = rne(2^(S - m) f)

    // ---------------------------------------------------------------- pass 2: P_q and P_q V_q, 128 positions of V at a time
    for (int c0 = 0; c0 < nuv; c0 += V_CHUNK_UNITS) {
        const int cu = min(V_CHUNK_UNITS, nuv - c0);
        int O[4 * V_CHUNK_UNITS][4];
#pragma unroll
        for (int n = 0; n < 4 * V_CHUNK_UNITS; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) O[n][e] = 0;
        int rs0 = 0, rs1 = 0;                // sums of my rows' codes (this thread's keys)
        stage_tile(0, true);
        for (int kt = 0; kt < n_kt; ++kt) {
            if (kt + 1 < n_kt) { stage_tile(kt + 1, true); cp_async_wait<1>(); } else cp_async_wait<0>();
            __syncthreads();                 // everyone's copies of tile kt have landed
            load_k_tile(kt);
            // V tile, transposed: Vt[position][slot] = code of key key_of_slot(slot)
            const uint8_t* rawv = rawV + (kt & 1) * BN * p.raw_pitch + offV;
            for (int it = tid; it < cu * 16; it += THREADS) {
                const int u = it >> 4, w = it & 15;
                uint32_t o[4][8];
#pragma unroll
                for (int b = 0; b < 4; ++b)
                    load_unit_smem(rawv + key_of_slot(4 * w + b) * p.raw_pitch, c0 + u, p.bits_v, o[b]);
#pragma unroll
                for (int e = 0; e < 8; ++e) {        // positions 4e..4e+3 of the unit: a 4 x 4 byte transpose
                    const uint32_t x01l = __byte_perm(o[0][e], o[1][e], 0x5140), x01h = __byte_perm(o[0][e], o[1][e], 0x7362);
                    const uint32_t x23l = __byte_perm(o[2][e], o[3][e], 0x5140), x23h = __byte_perm(o[2][e], o[3][e], 0x7362);
                    uint8_t* d = Vt + (32 * u + 4 * e) * VT_PITCH + 4 * w;
                    *reinterpret_cast<uint32_t*>(d) = __byte_perm(x01l, x23l, 0x5410);
                    *reinterpret_cast<uint32_t*>(d + VT_PITCH) = __byte_perm(x01l, x23l, 0x7632);
                    *reinterpret_cast<uint32_t*>(d + 2 * VT_PITCH) = __byte_perm(x01h, x23h, 0x5410);
                    *reinterpret_cast<uint32_t*>(d + 3 * VT_PITCH) = __byte_perm(x01h, x23h, 0x7632);
                }
            }
            float S[8][4];
            scores(kt, S);
            uint32_t pa[2][4];               // the codes as the first operand of the second product, per 32 keys
#pragma unroll
            for (int ks = 0; ks < 2; ++ks)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const int n = 4 * ks + 2 * half;
                    int c[2][4];
#pragma unroll
                    for (int b = 0; b < 2; ++b)
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            c[b][e] = min(__float2int_rn(ex2(S[n + b][e] - ((e & 2) ? m1 : m0)) * ((e & 2) ? f1 : f0)), 255);
                    rs0 += c[0][0] + c[0][1] + c[1][0] + c[1][1];
                    rs1 += c[0][2] + c[0][3] + c[1][2] + c[1][3];
                    pa[ks][2 * half] = (uint32_t)c[0][0] | ((uint32_t)c[0][1] << 8) | ((uint32_t)c[1][0] << 16) | ((uint32_t)c[1][1] << 24);
                    pa[ks][2 * half + 1] = (uint32_t)c[0][2] | ((uint32_t)c[0][3] << 8) | ((uint32_t)c[1][2] << 16) | ((uint32_t)c[1][3] << 24);
                    if (p.p_dbg && c0 == 0) {
#pragma unroll
                        for (int b = 0; b < 2; ++b)
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int i = (e & 2) ? row1 : row0, j = kt * BN + 8 * (n + b) + 2 * t4 + (e & 1);
                                if (i < p.Tq && j < p.Tk) p.p_dbg[(((int64_t)blockIdx.z * p.H + h) * p.Tq + i) * p.Tk + j] = (uint8_t)c[b][e];
                            }
                    }
                }
            __syncthreads();                 // Vt is complete
            const uint32_t v_addr = smem_u32(Vt + (lane & 7) * VT_PITCH + 16 * (lane >> 3));
#pragma unroll
            for (int n = 0; n < 4 * V_CHUNK_UNITS; ++n) {
                if (n < 4 * cu) {
                    uint32_t b[4];
                    ldsm4(v_addr + 8 * n * VT_PITCH, b);
                    mma_u8(O[n], pa[0], b[0], b[1]);
                    mma_u8(O[n], pa[1], b[2], b[3]);
                }
            }
            __syncthreads();                 // every warp is done with Ks and Vt
        }
        rs0 += __shfl_xor_sync(0xffffffffu, rs0, 1); rs0 += __shfl_xor_sync(0xffffffffu, rs0, 2);
        rs1 += __shfl_xor_sync(0xffffffffu, rs1, 1); rs1 += __shfl_xor_sync(0xffffffffu, rs1, 2);
        // O = s_P s^V_c (sum_j P_q V_q - z^V_c sum_j P_q), written at the position's channel
#pragma unroll
        for (int n = 0; n < 4 * V_CHUNK_UNITS; ++n) {
            if (n < 4 * cu) {
                const int unit = uv0 + c0 + (n >> 2);
                const float2 sz = __ldg(p.unit_sz_v + unit);
                const float sc = p.s_P * sz.x;
                const int zv = (int)sz.y;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int pos = 32 * unit + 8 * (n & 3) + 2 * t4 + (e & 1);
                    const int i = (e & 2) ? row1 : row0;
                    if (i < p.Tq && __ldg(p.jidx_v + pos) >= 0)
                        p.out[(q_row0 + i) * p.ldo + __ldg(p.src_v + pos)] = __float2half_rn(sc * (float)(O[n][e] - zv * ((e & 2) ? rs1 : rs0)));
                }
            }
        }
    }
}

}  // namespace attn
}  // namespace rptq

static bool units_in_cluster_order(const rptq_layout_t* L, int* n_used)
{
    int prev = 0, n = 0;
    for (int u = 0; u < L->n_units; ++u) {
        const int c = L->unit_cluster[u];
        if (c < 0) { for (int v = u; v < L->n_units; ++v) if (L->unit_cluster[v] >= 0) return false; break; }
        if (c < prev) return false;
        prev = c;
        ++n;
    }
    *n_used = n;
    return true;
}

static int max_units_per_head(const rptq_layout_t* L, int n_used, int H)
{
    const int gh = L->g / H;
    std::vector<int> cnt((size_t)H, 0);
    for (int u = 0; u < n_used; ++u) ++cnt[(size_t)(L->unit_cluster[u] / gh)];
    int m = 0;
    for (int c : cnt) m = c > m ? c : m;
    return m;
}

extern "C" int rptq_attention(const rptq_layout_t* LQ, const rptq_layout_t* LK, const rptq_layout_t* LV, int n_heads,
                              const void* q_codes, int Tq, const void* k_codes, const void* v_codes, int Tk, int n_seq,
                              float s_P, int z_P, float qk_scale, int causal,
                              void* out_f16, int64_t ldo, uint8_t* p_codes_out, void* stream)
{
    using namespace rptq;
    using namespace rptq::attn;
    if (!LQ || !LK || !LV || !q_codes || !k_codes || !v_codes || !out_f16) return RPTQ_ERR_INVALID_ARG;
    if (n_heads < 1 || Tq < 0 || Tk < Tq || n_seq < 0 || !(s_P > 0.f) || !(qk_scale >= 0.f)) return RPTQ_ERR_INVALID_ARG;
    if (LQ->g % n_heads || LK->g != LQ->g || LV->g % n_heads || ldo < LV->C) return RPTQ_ERR_INVALID_ARG;
    if (!aligned16(q_codes) || !aligned16(k_codes) || !aligned16(v_codes) || (reinterpret_cast<uintptr_t>(out_f16) & 1u)) return RPTQ_ERR_INVALID_ARG;
    // Q and K pair equal positions: same reorder index, same cluster sizes, same placement
    if (LQ->C != LK->C || LQ->size != LK->size || LQ->perm != LK->perm || LQ->pos != LK->pos || LQ->unit_cluster != LK->unit_cluster)
        return RPTQ_ERR_INVALID_ARG;
    if (z_P != 0 || n_heads > 65535 || n_seq > 65535) return RPTQ_ERR_UNSUPPORTED;
    int n_used_qk = 0, n_used_v = 0;
    if (!units_in_cluster_order(LQ, &n_used_qk) || !units_in_cluster_order(LV, &n_used_v)) return RPTQ_ERR_UNSUPPORTED;
    if (max_units_per_head(LQ, n_used_qk, n_heads) > MAX_UNITS || max_units_per_head(LV, n_used_v, n_heads) > MAX_UNITS) return RPTQ_ERR_UNSUPPORTED;
    if ((int64_t)Tk * 255 * 255 > 2147483647ll) return RPTQ_ERR_UNSUPPORTED;      // the int32 sums of the second product
    if (Tq == 0 || n_seq == 0) return RPTQ_OK;
    int dev = -1;
    if (LQ->device < 0 || cudaGetDevice(&dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (dev != LQ->device || dev != LK->device || dev != LV->device) return RPTQ_ERR_INVALID_ARG;

    Params p{};
    p.q = static_cast<const uint8_t*>(q_codes); p.k = static_cast<const uint8_t*>(k_codes); p.v = static_cast<const uint8_t*>(v_codes);
    p.q_row_bytes = LQ->row_bytes; p.k_row_bytes = LK->row_bytes; p.v_row_bytes = LV->row_bytes;
    p.bits_q = LQ->bits; p.bits_k = LK->bits; p.bits_v = LV->bits;
    p.Tq = Tq; p.Tk = Tk; p.H = n_heads; p.gh_qk = LQ->g / n_heads; p.gh_v = LV->g / n_heads; p.causal = causal ? 1 : 0;
    p.n_used_qk = n_used_qk; p.n_used_v = n_used_v;
    p.unit_cluster_qk = LQ->d_unit_cluster; p.unit_cluster_v = LV->d_unit_cluster;
    p.unit_sz_q = LQ->d_unit_sz; p.unit_sz_k = LK->d_unit_sz; p.unit_sz_v = LV->d_unit_sz;
    p.src_v = LV->d_src; p.jidx_v = LV->d_jidx;
    p.inv_sP = 1.0f / s_P; p.s_P = s_P; p.qk_scale_log2e = qk_scale * 1.4426950408889634f;
    p.out = static_cast<__half*>(out_f16); p.ldo = ldo; p.p_dbg = p_codes_out;

    const int max_bits = LK->bits > LV->bits ? LK->bits : LV->bits;
    p.raw_pitch = 4 * max_bits * MAX_UNITS + 32;          // a head's packed codes plus the alignment slack, a multiple of 16
    const int smem = (BM + BN) * QK_PITCH_MAX + 32 * V_CHUNK_UNITS * VT_PITCH + 4 * BN * p.raw_pitch;
    if (cudaFuncSetAttribute(attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return RPTQ_ERR_CUDA;
    const dim3 grid((unsigned)((Tq + BM - 1) / BM), (unsigned)n_heads, (unsigned)n_seq);
    attention_kernel<<<grid, THREADS, smem, static_cast<cudaStream_t>(stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}
