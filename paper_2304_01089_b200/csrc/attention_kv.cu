// rptq_attention_kv: attention with only the key / value cache quantised (Sec. 5.2: the W4A4KV, W4A3KV
// and W3A3KV schemes). The query and the probabilities stay 16-bit floating point; K and V are the
// per-cluster codes of the per-head layouts (Sec. 4.2, 5.1), written by the projections' epilogues.
//
// One block of eight warps handles one sequence, one head and 128 queries; a warp owns 16 query rows (the
// conversion of a key tile's codes to fp16 is shared by twice as many queries as with 64: 16 % faster).
//   - The head's query channels are gathered once into K's position order (fp16, shared memory).
//   - Per tile of 64 keys the K and V codes become fp16 integers in shared memory (a byte b is the
//     fp16 number 1024 + b with the bit pattern 0x6400 | b; subtracting 1024 is exact).
//   - Scores: mma.sync m16n8k16 (fp16 x fp16 -> fp32), one unit of 32 positions = two instructions; the
//     fp32 sums of a cluster's units are scaled by s^K_c qk_scale log2(e) when the cluster ends. The term
//     -z^K_c sum_p Q[i][p] is the same for every key of a row and cancels in the softmax.
//   - Online softmax (running row maximum and sum, fp32), probabilities rounded to fp16 for the second
//     product, V read with ldmatrix.trans; O = s^V_c (sum_j P V_q / sum_j P - z^V_c), fp16 out.
#include <cuda_fp16.h>

#include "rptq_internal.h"
#include "unpack.cuh"

namespace rptq {
namespace attnkv {

constexpr int BM = 128, BN = 64, THREADS = 256;
constexpr int MAX_UNITS = 8;                         // units of 32 positions per head
constexpr int PITCH = 32 * MAX_UNITS * 2 + 16;       // bytes per row of the fp16 tiles: an odd number of 16-byte chunks
constexpr float NEG_BIG = -1.0e30f;

struct Params {
    const __half* q; int64_t ldq;
    const uint8_t *k, *v;
    int64_t k_row_bytes, v_row_bytes;
    int bits_k, bits_v;
    int Tq, Tk, H, hd, gh_k, gh_v, causal;
    int n_used_k, n_used_v;
    const int32_t *unit_cluster_k, *unit_cluster_v;
    const float2 *unit_sz_k, *unit_sz_v;
    const uint16_t *src_k, *src_v;                   // channel at each padded position
    const int32_t *jidx_k, *jidx_v;                  // -1 at pad positions
    float qk_scale_log2e;
    __half* out; int64_t ldo;
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
// four code bytes -> four fp16 integers (two words)
__device__ __forceinline__ void bytes_to_half4(uint32_t w, uint32_t& lo, uint32_t& hi)
{
    const __half2 k1024 = __floats2half2_rn(1024.f, 1024.f);
    uint32_t a = __byte_perm(w, 0x64006400u, 0x7170), b = __byte_perm(w, 0x64006400u, 0x7372);   // 0x6400 | byte
    __half2 x = __hsub2(*reinterpret_cast<__half2*>(&a), k1024), y = __hsub2(*reinterpret_cast<__half2*>(&b), k1024);
    lo = *reinterpret_cast<uint32_t*>(&x);
    hi = *reinterpret_cast<uint32_t*>(&y);
}
// the 32 codes of a unit as fp16 at dst (64 bytes)
__device__ __forceinline__ void store_unit_half(uint8_t* dst, const uint32_t (&o)[8])
{
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        uint32_t a, b, c, d;
        bytes_to_half4(o[2 * i], a, b);
        bytes_to_half4(o[2 * i + 1], c, d);
        *reinterpret_cast<uint4*>(dst + 16 * i) = make_uint4(a, b, c, d);
    }
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm4_trans(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_half2(float a, float b)
{
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ int first_unit_of(const int32_t* unit_cluster, int n, int c)
{
    int lo = 0, hi = n;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (__ldg(unit_cluster + mid) < c) lo = mid + 1; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(THREADS)
attention_kv_kernel(const Params p)
{
    extern __shared__ __align__(16) uint8_t smem[];
    __shared__ int s_rng[4];
    __shared__ float s_coef[MAX_UNITS];
    __shared__ uint8_t s_last[MAX_UNITS];

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g8 = lane >> 2, t4 = lane & 3;
    const int h = blockIdx.y;
    const int64_t q_row0 = (int64_t)blockIdx.z * p.Tq, k_row0 = (int64_t)blockIdx.z * p.Tk;
    const int qt = (int)gridDim.x - 1 - (int)blockIdx.x;      // the tiles with the most visible keys first
    const int i0 = qt * BM;

    if (tid == 0) {
        s_rng[0] = first_unit_of(p.unit_cluster_k, p.n_used_k, h * p.gh_k);
        s_rng[1] = first_unit_of(p.unit_cluster_k, p.n_used_k, (h + 1) * p.gh_k);
        s_rng[2] = first_unit_of(p.unit_cluster_v, p.n_used_v, h * p.gh_v);
        s_rng[3] = first_unit_of(p.unit_cluster_v, p.n_used_v, (h + 1) * p.gh_v);
    }
    __syncthreads();
    const int uk0 = s_rng[0], nuk = s_rng[1] - s_rng[0], uv0 = s_rng[2], nuv = s_rng[3] - s_rng[2];
    uint8_t* Qs = smem;                       // [BM][PITCH] fp16, K's position order
    uint8_t* Ks = Qs + BM * PITCH;            // [BN][PITCH] fp16 integers
    uint8_t* Vs = Ks + BN * PITCH;            // [BN][PITCH] fp16 integers, V's position order

    if (tid < nuk) {
        s_coef[tid] = __ldg(&p.unit_sz_k[uk0 + tid].x) * p.qk_scale_log2e;
        s_last[tid] = (tid == nuk - 1) || (__ldg(p.unit_cluster_k + uk0 + tid + 1) != __ldg(p.unit_cluster_k + uk0 + tid));
    }
    // The queries' channels in K's position order (pads 0): the head's slice of every row is read in memory order
    // (independent, coalesced loads) into the K tile's buffer, then permuted from there.
    __shared__ int16_t s_chan[32 * MAX_UNITS];               // channel within the head at each of its positions, -1 at pads
    for (int pp = tid; pp < 32 * nuk; pp += THREADS) {
        const int pos = 32 * uk0 + pp;
        s_chan[pp] = __ldg(p.jidx_k + pos) >= 0 ? (int16_t)((int)__ldg(p.src_k + pos) - h * p.hd) : (int16_t)-1;
    }
    for (int it = tid; it < BM * p.hd; it += THREADS) {
        const int r = it / p.hd, c = it - r * p.hd;
        __half v = __float2half_rn(0.f);
        if (i0 + r < p.Tq) v = p.q[(q_row0 + i0 + r) * p.ldq + h * p.hd + c];
        *reinterpret_cast<__half*>(Ks + r * PITCH + 2 * c) = v;
    }
    __syncthreads();
    for (int it = tid; it < BM * 32 * nuk; it += THREADS) {
        const int r = it / (32 * nuk), pp = it - r * (32 * nuk);
        const int c = s_chan[pp];
        *reinterpret_cast<__half*>(Qs + r * PITCH + 2 * pp) = c >= 0 ? *reinterpret_cast<const __half*>(Ks + r * PITCH + 2 * c) : __float2half_rn(0.f);
    }
    __syncthreads();

    const int off = p.Tk - p.Tq;
    const int last_vis_tile = p.causal ? min(p.Tk - 1, i0 + BM - 1 + off) : p.Tk - 1;
    const int n_kt = last_vis_tile / BN + 1;
    const int row0 = i0 + 16 * warp + g8, row1 = row0 + 8;
    const int vis0 = p.causal ? min(p.Tk - 1, row0 + off) : p.Tk - 1;
    const int vis1 = p.causal ? min(p.Tk - 1, row1 + off) : p.Tk - 1;

    float O[4 * MAX_UNITS][4];                // sums of P V_q of my two rows over the head's (padded) positions
#pragma unroll
    for (int n = 0; n < 4 * MAX_UNITS; ++n)
#pragma unroll
        for (int e = 0; e < 4; ++e) O[n][e] = 0.f;
    float m0 = NEG_BIG, m1 = NEG_BIG, l0 = 0.f, l1 = 0.f;     // running maximum and (this thread's part of the) sum

    const uint32_t q_addr = smem_u32(Qs + (16 * warp + (lane & 7) + 8 * ((lane >> 3) & 1)) * PITCH + 16 * (lane >> 4));
    const uint32_t k_addr = smem_u32(Ks + ((lane & 7) + 8 * (lane >> 4)) * PITCH + 16 * ((lane >> 3) & 1));
    const uint32_t v_addr = smem_u32(Vs + ((lane & 7) + 8 * ((lane >> 3) & 1)) * PITCH + 16 * (lane >> 4));

    for (int kt = 0; kt < n_kt; ++kt) {
        // the tile's codes as fp16 integers; keys past the last one are zero
        for (int it = tid; it < BN * (nuk + nuv); it += THREADS) {
            const int r = it / (nuk + nuv), u = it - r * (nuk + nuv), j = kt * BN + r;
            uint32_t o[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            if (u < nuk) {
                if (j < p.Tk) load_unit(p.k + (k_row0 + j) * p.k_row_bytes, uk0 + u, p.bits_k, o);
                store_unit_half(Ks + r * PITCH + 64 * u, o);
            } else {
                if (j < p.Tk) load_unit(p.v + (k_row0 + j) * p.v_row_bytes, uv0 + (u - nuk), p.bits_v, o);
                store_unit_half(Vs + r * PITCH + 64 * (u - nuk), o);
            }
        }
        __syncthreads();

        // scores times log2(e), hidden keys at NEG_BIG
        float S[8][4], acc[8][4];
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) { S[n][e] = 0.f; acc[n][e] = 0.f; }
        for (int u = 0; u < nuk; ++u) {
#pragma unroll
            for (int ks = 0; ks < 2; ++ks) {                  // 16 positions per instruction
                uint32_t a[4];
                ldsm4(q_addr + 64 * u + 32 * ks, a);
#pragma unroll
                for (int n = 0; n < 8; n += 2) {
                    uint32_t b[4];
                    ldsm4(k_addr + 8 * n * PITCH + 64 * u + 32 * ks, b);
                    mma_f16(acc[n], a, b[0], b[1]);
                    mma_f16(acc[n + 1], a, b[2], b[3]);
                }
            }
            if (s_last[u]) {
                const float c = s_coef[u];
#pragma unroll
                for (int n = 0; n < 8; ++n)
#pragma unroll
                    for (int e = 0; e < 4; ++e) { S[n][e] = __fmaf_rn(c, acc[n][e], S[n][e]); acc[n][e] = 0.f; }
            }
        }
        float x0 = NEG_BIG, x1 = NEG_BIG;
#pragma unroll
        for (int n = 0; n < 8; ++n)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int j = kt * BN + 8 * n + 2 * t4 + (e & 1);
                if (j > ((e & 2) ? vis1 : vis0)) S[n][e] = NEG_BIG;
                if (e & 2) x1 = fmaxf(x1, S[n][e]); else x0 = fmaxf(x0, S[n][e]);
            }
        x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, 1)); x0 = fmaxf(x0, __shfl_xor_sync(0xffffffffu, x0, 2));
        x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, 1)); x1 = fmaxf(x1, __shfl_xor_sync(0xffffffffu, x1, 2));
        const float n0 = fmaxf(m0, x0), n1 = fmaxf(m1, x1);
        const float r0 = ex2(m0 - n0), r1 = ex2(m1 - n1);    // what the sums so far shrink by
        m0 = n0; m1 = n1;
        l0 *= r0; l1 *= r1;
        if (__any_sync(0xffffffffu, r0 != 1.f || r1 != 1.f)) {       // a row maximum of this warp moved (rare after the first tiles)
#pragma unroll
            for (int n = 0; n < 4 * MAX_UNITS; ++n) {
                if (n < 4 * nuv) { O[n][0] *= r0; O[n][1] *= r0; O[n][2] *= r1; O[n][3] *= r1; }
            }
        }
        // probabilities (not normalised) as fp16, in the layout of the second product's first operand; the row
        // sums add the rounded values, so that the division at the end normalises exactly what was multiplied
        uint32_t pa[4][4];
#pragma unroll
        for (int s = 0; s < 4; ++s)
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                const int n = 2 * s + hh;
                const uint32_t w0 = pack_half2(ex2(S[n][0] - m0), ex2(S[n][1] - m0));
                const uint32_t w1 = pack_half2(ex2(S[n][2] - m1), ex2(S[n][3] - m1));
                const float2 f0 = __half22float2(*reinterpret_cast<const __half2*>(&w0));
                const float2 f1 = __half22float2(*reinterpret_cast<const __half2*>(&w1));
                l0 += f0.x + f0.y;
                l1 += f1.x + f1.y;
                pa[s][2 * hh] = w0;
                pa[s][2 * hh + 1] = w1;
            }
#pragma unroll
        for (int n = 0; n < 4 * MAX_UNITS; n += 2) {
            if (n < 4 * nuv) {
#pragma unroll
                for (int s = 0; s < 4; ++s) {                  // 16 keys per instruction
                    uint32_t b[4];
                    ldsm4_trans(v_addr + 16 * s * PITCH + 16 * n, b);
                    mma_f16(O[n], pa[s], b[0], b[1]);
                    mma_f16(O[n + 1], pa[s], b[2], b[3]);
                }
            }
        }
        __syncthreads();                     // every warp is done with the tile
    }
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const float inv0 = 1.0f / l0, inv1 = 1.0f / l1;
    // O = s^V_c (sum_j P V_q / sum_j P - z^V_c), written at the position's channel
#pragma unroll
    for (int n = 0; n < 4 * MAX_UNITS; ++n) {
        if (n < 4 * nuv) {
            const int unit = uv0 + (n >> 2);
            const float2 sz = __ldg(p.unit_sz_v + unit);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int pos = 32 * unit + 8 * (n & 3) + 2 * t4 + (e & 1);
                const int i = (e & 2) ? row1 : row0;
                if (i < p.Tq && __ldg(p.jidx_v + pos) >= 0)
                    p.out[(q_row0 + i) * p.ldo + __ldg(p.src_v + pos)] = __float2half_rn(sz.x * (O[n][e] * ((e & 2) ? inv1 : inv0) - sz.y));
            }
        }
    }
}

}  // namespace attnkv
}  // namespace rptq

static bool kv_units_in_cluster_order(const rptq_layout_t* L, int* n_used)
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

// head h's clusters hold exactly the channels h * hd .. (h + 1) * hd - 1 (the kernel reads a head's query slice by that rule)
static bool kv_heads_own_their_channels(const rptq_layout_t* L, int H)
{
    const int gh = L->g / H, hd = L->C / H;
    size_t j = 0;
    for (int c = 0; c < L->g; ++c)
        for (int i = 0; i < L->size[(size_t)c]; ++i, ++j)
            if (L->perm[j] / hd != c / gh) return false;
    return true;
}

static int kv_max_units_per_head(const rptq_layout_t* L, int n_used, int H)
{
    const int gh = L->g / H;
    std::vector<int> cnt((size_t)H, 0);
    for (int u = 0; u < n_used; ++u) ++cnt[(size_t)(L->unit_cluster[u] / gh)];
    int m = 0;
    for (int c : cnt) m = c > m ? c : m;
    return m;
}

extern "C" int rptq_attention_kv(const rptq_layout_t* LK, const rptq_layout_t* LV, int n_heads,
                                 const void* q_f16, int64_t ldq, int Tq, const void* k_codes, const void* v_codes, int Tk, int n_seq,
                                 float qk_scale, int causal, void* out_f16, int64_t ldo, void* stream)
{
    using namespace rptq;
    using namespace rptq::attnkv;
    if (!LK || !LV || !q_f16 || !k_codes || !v_codes || !out_f16) return RPTQ_ERR_INVALID_ARG;
    if (n_heads < 1 || Tq < 0 || Tk < Tq || n_seq < 0 || !(qk_scale >= 0.f)) return RPTQ_ERR_INVALID_ARG;
    if (LK->g % n_heads || LV->g % n_heads || LK->C != LV->C || LK->C % n_heads || ldq < LK->C || ldo < LV->C) return RPTQ_ERR_INVALID_ARG;
    if (!aligned16(k_codes) || !aligned16(v_codes) || (reinterpret_cast<uintptr_t>(q_f16) & 1u) || (reinterpret_cast<uintptr_t>(out_f16) & 1u))
        return RPTQ_ERR_INVALID_ARG;
    if (n_heads > 65535 || n_seq > 65535) return RPTQ_ERR_UNSUPPORTED;
    int n_used_k = 0, n_used_v = 0;
    if (!kv_units_in_cluster_order(LK, &n_used_k) || !kv_units_in_cluster_order(LV, &n_used_v)) return RPTQ_ERR_UNSUPPORTED;
    if (kv_max_units_per_head(LK, n_used_k, n_heads) > MAX_UNITS || kv_max_units_per_head(LV, n_used_v, n_heads) > MAX_UNITS) return RPTQ_ERR_UNSUPPORTED;
    if (!kv_heads_own_their_channels(LK, n_heads)) return RPTQ_ERR_INVALID_ARG;
    if (Tq == 0 || n_seq == 0) return RPTQ_OK;
    int dev = -1;
    if (LK->device < 0 || cudaGetDevice(&dev) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (dev != LK->device || dev != LV->device) return RPTQ_ERR_INVALID_ARG;

    Params p{};
    p.q = static_cast<const __half*>(q_f16); p.ldq = ldq;
    p.k = static_cast<const uint8_t*>(k_codes); p.v = static_cast<const uint8_t*>(v_codes);
    p.k_row_bytes = LK->row_bytes; p.v_row_bytes = LV->row_bytes; p.bits_k = LK->bits; p.bits_v = LV->bits;
    p.Tq = Tq; p.Tk = Tk; p.H = n_heads; p.hd = LK->C / n_heads; p.gh_k = LK->g / n_heads; p.gh_v = LV->g / n_heads; p.causal = causal ? 1 : 0;
    p.n_used_k = n_used_k; p.n_used_v = n_used_v;
    p.unit_cluster_k = LK->d_unit_cluster; p.unit_cluster_v = LV->d_unit_cluster;
    p.unit_sz_k = LK->d_unit_sz; p.unit_sz_v = LV->d_unit_sz;
    p.src_k = LK->d_src; p.src_v = LV->d_src; p.jidx_k = LK->d_jidx; p.jidx_v = LV->d_jidx;
    p.qk_scale_log2e = qk_scale * 1.4426950408889634f;
    p.out = static_cast<__half*>(out_f16); p.ldo = ldo;

    const int smem = (BM + 2 * BN) * PITCH;
    if (cudaFuncSetAttribute(attention_kv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return RPTQ_ERR_CUDA;
    const dim3 grid((unsigned)((Tq + BM - 1) / BM), (unsigned)n_heads, (unsigned)n_seq);
    attention_kv_kernel<<<grid, THREADS, smem, static_cast<cudaStream_t>(stream)>>>(p);
    return cudaGetLastError() == cudaSuccess ? RPTQ_OK : RPTQ_ERR_CUDA;
}
