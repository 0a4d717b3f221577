/*
 * CPU oracle for the RPTQ hot path (reorder-based post-training quantisation, arXiv 2304.01089).
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain statement of what the GPU library must
 * compute. It is called from the test-suite, from the smoke check and from the benchmark's CPU
 * baseline leg, and from nowhere else. It shares no code, header, table or helper with the CUDA
 * library. Floating point is fp64 unless a function says otherwise.
 *
 * Every function cites the passage of the paper that it follows. Where the paper is silent the
 * reading taken is stated beside the code.
 *
 * Parity pins live in tests/test_oracle_*.py. Function with no independent pin:
 *   orc_kmeans  -- result quality is "parity unpinned" (the paper prints no clustering output);
 *                  its invariants (partition, non-increasing inertia, recovery of separated blobs)
 *                  are tested, and its output is only ever an input to both sides.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC (see oracle/build.py). No fast-math.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------------ */
/* Calibration side (host, off the hot path)                                                   */
/* ------------------------------------------------------------------------------------------ */

/* Eq. 3: per-channel minimum and maximum over all calibration samples and tokens.
 * y is [T][C] with T = B*N flattened. */
void orc_channel_minmax(const double* y, int64_t T, int C, double* x_min, double* x_max)
{
    for (int c = 0; c < C; ++c) {
        double lo = INFINITY, hi = -INFINITY;
        for (int64_t t = 0; t < T; ++t) {
            double v = y[t * C + c];
            if (v < lo) lo = v;
            if (v > hi) hi = v;
        }
        x_min[c] = lo;
        x_max[c] = hi;
    }
}

/* Eq. 2 (Min-Max method), taken literally: s = (max - min) / 2^k, z = -round((max + min)/(2 s)).
 * Eq. 1 states signed codes in [-2^(k-1), 2^(k-1)-1]; the library stores codes re-based to
 * [0, 2^k - 1], which shifts the zero point by 2^(k-1) and leaves s (x_q - z) unchanged.
 * round() is round-half-to-even. The paper is silent on max == min: s = 1 is used there. */
void orc_minmax_params(double x_min, double x_max, int k, double* s_out, int32_t* z_unsigned_out)
{
    double s = (x_max - x_min) / (double)(1 << k);
    if (!(s > 0.0)) s = 1.0;
    double z_signed = -nearbyint((x_max + x_min) / (2.0 * s));
    *s_out = s;
    *z_unsigned_out = (int32_t)z_signed + (1 << (k - 1));
}

/* Sec. 4.1: K-Means of the channels on the points (X_min,i , X_max,i) into g clusters.
 * The paper names the algorithm only. Reading: k-means++ seeding driven by the caller's uniform
 * draws u[0..g-1], then `iters` Lloyd iterations with squared Euclidean distance on the raw
 * points; ties go to the lowest centre index; a centre that loses all its points is re-seeded at
 * the point that lies farthest from its own centre. inertia[it] receives the sum of squared
 * distances measured in the assignment step of iteration it. Returns 0. */
int orc_kmeans(const double* pts, int n, int dim, int g, const double* u, int iters,
               int32_t* labels, double* centres, double* inertia)
{
    double* d2 = (double*)malloc(sizeof(double) * (size_t)n);
    int32_t* count = (int32_t*)malloc(sizeof(int32_t) * (size_t)g);
    if (!d2 || !count) return -1;

    /* seeding */
    int first = (int)floor(u[0] * n);
    if (first >= n) first = n - 1;
    memcpy(centres, pts + (size_t)first * dim, sizeof(double) * dim);
    for (int i = 0; i < n; ++i) d2[i] = INFINITY;
    for (int k = 1; k < g; ++k) {
        double total = 0.0;
        for (int i = 0; i < n; ++i) {
            double d = 0.0;
            for (int a = 0; a < dim; ++a) {
                double t = pts[(size_t)i * dim + a] - centres[(size_t)(k - 1) * dim + a];
                d += t * t;
            }
            if (d < d2[i]) d2[i] = d;
            total += d2[i];
        }
        double target = u[k] * total, run = 0.0;
        int pick = n - 1;
        for (int i = 0; i < n; ++i) {
            run += d2[i];
            if (run > target) { pick = i; break; }
        }
        memcpy(centres + (size_t)k * dim, pts + (size_t)pick * dim, sizeof(double) * dim);
    }

    for (int it = 0; it < iters; ++it) {
        /* assignment */
        double total = 0.0;
        for (int i = 0; i < n; ++i) {
            double best = INFINITY;
            int bk = 0;
            for (int k = 0; k < g; ++k) {
                double d = 0.0;
                for (int a = 0; a < dim; ++a) {
                    double t = pts[(size_t)i * dim + a] - centres[(size_t)k * dim + a];
                    d += t * t;
                }
                if (d < best) { best = d; bk = k; }
            }
            labels[i] = bk;
            d2[i] = best;
            total += best;
        }
        if (inertia) inertia[it] = total;
        /* re-seed empty centres at the farthest point, one at a time */
        for (int k = 0; k < g; ++k) count[k] = 0;
        for (int i = 0; i < n; ++i) count[labels[i]]++;
        for (int k = 0; k < g; ++k) {
            if (count[k] != 0) continue;
            int far = -1;
            double fd = -1.0;
            for (int i = 0; i < n; ++i)
                if (count[labels[i]] > 1 && d2[i] > fd) { fd = d2[i]; far = i; }
            if (far < 0) continue;              /* fewer distinct points than centres */
            count[labels[far]]--;
            labels[far] = k;
            count[k] = 1;
            d2[far] = 0.0;
        }
        /* update */
        for (int k = 0; k < g; ++k) {
            if (count[k] == 0) continue;
            for (int a = 0; a < dim; ++a) {
                double sum = 0.0;
                for (int i = 0; i < n; ++i)
                    if (labels[i] == k) sum += pts[(size_t)i * dim + a];
                centres[(size_t)k * dim + a] = sum / count[k];
            }
        }
    }
    free(d2);
    free(count);
    return 0;
}

/* Sec. 4.1: S = [S^1, ..., S^g], the concatenation of the clusters' channel index sets.
 * The paper leaves both orders open. Reading: clusters are ordered by ascending
 * (max - min) of their merged range, ties by ascending min, then by smallest member; channels
 * inside a cluster keep ascending index. Outputs: perm[C] (S), size[g] in the new cluster
 * order, and new_of_old[g] (new position of each input label). */
void orc_reorder_index(const int32_t* labels, const double* x_min, const double* x_max, int C, int g,
                       int32_t* perm, int32_t* size, int32_t* new_of_old)
{
    double* lo = (double*)malloc(sizeof(double) * g);
    double* hi = (double*)malloc(sizeof(double) * g);
    int32_t* firstm = (int32_t*)malloc(sizeof(int32_t) * g);
    int32_t* order = (int32_t*)malloc(sizeof(int32_t) * g);
    int32_t* cnt = (int32_t*)calloc(g, sizeof(int32_t));
    for (int k = 0; k < g; ++k) { lo[k] = INFINITY; hi[k] = -INFINITY; firstm[k] = C; order[k] = k; }
    for (int c = 0; c < C; ++c) {
        int k = labels[c];
        cnt[k]++;
        if (x_min[c] < lo[k]) lo[k] = x_min[c];
        if (x_max[c] > hi[k]) hi[k] = x_max[c];
        if (c < firstm[k]) firstm[k] = c;
    }
    /* insertion sort of the cluster ids; empty clusters go last, in label order */
    for (int i = 1; i < g; ++i) {
        int k = order[i], j = i - 1;
        for (; j >= 0; --j) {
            int q = order[j];
            int q_before_k;
            if (cnt[q] == 0 || cnt[k] == 0) q_before_k = (cnt[k] == 0) ? 1 : 0;
            else {
                double rq = hi[q] - lo[q], rk = hi[k] - lo[k];
                if (rq != rk) q_before_k = rq < rk;
                else if (lo[q] != lo[k]) q_before_k = lo[q] < lo[k];
                else q_before_k = firstm[q] < firstm[k];
            }
            if (q_before_k) break;
            order[j + 1] = q;
        }
        order[j + 1] = k;
    }
    int pos = 0;
    for (int r = 0; r < g; ++r) {
        int k = order[r];
        new_of_old[k] = r;
        size[r] = cnt[k];
        for (int c = 0; c < C; ++c)
            if (labels[c] == k) perm[pos++] = c;
    }
    free(lo); free(hi); free(firstm); free(order); free(cnt);
}

/* ------------------------------------------------------------------------------------------ */
/* Padded cluster-segment layout shared by activations and weights                             */
/* ------------------------------------------------------------------------------------------ */

/* The paper has no padding; the hardware contraction step is 32 codes wide and the staging block
 * 128, so each cluster segment is padded to a multiple of 32 and the row to a multiple of 128.
 * seg_off[c] is the first padded position of cluster c, seg_off[g] the end of the last segment.
 * Returns K_pad. Pad positions hold activation code 0 and weight code 0. */
int32_t orc_segment_offsets(const int32_t* size, int g, int32_t* seg_off)
{
    int32_t off = 0;
    for (int c = 0; c < g; ++c) {
        seg_off[c] = off;
        off += (size[c] + 31) / 32 * 32;
    }
    seg_off[g] = off;
    int32_t k_pad = (off + 127) / 128 * 128;
    return k_pad < 128 ? 128 : k_pad;
}

/* ------------------------------------------------------------------------------------------ */
/* Hot path, step by step                                                                      */
/* ------------------------------------------------------------------------------------------ */

/* Sec. 4.2 "layer norm operation". The paper does not print the formula; the standard one is
 * used: mu = mean(x), var = mean((x-mu)^2) (biased), y = (x-mu)/sqrt(var+eps)*gamma + beta.
 * x[M][C], gamma[C], beta[C] are the fp16 inputs widened exactly to fp64 by the caller. */
void orc_layernorm(const double* x, const double* gamma, const double* beta, int64_t M, int C,
                   double eps, double* y)
{
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        const double* xr = x + m * C;
        double sum = 0.0;
        for (int c = 0; c < C; ++c) sum += xr[c];
        double mu = sum / C;
        double sq = 0.0;
        for (int c = 0; c < C; ++c) sq += (xr[c] - mu) * (xr[c] - mu);
        double rstd = 1.0 / sqrt(sq / C + eps);
        for (int c = 0; c < C; ++c) y[m * C + c] = (xr[c] - mu) * rstd * gamma[c] + beta[c];
    }
}

/* Sec. 4.1 reorder: X~[:, i] = X[:, S_i].  y[M][C] -> y_r[M][C]. */
void orc_reorder(const double* y, int64_t M, int C, const int32_t* perm, double* y_r)
{
    for (int64_t m = 0; m < M; ++m)
        for (int j = 0; j < C; ++j) y_r[m * C + j] = y[m * C + perm[j]];
}

/* Eq. 1 applied per cluster (Appendix "Computation under cluster-based quantization":
 * X~_q,i = Q_k(X~_i, s_i, z_i)), codes re-based to [0, 2^k - 1]:
 *     q = clamp(round(x / s_c) + z_c, 0, 2^k - 1),   round = half-to-even.
 * Input y_r[M][C] is already in reordered channel order; output codes[M][K_pad] (one byte per
 * code) uses the padded segment layout, pad positions = 0. A NaN input gives code 0. */
void orc_quantize_clusters(const double* y_r, int64_t M, int C, int g, const int32_t* size,
                           const double* scale, const int32_t* zero, int k, int32_t K_pad,
                           uint8_t* codes)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
    const double qmax = (double)((1 << k) - 1);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        uint8_t* row = codes + m * K_pad;
        memset(row, 0, (size_t)K_pad);
        int j = 0;
        for (int c = 0; c < g; ++c) {
            for (int i = 0; i < size[c]; ++i, ++j) {
                double q = nearbyint(y_r[m * C + j] / scale[c]) + (double)zero[c];
                if (!(q > 0.0)) q = 0.0;         /* also catches NaN */
                if (q > qmax) q = qmax;
                row[seg_off[c] + i] = (uint8_t)q;
            }
        }
    }
    free(seg_off);
}

/* The same quantiser with the decision taken from fp32 operands, as the GPU kernel takes it:
 * Eq. 1's x / s is evaluated as the product of the fp32 value y and the fp32 reciprocal
 * inv_s = (float)(1.0 / (double)s), and that product is rounded ONCE, half to even, to an integer
 * (the product of two fp32 numbers is exact in fp64, so nearbyint of the fp64 product is that
 * single rounding). Then q = clamp(r + z, 0, 2^k - 1). Input: fp32 LayerNorm outputs, reordered.
 * With identical inputs the codes must match the GPU's bit for bit. */
void orc_quantize_clusters_f32(const float* y_r, int64_t M, int C, int g, const int32_t* size,
                               const float* scale, const int32_t* zero, int k, int32_t K_pad,
                               uint8_t* codes)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
    const double qmax = (double)((1 << k) - 1);
    for (int64_t m = 0; m < M; ++m) {
        uint8_t* row = codes + m * K_pad;
        memset(row, 0, (size_t)K_pad);
        int j = 0;
        for (int c = 0; c < g; ++c) {
            const float inv_s = (float)(1.0 / (double)scale[c]);
            for (int i = 0; i < size[c]; ++i, ++j) {
                double q = nearbyint((double)y_r[m * C + j] * (double)inv_s) + (double)zero[c];
                if (!(q > 0.0)) q = 0.0;
                if (q > qmax) q = qmax;
                row[seg_off[c] + i] = (uint8_t)q;
            }
        }
    }
    free(seg_off);
}

/* De-quantisation, Eq. 1 text: x^ = s (x_q - z), per cluster, padded layout -> [M][C] reordered. */
void orc_dequantize_clusters(const uint8_t* codes, int64_t M, int C, int g, const int32_t* size,
                             const double* scale, const int32_t* zero, int32_t K_pad, double* x_hat)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
    for (int64_t m = 0; m < M; ++m) {
        int j = 0;
        for (int c = 0; c < g; ++c)
            for (int i = 0; i < size[c]; ++i, ++j)
                x_hat[m * C + j] = scale[c] * ((double)codes[m * K_pad + seg_off[c] + i] - (double)zero[c]);
    }
    free(seg_off);
}

/* ------------------------------------------------------------------------------------------ */
/* Packed storage (Appendix: 3-bit values are stored narrow and computed as wider types).      */
/* The bit layout is not the paper's; it is the library's documented private format, written   */
/* here from the format description, element by element.                                       */
/*   8 bit: one byte per code.                                                                 */
/*   4 bit: 32-bit little-endian word w of a row holds codes 8w..8w+7; byte i (0..3) carries   */
/*          code 8w+i in bits 0-3 and code 8w+4+i in bits 4-7.                                 */
/*   3 bit: 32 codes -> three words. Word j (0..2) carries codes 8j..8j+7 of the group as in   */
/*          the 4-bit layout (3 significant bits per nibble). The spare top bit of nibble t    */
/*          (t = i for the low nibble of byte i, 4+i for the high nibble) of word j carries    */
/*          bit j of code 24+t.                                                                */
/* ------------------------------------------------------------------------------------------ */

int64_t orc_row_bytes(int32_t K_pad, int k) { return (int64_t)K_pad * k / 8; }

static void put_nibble(uint8_t* row_words, int word, int t, unsigned v)
{
    int byte = word * 4 + (t & 3);
    int shift = (t >> 2) * 4;
    row_words[byte] = (uint8_t)(row_words[byte] | (v << shift));
}

static unsigned get_nibble(const uint8_t* row_words, int word, int t)
{
    int byte = word * 4 + (t & 3);
    int shift = (t >> 2) * 4;
    return (row_words[byte] >> shift) & 0xFu;
}

void orc_pack_codes(const uint8_t* codes, int64_t M, int32_t K_pad, int k, uint8_t* packed)
{
    int64_t rb = orc_row_bytes(K_pad, k);
    memset(packed, 0, (size_t)(M * rb));
    for (int64_t m = 0; m < M; ++m) {
        const uint8_t* src = codes + m * K_pad;
        uint8_t* dst = packed + m * rb;
        if (k == 8) {
            memcpy(dst, src, (size_t)K_pad);
        } else if (k == 4) {
            for (int p = 0; p < K_pad; ++p) put_nibble(dst, p / 8, p % 8, src[p] & 0xFu);
        } else { /* k == 3 */
            for (int p = 0; p < K_pad; ++p) {
                int grp = p / 32, e = p % 32;
                unsigned v = src[p] & 0x7u;
                if (e < 24) {
                    put_nibble(dst, grp * 3 + e / 8, e % 8, v);
                } else {
                    for (int j = 0; j < 3; ++j)
                        put_nibble(dst, grp * 3 + j, e - 24, ((v >> j) & 1u) << 3);
                }
            }
        }
    }
}

void orc_unpack_codes(const uint8_t* packed, int64_t M, int32_t K_pad, int k, uint8_t* codes)
{
    int64_t rb = orc_row_bytes(K_pad, k);
    for (int64_t m = 0; m < M; ++m) {
        const uint8_t* src = packed + m * rb;
        uint8_t* dst = codes + m * K_pad;
        if (k == 8) {
            memcpy(dst, src, (size_t)K_pad);
        } else if (k == 4) {
            for (int p = 0; p < K_pad; ++p) dst[p] = (uint8_t)get_nibble(src, p / 8, p % 8);
        } else {
            for (int p = 0; p < K_pad; ++p) {
                int grp = p / 32, e = p % 32;
                if (e < 24) {
                    dst[p] = (uint8_t)(get_nibble(src, grp * 3 + e / 8, e % 8) & 0x7u);
                } else {
                    unsigned v = 0;
                    for (int j = 0; j < 3; ++j)
                        v |= ((get_nibble(src, grp * 3 + j, e - 24) >> 3) & 1u) << j;
                    dst[p] = (uint8_t)v;
                }
            }
        }
    }
}

/* Signed 4-bit weight codes use the 4-bit word layout above with two's-complement nibbles, stored
 * tile-major (the library's documented format): tile (i, kb) = output rows 128i..128i+127, padded
 * positions 128kb..128kb+127, as 128 rows of 64 bytes; tiles ordered [i][kb], kb fastest; rows
 * beyond N in the last tile are zero. Buffer size: roundup128(N) * K_pad / 2 bytes. */
int64_t orc_weight_codes_bytes(int64_t N, int32_t K_pad) { return (N + 127) / 128 * 128 * (int64_t)(K_pad / 2); }

static uint8_t* weight_piece(uint8_t* base, int64_t n, int kb, int32_t K_pad)
{
    int64_t tile = (n / 128) * (K_pad / 128) + kb;
    return base + tile * 8192 + (n % 128) * 64;
}

void orc_pack_weight_codes(const int8_t* w, int64_t N, int32_t K_pad, uint8_t* packed)
{
    memset(packed, 0, (size_t)orc_weight_codes_bytes(N, K_pad));
    for (int64_t n = 0; n < N; ++n)
        for (int p = 0; p < K_pad; ++p) {
            int q = p % 128;
            put_nibble(weight_piece(packed, n, p / 128, K_pad), q / 8, q % 8, (unsigned)w[n * K_pad + p] & 0xFu);
        }
}

void orc_unpack_weight_codes(const uint8_t* packed, int64_t N, int32_t K_pad, int8_t* w)
{
    for (int64_t n = 0; n < N; ++n)
        for (int p = 0; p < K_pad; ++p) {
            int q = p % 128;
            int v = (int)get_nibble(weight_piece((uint8_t*)packed, n, p / 128, K_pad), q / 8, q % 8);
            w[n * K_pad + p] = (int8_t)(v >= 8 ? v - 16 : v);
        }
}

/* ------------------------------------------------------------------------------------------ */
/* Weights (Sec. 4.2: columns of W follow the input reorder index, rows the output index)      */
/* ------------------------------------------------------------------------------------------ */

/* W[N][C] is in the PyTorch [out][in] orientation, so Y = X W^T and "columns (dimension C1)"
 * are the input channels. Weight quantisation here is round-to-nearest, symmetric, one scale
 * per output channel (the paper itself uses GPTQ, which needs model Hessians):
 *     s_w[n] = max_k |W[n,k]| / 7  (1 when the row is zero),  w_q = clamp(rne(W / s_w), -8, 7),
 * both evaluated in IEEE fp32 because they decide integers and the library decides them in
 * fp32. "Rows (dimension C2) based on the output activation reorder index": output row r of
 * w_codes is original row out_perm[r] for r < N_pad, or a zero row with s_w = 1 where
 * out_perm[r] < 0 (the pad positions of the next site's padded layout); with out_perm NULL, row r
 * is original row r for r < N and zero beyond. Column layout: padded cluster segments, pads = 0.
 * wsum[c][r] = sum over the real channels of cluster c of w_q. */
void orc_weight_quantize(const float* W, int64_t N, int C, int g, const int32_t* perm,
                         const int32_t* size, const int32_t* out_perm, int64_t N_pad, int32_t K_pad,
                         int8_t* w_codes, float* s_w, int32_t* wsum)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
    memset(w_codes, 0, (size_t)(N_pad * K_pad));
    for (int64_t r = 0; r < N_pad; ++r) {
        s_w[r] = 1.0f;
        for (int c = 0; c < g; ++c) wsum[(int64_t)c * N_pad + r] = 0;
    }
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N_pad; ++r) {
        int64_t n = out_perm ? out_perm[r] : (r < N ? r : -1);
        if (n < 0) continue;
        const float* wr = W + n * C;
        float amax = 0.0f;
        for (int kk = 0; kk < C; ++kk) {
            float a = fabsf(wr[kk]);
            if (a > amax) amax = a;
        }
        volatile float s = amax > 0.0f ? amax / 7.0f : 1.0f;
        s_w[r] = s;
        int j = 0;
        for (int c = 0; c < g; ++c) {
            int32_t acc = 0;
            for (int i = 0; i < size[c]; ++i, ++j) {
                volatile float t = wr[perm[j]] / s;
                float q = rintf(t);
                if (q < -8.0f) q = -8.0f;
                if (q > 7.0f) q = 7.0f;
                w_codes[r * K_pad + seg_off[c] + i] = (int8_t)q;
                acc += (int32_t)q;
            }
            wsum[(int64_t)c * N_pad + r] = acc;
        }
    }
    free(seg_off);
}

/* ------------------------------------------------------------------------------------------ */
/* Cluster-segmented integer matmul (Appendix, second method)                                  */
/* ------------------------------------------------------------------------------------------ */

/* Raw per-cluster integer products  acc_c[m][n] = sum_{k in segment c} X_q[m][k] * W_q[n][k].
 * acc is [g][M][N] int64. Pad positions contribute 0 because the weight pads are 0. */
void orc_cluster_acc(const uint8_t* a_codes, int64_t M, const int8_t* w_codes, int64_t N,
                     int32_t K_pad, int g, const int32_t* size, int64_t* acc)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n)
            for (int c = 0; c < g; ++c) {
                int64_t s = 0;
                for (int p = seg_off[c]; p < seg_off[c] + size[c]; ++p)
                    s += (int64_t)a_codes[m * K_pad + p] * (int64_t)w_codes[n * K_pad + p];
                acc[((int64_t)c * M + m) * N + n] = s;
            }
    free(seg_off);
}

/* Appendix, second method. The printed per-cluster expression omits the sums; written out for
 * one output element it is
 *   Y_q,i[m][n] = sum_k (X_q[m][k] - z^X_i)(W_q[n][k] - z^W_i)
 *               = sum X_q W_q - z^X_i sum_k W_q - z^W_i sum_k X_q + n_i z^X_i z^W_i ,
 * and Y = sum_i s^X_i s^W_i Y_q,i. With symmetric per-output-channel weights (z^W = 0,
 * s^W_i = s_w[n] for every i) this is
 *   Y[m][n] = s_w[n] * sum_i s_i * (acc_i[m][n] - z_i * Wsum_i[n])        (clusters ascending)
 * optionally followed by + bias[n] and ReLU (the paper is silent on both; OPT has biases and
 * a ReLU after FC1). Returns the number of accumulators that do not fit in int32 (must be 0
 * for the hardware path to be exact). */
int64_t orc_cluster_gemm(const uint8_t* a_codes, int64_t M, const int8_t* w_codes, int64_t N,
                         int32_t K_pad, int g, const int32_t* size, const double* scale,
                         const int32_t* zero, const float* s_w, const int32_t* wsum, int64_t ld_wsum,
                         const float* bias, int relu, double* y)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
    int64_t overflow = 0;
#pragma omp parallel for schedule(static) reduction(+ : overflow)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double total = 0.0;
            for (int c = 0; c < g; ++c) {
                int64_t acc = 0;
                for (int p = seg_off[c]; p < seg_off[c] + size[c]; ++p)
                    acc += (int64_t)a_codes[m * K_pad + p] * (int64_t)w_codes[n * K_pad + p];
                if (acc > INT32_MAX || acc < INT32_MIN) overflow++;
                total += scale[c] * (double)(acc - (int64_t)zero[c] * wsum[(int64_t)c * ld_wsum + n]);
            }
            double v = (double)s_w[n] * total;
            if (bias) v += (double)bias[n];
            if (relu && v < 0.0) v = 0.0;
            y[m * N + n] = v;
        }
    free(seg_off);
    return overflow;
}

/* Appendix, first method: de-quantise both operands, then a floating-point product
 * Y = X^ W^T with X^ = s_i (X_q - z_i) and W^ = s_w W_q. Used as the cross-check of the
 * integer method (they are algebraically identical). */
void orc_dequant_matmul(const uint8_t* a_codes, int64_t M, const int8_t* w_codes, int64_t N,
                        int32_t K_pad, int g, const int32_t* size, const double* scale,
                        const int32_t* zero, const float* s_w, double* y)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double s = 0.0;
            for (int c = 0; c < g; ++c)
                for (int p = seg_off[c]; p < seg_off[c] + size[c]; ++p) {
                    double xh = scale[c] * ((double)a_codes[m * K_pad + p] - (double)zero[c]);
                    double wh = (double)s_w[n] * (double)w_codes[n * K_pad + p];
                    s += xh * wh;
                }
            y[m * N + n] = s;
        }
    free(seg_off);
}

/* ------------------------------------------------------------------------------------------ */
/* Per-cluster asymmetric weight parameters (Appendix, W~_q,i = Q_k(W~_i, s^W_i, z^W_i))       */
/* ------------------------------------------------------------------------------------------ */

/* Appendix: the weights of an output channel get one asymmetric (scale, zero point) pair per input
 * cluster. For output row r and input cluster i the parameters come from the Min-Max method
 * (Eq. 2, taken literally as for the activations) over the row's weights of that cluster, and the
 * codes from Eq. 1 re-based to [0, 2^k - 1]. (The paper obtains the codes with GPTQ, which needs a
 * trained model's Hessians; round-to-nearest is used here.) Everything that decides an integer is
 * evaluated in IEEE fp32, as in orc_weight_quantize.
 *   w_codes [N_pad][K_pad] unsigned codes in the padded cluster segments, pad positions 0
 *   s_w, z_w, wsum [g][N_pad]: scale, zero point (for the re-based codes) and the sum of the codes
 *   over the real channels of the cluster. Empty clusters and rows r >= N: s = 1, z = 0, sum 0. */
void orc_weight_quantize_clustered(const float* W, int64_t N, int C, int g, int k, const int32_t* perm,
                                   const int32_t* size, int64_t N_pad, int32_t K_pad,
                                   uint8_t* w_codes, float* s_w, int32_t* z_w, int32_t* wsum)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
    memset(w_codes, 0, (size_t)(N_pad * K_pad));
    const float qmax = (float)((1 << k) - 1);
    for (int64_t r = 0; r < N_pad; ++r)
        for (int c = 0; c < g; ++c) {
            s_w[(int64_t)c * N_pad + r] = 1.0f;
            z_w[(int64_t)c * N_pad + r] = 0;
            wsum[(int64_t)c * N_pad + r] = 0;
        }
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < N; ++r) {
        const float* wr = W + r * C;
        int j0 = 0;
        for (int c = 0; c < g; j0 += size[c], ++c) {
            if (size[c] == 0) continue;
            float lo = INFINITY, hi = -INFINITY;
            for (int i = 0; i < size[c]; ++i) {
                float v = wr[perm[j0 + i]];
                if (v < lo) lo = v;
                if (v > hi) hi = v;
            }
            volatile float s = (hi - lo) / (float)(1 << k);           /* Eq. 2, denominator 2^k */
            if (!(s > 0.0f)) s = 1.0f;
            volatile float mid = (hi + lo) / (2.0f * s);
            const int32_t z = (1 << (k - 1)) - (int32_t)rintf(mid);    /* re-based zero point */
            int32_t acc = 0;
            for (int i = 0; i < size[c]; ++i) {
                volatile float t = wr[perm[j0 + i]] / s;
                float q = rintf(t) + (float)z;                         /* Eq. 1 */
                if (q < 0.0f) q = 0.0f;
                if (q > qmax) q = qmax;
                w_codes[r * K_pad + seg_off[c] + i] = (uint8_t)q;
                acc += (int32_t)q;
            }
            s_w[(int64_t)c * N_pad + r] = s;
            z_w[(int64_t)c * N_pad + r] = z;
            wsum[(int64_t)c * N_pad + r] = acc;
        }
    }
    free(seg_off);
}

/* Sums of the activation codes over the real positions of each cluster, xsum[m][c] = sum_{k in
 * S^c} X_q[m][k]: the third term of the second method needs them. */
void orc_code_rowsums(const uint8_t* a_codes, int64_t M, int32_t K_pad, int g, const int32_t* size, int32_t* xsum)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
    for (int64_t m = 0; m < M; ++m)
        for (int c = 0; c < g; ++c) {
            int32_t s = 0;
            for (int p = seg_off[c]; p < seg_off[c] + size[c]; ++p) s += a_codes[m * K_pad + p];
            xsum[m * g + c] = s;
        }
    free(seg_off);
}

/* Appendix, second method, all four terms (the printed expression omits the sums and the cluster
 * size; written out for one output element):
 *   Y_q,i[m][n] = sum_k X_q W_q - z^X_i sum_k W_q - z^W_i[n] sum_k X_q + n_i z^X_i z^W_i[n]
 *   Y[m][n]     = sum_i s^X_i s^W_i[n] Y_q,i[m][n]                       (clusters ascending)
 * with every sum over the n_i real channels of cluster i, then + bias[n] and ReLU if asked for. */
void orc_cluster_gemm_asym(const uint8_t* a_codes, int64_t M, const uint8_t* w_codes, int64_t N,
                           int32_t K_pad, int g, const int32_t* size, const double* scale,
                           const int32_t* zero, const float* s_w, const int32_t* z_w, int64_t ld,
                           const float* bias, int relu, double* y)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double total = 0.0;
            for (int c = 0; c < g; ++c) {
                int64_t xw = 0, sum_w = 0, sum_x = 0;
                for (int p = seg_off[c]; p < seg_off[c] + size[c]; ++p) {
                    const int64_t xq = a_codes[m * K_pad + p], wq = w_codes[n * K_pad + p];
                    xw += xq * wq;
                    sum_w += wq;
                    sum_x += xq;
                }
                const int64_t zx = zero[c], zw = z_w[(int64_t)c * ld + n];
                const int64_t yq = xw - zx * sum_w - zw * sum_x + (int64_t)size[c] * zx * zw;
                total += scale[c] * (double)s_w[(int64_t)c * ld + n] * (double)yq;
            }
            if (bias) total += (double)bias[n];
            if (relu && total < 0.0) total = 0.0;
            y[m * N + n] = total;
        }
    free(seg_off);
}

/* Appendix, first method with the same parameters: X^ = s^X_i (X_q - z^X_i), W^ = s^W_i[n] (W_q -
 * z^W_i[n]), Y = X^ W^T in floating point. The cross-check of orc_cluster_gemm_asym. */
void orc_dequant_matmul_asym(const uint8_t* a_codes, int64_t M, const uint8_t* w_codes, int64_t N,
                             int32_t K_pad, int g, const int32_t* size, const double* scale,
                             const int32_t* zero, const float* s_w, const int32_t* z_w, int64_t ld, double* y)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double s = 0.0;
            for (int c = 0; c < g; ++c)
                for (int p = seg_off[c]; p < seg_off[c] + size[c]; ++p) {
                    double xh = scale[c] * ((double)a_codes[m * K_pad + p] - (double)zero[c]);
                    double wh = (double)s_w[(int64_t)c * ld + n] * ((double)w_codes[n * K_pad + p] - (double)z_w[(int64_t)c * ld + n]);
                    s += xh * wh;
                }
            y[m * N + n] = s;
        }
    free(seg_off);
}

/* ------------------------------------------------------------------------------------------ */
/* First method with de-quantised operands of limited precision                                */
/* ------------------------------------------------------------------------------------------ */

/* round-to-nearest-even of an fp32 value to the bfloat16 format (8 bits of significand) */
static float bf16_rne(float v)
{
    uint32_t u;
    memcpy(&u, &v, 4);
    if ((u & 0x7F800000u) != 0x7F800000u) u += 0x7FFFu + ((u >> 16) & 1u);
    u &= 0xFFFF0000u;
    memcpy(&v, &u, 4);
    return v;
}

/* Appendix, first method, as a 16-bit floating-point matrix product computes it: the de-quantised
 * activation X^ = s_c (X_q - z_c) is formed in fp32 (one multiply of the fp32 scale with the exact
 * integer difference) and rounded to bfloat16; the weight operand is the integer code W_q, which
 * bfloat16 holds exactly, and its scale s_w[n] multiplies the finished sum (W^ = s_w W_q, so that
 * X^ W^ = s_w sum X^ W_q). The sum itself is exact here. Optional bias and ReLU as elsewhere. */
void orc_dequant_matmul_bf16(const uint8_t* a_codes, int64_t M, const int8_t* w_codes, int64_t N,
                             int32_t K_pad, int g, const int32_t* size, const float* scale32,
                             const int32_t* zero, const float* s_w, const float* bias, int relu, double* y)
{
    int32_t* seg_off = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size, g, seg_off);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
        for (int64_t n = 0; n < N; ++n) {
            double s = 0.0;
            for (int c = 0; c < g; ++c)
                for (int p = seg_off[c]; p < seg_off[c] + size[c]; ++p) {
                    volatile float xh = scale32[c] * (float)((int32_t)a_codes[m * K_pad + p] - zero[c]);
                    s += (double)bf16_rne(xh) * (double)w_codes[n * K_pad + p];
                }
            double v = (double)s_w[n] * s;
            if (bias) v += (double)bias[n];
            if (relu && v < 0.0) v = 0.0;
            y[m * N + n] = v;
        }
    free(seg_off);
}

/* ------------------------------------------------------------------------------------------ */
/* Attention sites (reorders R2 and R3)                                                        */
/* ------------------------------------------------------------------------------------------ */

/* Sec. 4.2: the query and the key of a head share one reorder index, so the products over the head's
 * channels pair equal positions; Sec. 5.1: R2 and R3 are computed per head, every cluster has its own
 * asymmetric parameters, and the softmax output is quantised at 8 bits. Self-attention of H heads on
 * quantised Q, K and V, as its definition on the de-quantised operands (Eq. 1):
 *   head h owns clusters h*gh .. h*gh + gh - 1 of both layouts (Q and K: size_qk; V: size_v);
 *   Q^ = sQ_c (Qq - zQ_c), K^ = sK_c (Kq - zK_c), V^ = sV_c (Vq - zV_c) on the clusters' real positions;
 *   A[i][j] = qk_scale * sum over the head's positions of Q^[i][p] K^[j][p];
 *   key j is visible to query i when causal == 0 or j <= i + (Tk - Tq) (the queries are the last Tq
 *   of the Tk tokens);
 *   P[i][.] = softmax of A[i][.] over the visible keys, 0 at the hidden ones;
 *   Pq = clamp(round_half_even(P / s_P) + z_P, 0, 255), P^ = s_P (Pq - z_P);
 *   O[i][p] = sum_j P^[i][j] V^[j][p] for every real position p of the head in V's layout.
 * Codes are given at padded positions (q, k: [T][K_pad_qk]; v: [Tk][K_pad_v]); out is [Tq][K_pad_v]
 * with 0 at pad positions. p_codes, if not NULL, receives Pq as [H][Tq][Tk].
 * The paper does not say where the 1/sqrt(d) of the scores is applied; it is a factor of the scores here. */
void orc_attention(const uint8_t* q_codes, const uint8_t* k_codes, const uint8_t* v_codes,
                   int64_t Tq, int64_t Tk, int H, int gh,
                   int32_t K_pad_qk, const int32_t* size_qk, const double* sQ, const int32_t* zQ,
                   const double* sK, const int32_t* zK,
                   int32_t K_pad_v, const int32_t* size_v, const double* sV, const int32_t* zV,
                   double s_P, int32_t z_P, double qk_scale, int causal, double* out, uint8_t* p_codes)
{
    const int g = H * gh;
    int32_t* off_qk = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    int32_t* off_v = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size_qk, g, off_qk);
    orc_segment_offsets(size_v, g, off_v);
    memset(out, 0, sizeof(double) * (size_t)Tq * (size_t)K_pad_v);
#pragma omp parallel for schedule(dynamic, 4) collapse(2)
    for (int h = 0; h < H; ++h)
        for (int64_t i = 0; i < Tq; ++i) {
            double* A = (double*)malloc(sizeof(double) * (size_t)Tk);
            const int64_t last = causal ? i + (Tk - Tq) : Tk - 1;      /* last visible key */
            double top = -INFINITY;
            for (int64_t j = 0; j <= last; ++j) {
                double a = 0.0;
                for (int c = h * gh; c < (h + 1) * gh; ++c)
                    for (int p = off_qk[c]; p < off_qk[c] + size_qk[c]; ++p) {
                        const double qh = sQ[c] * ((double)q_codes[i * K_pad_qk + p] - (double)zQ[c]);
                        const double kh = sK[c] * ((double)k_codes[j * K_pad_qk + p] - (double)zK[c]);
                        a += qh * kh;
                    }
                A[j] = qk_scale * a;
                if (A[j] > top) top = A[j];
            }
            double denom = 0.0;
            for (int64_t j = 0; j <= last; ++j) denom += exp(A[j] - top);
            for (int64_t j = 0; j < Tk; ++j) {
                const double pr = j <= last ? exp(A[j] - top) / denom : 0.0;
                double code = nearbyint(pr / s_P) + (double)z_P;       /* default rounding mode: half to even */
                if (code < 0.0) code = 0.0;
                if (code > 255.0) code = 255.0;
                if (p_codes) p_codes[((int64_t)h * Tq + i) * Tk + j] = (uint8_t)code;
                A[j] = s_P * (code - (double)z_P);                     /* P^ */
            }
            for (int c = h * gh; c < (h + 1) * gh; ++c)
                for (int p = off_v[c]; p < off_v[c] + size_v[c]; ++p) {
                    double o = 0.0;
                    for (int64_t j = 0; j < Tk; ++j)
                        o += A[j] * (sV[c] * ((double)v_codes[j * K_pad_v + p] - (double)zV[c]));
                    out[i * K_pad_v + p] = o;
                }
            free(A);
        }
    free(off_qk);
    free(off_v);
}

/* The last step of orc_attention alone, on given softmax codes (p_codes [H][Tq][Tk]):
 *   O[i][p] = sum_j s_P (Pq[i][j] - z_P) sV_c (Vq[j][p] - zV_c)
 * for comparing an implementation whose softmax codes differ from orc_attention's by a rounding. */
void orc_attention_output(const uint8_t* p_codes, const uint8_t* v_codes, int64_t Tq, int64_t Tk, int H, int gh,
                          int32_t K_pad_v, const int32_t* size_v, const double* sV, const int32_t* zV,
                          double s_P, int32_t z_P, double* out)
{
    const int g = H * gh;
    int32_t* off_v = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size_v, g, off_v);
    memset(out, 0, sizeof(double) * (size_t)Tq * (size_t)K_pad_v);
#pragma omp parallel for schedule(dynamic, 4) collapse(2)
    for (int h = 0; h < H; ++h)
        for (int64_t i = 0; i < Tq; ++i)
            for (int c = h * gh; c < (h + 1) * gh; ++c)
                for (int p = off_v[c]; p < off_v[c] + size_v[c]; ++p) {
                    double o = 0.0;
                    for (int64_t j = 0; j < Tk; ++j)
                        o += s_P * ((double)p_codes[((int64_t)h * Tq + i) * Tk + j] - (double)z_P) *
                             (sV[c] * ((double)v_codes[j * K_pad_v + p] - (double)zV[c]));
                    out[i * K_pad_v + p] = o;
                }
    free(off_v);
}

/* Sec. 5.2, the schemes that quantise only the key / value cache (W4A4KV, W4A3KV, W3A3KV): the query
 * and the softmax output stay 16-bit floating point, the cached keys and values are per-cluster codes
 * of the per-head layouts. Attention as its definition on the de-quantised cache:
 *   K^[j][ch] = sK_c (Kq - zK_c), V^ likewise;  A[i][j] = qk_scale * sum over the head's channels of Q[i][ch] K^[j][ch];
 *   visibility as in orc_attention;  P = softmax over the visible keys;  O[i][p] = sum_j P[i][j] V^[j][p].
 * q is [Tq][C] in the ORIGINAL channel order (head h owns channels h * C / H ..); ch_of_pos_k[K_pad_k]
 * gives the channel at each padded position of K's layout (-1 at pads). out is [Tq][K_pad_v], 0 at pads.
 * Nothing is rounded here: the 16-bit roundings of an implementation are the caller's tolerance. */
void orc_attention_kv(const double* q, int C, const int32_t* ch_of_pos_k, const uint8_t* k_codes, const uint8_t* v_codes,
                      int64_t Tq, int64_t Tk, int H, int gh,
                      int32_t K_pad_k, const int32_t* size_k, const double* sK, const int32_t* zK,
                      int32_t K_pad_v, const int32_t* size_v, const double* sV, const int32_t* zV,
                      double qk_scale, int causal, double* out)
{
    const int g = H * gh;
    int32_t* off_k = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    int32_t* off_v = (int32_t*)malloc(sizeof(int32_t) * (g + 1));
    orc_segment_offsets(size_k, g, off_k);
    orc_segment_offsets(size_v, g, off_v);
    memset(out, 0, sizeof(double) * (size_t)Tq * (size_t)K_pad_v);
#pragma omp parallel for schedule(dynamic, 4) collapse(2)
    for (int h = 0; h < H; ++h)
        for (int64_t i = 0; i < Tq; ++i) {
            double* A = (double*)malloc(sizeof(double) * (size_t)Tk);
            const int64_t last = causal ? i + (Tk - Tq) : Tk - 1;
            double top = -INFINITY;
            for (int64_t j = 0; j <= last; ++j) {
                double a = 0.0;
                for (int c = h * gh; c < (h + 1) * gh; ++c)
                    for (int p = off_k[c]; p < off_k[c] + size_k[c]; ++p)
                        a += q[i * C + ch_of_pos_k[p]] * (sK[c] * ((double)k_codes[j * K_pad_k + p] - (double)zK[c]));
                A[j] = qk_scale * a;
                if (A[j] > top) top = A[j];
            }
            double denom = 0.0;
            for (int64_t j = 0; j <= last; ++j) denom += exp(A[j] - top);
            for (int64_t j = 0; j < Tk; ++j) A[j] = j <= last ? exp(A[j] - top) / denom : 0.0;
            for (int c = h * gh; c < (h + 1) * gh; ++c)
                for (int p = off_v[c]; p < off_v[c] + size_v[c]; ++p) {
                    double o = 0.0;
                    for (int64_t j = 0; j < Tk; ++j)
                        o += A[j] * (sV[c] * ((double)v_codes[j * K_pad_v + p] - (double)zV[c]));
                    out[i * K_pad_v + p] = o;
                }
            free(A);
        }
    free(off_k);
    free(off_v);
}
