/*
 * rptq.h -- C boundary of the B200 (sm_100a) library for the hot path of RPTQ, reorder-based
 * post-training quantisation (arXiv 2304.01089).
 *
 * The two calls of the hot path, and the small amount of host logic around them:
 *
 *   rptq_ln_reorder_quant   LayerNorm -> channel reorder -> per-cluster quantise -> packed codes
 *   rptq_cluster_gemm       packed activation codes x packed int4 weights, integer products per
 *                           cluster segment on the tensor cores, floating-point epilogue (calls
 *                           with at most 16 tokens run a second kernel with the same arithmetic)
 * Further down: the same product with per-cluster asymmetric weights or as a de-quantised
 * bfloat16 product, attention on quantised Q / K / V, calibration on the device, and aids for
 * tests and measurement.
 *
 * Conventions
 *   - Every function returns an int status: RPTQ_OK or a negative RPTQ_ERR_* value. Nothing
 *     throws, aborts or prints.
 *   - "dev" pointers are device global memory of the device that was current when the layout
 *     was created; "host" pointers are ordinary host memory. The caller owns every buffer. The
 *     library allocates device memory only inside rptq_layout_create (small tables) and for one
 *     lazily created status word per device.
 *   - Kernel launches are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is the
 *     default stream). A layout handle is immutable after creation and may be used from several
 *     streams at once.
 *   - dev pointers must be 16-byte aligned.
 *
 * Notation (paper, Sec. 4.1 and Appendix "Computation under cluster-based quantization"):
 *   M tokens, C channels, g clusters, k (here `bits`) activation bits, N output channels,
 *   S = [S^1 .. S^g] the reorder index, n_c = |S^c|, (s_c, z_c) the quantisation parameters of
 *   cluster c.
 *
 * Padded layout (not in the paper; the tensor-core contraction step is 32 codes wide and operands
 * are staged in blocks of 128): a row of codes is K_pad/32 units of 32 positions. Cluster c owns
 * roundup32(n_c)/32 units, filled in order, so only its last unit can hold pad positions (at the
 * end). WHICH channel of the cluster sits at which of the cluster's positions is the library's
 * choice (all of them share s_c and z_c; the choice spreads a warp's shared-memory reads in
 * rptq_ln_reorder_quant over the banks): rptq_layout_padded_index reports it. K_pad = max(128, roundup128(sum_c roundup32(n_c))); the units
 * left over at the end of the row belong to no cluster. Pad positions hold activation code 0 and
 * weight code 0. Two unit orders:
 *   RPTQ_ORDER_CONTIGUOUS   the clusters' units follow one another in the order of S, so cluster
 *                           c occupies n_c of the positions seg_off[c] .. seg_off[c] + roundup32(n_c) - 1
 *                           with seg_off[c] = sum_{c' < c} roundup32(n_c');
 *   RPTQ_ORDER_INTERLEAVED  clusters of one or two units are placed between the units of the
 *                           larger clusters, one after every seven larger-cluster units (those left
 *                           over follow at the end); a larger cluster's units keep their order
 *                           but are no longer adjacent. The GEMM drains one accumulator per
 *                           cluster, and a run of very small clusters leaves the tensor cores
 *                           waiting for those drains; spread out, each drain runs under the
 *                           surrounding cluster's products. Falls back to the contiguous order
 *                           when there are fewer than two small clusters or no larger one.
 * rptq_layout_query and rptq_layout_padded_index report where everything went.
 *
 * Packed storage, format version 2 (private to this library; read it back with the *_unpack_host
 * helpers). A row of K_pad codes takes K_pad*bits/8 bytes:
 *   8 bit  one byte per code;
 *   4 bit  32-bit little-endian word w holds codes 8w..8w+7: byte i (0..3) carries code 8w+i in
 *          bits 0-3 and code 8w+4+i in bits 4-7;
 *   3 bit  32 codes take three words; word j carries codes 8j..8j+7 of the group as in the 4-bit
 *          layout, and bit 3 of nibble t of word j carries bit j of code 24+t (nibble t = low
 *          nibble of byte t for t < 4, high nibble of byte t-4 otherwise).
 * Weight codes are signed 4-bit two's-complement nibbles in the 4-bit word layout, stored tile-major
 * so that one staging block is one contiguous 8 KiB copy: tile (i, kb) holds output rows
 * 128i..128i+127 and padded positions 128kb..128kb+127 as 128 rows of 64 bytes; tiles are ordered
 * [i][kb] with kb fastest. Rows beyond N_pad in the last tile are zero. The buffer therefore has
 * rptq_weight_codes_bytes(K_pad, N_pad) = roundup128(N_pad) * K_pad / 2 bytes.
 */
#ifndef RPTQ_H_
#define RPTQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    RPTQ_OK = 0,
    RPTQ_ERR_INVALID_ARG = -1,     /* null pointer, negative size, misaligned pointer, bad stride */
    RPTQ_ERR_UNSUPPORTED = -2,     /* a size or option outside what the kernels handle */
    RPTQ_ERR_NOT_BIJECTION = -3,   /* perm is not a permutation of 0..C-1, or sizes do not sum to C */
    RPTQ_ERR_CUDA = -4,            /* a CUDA runtime or driver call failed */
    RPTQ_ERR_DEVICE_TIMEOUT = -5,  /* a bounded wait inside a kernel ran out (see rptq_get_device_status) */
    RPTQ_ERR_ALLOC = -6            /* host or device allocation failed */
};

enum { RPTQ_OUT_F32 = 0, RPTQ_OUT_F16 = 1, RPTQ_OUT_CODES = 2 };
enum { RPTQ_ACT_NONE = 0, RPTQ_ACT_RELU = 1 };
enum { RPTQ_FORMAT_VERSION = 2 };
enum { RPTQ_ORDER_CONTIGUOUS = 0, RPTQ_ORDER_INTERLEAVED = 1 };

typedef struct rptq_layout rptq_layout_t;

/*
 * Sec. 4.1: the reorder index S (concatenated cluster index sets) with one (s_c, z_c) per
 * cluster (Sec. 5.1: per-cluster asymmetric parameters), for a site with C channels quantised
 * to `bits` in {3, 4, 8}.
 *   perm_host[C]     S: reordered position j holds original channel perm_host[j]; must be a
 *                    permutation of 0..C-1 (else RPTQ_ERR_NOT_BIJECTION).
 *   cluster_size[g]  n_c >= 0 in the order the clusters appear in S; must sum to C.
 *   scale_host[g]    s_c > 0 and finite.
 *   zero_host[g]     z_c for codes re-based to [0, 2^bits - 1] (Eq. 1 states the signed range
 *                    [-2^(k-1), 2^(k-1)-1]; adding 2^(k-1) to both code and zero point leaves
 *                    s (x_q - z) unchanged). |z_c| < 2^21.
 *   order            RPTQ_ORDER_CONTIGUOUS or RPTQ_ORDER_INTERLEAVED (see "Padded layout" above).
 *                    Codes, packed weights and layouts of different orders do not mix.
 * Limits: C a multiple of 8, 8 <= C <= 65528, 1 <= g <= 4096, K_pad <= 65408; otherwise
 * RPTQ_ERR_UNSUPPORTED. On success *out owns small device tables on the current device; free it
 * with rptq_layout_destroy. All four arrays are copied.
 */
int rptq_layout_create(rptq_layout_t** out, int C, int g, int bits,
                       const int32_t* perm_host, const int32_t* cluster_size,
                       const float* scale_host, const int32_t* zero_host, int order);

/* Sizes of the padded layout. Any output pointer may be NULL. unit_cluster_out receives K_pad/32
 * ints: the cluster that owns each unit of 32 positions, -1 for the units past the last cluster. */
int rptq_layout_query(const rptq_layout_t* L, int* K_pad, int64_t* row_bytes, int32_t* unit_cluster_out);

/* padded_index[K_pad]: the original channel held by each padded position, -1 for pad positions. */
int rptq_layout_padded_index(const rptq_layout_t* L, int32_t* padded_index);

/* Frees the handle and its device tables. Work that uses it must have completed. NULL is OK. */
int rptq_layout_destroy(rptq_layout_t* L);

/*
 * Sec. 4.2: LayerNorm with the channel reorder fused into its write, followed by the cluster
 * quantiser of the Appendix, X~_q,c = Q_k(X~_c, s_c, z_c) with Q_k of Eq. 1:
 *   mu = mean_c x[m][c], var = mean_c (x[m][c]-mu)^2, y[c] = (x[m][c]-mu)/sqrt(var+eps)*gamma[c]+beta[c]
 *   (fp32 arithmetic on fp16 inputs), then for reordered position j in cluster c
 *   q = clamp(rne(y[S_j] / s_c) + z_c, 0, 2^bits - 1)
 * where y / s_c is evaluated as the exact product of y (fp32) and the fp32 reciprocal
 * (float)(1.0/(double)s_c), rounded once, half to even, to an integer.
 *   x      dev fp16 [M][ldx], ldx >= C, ldx a multiple of 8
 *   gamma  dev fp16 [C], beta dev fp16 [C]  (original channel order)
 *   codes  dev, M rows of row_bytes bytes, packed as described above; every byte is written
 *   y_dbg  NULL, or dev fp32 [M][C]: receives the LayerNorm outputs in reordered channel order
 *          (the values the codes were decided from)
 * M >= 0 (M == 0 launches nothing). Non-finite inputs give in-range codes, not an error.
 */
int rptq_ln_reorder_quant(const rptq_layout_t* L, const void* x, int64_t ldx, const void* gamma,
                          const void* beta, float eps, int M, void* codes, float* y_dbg, void* stream);

/*
 * Sec. 4.2: the weight's columns (dimension C1, input channels) follow the reorder index of the
 * site that feeds the layer, its rows (dimension C2, output channels) the index of the site that
 * reads its output; done once before deployment, on the host. W_host is fp32 [N][C] in the [out][in]
 * orientation (Y = X W^T). Weights are quantised round-to-nearest, symmetric, one scale per output
 * channel (the paper uses GPTQ, which needs a trained model's statistics):
 *   s_w[n] = max_k |W[n][k]| / 7 (1 if the row is zero), w_q = clamp(rne(W / s_w), -8, 7), in fp32.
 *   N_pad         >= N, the number of output rows written
 *   out_perm      NULL: output row r is original row r for r < N and a zero row (s_w = 1) beyond.
 *                 Otherwise host int32 [N_pad]: output row r is original row out_perm[r], or a zero
 *                 row where out_perm[r] < 0; no original row may appear twice. With the array that
 *                 rptq_layout_padded_index gives for the next site, the output channels come out in
 *                 that site's padded cluster order and rptq_cluster_gemm can re-quantise them in place.
 *   w_codes_host  host, rptq_weight_codes_bytes(K_pad, N_pad) bytes (tile-major packed signed nibbles)
 *   s_w           host fp32 [N_pad]
 *   wsum          host int32 [g][N_pad]: Wsum_c[r] = sum of w_q over the channels of cluster c
 * Runs on the calling thread plus OpenMP workers; touches no device.
 */
int rptq_weight_pack(const rptq_layout_t* Lin, const float* W_host, int N, const int32_t* out_perm,
                     int N_pad, void* w_codes_host, float* s_w, int32_t* wsum);

/*
 * Appendix, second computation method, with symmetric per-output-channel weights (z^W = 0):
 *   acc_c[m][n] = sum_{k in segment c} X_q[m][k] * W_q[n][k]                (int32, exact)
 *   y[m][n]     = s_w[n] * sum_c s_c * (acc_c[m][n] - z_c * Wsum_c[n])  (+ bias[n]) (ReLU)
 * in fp32, optionally re-quantised for the next layer (Sec. 4.2: the output channel order is
 * that of the weight's rows, so a following reordered site reads it without an explicit reorder).
 *   a_codes  dev, M rows of Lin.row_bytes bytes (as written by rptq_ln_reorder_quant or by this
 *            function with RPTQ_OUT_CODES)
 *   w_codes  dev, rptq_weight_codes_bytes(Lin.K_pad, N_pad) bytes; s_w dev fp32 [N_pad]; wsum dev
 *            int32 [g][N_pad] (as produced by rptq_weight_pack and copied to the device); N_pad = ld_w >= N
 *   bias     NULL or dev fp32 [N_pad]
 *   act      RPTQ_ACT_NONE or RPTQ_ACT_RELU
 *   y_dtype  RPTQ_OUT_F32 / RPTQ_OUT_F16: y is dev [M][ldy] of that type (ldy >= N, in elements,
 *            ldy*sizeof(type) a multiple of 16).
 *            RPTQ_OUT_CODES: Lout must be given with Lout.K_pad == N; column n of the result is
 *            padded position n of Lout's layout; y receives M rows of Lout.row_bytes bytes of
 *            packed codes q' = clamp(rne(v / s'_c') + z'_c'), pad positions 0; ldy is ignored.
 *   Lout     NULL unless y_dtype == RPTQ_OUT_CODES
 * Limits: Lin.g <= 1024 and Lin.K_pad <= 65536 (the kernel keeps the per-cluster tables in shared
 * memory); beyond them RPTQ_ERR_UNSUPPORTED.
 */
int rptq_cluster_gemm(const rptq_layout_t* Lin, const void* a_codes, int M, const void* w_codes,
                      const float* s_w, const int32_t* wsum, int64_t ld_w, const void* bias, int N,
                      int act, const rptq_layout_t* Lout, void* y, int y_dtype, int64_t ldy,
                      void* stream);

/*
 * Appendix, first computation method: de-quantise both operands, then one floating-point product,
 *   X^ = s_c (X_q - z_c),  W^ = s_w[n] W_q,  y = X^ W^T  (+ bias[n]) (ReLU)
 * as a bfloat16 tensor-core product with fp32 accumulation: X^ is formed in fp32 (one multiply of
 * s_c with the exact integer difference) and rounded to bfloat16 in shared memory; the weight codes
 * are exact in bfloat16 and s_w[n] multiplies the finished fp32 sum. One accumulator per output
 * tile, no per-cluster accumulators: the workload for hardware or precisions where draining an
 * accumulator per cluster costs more than the 16-bit product. Against the second method
 * (rptq_cluster_gemm) the result differs by the bfloat16 rounding of X^ (2^-9 relative per operand).
 * Arguments as for rptq_cluster_gemm (same packed activation codes and packed weights; wsum is not
 * needed); y_dtype RPTQ_OUT_F32 or RPTQ_OUT_F16.
 */
int rptq_dequant_gemm(const rptq_layout_t* Lin, const void* a_codes, int M, const void* w_codes,
                      const float* s_w, int64_t ld_w, const void* bias, int N, int act,
                      void* y, int y_dtype, int64_t ldy, void* stream);

/*
 * Appendix: the weights of an output channel get one asymmetric (scale, zero point) pair per input
 * cluster, W~_q,i = Q_k(W~_i, s^W_i, z^W_i), the paper's own weight scheme (it finds the codes
 * with GPTQ; here round-to-nearest). For output row r and input cluster c with n_c > 0, in fp32:
 *   s = (max - min) / 16 over the row's weights of the cluster (1 if max == min)       [Eq. 2, k = 4]
 *   z = 8 - rne((max + min) / (2 s)),   W_q = clamp(rne(W / s) + z, 0, 15)           [Eq. 1, re-based]
 * The packed buffer has the format and size of rptq_weight_pack's; the stored nibble is W_q - 8.
 *   s_w, z_w, wsum  host [g][N_pad]: scale, zero point of the codes in [0, 15], sum of the codes over
 *                   the cluster's channels. Empty clusters and rows r >= N: s = 1, z = 0, sum 0.
 */
int rptq_weight_pack_clustered(const rptq_layout_t* Lin, const float* W_host, int N, int N_pad,
                               void* w_codes_host, float* s_w, int32_t* z_w, int32_t* wsum);

/*
 * xsum[m][c] = sum of the activation codes of token m over the positions of cluster c (int32, dev
 * [M][g]): the factor of z^W_c in the second computation method of the Appendix.
 *   codes  dev, M rows of L.row_bytes bytes as written by rptq_ln_reorder_quant or an RPTQ_OUT_CODES GEMM
 * g <= 8192.
 */
int rptq_code_rowsums(const rptq_layout_t* L, const void* codes, int M, int32_t* xsum, void* stream);

/*
 * Appendix, second computation method with all four terms (the printed expression leaves the sums
 * and the cluster size out):
 *   Y_q,c[m][n] = sum_k X_q W_q - z^X_c sum_k W_q - z^W_c[n] sum_k X_q + n_c z^X_c z^W_c[n]   (k over cluster c)
 *   y[m][n]     = sum_c s^X_c s^W_c[n] Y_q,c[m][n]  (+ bias[n]) (ReLU), re-quantised if asked for
 * with the integer products exact on the tensor cores and the rest in fp32. Arguments as for
 * rptq_cluster_gemm, except:
 *   xsum           dev int32 [M][g] from rptq_code_rowsums on a_codes
 *   w_codes, s_w, z_w, wsum  as produced by rptq_weight_pack_clustered and copied to the device; the
 *                  three tables are [g][ld_w] with ld_w = N_pad a multiple of 4
 */
int rptq_cluster_gemm_clustered(const rptq_layout_t* Lin, const void* a_codes, int M, const int32_t* xsum,
                                const void* w_codes, const float* s_w, const int32_t* z_w, const int32_t* wsum,
                                int64_t ld_w, const void* bias, int N, int act, const rptq_layout_t* Lout,
                                void* y, int y_dtype, int64_t ldy, void* stream);

/*
 * The same operation as rptq_cluster_gemm, arguments and results included, for callers that must
 * not allocate device memory. (The paper has no counterpart; this is a property of the library.)
 * Who needs it: a process whose device memory is owned wholesale by its own pool -- an inference
 * server that reserves the whole GPU at start-up, or a job running under a fixed memory budget --
 * cannot let a library call cudaMalloc behind its back, and code that is recording work on a
 * stream cannot afford a call that allocates on first use. rptq_cluster_gemm does allocate once,
 * lazily (its status word); this entry point never does: it calls no cudaMalloc, cudaFree or
 * allocating library routine.
 * What it uses instead: a table of one float per output column (the zero-point correction
 * sum_c s_c z_c Wsum_c[n], computed by a small kernel on `stream` just before the GEMM) that lives
 * in a static device array of RPTQ_NOALLOC_MAX_N floats. Every device that loads the library
 * holds these 256 KiB until the process exits.
 *   - N > RPTQ_NOALLOC_MAX_N returns RPTQ_ERR_UNSUPPORTED and launches nothing.
 *   - The first call on a device looks up the table's device address (a host-side query, no
 *     allocation); make that first call outside any stream capture.
 *   - All calls on a device share the one table. Each call rewrites the N entries it will read
 *     before it reads them, so nothing has to be cleared; but two calls that can overlap on the
 *     GPU (different streams, no dependency) race on it. Serialise them.
 *   - A bounded wait that runs out inside the kernel leaves y undefined as in rptq_cluster_gemm,
 *     but is not recorded anywhere: this variant has no status word.
 */
enum { RPTQ_NOALLOC_MAX_N = 65536 };
int rptq_cluster_gemm_noalloc(const rptq_layout_t* Lin, const void* a_codes, int M, const void* w_codes,
                              const float* s_w, const int32_t* wsum, int64_t ld_w, const void* bias, int N,
                              int act, const rptq_layout_t* Lout, void* y, int y_dtype, int64_t ldy,
                              void* stream);

/*
 * Raw per-cluster integer accumulators of an output window (Appendix, X~_q,c W~_q,c before
 * de-quantisation), computed with plain integer instructions and no tensor cores:
 *   acc[c][m - m0][n - n0] = acc_c[m][n],  m0 <= m < m1 <= M, n0 <= n < n1 <= N
 * acc is dev int32 [g][m1-m0][n1-n0].
 */
int rptq_cluster_gemm_debug_acc(const rptq_layout_t* Lin, const void* a_codes, int M,
                                const void* w_codes, int N, int m0, int m1, int n0, int n1,
                                int32_t* acc, void* stream);

/* Host-side readers of the packed formats (format version 2): one byte per code out. */
int rptq_codes_unpack_host(int K_pad, int bits, const void* packed_host, int64_t M, uint8_t* codes_host);
int rptq_codes_pack_host(int K_pad, int bits, const uint8_t* codes_host, int64_t M, void* packed_host);
int rptq_weight_unpack_host(int K_pad, const void* packed_host, int64_t N, int8_t* w_host);
int64_t rptq_weight_codes_bytes(int K_pad, int64_t N_pad);

/*
 * Kernels never spin without a limit: a wait that runs out records RPTQ_ERR_DEVICE_TIMEOUT in a
 * device status word, lets the block drain and return, and leaves the output undefined. This call
 * synchronises the current device, returns that device's word in *status (RPTQ_OK if nothing
 * happened) and clears it. Each device has its own word.
 */
int rptq_get_device_status(int* status);

/*
 * Calibration on the device (Sec. 4.1), off the hot path.
 *
 * Eq. 3 at a LayerNorm site: x_min[c], x_max[c] = minimum and maximum of the LayerNorm output of
 * channel c over T calibration tokens (LayerNorm in fp32 with the arithmetic of
 * rptq_ln_reorder_quant). x dev fp16 [T][ldx], gamma / beta dev fp16 [C], x_min / x_max dev fp32 [C]
 * (overwritten). C <= 16384.
 */
int rptq_ln_channel_minmax(const void* x, int64_t ldx, const void* gamma, const void* beta, float eps,
                           int T, int C, float* x_min, float* x_max, void* stream);

/*
 * Sec. 4.1: K-Means of n points (the channels' (min, max) pairs: dim = 2; Sec. 4.2 clusters Q and K
 * together on (Q_max, Q_min, K_max, K_min): dim = 4) into g clusters. The paper names the algorithm
 * only; the steps are: k-means++ seeding driven by the uniform draws u[0..g-1] (u[0] picks the first
 * centre, u[k] the point at which the running sum of squared distances to the nearest chosen centre
 * passes u[k] times its total), then `iters` Lloyd iterations with squared Euclidean distance in fp64,
 * ties to the lowest centre, a centre without points re-seeded at the point farthest from its own
 * centre. All sums run in point order, so a sequential program taking the same steps gives the same
 * labels.
 *   pts dev fp64 [n][dim], u dev fp64 [g], labels dev int32 [n], centres dev fp64 [g][dim],
 *   inertia NULL or dev fp64 [iters] (sum of squared distances at each assignment step),
 *   workspace dev, rptq_kmeans_workspace_bytes(n, g) bytes, 8-byte aligned. dim <= 8.
 * One thread block does all of it: seconds for tens of thousands of points and hundreds of clusters.
 */
int64_t rptq_kmeans_workspace_bytes(int n, int g);
int rptq_kmeans(const double* pts, int n, int dim, int g, const double* u, int iters, int32_t* labels,
                double* centres, double* inertia, void* workspace, void* stream);

/*
 * Measurement aid (the paper has no counterpart): launches, on `stream`, a kernel that issues the
 * cluster GEMM's own tensor-core instruction -- tcgen05.mma kind::i8 over CTA pairs, 256 x 256 x 32,
 * unsigned x signed 8-bit into int32 -- back to back on operands resident in shared memory, with no
 * loads, unpacking or epilogue, on every SM pair of the current device: n_batches batches of 32
 * instructions per pair. Time the launch with events on `stream`; *ops_out receives the integer
 * operations it performs (2 * 256 * 256 * 32 per instruction), so ops / time is the int8 tensor
 * ceiling of this device at the clocks it ran at.
 *   failed_dev  dev int, zero before the call: set to 1 if a bounded wait inside the kernel ran out
 *   n_batches   1 .. 2^20 (2000 is a few milliseconds)
 */
int rptq_probe_int8_peak(int n_batches, int* failed_dev, double* ops_out, void* stream);

/*
 * Self-test of the give-up path of rptq_ln_reorder_quant (the paper has no counterpart): the same
 * launch with every row's barrier told to expect 16 bytes more than its copy delivers and a wait
 * budget of ten million cycles (~5 ms). The waits run out, RPTQ_ERR_DEVICE_TIMEOUT is recorded in the
 * device's status word, the blocks drain and the kernel returns after some tens of milliseconds;
 * `codes` (M rows of row_bytes bytes) receives undefined bytes. Nothing faults or spins without a
 * limit; the context stays usable. Arguments as for rptq_ln_reorder_quant.
 */
int rptq_selftest_ln_timeout(const rptq_layout_t* L, const void* x, int64_t ldx, const void* gamma,
                             const void* beta, float eps, int M, void* codes, void* stream);

/*
 * Sec. 4.2 and 5.1: self-attention on quantised Q, K and V. The query and the key of a head are
 * multiplied position by position, so they share one reorder index (their channels are clustered
 * together, on the points (Q max, Q min, K max, K min)); the attention sites are reordered per
 * head; the softmax output is quantised at 8 bits. For head h, query i, key j:
 *   A[i][j]  = qk_scale * sum_c s^Q_c s^K_c sum_{p in c} (Q_q[i][p] - z^Q_c)(K_q[j][p] - z^K_c)
 *              (integer products per cluster segment of the head on the tensor cores, fp32 scaling)
 *   key j is visible to query i when causal == 0 or j <= i + (Tk - Tq)
 *   P        = softmax of A over the visible keys (fp32),  P_q = min(rne(P / s_P), 255)
 *   O[i][ch] = s_P s^V_c (sum_j P_q[i][j] V_q[j][p] - z^V_c sum_j P_q[i][j])   for V's position p of channel ch
 *              (integer sums, exact), written as fp16.
 * Layouts: LQ, LK, LV have n_heads * (clusters per head) clusters in RPTQ_ORDER_CONTIGUOUS order, head h
 * owning clusters h * g / n_heads .. (h + 1) * g / n_heads - 1 and the channels h * d .. (h + 1) * d - 1;
 * LQ and LK must have the same reorder index and cluster sizes (their scales and zero points differ).
 * A head may take at most 8 units of 32 positions in each layout.
 *   n_seq    sequences in the call, each with Tq queries and Tk keys; their rows follow one another
 *   q_codes  dev, n_seq * Tq rows of LQ.row_bytes bytes (as an RPTQ_OUT_CODES GEMM writes them)
 *   k_codes, v_codes  dev, n_seq * Tk rows of LK.row_bytes / LV.row_bytes bytes: the quantised key / value cache
 *   s_P, z_P Eq. 1 parameters of the softmax output for codes in [0, 255]; z_P must be 0 (Eq. 2 on a
 *            range that starts at 0 gives exactly that), otherwise RPTQ_ERR_UNSUPPORTED
 *   out_f16  dev fp16 [n_seq * Tq][ldo], ldo >= LV.C: channel ch of query row i at out[i * ldo + ch]
 *   p_codes_out  NULL, or dev uint8 [n_seq][n_heads][Tq][Tk]: receives P_q at the visible keys of key tiles
 *            that hold a visible key (a test aid; clear it before the call)
 * Tk >= Tq; Tk * 255 * 255 < 2^31; n_seq, n_heads <= 65535. Row-constant terms of A cancel in the softmax and are not formed.
 */
int rptq_attention(const rptq_layout_t* LQ, const rptq_layout_t* LK, const rptq_layout_t* LV, int n_heads,
                   const void* q_codes, int Tq, const void* k_codes, const void* v_codes, int Tk, int n_seq,
                   float s_P, int z_P, float qk_scale, int causal,
                   void* out_f16, int64_t ldo, uint8_t* p_codes_out, void* stream);

/*
 * Sec. 5.2, the schemes that quantise only the key / value cache (W4A4KV, W4A3KV, W3A3KV): the query and
 * the softmax output stay 16-bit floating point; the cached keys and values are per-cluster codes of the
 * per-head layouts LK and LV (as for rptq_attention; K's layout is the one Q and K were clustered for). For
 * head h, query i, key j:
 *   A[i][j]  = qk_scale * sum_c s^K_c sum_{p in c} Q[i][ch(p)] (K_q[j][p] - z^K_c)     ch(p): the channel at K's position p
 *   P        = softmax of A over the visible keys (as for rptq_attention), fp32, rounded to fp16 for the second product
 *   O[i][ch] = s^V_c (sum_j P[i][j] V_q[j][p] / sum_j P[i][j] - z^V_c)                 fp16
 * fp16 x fp16 products with fp32 sums on the tensor cores (the codes are exact in fp16).
 *   q_f16    dev fp16 [n_seq * Tq][ldq], ldq >= C, original channel order (head h owns channels h * C / n_heads ..)
 *   k_codes, v_codes  dev, n_seq * Tk rows of LK.row_bytes / LV.row_bytes bytes
 *   out_f16  dev fp16 [n_seq * Tq][ldo], ldo >= C, original channel order
 * Limits as for rptq_attention (eight units per head and layout, Tk >= Tq, n_seq, n_heads <= 65535).
 */
int rptq_attention_kv(const rptq_layout_t* LK, const rptq_layout_t* LV, int n_heads,
                      const void* q_f16, int64_t ldq, int Tq, const void* k_codes, const void* v_codes, int Tk, int n_seq,
                      float qk_scale, int causal, void* out_f16, int64_t ldo, void* stream);

const char* rptq_status_string(int status);
int rptq_format_version(void);

#ifdef __cplusplus
}
#endif
#endif /* RPTQ_H_ */
