// Host side of librptq.so: the layout handle (reorder index S with per-cluster parameters,
// Sec. 4.1), the offline weight preparation (Sec. 4.2), the packed-format readers and the
// device status word.
#include <cmath>
#include <cstring>
#include <mutex>
#include <new>

#include <algorithm>

#include "rptq_internal.h"

namespace rptq {

// One status word per device, allocated on first use with that device current: a kernel that gives
// up a wait writes to the word of the device it runs on.
constexpr int kMaxDevices = 64;
static std::mutex g_status_mutex;
static int* g_status_word[kMaxDevices] = {};

int* device_status_word()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_status_mutex);
    if (g_status_word[dev] == nullptr) {
        int* p = nullptr;
        if (cudaMalloc(&p, 256) != cudaSuccess) return nullptr;
        if (cudaMemset(p, 0, 256) != cudaSuccess) { cudaFree(p); return nullptr; }
        g_status_word[dev] = p;
    }
    return g_status_word[dev];
}

template <class T>
static int upload(T** dst, const T* src, size_t n)
{
    if (n == 0) n = 1;
    if (cudaMalloc(reinterpret_cast<void**>(dst), n * sizeof(T)) != cudaSuccess) return RPTQ_ERR_ALLOC;
    if (src && cudaMemcpy(*dst, src, n * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess) return RPTQ_ERR_CUDA;
    return RPTQ_OK;
}

// ---- packed formats, word at a time ------------------------------------------------------------
// 4-bit: word = lo | hi << 4 where lo holds codes 0..3 one per byte and hi codes 4..7.
static inline uint32_t word_of_bytes(const uint8_t* c) { return c[0] | (c[1] << 8) | (c[2] << 16) | ((uint32_t)c[3] << 24); }

static void pack_row(const uint8_t* codes, int K_pad, int bits, uint8_t* out)
{
    if (bits == 8) { std::memcpy(out, codes, (size_t)K_pad); return; }
    uint32_t* w = reinterpret_cast<uint32_t*>(out);
    if (bits == 4) {
        for (int i = 0; i < K_pad / 8; ++i)
            w[i] = (word_of_bytes(codes + 8 * i) & 0x0F0F0F0Fu) | ((word_of_bytes(codes + 8 * i + 4) & 0x0F0F0F0Fu) << 4);
        return;
    }
    for (int grp = 0; grp < K_pad / 32; ++grp) {
        const uint8_t* c = codes + 32 * grp;
        uint32_t tail = (word_of_bytes(c + 24) & 0x07070707u) | ((word_of_bytes(c + 28) & 0x07070707u) << 4);
        for (int j = 0; j < 3; ++j) {
            uint32_t body = (word_of_bytes(c + 8 * j) & 0x07070707u) | ((word_of_bytes(c + 8 * j + 4) & 0x07070707u) << 4);
            w[3 * grp + j] = body | (((tail >> j) & 0x11111111u) << 3);
        }
    }
}

static inline void bytes_of_word(uint32_t v, uint8_t* c) { c[0] = v; c[1] = v >> 8; c[2] = v >> 16; c[3] = v >> 24; }

static void unpack_row(const uint8_t* in, int K_pad, int bits, uint8_t* codes)
{
    if (bits == 8) { std::memcpy(codes, in, (size_t)K_pad); return; }
    const uint32_t* w = reinterpret_cast<const uint32_t*>(in);
    if (bits == 4) {
        for (int i = 0; i < K_pad / 8; ++i) {
            bytes_of_word(w[i] & 0x0F0F0F0Fu, codes + 8 * i);
            bytes_of_word((w[i] >> 4) & 0x0F0F0F0Fu, codes + 8 * i + 4);
        }
        return;
    }
    for (int grp = 0; grp < K_pad / 32; ++grp) {
        uint32_t tail = 0;
        for (int j = 0; j < 3; ++j) {
            uint32_t v = w[3 * grp + j];
            bytes_of_word(v & 0x07070707u, codes + 32 * grp + 8 * j);
            bytes_of_word((v >> 4) & 0x07070707u, codes + 32 * grp + 8 * j + 4);
            tail |= ((v >> 3) & 0x11111111u) << j;
        }
        bytes_of_word(tail & 0x07070707u, codes + 32 * grp + 24);
        bytes_of_word((tail >> 4) & 0x07070707u, codes + 32 * grp + 28);
    }
}

}  // namespace rptq

using namespace rptq;

extern "C" {

int rptq_format_version(void) { return RPTQ_FORMAT_VERSION; }

const char* rptq_status_string(int status)
{
    switch (status) {
        case RPTQ_OK: return "ok";
        case RPTQ_ERR_INVALID_ARG: return "invalid argument";
        case RPTQ_ERR_UNSUPPORTED: return "unsupported size or option";
        case RPTQ_ERR_NOT_BIJECTION: return "reorder index is not a bijection";
        case RPTQ_ERR_CUDA: return "CUDA call failed";
        case RPTQ_ERR_DEVICE_TIMEOUT: return "bounded wait inside a kernel ran out";
        case RPTQ_ERR_ALLOC: return "allocation failed";
        default: return "unknown status";
    }
}

int rptq_get_device_status(int* status)
{
    if (!status) return RPTQ_ERR_INVALID_ARG;
    int* word = device_status_word();
    if (!word) return RPTQ_ERR_ALLOC;
    if (cudaDeviceSynchronize() != cudaSuccess) return RPTQ_ERR_CUDA;
    int v = 0;
    if (cudaMemcpy(&v, word, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return RPTQ_ERR_CUDA;
    if (v != 0 && cudaMemset(word, 0, sizeof(int)) != cudaSuccess) return RPTQ_ERR_CUDA;
    *status = v;
    return RPTQ_OK;
}

int rptq_layout_create(rptq_layout_t** out, int C, int g, int bits, const int32_t* perm_host,
                       const int32_t* cluster_size, const float* scale_host, const int32_t* zero_host, int order)
{
    if (!out) return RPTQ_ERR_INVALID_ARG;
    *out = nullptr;
    if (!perm_host || !cluster_size || !scale_host || !zero_host) return RPTQ_ERR_INVALID_ARG;
    if (order != RPTQ_ORDER_CONTIGUOUS && order != RPTQ_ORDER_INTERLEAVED) return RPTQ_ERR_INVALID_ARG;
    if (C <= 0 || g <= 0) return RPTQ_ERR_INVALID_ARG;
    if (bits != 3 && bits != 4 && bits != 8) return RPTQ_ERR_UNSUPPORTED;
    if (C % 8 != 0 || C < 8 || C > 65528 || g > 4096) return RPTQ_ERR_UNSUPPORTED;

    // S must be a bijection and the sizes must tile it
    std::vector<uint8_t> seen((size_t)C, 0);
    for (int j = 0; j < C; ++j) {
        int32_t c = perm_host[j];
        if (c < 0 || c >= C || seen[c]) return RPTQ_ERR_NOT_BIJECTION;
        seen[c] = 1;
    }
    int64_t total = 0, padded = 0;
    for (int c = 0; c < g; ++c) {
        if (cluster_size[c] < 0) return RPTQ_ERR_INVALID_ARG;
        total += cluster_size[c];
        padded += (cluster_size[c] + 31) / 32 * 32;
        if (!(scale_host[c] > 0.0f) || !std::isfinite(scale_host[c])) return RPTQ_ERR_INVALID_ARG;
        if (zero_host[c] <= -(1 << 21) || zero_host[c] >= (1 << 21)) return RPTQ_ERR_UNSUPPORTED;
    }
    if (total != C) return RPTQ_ERR_NOT_BIJECTION;
    int64_t k_pad = (padded + 127) / 128 * 128;
    if (k_pad < 128) k_pad = 128;
    if (k_pad > 65408) return RPTQ_ERR_UNSUPPORTED;

    rptq_layout* L = new (std::nothrow) rptq_layout();
    if (!L) return RPTQ_ERR_ALLOC;
    L->C = C; L->g = g; L->bits = bits; L->K_pad = (int)k_pad;
    L->row_bytes = k_pad * bits / 8;
    L->n_units = (int)(k_pad / 32);
    L->perm.assign(perm_host, perm_host + C);
    L->size.assign(cluster_size, cluster_size + g);
    L->scale.assign(scale_host, scale_host + g);
    L->zero.assign(zero_host, zero_host + g);
    // Without a CUDA device the handle is host-only: rptq_weight_pack and rptq_layout_query work,
    // kernel launches report RPTQ_ERR_CUDA.
    int n_dev = 0;
    const bool have_device = cudaGetDeviceCount(&n_dev) == cudaSuccess && n_dev > 0;
    if (!have_device) (void)cudaGetLastError();
    if (have_device && cudaGetDevice(&L->device) != cudaSuccess) { delete L; return RPTQ_ERR_CUDA; }

    // ---- unit order: a list of runs (cluster, first unit within the cluster, units)
    struct Run { int c, u0, nu; };
    std::vector<Run> runs;
    std::vector<int> n_units_of((size_t)g), j_start((size_t)g);
    {
        int j = 0;
        for (int c = 0; c < g; ++c) { n_units_of[c] = (cluster_size[c] + 31) / 32; j_start[c] = j; j += cluster_size[c]; }
    }
    constexpr int kSmallUnits = 2, kGap = 7;
    std::vector<int> small, big;
    for (int c = 0; c < g; ++c) {
        if (n_units_of[c] == 0) continue;
        (n_units_of[c] <= kSmallUnits ? small : big).push_back(c);
    }
    if (order == RPTQ_ORDER_INTERLEAVED && small.size() >= 2 && !big.empty()) {
        size_t next_small = 0;
        int since = 0;                       // larger-cluster units since the last small cluster
        for (int c : big) {
            int u = 0;
            while (u < n_units_of[c]) {
                const int take = std::min(n_units_of[c] - u, kGap - since);
                runs.push_back({c, u, take});
                u += take; since += take;
                if (since == kGap) {
                    if (next_small < small.size()) { const int t = small[next_small++]; runs.push_back({t, 0, n_units_of[t]}); }
                    since = 0;
                }
            }
        }
        for (; next_small < small.size(); ++next_small) { const int t = small[next_small]; runs.push_back({t, 0, n_units_of[t]}); }
    } else {
        for (int c = 0; c < g; ++c) if (n_units_of[c] > 0) runs.push_back({c, 0, n_units_of[c]});
    }

    std::vector<uint16_t> src((size_t)k_pad, 0);                 // channel read for each position (at pads: any, the code is masked)
    std::vector<int32_t> jidx((size_t)k_pad, -1);                // reordered index at each position, -1 at pads
    std::vector<UnitInfo> unit((size_t)L->n_units);
    std::vector<uint8_t> flags((size_t)L->n_units, STEP_SKIP);
    std::vector<float> seg_scale, cl_sz((size_t)g), cl_n((size_t)g);
    std::vector<int32_t> seg_cluster;
    std::vector<uint8_t> seg_buf;
    L->unit_cluster.assign((size_t)L->n_units, -1);
    L->pos.assign((size_t)C, 0);
    for (auto& u : unit) { u.inv_s = 1.0f; u.zc = 0 - 0x4B400000; u.j0 = 0; u.nvalid = 0; }
    for (int c = 0; c < g; ++c) { cl_sz[c] = scale_host[c] * (float)zero_host[c]; cl_n[c] = (float)cluster_size[c]; }
    // Accumulator of each cluster: the one that is not held by a cluster still under way; when
    // both are free, the one whose last cluster ended longer ago (its drain has had more time).
    int last_end[2] = {-2, -1};              // unit index at which each accumulator's last cluster ended
    std::vector<int> buf_of((size_t)g, -1);
    int open_buf = -1, open_cluster = -1, cur = 0;
    for (const Run& r : runs) {
        const int c = r.c, n = cluster_size[c];
        const float inv_s = (float)(1.0 / (double)scale_host[c]);
        for (int k = 0; k < r.nu; ++k, ++cur) {
            const int uc = r.u0 + k;         // unit within the cluster
            uint8_t f = 0;
            if (uc == 0) {
                f |= STEP_FIRST;
                if (open_cluster >= 0 && open_cluster != c) buf_of[c] = 1 - open_buf;
                else buf_of[c] = last_end[0] <= last_end[1] ? 0 : 1;
                if (n_units_of[c] > r.nu) { open_cluster = c; open_buf = buf_of[c]; }   // continues in later runs
            }
            if (uc == n_units_of[c] - 1) {
                f |= STEP_LAST;
                last_end[buf_of[c]] = cur;
                seg_scale.push_back(scale_host[c]);
                seg_buf.push_back((uint8_t)buf_of[c]);
                seg_cluster.push_back(c);
                L->n_seg++;
                if (open_cluster == c) { open_cluster = -1; open_buf = -1; }
            }
            if (buf_of[c]) f |= STEP_BUF;
            flags[cur] = f;
            L->unit_cluster[cur] = c;
            UnitInfo& ui = unit[cur];
            ui.inv_s = inv_s;
            ui.zc = zero_host[c] - 0x4B400000;
            ui.j0 = j_start[c] + 32 * uc;
            ui.nvalid = (n - 32 * uc) < 32 ? (n - 32 * uc) : 32;
        }
    }
    // ---- which channel of a cluster goes to which of the cluster's positions. All channels of a
    // cluster share (s_c, z_c), so any assignment is the same quantisation. rptq_ln_reorder_quant
    // gives every unit to one thread, and the 32 threads of a warp (32 consecutive units) read
    // element e of their units in the same instruction, from the raw fp16 row in shared memory:
    // channel ch sits in bank (ch / 2) mod 32. Rows of 32 such reads are filled greedily with
    // channels from 32 different banks, always from the fullest bank of the lane's cluster.
    {
        std::vector<std::vector<int>> pool((size_t)g * 32);          // [cluster][bank]: reordered indices j, descending
        for (int c = 0; c < g; ++c)
            for (int i = cluster_size[c] - 1; i >= 0; --i) {
                const int j = j_start[c] + i;
                pool[(size_t)c * 32 + ((perm_host[j] >> 1) & 31)].push_back(j);
            }
        for (int w0 = 0; w0 < L->n_units; w0 += 32)
            for (int e = 0; e < 32; ++e) {
                uint32_t used = 0;
                int first_real = -1;             // channel read by the first lane that has an element e
                for (int l = 0; l < 32 && w0 + l < L->n_units; ++l) {
                    const int u = w0 + l, c = L->unit_cluster[u];
                    if (c < 0 || e >= unit[u].nvalid) continue;
                    int best = -1, any = -1;
                    size_t best_n = 0, any_n = 0;
                    for (int b = 0; b < 32; ++b) {
                        const size_t n_b = pool[(size_t)c * 32 + b].size();
                        if (n_b > any_n) { any_n = n_b; any = b; }
                        if (!((used >> b) & 1u) && n_b > best_n) { best_n = n_b; best = b; }
                    }
                    const int b = best >= 0 ? best : any;
                    std::vector<int>& from = pool[(size_t)c * 32 + b];
                    const int j = from.back();
                    from.pop_back();
                    used |= 1u << b;
                    L->pos[j] = u * 32 + e;
                    src[u * 32 + e] = (uint16_t)perm_host[j];
                    jidx[u * 32 + e] = j;
                    if (first_real < 0) first_real = perm_host[j];
                }
                // Lanes whose unit has no element e still execute the read; their codes are masked
                // to zero afterwards, so they read what another lane reads (a broadcast costs nothing).
                for (int l = 0; l < 32 && w0 + l < L->n_units; ++l)
                    if (e >= unit[w0 + l].nvalid) src[(w0 + l) * 32 + e] = (uint16_t)(first_real < 0 ? 0 : first_real);
            }
    }

    if (!have_device) { *out = L; return RPTQ_OK; }
    int rc = upload(&L->d_src, src.data(), src.size());
    if (rc == RPTQ_OK) rc = upload(&L->d_jidx, jidx.data(), jidx.size());
    if (rc == RPTQ_OK) rc = upload(&L->d_unit, unit.data(), unit.size());
    if (rc == RPTQ_OK) rc = upload(&L->d_step_flags, flags.data(), flags.size());
    if (rc == RPTQ_OK) rc = upload(&L->d_seg_scale, seg_scale.data(), seg_scale.size());
    if (rc == RPTQ_OK) rc = upload(&L->d_cl_sz, cl_sz.data(), cl_sz.size());
    if (rc == RPTQ_OK) rc = upload(&L->d_seg_buf, seg_buf.data(), seg_buf.size());
    if (rc == RPTQ_OK) rc = upload(&L->d_cl_n, cl_n.data(), cl_n.size());
    if (rc == RPTQ_OK) rc = upload(&L->d_seg_cluster, seg_cluster.data(), seg_cluster.size());
    std::vector<float2> unit_sz((size_t)L->n_units, make_float2(1.0f, 0.0f));
    for (int u = 0; u < L->n_units; ++u)
        if (L->unit_cluster[u] >= 0) unit_sz[u] = make_float2(scale_host[L->unit_cluster[u]], (float)zero_host[L->unit_cluster[u]]);
    if (rc == RPTQ_OK) rc = upload(&L->d_unit_sz, unit_sz.data(), unit_sz.size());
    if (rc == RPTQ_OK) rc = upload(&L->d_unit_cluster, L->unit_cluster.data(), L->unit_cluster.size());
    if (rc != RPTQ_OK) { rptq_layout_destroy(L); return rc; }
    *out = L;
    return RPTQ_OK;
}

int rptq_layout_query(const rptq_layout_t* L, int* K_pad, int64_t* row_bytes, int32_t* unit_cluster_out)
{
    if (!L) return RPTQ_ERR_INVALID_ARG;
    if (K_pad) *K_pad = L->K_pad;
    if (row_bytes) *row_bytes = L->row_bytes;
    if (unit_cluster_out) std::memcpy(unit_cluster_out, L->unit_cluster.data(), sizeof(int32_t) * (size_t)L->n_units);
    return RPTQ_OK;
}

int rptq_layout_padded_index(const rptq_layout_t* L, int32_t* padded_index)
{
    if (!L || !padded_index) return RPTQ_ERR_INVALID_ARG;
    for (int p = 0; p < L->K_pad; ++p) padded_index[p] = -1;
    for (int j = 0; j < L->C; ++j) padded_index[L->pos[j]] = L->perm[j];
    return RPTQ_OK;
}

int rptq_layout_destroy(rptq_layout_t* L)
{
    if (!L) return RPTQ_OK;
    cudaFree(L->d_src);
    cudaFree(L->d_jidx);
    cudaFree(L->d_unit);
    cudaFree(L->d_step_flags);
    cudaFree(L->d_seg_scale);
    cudaFree(L->d_cl_sz);
    cudaFree(L->d_seg_buf);
    cudaFree(L->d_cl_n);
    cudaFree(L->d_seg_cluster);
    cudaFree(L->d_unit_sz);
    cudaFree(L->d_unit_cluster);
    delete L;
    return RPTQ_OK;
}

int rptq_codes_pack_host(int K_pad, int bits, const uint8_t* codes_host, int64_t M, void* packed_host)
{
    if (!codes_host || !packed_host || M < 0 || K_pad <= 0 || K_pad % 128) return RPTQ_ERR_INVALID_ARG;
    if (bits != 3 && bits != 4 && bits != 8) return RPTQ_ERR_UNSUPPORTED;
    const int64_t rb = (int64_t)K_pad * bits / 8;
    for (int64_t m = 0; m < M; ++m) pack_row(codes_host + m * K_pad, K_pad, bits, static_cast<uint8_t*>(packed_host) + m * rb);
    return RPTQ_OK;
}

int rptq_codes_unpack_host(int K_pad, int bits, const void* packed_host, int64_t M, uint8_t* codes_host)
{
    if (!codes_host || !packed_host || M < 0 || K_pad <= 0 || K_pad % 128) return RPTQ_ERR_INVALID_ARG;
    if (bits != 3 && bits != 4 && bits != 8) return RPTQ_ERR_UNSUPPORTED;
    const int64_t rb = (int64_t)K_pad * bits / 8;
    for (int64_t m = 0; m < M; ++m) unpack_row(static_cast<const uint8_t*>(packed_host) + m * rb, K_pad, bits, codes_host + m * K_pad);
    return RPTQ_OK;
}

int64_t rptq_weight_codes_bytes(int K_pad, int64_t N_pad)
{
    if (K_pad <= 0 || K_pad % 128 || N_pad < 0) return RPTQ_ERR_INVALID_ARG;
    return (N_pad + 127) / 128 * 128 * (int64_t)(K_pad / 2);
}

int rptq_weight_unpack_host(int K_pad, const void* packed_host, int64_t N, int8_t* w_host)
{
    if (!w_host || !packed_host || N < 0 || K_pad <= 0 || K_pad % 128) return RPTQ_ERR_INVALID_ARG;
    const int n_kb = K_pad / 128;
    for (int64_t n = 0; n < N; ++n) {
        uint8_t* dst = reinterpret_cast<uint8_t*>(w_host) + n * K_pad;
        for (int kb = 0; kb < n_kb; ++kb)     // one 64-byte piece of the row per tile
            unpack_row(static_cast<const uint8_t*>(packed_host) + weight_tile_offset(n, kb, n_kb), 128, 4, dst + 128 * kb);
        for (int p = 0; p < K_pad; ++p) dst[p] = (uint8_t)((dst[p] ^ 8u) - 8u);   // sign-extend the nibble
    }
    return RPTQ_OK;
}

int rptq_weight_pack(const rptq_layout_t* Lin, const float* W_host, int N, const int32_t* out_perm,
                     int N_pad, void* w_codes_host, float* s_w, int32_t* wsum)
{
    if (!Lin || !W_host || !w_codes_host || !s_w || !wsum) return RPTQ_ERR_INVALID_ARG;
    if (N <= 0 || N_pad < N) return RPTQ_ERR_INVALID_ARG;
    const int C = Lin->C, g = Lin->g, K_pad = Lin->K_pad;
    if (out_perm) {
        std::vector<uint8_t> seen((size_t)N, 0);
        for (int r = 0; r < N_pad; ++r) {
            if (out_perm[r] < 0) continue;
            if (out_perm[r] >= N || seen[out_perm[r]]) return RPTQ_ERR_NOT_BIJECTION;
            seen[out_perm[r]] = 1;
        }
    }
    const int n_kb = K_pad / 128;
    const int rows_stored = (N_pad + 127) / 128 * 128;        // the last tile is filled with zero rows
    uint8_t* packed = static_cast<uint8_t*>(w_codes_host);
    int failed = 0;            // set by any worker that meets a non-finite weight (atomic write)
#pragma omp parallel
    {
        std::vector<uint8_t> row((size_t)K_pad), row_packed((size_t)K_pad / 2);
#pragma omp for schedule(static)
        for (int r = 0; r < rows_stored; ++r) {
            if (r >= N_pad) {
                for (int kb = 0; kb < n_kb; ++kb) std::memset(packed + weight_tile_offset(r, kb, n_kb), 0, 64);
                continue;
            }
            std::memset(row.data(), 0, (size_t)K_pad);
            float s = 1.0f;
            const int src_row = out_perm ? out_perm[r] : (r < N ? r : -1);
            if (src_row >= 0) {
                const float* w = W_host + (int64_t)src_row * C;
                float amax = 0.0f;
                for (int k = 0; k < C; ++k) amax = fmaxf(amax, fabsf(w[k]));
                if (!std::isfinite(amax)) {
#pragma omp atomic write
                    failed = 1;
                }
                if (amax > 0.0f) s = amax / 7.0f;
                int j = 0;
                for (int c = 0; c < g; ++c) {
                    int32_t sum = 0;
                    for (int i = 0; i < Lin->size[c]; ++i, ++j) {
                        float q = rintf(w[Lin->perm[j]] / s);
                        q = fminf(fmaxf(q, -8.0f), 7.0f);
                        const int qi = (int)q;
                        sum += qi;
                        row[Lin->pos[j]] = (uint8_t)(qi & 0xF);
                    }
                    wsum[(int64_t)c * N_pad + r] = sum;
                }
            } else {
                for (int c = 0; c < g; ++c) wsum[(int64_t)c * N_pad + r] = 0;
            }
            s_w[r] = s;
            pack_row(row.data(), K_pad, 4, row_packed.data());
            for (int kb = 0; kb < n_kb; ++kb) std::memcpy(packed + weight_tile_offset(r, kb, n_kb), row_packed.data() + 64 * kb, 64);
        }
    }
    return failed ? RPTQ_ERR_INVALID_ARG : RPTQ_OK;
}

int rptq_weight_pack_clustered(const rptq_layout_t* Lin, const float* W_host, int N, int N_pad,
                               void* w_codes_host, float* s_w, int32_t* z_w, int32_t* wsum)
{
    if (!Lin || !W_host || !w_codes_host || !s_w || !z_w || !wsum) return RPTQ_ERR_INVALID_ARG;
    if (N <= 0 || N_pad < N) return RPTQ_ERR_INVALID_ARG;
    const int C = Lin->C, g = Lin->g, K_pad = Lin->K_pad;
    const int n_kb = K_pad / 128;
    const int rows_stored = (N_pad + 127) / 128 * 128;
    uint8_t* packed = static_cast<uint8_t*>(w_codes_host);
    std::vector<int> j_start((size_t)g);
    for (int c = 0, j = 0; c < g; ++c) { j_start[c] = j; j += Lin->size[c]; }
    int failed = 0;
#pragma omp parallel
    {
        std::vector<uint8_t> row((size_t)K_pad), row_packed((size_t)K_pad / 2);
#pragma omp for schedule(static)
        for (int r = 0; r < rows_stored; ++r) {
            if (r >= N_pad) {
                for (int kb = 0; kb < n_kb; ++kb) std::memset(packed + weight_tile_offset(r, kb, n_kb), 0, 64);
                continue;
            }
            // positions that hold no channel, and rows past N, store code 8 (the nibble 0)
            std::memset(row.data(), 0, (size_t)K_pad);
            for (int c = 0; c < g; ++c) {
                float s = 1.0f;
                int32_t z = 0, sum = 0;
                const int n_c = Lin->size[c];
                if (r < N && n_c > 0) {
                    const float* w = W_host + (int64_t)r * C;
                    float lo = INFINITY, hi = -INFINITY;
                    for (int i = 0; i < n_c; ++i) {
                        const float v = w[Lin->perm[j_start[c] + i]];
                        lo = fminf(lo, v); hi = fmaxf(hi, v);
                    }
                    if (!std::isfinite(lo) || !std::isfinite(hi)) {
#pragma omp atomic write
                        failed = 1;
                    }
                    s = (hi - lo) / 16.0f;                              // Eq. 2, k = 4
                    if (!(s > 0.0f)) s = 1.0f;
                    const float mid = (hi + lo) / (2.0f * s);
                    z = 8 - (int32_t)rintf(mid);
                    for (int i = 0; i < n_c; ++i) {
                        const int j = j_start[c] + i;
                        float q = rintf(w[Lin->perm[j]] / s) + (float)z;   // Eq. 1
                        q = fminf(fmaxf(q, 0.0f), 15.0f);
                        const int qi = (int)q;
                        sum += qi;
                        row[Lin->pos[j]] = (uint8_t)((qi - 8) & 0xF);
                    }
                }
                s_w[(int64_t)c * N_pad + r] = s;
                z_w[(int64_t)c * N_pad + r] = z;
                wsum[(int64_t)c * N_pad + r] = sum;
            }
            pack_row(row.data(), K_pad, 4, row_packed.data());
            for (int kb = 0; kb < n_kb; ++kb) std::memcpy(packed + weight_tile_offset(r, kb, n_kb), row_packed.data() + 64 * kb, 64);
        }
    }
    return failed ? RPTQ_ERR_INVALID_ARG : RPTQ_OK;
}

}  // extern "C"
