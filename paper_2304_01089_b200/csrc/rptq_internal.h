// Internal declarations shared by the translation units of librptq.so. Not part of the C boundary.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "rptq.h"

namespace rptq {

// One entry per group of 32 padded positions ("unit"). A unit belongs to one cluster.
struct UnitInfo {
    float inv_s;      // (float)(1.0 / (double)s_c)
    int32_t zc;       // z_c - 0x4B400000: added to the bit pattern of (t + 1.5*2^23)
    int32_t j0;       // reordered channel index of the unit's first position
    int32_t nvalid;   // real (non-pad) positions in the unit, 0..32; real ones come first
};
static_assert(sizeof(UnitInfo) == 16, "UnitInfo is loaded as one 16-byte vector");

// Flags of one contraction step (32 consecutive padded positions) along K.
// FIRST / LAST: first / last step of its cluster (a cluster's steps need not be adjacent); SKIP: no
// cluster; BUF: which of the two accumulators the cluster uses.
enum : uint8_t { STEP_FIRST = 1, STEP_LAST = 2, STEP_SKIP = 4, STEP_BUF = 8 };

constexpr int kMaxGemmSegments = 1024;

// Byte offset of the 64-byte piece (row n, K block kb) in the tile-major packed weight buffer.
__host__ __device__ inline int64_t weight_tile_offset(int64_t n, int kb, int n_kb) { return ((n >> 7) * n_kb + kb) * 8192 + (n & 127) * 64; }

}  // namespace rptq

struct rptq_layout {
    int C = 0, g = 0, bits = 0, K_pad = 0, device = -1;
    int64_t row_bytes = 0;
    int n_units = 0;   // K_pad / 32
    int n_seg = 0;     // clusters with n_c > 0
    std::vector<int32_t> perm, size, zero;
    std::vector<int32_t> pos;            // [C]       padded position of reordered channel j
    std::vector<int32_t> unit_cluster;   // [n_units] owning cluster, -1 past the last cluster
    std::vector<float> scale;
    // device tables
    uint16_t* d_src = nullptr;          // [K_pad] channel read for each padded position (at pads: some channel, the code is masked)
    int32_t* d_jidx = nullptr;          // [K_pad] reordered index at each padded position, -1 at pads
    rptq::UnitInfo* d_unit = nullptr;   // [n_units]
    uint8_t* d_step_flags = nullptr;    // [n_units]
    float* d_seg_scale = nullptr;       // [n_seg]  s_c of the non-empty clusters, in the order their last steps come
    uint8_t* d_seg_buf = nullptr;       // [n_seg]  the accumulator each of them uses, same order
    float* d_cl_sz = nullptr;           // [g]      s_c * z_c
    float* d_cl_n = nullptr;            // [g]      n_c
    int32_t* d_seg_cluster = nullptr;   // [n_seg]  the cluster of each entry of d_seg_scale
    float2* d_unit_sz = nullptr;        // [n_units] {s_c, (float) z_c} of the unit's cluster ({1, 0} where there is none)
    int32_t* d_unit_cluster = nullptr;  // [n_units]
};

namespace rptq {

// The cluster GEMM for at most 16 tokens (small_m_gemm.cu).
struct SmallMParams {
    const uint8_t* a; int64_t a_row_bytes; int M, K_pad, n_units, n_kb;
    const uint8_t* w; int n_wtiles;
    const uint8_t* step_flags; const int32_t* unit_cluster; const float2* unit_sz; const float* cl_sz; int g;
    const float* corr; const float* s_w; const int32_t* wsum; int64_t ld_w; const float* bias;
    int N, act, y_dtype; void* y; int64_t ldy; int* status;
};
namespace smallm {
bool fits(int M, int bits, int K_pad);
int launch(const SmallMParams& p, int bits, cudaStream_t st);
}

int* device_status_word();   // lazily allocated device int, RPTQ_OK when clear; nullptr on failure

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace rptq
