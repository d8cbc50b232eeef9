// Shared declarations of the LQ-LoRA CUDA library: configuration checks, the packed-code
// addressing rule, code-book tables and small device helpers.  Product code only; the CPU
// oracle shares nothing with this file.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lqlora.h"

namespace lq {

constexpr int kTileRows = 128;   // rows of a packed tile
constexpr int kTileCols = 64;    // columns of a packed tile
constexpr int kSlabRows = 32;    // rows of a slab (one warp's worth)
// 2^(b1-1) - 1 positive levels of the b1-bit round-to-nearest quantizer of the block scales (Sec. 2.2, Sec. 3.2)
__host__ __device__ inline int scale_levels(int b1) { return (1 << (b1 - 1)) - 1; }
// Second-level scale formats (the b2 field): 32 = fp32, 16 = IEEE fp16, -16 = bfloat16 (Table 1 of Sec. 3.2)
constexpr int kB2Fp32 = 32, kB2Fp16 = 16, kB2Bf16 = -16;
constexpr int kStatusBytes = 256;  // status word area at the start of a linear workspace

// Index of a code width in the table arrays.
__host__ __device__ inline int bits_index(int b0) { return b0 == 2 ? 0 : b0 == 3 ? 1 : b0 == 4 ? 2 : 3; }

inline int ilog2(int x) { int l = 0; while ((1 << l) < x) ++l; return l; }
inline bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

inline int check_config(const lqlora_config* c) {
    if (!c) return LQLORA_ERR_NULL_POINTER;
    if (!(c->b0 == 2 || c->b0 == 3 || c->b0 == 4 || c->b0 == 8)) return LQLORA_ERR_INVALID_CONFIG;
    if (!is_pow2(c->B0) || c->B0 < 16 || c->B0 > 256) return LQLORA_ERR_INVALID_CONFIG;
    if (!is_pow2(c->B1) || c->B1 < 16 || c->B1 > 4096) return LQLORA_ERR_INVALID_CONFIG;
    if (!(c->b1 == 2 || c->b1 == 3 || c->b1 == 4 || c->b1 == 8)) return LQLORA_ERR_INVALID_CONFIG;
    if (!(c->b2 == kB2Fp32 || c->b2 == kB2Fp16 || c->b2 == kB2Bf16)) return LQLORA_ERR_INVALID_CONFIG;
    return LQLORA_OK;
}

inline int check_shape(int64_t N, int64_t K, const lqlora_config* c) {
    if (N <= 0 || K <= 0) return LQLORA_ERR_INVALID_SHAPE;
    if (K % kTileCols != 0 || K % c->B0 != 0) return LQLORA_ERR_INVALID_SHAPE;
    if (N > (int64_t(1) << 30) || K > (int64_t(1) << 30)) return LQLORA_ERR_INVALID_SHAPE;
    return LQLORA_OK;
}

// The kernels read one scale code per byte and fp32 second-level scales; any other storage form (b1 < 8, 16-bit v) is
// expanded into scratch first.
inline bool packed_scales(const lqlora_config* c) { return c->b1 != 8 || c->b2 != kB2Fp32; }

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Device-side view of a quantized matrix.  sc / v are the arrays the kernels read: one code per byte and fp32 (the
// matrix's own arrays for b1 = 8, b2 = fp32; expanded copies otherwise, see expand_scales).
struct QView {
    const uint32_t* codes;
    const uint8_t* sc;     // s^ [N * KB]
    const float* v;        // v  [ngrp]
    float levels;          // 2^(b1-1) - 1
    int b1, b2;            // storage form of sc / v as this view holds them (8 / fp32 once expanded)
    int N, K;
    int b0, B0, B1;
    int logB0, logB1;
    int KB;                // blocks per row  = K / B0
    int ktiles;            // 64-column tiles per row = K / 64
    int ntiles;            // 128-row tiles = ceil(N / 128)
};

inline QView make_view(const lqlora_qmatrix* q) {
    QView v;
    v.codes = static_cast<const uint32_t*>(q->codes);
    v.sc = q->scale_codes;
    v.v = q->scale2;
    v.N = static_cast<int>(q->N);
    v.K = static_cast<int>(q->K);
    v.b0 = q->cfg.b0; v.B0 = q->cfg.B0; v.B1 = q->cfg.B1;
    v.levels = static_cast<float>(scale_levels(q->cfg.b1));
    v.b1 = q->cfg.b1; v.b2 = q->cfg.b2;
    v.logB0 = ilog2(v.B0); v.logB1 = ilog2(v.B1);
    v.KB = v.K / v.B0;
    v.ktiles = v.K / kTileCols;
    v.ntiles = (v.N + kTileRows - 1) / kTileRows;
    return v;
}

// First 32-bit word of the slab holding (row, 64-column tile kt): tiles in row-major tile order,
// four slabs of 32 rows per tile, 64*b0 words per slab.
__host__ __device__ inline size_t slab_word_base(int row, int kt, int ktiles, int b0) {
    const size_t tile = static_cast<size_t>(row >> 7) * ktiles + kt;
    return (tile * 4 + ((row >> 5) & 3)) * static_cast<size_t>(64 * b0);
}
// Word w of the 32-code group g of `row` inside the slab of 64-column tile kt.  The 32 rows of a word
// plane are rotated by 8 g + 16 (kt % 2) positions, so that threads that read the same four rows from
// the two groups of two neighbouring tiles (the access pattern of the decode kernels) hit different
// shared-memory banks; a rotation by a multiple of four keeps aligned groups of four rows together.
__host__ __device__ inline int slab_row_slot(int row, int g, int kt) { return (row + 8 * g + 16 * (kt & 1)) & 31; }
__host__ __device__ inline int slab_word_offset(int row, int g, int w, int b0, int kt) {
    return (g * b0 + w) * 32 + slab_row_slot(row, g, kt);
}

// Bit layout of the 32 codes c[0..31] of one (row, 32-column group) inside its b0 words.  Every
// word is a string of eight 4-bit fields ("selectors") so that a byte-permute instruction can use
// it directly as a table index for eight weights:
//   b0 = 4: word w holds codes 8w .. 8w+7, code 8w+i in field i (bits [4i, 4i+4));
//   b0 = 3: word w (0..2) holds code 8w+i in the low three bits of field i; the top bit of field i
//           of word w is bit w of code 24+i;
//   b0 = 2: word w (0..1) holds code 16w+i in the low two bits of field i and code 16w+8+i in its
//           high two bits;
//   b0 = 8: word w holds codes 4w .. 4w+3, one per byte.
template <int B>
__host__ __device__ __forceinline__ void deposit_code(uint32_t* w, int j, uint32_t c) {
    if constexpr (B == 4) w[j >> 3] |= c << (4 * (j & 7));
    else if constexpr (B == 8) w[j >> 2] |= c << (8 * (j & 3));
    else if constexpr (B == 2) w[j >> 4] |= c << (4 * (j & 7) + 2 * ((j >> 3) & 1));
    else {
        if (j < 24) w[j >> 3] |= c << (4 * (j & 7));
        else {
            const int i = j - 24;
            w[0] |= (c & 1u) << (4 * i + 3);
            w[1] |= ((c >> 1) & 1u) << (4 * i + 3);
            w[2] |= ((c >> 2) & 1u) << (4 * i + 3);
        }
    }
}
// Code j (0..31) of a group whose b0 words are in `w`.
template <int B>
__host__ __device__ __forceinline__ uint32_t extract_code(const uint32_t* w, int j) {
    if constexpr (B == 4) return (w[j >> 3] >> (4 * (j & 7))) & 15u;
    else if constexpr (B == 8) return (w[j >> 2] >> (8 * (j & 3))) & 255u;
    else if constexpr (B == 2) return (w[j >> 4] >> (4 * (j & 7) + 2 * ((j >> 3) & 1))) & 3u;
    else {
        if (j < 24) return (w[j >> 3] >> (4 * (j & 7))) & 7u;
        const int sh = 4 * (j - 24) + 3;
        return ((w[0] >> sh) & 1u) | (((w[1] >> sh) & 1u) << 1) | (((w[2] >> sh) & 1u) << 2);
    }
}

// s~ = fl32(float(s^) * fl32(v / levels)),  levels = 2^(b1-1) - 1 (127 for 8-bit scale codes)
__device__ __forceinline__ float block_scale(uint8_t sc, float v, float levels) {
    return __fmul_rn(static_cast<float>(sc), __fdiv_rn(v, levels));
}

__device__ __forceinline__ float bf16_bits_to_float(uint16_t b) { return __uint_as_float(static_cast<uint32_t>(b) << 16); }

// Tables (index 0..3 for b0 = 2, 3, 4, 8): code book and the round-down fp32 midpoints between
// neighbouring code-book entries (x > midpoint  <=>  x > threshold for fp32 x).
__constant__ float c_codebook[4][256];
__constant__ float c_threshold[4][256];
// 2- and 3-bit encoder: fl(0.5 - threshold * kSatScale) per threshold; saturate(x * kSatScale + bias) is 0 below the
// threshold, 1 above it and in between only within 0.5 / kSatScale = 9.5e-7 of it.
constexpr float kSatScale = 524288.0f;
__constant__ float c_satbias[2][8];

// Bin table for the nearest-code search of the encoder: [-1, 1] is cut into `nb` equal bins chosen so that every
// bin holds at most one threshold and no threshold lies near a bin edge.  Entry k = (threshold in the bin or +inf,
// number of thresholds below the bin); entry nb serves x slightly above 1.
constexpr int kMaxBins = 1280;
struct BinEntry { float thr; int base; };
__device__ BinEntry g_bins[4][kMaxBins + 1];
__constant__ int c_nbins[4];

int ensure_tables();                 // uploads the tables to the current device once; LQLORA_OK or error
const float* host_codebook(int b0);  // 2^b0 floats
void count_launch(int n = 1);

}  // namespace lq
