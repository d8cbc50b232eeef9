// Quantize(A, c) of Sec. 3.2 on the GPU: block absmax, nearest NormalFloat code, bit packing,
// 8-bit round-to-nearest quantization of the absmax values; plus the unpack / dequantize
// exports used for parity checks.
#pragma once

#include <cuda_fp16.h>

#include "common.cuh"

namespace lq {

// ---------------------------------------------------------------------------------------
// Nearest code by counting thresholds below x (thresholds ascending; a tie x == midpoint is
// not "above", so it goes to the lower index).
// ---------------------------------------------------------------------------------------
template <int B>
__device__ __forceinline__ uint32_t nearest_code(float x, const float* __restrict__ th_smem) {
    if constexpr (B <= 4) {
        uint32_t c = 0;
#pragma unroll
        for (int i = 0; i < (1 << B) - 1; ++i) c += (x > c_threshold[B == 2 ? 0 : B == 3 ? 1 : 2][i]) ? 1u : 0u;
        return c;
    } else {
        uint32_t c = 0;
#pragma unroll
        for (int step = 128; step >= 1; step >>= 1)
            if (x > th_smem[c + step - 1]) c += step;   // th_smem[255] = +inf, never exceeded
        return c;
    }
}

// Fast search for 2- and 3-bit codes without compares or selects (the compare / select pipe is the encoder's
// bottleneck; this runs on the fused-multiply-add pipe).  For x^ and threshold T_k, f_k = saturate(x^ * S + b_k) with
// S = kSatScale, b_k = fl(0.5 - T_k S) is exactly 0 when x^ < T_k - 0.5/S, exactly 1 when x^ > T_k + 0.5/S, so the code
// is f_1 + ... + f_n whenever x^ is not that close to a threshold.  The sum starts from a power of two chosen so that
// the code lands in the mantissa bits that are the code's field of the packed word, seven bits above the bottom of the
// word's 16-bit half: all bits below the field are zero unless some f_k was fractional (to 2^-8), i.e. unless x^ lies
// within (0.5 - 2^-8 - 2^-5) / S = 8.9e-7 of a threshold (2^-5 bounds the rounding of b_k) -- more than the 2.4e-7 that x^ can
// differ from the quotient.  Those bits are collected in `danger`; the caller then decides every code of the thread
// exactly.  field_bits: position p (0, 2, .. 14) of the field in its half-word.
template <int B>
__device__ __forceinline__ uint32_t sat_count(float xh, float start) {
    float acc = start;
#pragma unroll
    for (int k = 0; k < (1 << B) - 1; ++k) {
        float f;
        asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(f) : "f"(xh), "f"(kSatScale), "f"(c_satbias[B - 2][k]));
        acc += f;
    }
    return __float_as_uint(acc);
}
// The B words of 32 codes from u * (r_lo | r_hi), layout of deposit_code<B>.
template <int B>
__device__ __forceinline__ void sat_encode(const float (&u)[32], float r_lo, float r_hi, uint32_t (&words)[B], uint32_t& danger) {
    static_assert(B == 2 || B == 3, "2- and 3-bit codes");
    constexpr uint32_t cmask = (1u << B) - 1u;
    if constexpr (B == 3) {
        uint32_t V = 0;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            uint32_t H[2] = {0u, 0u};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int jj = 0; jj < 4; ++jj) {
                    const int j = 8 * w + 4 * h + jj, p = 4 * jj;
                    const uint32_t bits = sat_count<3>(u[j] * ((j < 16) ? r_lo : r_hi), static_cast<float>(1u << (16 - p)));
                    H[h] |= bits & (cmask << (7 + p));
                    danger |= bits & ((1u << (7 + p)) - 1u);
                }
            }
            const uint32_t word = (H[0] >> 7) | (H[1] << 9);
            if (w < 3) words[w] = word;
            else V = word;                 // codes 24..31 as 4-bit fields: their bits go to the spare fourth bits
        }
        words[0] |= (V & 0x11111111u) << 3;
        words[1] |= ((V >> 1) & 0x11111111u) << 3;
        words[2] |= ((V >> 2) & 0x11111111u) << 3;
    } else {
#pragma unroll
        for (int w = 0; w < 2; ++w) {
            uint32_t H[2] = {0u, 0u};
#pragma unroll
            for (int h = 0; h < 2; ++h) {
#pragma unroll
                for (int t2 = 0; t2 < 8; ++t2) {
                    const int j = 16 * w + (t2 >> 2) * 8 + 4 * h + (t2 & 3), p = 4 * (t2 & 3) + 2 * (t2 >> 2);
                    const uint32_t bits = sat_count<2>(u[j] * ((j < 16) ? r_lo : r_hi), static_cast<float>(1u << (16 - p)));
                    H[h] |= bits & (cmask << (7 + p));
                    danger |= bits & ((1u << (7 + p)) - 1u);
                }
            }
            words[w] = (H[0] >> 7) | (H[1] << 9);
        }
    }
}

// Reciprocal used by the fast searches: 0 for an all-zero block (x^ = 0 gives the zero code), NaN for block maxima
// whose reciprocal is not a normal number (every element then takes the exact route).
__device__ __forceinline__ float search_reciprocal(float s) {
    if (s == 0.0f) return 0.0f;
    if (!(s > 1e-30f && s < 1e30f)) return __int_as_float(0x7fc00000);
    return __fdiv_rn(1.0f, s);
}

// One CTA: 32 rows x 256 columns.  Thread (row = tid % 32, grp = tid / 32) owns 32 consecutive
// columns of one row: it finds the block absmax (with its neighbours through shared memory when
// B0 > 32), the 32 codes, and writes the b0 words of its group to the packed slab.
template <int B>
__global__ void __launch_bounds__(256) encode_codes_kernel(const float* __restrict__ W, uint32_t* __restrict__ codes,
                                                           float* __restrict__ absmax, int N, int K, int B0, int logB0) {
    __shared__ float red[8][33];
    __shared__ __align__(16) float4 tile[8][32 * 8];   // per warp: 32 rows x 32 columns
    __shared__ float th8[256];
    __shared__ float2 bins[kMaxBins + 1];        // (threshold of the bin or +inf, number of thresholds below the bin)
    if constexpr (B == 8) {
        th8[threadIdx.x] = c_threshold[3][threadIdx.x];
    }
    // 4- and 8-bit codes (15 / 255 thresholds) find their code through a bin table; 2- and 3-bit codes by a binary
    // search among constants
    constexpr bool kUseBins = (B >= 4);
    const int nb = kUseBins ? c_nbins[bits_index(B)] : 0;
    if constexpr (kUseBins) {
        for (int i = threadIdx.x; i <= nb; i += 256) {
            const BinEntry e = g_bins[bits_index(B)][i];       // global memory: coalesced (the constant bank would serialize the lanes)
            bins[i] = make_float2(e.thr, __int_as_float(e.base));
        }
    }
    const float bin_scale = 0.5f * static_cast<float>(nb);
    const int rl = threadIdx.x & 31, grp = threadIdx.x >> 5;
    const int row = blockIdx.x * 32 + rl;
    const int k0 = blockIdx.y * 256 + grp * 32;
    const bool live = (k0 < K);
    const bool real = live && (row < N);

    // A warp owns 32 rows x 32 columns.  It loads them coalesced (a load instruction covers four rows of 128 bytes),
    // passes them through its own shared-memory tile (16-byte chunks swizzled by row, conflict-free both ways) and
    // each lane reads back the 32 columns of one row.
    float u[32];
    {
        float4* mine = tile[grp];
        const int lr = rl >> 3, ch = rl & 7;
        float4 t[8];
        if (live && blockIdx.x * 32 + 32 <= N) {
            // all 32 rows exist: one pointer, constant strides
            const float4* src = reinterpret_cast<const float4*>(W + static_cast<size_t>(blockIdx.x * 32 + lr) * K + k0) + ch;
            const size_t stride = static_cast<size_t>(K);            // four rows, in float4
#pragma unroll
            for (int i = 0; i < 8; ++i) t[i] = __ldg(src + i * stride);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int rr = blockIdx.x * 32 + 4 * i + lr;
                t[i] = (live && rr < N) ? __ldg(reinterpret_cast<const float4*>(W + static_cast<size_t>(rr) * K + k0) + ch)
                                        : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            }
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = 4 * i + lr;
            mine[r * 8 + (ch ^ (r & 7))] = t[i];
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 v = mine[rl * 8 + (i ^ (rl & 7))];
            u[4 * i] = v.x; u[4 * i + 1] = v.y; u[4 * i + 2] = v.z; u[4 * i + 3] = v.w;
        }
    }
    // absmax of each 16-wide half
    float m0 = 0.0f, m1 = 0.0f;
#pragma unroll
    for (int i = 0; i < 16; ++i) { m0 = fmaxf(m0, fabsf(u[i])); m1 = fmaxf(m1, fabsf(u[16 + i])); }
    if constexpr (B >= 4) __syncthreads();       // the search tables in shared memory are complete
    float s_lo, s_hi;   // block absmax for columns 0..15 and 16..31 of this thread's group
    if (B0 == 16) { s_lo = m0; s_hi = m1; }
    else if (B0 == 32) { s_lo = s_hi = fmaxf(m0, m1); }
    else {
        // blocks wider than a thread's 32 columns: the maxima of the neighbouring groups come through shared memory
        red[grp][rl] = fmaxf(m0, m1);
        __syncthreads();
        const int span = B0 >> 5, g0 = grp & ~(span - 1);
        float m = 0.0f;
        for (int i = 0; i < span; ++i) m = fmaxf(m, red[g0 + i][rl]);
        s_lo = s_hi = m;
    }
    if (real) {
        const int KB = K >> logB0;
        if (B0 == 16) {
            *reinterpret_cast<float2*>(absmax + static_cast<size_t>(row) * KB + (k0 >> 4)) = make_float2(s_lo, s_hi);   // KB, k0 / 16 even
        } else if ((k0 & (B0 - 1)) == 0) {
            absmax[static_cast<size_t>(row) * KB + (k0 >> logB0)] = s_lo;
        }
    }
    if (!live) return;

    constexpr uint32_t zero_code = (1u << (B - 1)) - 1u;
    uint32_t words[B];
#pragma unroll
    for (int i = 0; i < B; ++i) words[i] = 0u;
    // Fast search: x^ = u * fl(1/s) is within 2 ulp (2.4e-7) of the quotient fl(u/s) that defines the code.  The code
    // is found from x^ (bin table: the bin of x^ holds at most one threshold, code = thresholds below the bin plus
    // (x^ > threshold); 2/3-bit codes: binary search).  When x^ comes within 1e-6 of a threshold it was compared with
    // (or is not a number in [-1, 1]) the decision is taken exactly, with the IEEE quotient and the full search.  No
    // threshold lies that close to a bin edge (the bin count is chosen on the host for the largest clearance), so
    // the two routes agree.
    const float r_lo = search_reciprocal(s_lo);
    const float r_hi = search_reciprocal(s_hi);
    if constexpr (B <= 3) {
        // codes by saturating arithmetic; exact route for the whole thread when some x^ came close to a threshold or a
        // reciprocal is not a normal number
        uint32_t danger = (r_lo == r_lo && r_hi == r_hi) ? 0u : 1u;
        if (danger == 0u) sat_encode<B>(u, r_lo, r_hi, words, danger);
        if (danger != 0u) {
#pragma unroll
            for (int i = 0; i < B; ++i) words[i] = 0u;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float s = (j < 16) ? s_lo : s_hi;
                uint32_t c = zero_code;
                if (s != 0.0f) c = nearest_code<B>(__fdiv_rn(u[j], s), th8);
                deposit_code<B>(words, j, c);
            }
        }
    } else {
        // Bin table: the bin of x^ holds at most one threshold, code = thresholds below the bin plus (x^ > threshold).
        // First all 32 codes without a branch (32 independent chains for the scheduler), keeping the smallest distance
        // between an x^ and the threshold it was compared with; only a thread where that distance is within 1e-6 (or a
        // reciprocal is not a normal number) goes through its elements again and decides the close ones exactly.
        float margin = (r_lo == r_lo && r_hi == r_hi) ? 1.0f : 0.0f;
        if (margin != 0.0f) {
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float xh = u[j] * ((j < 16) ? r_lo : r_hi);
                const uint32_t k = min(__float2uint_rd(fmaf(xh, bin_scale, bin_scale)), static_cast<uint32_t>(nb));
                const float2 e = bins[k];
                deposit_code<B>(words, j, static_cast<uint32_t>(__float_as_int(e.y)) + ((xh > e.x) ? 1u : 0u));
                margin = fminf(margin, fabsf(xh - e.x));
            }
        }
        if (!(margin > 1e-6f)) {
#pragma unroll
            for (int i = 0; i < B; ++i) words[i] = 0u;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float s = (j < 16) ? s_lo : s_hi, r = (j < 16) ? r_lo : r_hi;
                const float xh = u[j] * r;
                const uint32_t k = min(__float2uint_rd(fmaf(xh, bin_scale, bin_scale)), static_cast<uint32_t>(nb));
                const float2 e = bins[k];
                uint32_t c = static_cast<uint32_t>(__float_as_int(e.y)) + ((xh > e.x) ? 1u : 0u);
                if (!(fabsf(xh - e.x) > 1e-6f) || !(r == r)) {
                    c = zero_code;
                    if (s != 0.0f) c = nearest_code<B>(__fdiv_rn(u[j], s), th8);
                }
                deposit_code<B>(words, j, c);
            }
        }
    }
    uint32_t* dst = codes + slab_word_base(row, k0 >> 6, K >> 6, B);
    const int g = (k0 >> 5) & 1;
#pragma unroll
    for (int w = 0; w < B; ++w) dst[slab_word_offset(row, g, w, B, k0 >> 6)] = words[w];
}

// One warp per second-level group (eight groups per CTA): v_g = max s_i, s^_i = clamp(rint(s_i / (v_g / levels)), 0, levels).
// The quotient is found without a division where that is safe: t = fl(s_i * fl(1 / sigma) + 3072) holds the quotient in
// fixed point with 12 fraction bits (s_i <= v_g, so it is at most levels <= 127 and t stays in [2048, 4096)); its error
// against fl(s_i / sigma) is below 2^-13 + 1.2e-5, so rounding the fixed-point value half up gives rint of the IEEE
// quotient unless the fraction lies within 2^-12 of one half; those elements (0.07 %) take the IEEE division.
__device__ __forceinline__ uint32_t scale_code_exact(float a, float sigma, float levels) {
    return static_cast<uint32_t>(fminf(fmaxf(rintf(__fdiv_rn(a, sigma)), 0.0f), levels));
}
__device__ __forceinline__ uint32_t scale_code(float a, float sigma, float rsigma, float levels, bool fast) {
    if (fast) {
        const uint32_t bits = __float_as_uint(fmaf(a, rsigma, 3072.0f));
        if ((bits & 0xFFFu) - 0x7FFu > 2u) return ((bits + 0x800u) >> 12) & 0xFFu;
    }
    return scale_code_exact(a, sigma, levels);
}
// Groups of up to 256 blocks: a warp owns a span of 256 consecutive blocks (whole groups: spans and groups are aligned),
// four pairs of blocks per lane, all loaded before anything else happens (the kernel is bound by memory latency: the
// maxima, the quotients and the stores come from registers).  A group is a run of lanes of one load (B1 <= 64), two loads
// (128) or all four (256).
__global__ void __launch_bounds__(256) encode_scales_span_kernel(const float* __restrict__ absmax, uint8_t* __restrict__ sc,
                                                                 float* __restrict__ v, long long nblk, long long ngrp, int B1, int logB1,
                                                                 float levels) {
    const long long base = (static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5)) * 256;
    if (base >= nblk) return;
    const int lane = threadIdx.x & 31;
    float2 a[4];
    float m[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const long long blk = base + 2 * (e * 32 + lane);
        a[e] = make_float2(0.0f, 0.0f);
        if (blk + 1 < nblk) a[e] = *reinterpret_cast<const float2*>(absmax + blk);
        else if (blk < nblk) a[e].x = absmax[blk];
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) m[e] = fmaxf(a[e].x, a[e].y);
    const int seg = (B1 >= 64) ? 32 : (B1 >> 1);           // lanes of one load that share a group
    for (int o = seg >> 1; o > 0; o >>= 1) {
#pragma unroll
        for (int e = 0; e < 4; ++e) m[e] = fmaxf(m[e], __shfl_xor_sync(0xffffffffu, m[e], o));
    }
    if (B1 >= 128) {
        m[0] = m[1] = fmaxf(m[0], m[1]);
        m[2] = m[3] = fmaxf(m[2], m[3]);
    }
    if (B1 == 256) m[0] = m[1] = m[2] = m[3] = fmaxf(m[0], m[2]);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const long long blk = base + 2 * (e * 32 + lane);
        const float vg = m[e];
        if ((blk & (B1 - 1)) == 0 && blk < nblk) v[blk >> logB1] = vg;
        uint32_t c0 = 0u, c1 = 0u;
        if (vg != 0.0f) {
            const float sigma = __fdiv_rn(vg, levels);
            const bool fast = sigma > 1e-30f && sigma < 1e30f;
            const float rsigma = fast ? __fdiv_rn(1.0f, sigma) : 0.0f;
            c0 = scale_code(a[e].x, sigma, rsigma, levels, fast);
            c1 = scale_code(a[e].y, sigma, rsigma, levels, fast);
        }
        if (blk + 1 < nblk) *reinterpret_cast<uint16_t*>(sc + blk) = static_cast<uint16_t>(c0 | (c1 << 8));
        else if (blk < nblk) sc[blk] = static_cast<uint8_t>(c0);
    }
    (void)ngrp;
}

// Larger groups: one warp per group.
__global__ void __launch_bounds__(256) encode_scales_kernel(const float* __restrict__ absmax, uint8_t* __restrict__ sc,
                                                            float* __restrict__ v, long long nblk, long long ngrp, int B1, float levels) {
    const long long g = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
    if (g >= ngrp) return;
    const int lane = threadIdx.x & 31;
    const long long lo = g * B1;                          // a multiple of 16: pairs of blocks are 8-byte aligned
    const int n = static_cast<int>((lo + B1 < nblk) ? B1 : nblk - lo);
    const float2* __restrict__ a2 = reinterpret_cast<const float2*>(absmax + lo);
    float m = 0.0f;
    for (int i = lane; 2 * i + 1 < n; i += 32) {
        const float2 a = a2[i];
        m = fmaxf(m, fmaxf(a.x, a.y));
    }
    if ((n & 1) && lane == 0) m = fmaxf(m, absmax[lo + n - 1]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const float vg = m;
    if (lane == 0) v[g] = vg;
    uint16_t* __restrict__ sc2 = reinterpret_cast<uint16_t*>(sc + lo);
    if (vg == 0.0f) {
        for (int i = lane; 2 * i + 1 < n; i += 32) sc2[i] = 0;
        if ((n & 1) && lane == 0) sc[lo + n - 1] = 0;
        return;
    }
    const float sigma = __fdiv_rn(vg, levels);
    const bool fast = sigma > 1e-30f && sigma < 1e30f;
    const float rsigma = fast ? __fdiv_rn(1.0f, sigma) : 0.0f;
    for (int i = lane; 2 * i + 1 < n; i += 32) {
        const float2 a = a2[i];
        const uint32_t c0 = scale_code(a.x, sigma, rsigma, levels, fast), c1 = scale_code(a.y, sigma, rsigma, levels, fast);
        sc2[i] = static_cast<uint16_t>(c0 | (c1 << 8));
    }
    if ((n & 1) && lane == 0) sc[lo + n - 1] = static_cast<uint8_t>(scale_code_exact(absmax[lo + n - 1], sigma, levels));
}

// Storage forms of the scales (Table 1 of Sec. 3.2).  b1 < 8: the codes form a bit stream of b1 bits each, code i in
// bits [i b1, (i + 1) b1) of the little-endian byte stream (eight codes = b1 bytes); cast(v, b2): fp16 or bf16 numbers
// (round to nearest even).  One thread packs / expands eight codes; the second-level scales go one per thread.
__global__ void pack_scales_kernel(const uint8_t* __restrict__ sc8, const float* __restrict__ v32, uint8_t* __restrict__ sc_out,
                                   void* __restrict__ v_out, long long nblk, long long ngrp, int b1, int b2) {
    const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t * 8 < nblk) {
        if (b1 == 8) {
            for (int i = 0; i < 8 && t * 8 + i < nblk; ++i) sc_out[t * 8 + i] = sc8[t * 8 + i];
        } else {
            unsigned long long word = 0ull;
            for (int i = 0; i < 8; ++i)
                if (t * 8 + i < nblk) word |= static_cast<unsigned long long>(sc8[t * 8 + i]) << (i * b1);
            for (int j = 0; j < b1; ++j) sc_out[t * b1 + j] = static_cast<uint8_t>(word >> (8 * j));
        }
    }
    if (t < ngrp) {
        if (b2 == kB2Fp32) static_cast<float*>(v_out)[t] = v32[t];
        else if (b2 == kB2Fp16) static_cast<__half*>(v_out)[t] = __float2half_rn(v32[t]);
        else static_cast<__nv_bfloat16*>(v_out)[t] = __float2bfloat16_rn(v32[t]);
    }
}
__global__ void expand_scales_kernel(const uint8_t* __restrict__ sc_in, const void* __restrict__ v_in, uint8_t* __restrict__ sc8,
                                     float* __restrict__ v32, long long nblk, long long ngrp, int b1, int b2) {
    const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (t * 8 < nblk) {
        if (b1 == 8) {
            for (int i = 0; i < 8 && t * 8 + i < nblk; ++i) sc8[t * 8 + i] = sc_in[t * 8 + i];
        } else {
            unsigned long long word = 0ull;
            for (int j = 0; j < b1; ++j) word |= static_cast<unsigned long long>(sc_in[t * b1 + j]) << (8 * j);
            for (int i = 0; i < 8; ++i)
                if (t * 8 + i < nblk) sc8[t * 8 + i] = static_cast<uint8_t>((word >> (i * b1)) & ((1u << b1) - 1u));
        }
    }
    if (t < ngrp) {
        if (b2 == kB2Fp32) v32[t] = static_cast<const float*>(v_in)[t];
        else if (b2 == kB2Fp16) v32[t] = __half2float(static_cast<const __half*>(v_in)[t]);
        else v32[t] = __bfloat162float(static_cast<const __nv_bfloat16*>(v_in)[t]);
    }
}

// Bytes of scratch an expanded copy of the scales takes, and the expansion itself: returns the view the kernels read.
inline size_t expanded_scale_bytes(int64_t N, int64_t K, const lqlora_config* c) {
    if (!packed_scales(c)) return 0;
    const int64_t nblk = N * K / c->B0, ngrp = (nblk + c->B1 - 1) / c->B1;
    return (static_cast<size_t>(nblk) + 255) / 256 * 256 + (static_cast<size_t>(ngrp) * 4 + 255) / 256 * 256;
}
inline cudaError_t expand_scales(const lqlora_qmatrix* q, QView* view, char* scratch, cudaStream_t st) {
    *view = make_view(q);
    if (!packed_scales(&q->cfg)) return cudaSuccess;
    const long long nblk = static_cast<long long>(q->N) * q->K / q->cfg.B0, ngrp = (nblk + q->cfg.B1 - 1) / q->cfg.B1;
    uint8_t* sc8 = reinterpret_cast<uint8_t*>(scratch);
    float* v32 = reinterpret_cast<float*>(scratch + (static_cast<size_t>(nblk) + 255) / 256 * 256);
    const long long threads = (nblk + 7) / 8 > ngrp ? (nblk + 7) / 8 : ngrp;
    expand_scales_kernel<<<static_cast<unsigned>((threads + 255) / 256), 256, 0, st>>>(q->scale_codes, q->scale2, sc8, v32, nblk, ngrp,
                                                                                   q->cfg.b1, q->cfg.b2);
    count_launch(1);
    view->sc = sc8;
    view->v = v32;
    view->b1 = 8;
    view->b2 = kB2Fp32;
    return cudaGetLastError();
}

// Scale code of block `blk` and second-level scale of group `g` in whatever form the view holds them.
__device__ __forceinline__ uint32_t load_scale_code(const QView& q, long long blk) {
    if (q.b1 == 8) return q.sc[blk];
    const long long bit = blk * q.b1;
    const long long byte = bit >> 3;
    const int sh = static_cast<int>(bit & 7);
    uint32_t w = q.sc[byte];
    if (sh + q.b1 > 8) w |= static_cast<uint32_t>(q.sc[byte + 1]) << 8;
    return (w >> sh) & ((1u << q.b1) - 1u);
}
__device__ __forceinline__ float load_scale2(const QView& q, long long g) {
    if (q.b2 == kB2Fp32) return q.v[g];
    if (q.b2 == kB2Fp16) return __half2float(reinterpret_cast<const __half*>(q.v)[g]);
    return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(q.v)[g]);
}

// Thread per (row, 32-column group): unpack to one code per byte and / or dequantize (any storage form of the scales).
template <int B>
__global__ void __launch_bounds__(256) export_kernel(QView q, uint8_t* __restrict__ codes_out, float* __restrict__ deq32,
                                                     __nv_bfloat16* __restrict__ deq16) {
    const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    const int groups_per_row = q.K >> 5;
    // consecutive threads -> consecutive rows of one slab (coalesced packed reads)
    const int rl = static_cast<int>(t & 31);
    const long long rest = t >> 5;
    const int grp = static_cast<int>(rest % groups_per_row);
    const int row = static_cast<int>(rest / groups_per_row) * 32 + rl;
    if (row >= q.N) return;
    const int k0 = grp * 32;
    const uint32_t* src = q.codes + slab_word_base(row, k0 >> 6, q.ktiles, B);
    uint32_t w[B];
#pragma unroll
    for (int i = 0; i < B; ++i) w[i] = src[slab_word_offset(row, (k0 >> 5) & 1, i, B, k0 >> 6)];
    const size_t out = static_cast<size_t>(row) * q.K + k0;
    const float* cb = c_codebook[bits_index(B)];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        const uint32_t c = extract_code<B>(w, j);
        if (codes_out) codes_out[out + j] = static_cast<uint8_t>(c);
        if (deq32 || deq16) {
            const long long blk = static_cast<long long>(row) * q.KB + ((k0 + j) >> q.logB0);
            const float st = block_scale(static_cast<uint8_t>(load_scale_code(q, blk)), load_scale2(q, blk >> q.logB1), q.levels);
            const float wv = __fmul_rn(cb[c], st);
            if (deq32) deq32[out + j] = wv;
            if (deq16) deq16[out + j] = __float2bfloat16_rn(wv);
        }
    }
}

inline void launch_encode_scales(const float* absmax, uint8_t* sc, float* v, long long nblk, long long ngrp, int B1, float levels, cudaStream_t st) {
    if (B1 <= 256) {
        const long long spans = (nblk + 255) / 256;
        encode_scales_span_kernel<<<static_cast<unsigned>((spans + 7) / 8), 256, 0, st>>>(absmax, sc, v, nblk, ngrp, B1, ilog2(B1), levels);
    } else {
        encode_scales_kernel<<<static_cast<unsigned>((ngrp + 7) / 8), 256, 0, st>>>(absmax, sc, v, nblk, ngrp, B1, levels);
    }
}

template <int B>
inline cudaError_t launch_encode(const float* W, const lqlora_qmatrix* out, float* absmax, cudaStream_t st) {
    const int N = static_cast<int>(out->N), K = static_cast<int>(out->K);
    const int Np = (N + kTileRows - 1) / kTileRows * kTileRows;
    dim3 grid(Np / 32, (K + 255) / 256);
    encode_codes_kernel<B><<<grid, 256, 0, st>>>(W, static_cast<uint32_t*>(out->codes), absmax, N, K, out->cfg.B0,
                                                 ilog2(out->cfg.B0));
    const long long nblk = static_cast<long long>(N) * K / out->cfg.B0;
    const long long ngrp = (nblk + out->cfg.B1 - 1) / out->cfg.B1;
    const float levels = static_cast<float>(scale_levels(out->cfg.b1));
    if (!packed_scales(&out->cfg)) {
        launch_encode_scales(absmax, out->scale_codes, out->scale2, nblk, ngrp, out->cfg.B1, levels, st);
        count_launch(2);
        return cudaGetLastError();
    }
    // other storage forms: byte codes and fp32 scales into the scratch behind the absmax values, then packed / cast
    char* tail = reinterpret_cast<char*>(absmax) + (static_cast<size_t>(nblk) * sizeof(float) + 255) / 256 * 256;
    uint8_t* sc8 = reinterpret_cast<uint8_t*>(tail);
    float* v32 = reinterpret_cast<float*>(tail + (static_cast<size_t>(nblk) + 255) / 256 * 256);
    launch_encode_scales(absmax, sc8, v32, nblk, ngrp, out->cfg.B1, levels, st);
    const long long threads = (nblk + 7) / 8 > ngrp ? (nblk + 7) / 8 : ngrp;
    pack_scales_kernel<<<static_cast<unsigned>((threads + 255) / 256), 256, 0, st>>>(sc8, v32, out->scale_codes, out->scale2, nblk, ngrp,
                                                                                 out->cfg.b1, out->cfg.b2);
    count_launch(3);
    return cudaGetLastError();
}

template <int B>
inline cudaError_t launch_export(const QView& q, uint8_t* codes_out, float* deq32, void* deq16, cudaStream_t st) {
    const long long total = static_cast<long long>((q.N + 31) / 32 * 32) * (q.K >> 5);
    export_kernel<B><<<static_cast<unsigned>((total + 255) / 256), 256, 0, st>>>(q, codes_out, deq32,
                                                                               static_cast<__nv_bfloat16*>(deq16));
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace lq
