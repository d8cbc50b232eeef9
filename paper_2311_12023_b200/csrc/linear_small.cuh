// Weight-streaming kernels for few rows of X (decode-like M): every packed word is read once
// with 128-bit coalesced loads, dequantized in registers and multiplied with the activations;
// the contraction is split across warps / CTAs and reduced through fp32 partial sums.
#pragma once

#include "common.cuh"
#include "linear_decode.cuh"

namespace lq {

// T[m][j] = bf16( sum_c A[m][c] * F(j, c) ),  F(j, c) = F[j * fj + c * fc]
// forward:  A = X [M, K],  F = L2 [r, K] (fj = K, fc = 1)        -> T = X L2^T
// backward: A = dY [M, N], F = L1 [N, r] (fj = 1, fc = r)        -> T = dY L1
// One CTA per row m; warp w handles j = w, w + 8, ...; lanes stride over c.
__global__ void __launch_bounds__(256) lowrank_pre_kernel(const __nv_bfloat16* __restrict__ A, const __nv_bfloat16* __restrict__ F,
                                                          __nv_bfloat16* __restrict__ T, int C, int r, long long fj, long long fc) {
    const int m = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const __nv_bfloat16* a = A + static_cast<size_t>(m) * C;
    for (int j = warp; j < r; j += 8) {
        float acc = 0.0f;
        for (int c = lane; c < C; c += 32)
            acc = fmaf(__bfloat162float(a[c]), __bfloat162float(F[j * fj + c * fc]), acc);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (lane == 0) T[static_cast<size_t>(m) * r + j] = __float2bfloat16_rn(acc);
    }
}

// out[m][c] = bf16( sum_s P[s][m][c] + sum_j T[m][j] * F(c, j) ),  F(c, j) = F[c * fc + j * fj]
__global__ void __launch_bounds__(256) finalize_kernel(const float* __restrict__ P, int splits, const __nv_bfloat16* __restrict__ T,
                                                       const __nv_bfloat16* __restrict__ F, __nv_bfloat16* __restrict__ out,
                                                       int M, int C, int r, long long fc, long long fj) {
    const long long idx = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
    if (idx >= static_cast<long long>(M) * C) return;
    const int m = static_cast<int>(idx / C), c = static_cast<int>(idx % C);
    float acc = 0.0f;
    for (int s = 0; s < splits; ++s) acc += P[(static_cast<size_t>(s) * M + m) * C + c];
    float lr = 0.0f;
    for (int j = 0; j < r; ++j)
        lr = fmaf(__bfloat162float(T[static_cast<size_t>(m) * r + j]), __bfloat162float(F[c * fc + j * fj]), lr);
    out[idx] = __float2bfloat16_rn(acc + lr);
}

// Loads the b0 words of (4 consecutive rows, one 32-column group) as b0 128-bit loads.
template <int B>
__device__ __forceinline__ void load_group4(const uint32_t* __restrict__ slab, int g, int row4, uint4 (&w)[B]) {
#pragma unroll
    for (int i = 0; i < B; ++i)
        w[i] = __ldg(reinterpret_cast<const uint4*>(slab + (g * B + i) * 32 + row4));
}

template <int B>
__device__ __forceinline__ void row_words(const uint4 (&w)[B], int r, uint32_t (&out)[B + 1]) {
#pragma unroll
    for (int i = 0; i < B; ++i) out[i] = (r == 0) ? w[i].x : (r == 1) ? w[i].y : (r == 2) ? w[i].z : w[i].w;
    out[B] = 0u;
}

// Forward: one warp = 32 rows of Q x a slice of K.  Lane (kq = lane % 4, rq = lane / 4) owns rows
// 4rq .. 4rq+3 and columns 32kq .. 32kq+31 of each 128-column window.
template <int B, int MT>
__global__ void __launch_bounds__(128) small_fwd_kernel(QView q, const __nv_bfloat16* __restrict__ X, float* __restrict__ P,
                                                        int M, int windows_per_split) {
    __shared__ float cb[1 << B];
    for (int i = threadIdx.x; i < (1 << B); i += blockDim.x) cb[i] = c_codebook[bits_index(B)][i];
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kq = lane & 3, rq = lane >> 2;
    const int rowgroup = blockIdx.x * 4 + warp;
    if (rowgroup * 32 >= q.N) return;
    const int split = blockIdx.y;
    const int m0 = blockIdx.z * MT;
    const int nwin = q.K >> 7;
    const int w_lo = split * windows_per_split;
    const int w_hi = min(nwin, w_lo + windows_per_split);
    const int row0 = rowgroup * 32 + 4 * rq;

    float acc[4][MT];
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int m = 0; m < MT; ++m) acc[r][m] = 0.0f;

    for (int win = w_lo; win < w_hi; ++win) {
        const int kbase = win * 128 + 32 * kq;
        if (kbase >= q.K) continue;          // K is a multiple of 64: the last window may be half empty
        const uint32_t* slab = q.codes + slab_word_base(rowgroup * 32, kbase >> 6, q.ktiles, B);
        uint4 w[B];
        load_group4<B>(slab, (kbase >> 5) & 1, slab_row_slot(4 * rq, (kbase >> 5) & 1, kbase >> 6), w);
        // activations of this lane's 32 columns
        float x[MT][32];
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            if (m0 + m < M) {
                const uint4* xp = reinterpret_cast<const uint4*>(X + static_cast<size_t>(m0 + m) * q.K + kbase);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 t = __ldg(xp + i);
                    const uint32_t tt[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        x[m][8 * i + 2 * e] = __uint_as_float(tt[e] << 16);
                        x[m][8 * i + 2 * e + 1] = __uint_as_float(tt[e] & 0xffff0000u);
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) x[m][j] = 0.0f;
            }
        }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int row = row0 + r;
            uint32_t rw[B + 1];
            row_words<B>(w, r, rw);
            float s_lo = 0.0f, s_hi = 0.0f;
            if (row < q.N) {
                const long long blk = static_cast<long long>(row) * q.KB + (kbase >> q.logB0);
                s_lo = block_scale(q.sc[blk], q.v[blk >> q.logB1], q.levels);
                s_hi = s_lo;
                if (q.B0 == 16) s_hi = block_scale(q.sc[blk + 1], q.v[(blk + 1) >> q.logB1], q.levels);
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float wv = __fmul_rn(cb[extract_code<B>(rw, j)], j < 16 ? s_lo : s_hi);
                const float w16 = __bfloat162float(__float2bfloat16_rn(wv));
#pragma unroll
                for (int m = 0; m < MT; ++m) acc[r][m] = fmaf(w16, x[m][j], acc[r][m]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            float a = acc[r][m];
            a += __shfl_xor_sync(0xffffffffu, a, 1);
            a += __shfl_xor_sync(0xffffffffu, a, 2);
            if (kq == 0 && row0 + r < q.N && m0 + m < M)
                P[(static_cast<size_t>(split) * M + (m0 + m)) * q.N + row0 + r] = a;
        }
}

// Backward: one warp = a 128-column window of Q x a slice of the rows (the contraction runs over
// rows).  Same lane ownership; each lane keeps 32 column sums per row of dY.
template <int B, int MT>
__global__ void __launch_bounds__(128) small_bwd_kernel(QView q, const __nv_bfloat16* __restrict__ dY, float* __restrict__ P,
                                                        int M, int rowgroups_per_split) {
    __shared__ float cb[1 << B];
    for (int i = threadIdx.x; i < (1 << B); i += blockDim.x) cb[i] = c_codebook[bits_index(B)][i];
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kq = lane & 3, rq = lane >> 2;
    const int win = blockIdx.x * 4 + warp;
    if (win * 128 >= q.K) return;
    const int split = blockIdx.y;
    const int m0 = blockIdx.z * MT;
    const int ngroups = (q.N + 31) >> 5;
    const int g_lo = split * rowgroups_per_split;
    const int g_hi = min(ngroups, g_lo + rowgroups_per_split);
    const int kbase = win * 128 + 32 * kq;

    float acc[MT][32];
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int j = 0; j < 32; ++j) acc[m][j] = 0.0f;

    const bool kact = kbase < q.K;           // K is a multiple of 64: the last window may be half empty
    for (int rg = g_lo; rg < g_hi && kact; ++rg) {
        const uint32_t* slab = q.codes + slab_word_base(rg * 32, kbase >> 6, q.ktiles, B);
        uint4 w[B];
        load_group4<B>(slab, (kbase >> 5) & 1, slab_row_slot(4 * rq, (kbase >> 5) & 1, kbase >> 6), w);
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int row = rg * 32 + 4 * rq + r;
            if (row >= q.N) continue;
            uint32_t rw[B + 1];
            row_words<B>(w, r, rw);
            const long long blk = static_cast<long long>(row) * q.KB + (kbase >> q.logB0);
            const float s_lo = block_scale(q.sc[blk], q.v[blk >> q.logB1], q.levels);
            float s_hi = s_lo;
            if (q.B0 == 16) s_hi = block_scale(q.sc[blk + 1], q.v[(blk + 1) >> q.logB1], q.levels);
            float g[MT];
#pragma unroll
            for (int m = 0; m < MT; ++m)
                g[m] = (m0 + m < M) ? __bfloat162float(dY[static_cast<size_t>(m0 + m) * q.N + row]) : 0.0f;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float wv = __fmul_rn(cb[extract_code<B>(rw, j)], j < 16 ? s_lo : s_hi);
                const float w16 = __bfloat162float(__float2bfloat16_rn(wv));
#pragma unroll
                for (int m = 0; m < MT; ++m) acc[m][j] = fmaf(g[m], w16, acc[m][j]);
            }
        }
    }
#pragma unroll
    for (int m = 0; m < MT; ++m)
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            float a = acc[m][j];
            a += __shfl_xor_sync(0xffffffffu, a, 4);
            a += __shfl_xor_sync(0xffffffffu, a, 8);
            a += __shfl_xor_sync(0xffffffffu, a, 16);
            acc[m][j] = a;
        }
    if (rq == 0 && kact) {
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (m0 + m < M) {
                float4* dst = reinterpret_cast<float4*>(P + (static_cast<size_t>(split) * M + (m0 + m)) * q.K + kbase);
#pragma unroll
                for (int i = 0; i < 8; ++i) dst[i] = make_float4(acc[m][4 * i], acc[m][4 * i + 1], acc[m][4 * i + 2], acc[m][4 * i + 3]);
            }
    }
}

struct SmallPlan {
    int splits;
    int per_split;
    size_t t_bytes;      // rank-r intermediate
    size_t p_bytes;      // fp32 partial sums
};

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Forward splits K in 128-column windows, backward splits N in 32-row groups.
inline SmallPlan small_plan(int64_t N, int64_t K, int r, int64_t M, bool backward) {
    SmallPlan p;
    const int64_t units = backward ? (N + 31) / 32 : K / 128 + ((K % 128) ? 1 : 0);
    const int64_t outer = backward ? (K + 127) / 128 : (N + 31) / 32;
    int64_t want = (148 * 16 + outer - 1) / outer;
    if (want < 1) want = 1;
    if (want > units) want = units;
    p.per_split = static_cast<int>((units + want - 1) / want);
    p.splits = static_cast<int>((units + p.per_split - 1) / p.per_split);
    p.t_bytes = round_up(static_cast<size_t>(M) * (r > 0 ? r : 1) * 2, 256);
    p.p_bytes = round_up(static_cast<size_t>(p.splits) * M * (backward ? K : N) * 4, 256);
    return p;
}

template <int B>
inline cudaError_t launch_small(const QView& q, const void* L1, const void* L2, int r, const void* A, int M, void* out,
                                char* ws, bool backward, cudaStream_t st) {
    const SmallPlan p = small_plan(q.N, q.K, r, M, backward);
    __nv_bfloat16* T = reinterpret_cast<__nv_bfloat16*>(ws + kStatusBytes);
    float* P = reinterpret_cast<float*>(ws + kStatusBytes + p.t_bytes);
    const __nv_bfloat16* a = static_cast<const __nv_bfloat16*>(A);
    const __nv_bfloat16* l1 = static_cast<const __nv_bfloat16*>(L1);
    const __nv_bfloat16* l2 = static_cast<const __nv_bfloat16*>(L2);
    int launches = 0;
    if (!backward) {
        if (r > 0) { lowrank_pre_kernel<<<M, 256, 0, st>>>(a, l2, T, q.K, r, q.K, 1); ++launches; }
        constexpr int MT = 4;
        dim3 grid(((q.N + 31) / 32 + 3) / 4, p.splits, (M + MT - 1) / MT);
        small_fwd_kernel<B, MT><<<grid, 128, 0, st>>>(q, a, P, M, p.per_split);
        const long long tot = static_cast<long long>(M) * q.N;
        finalize_kernel<<<static_cast<unsigned>((tot + 255) / 256), 256, 0, st>>>(P, p.splits, T, l1,
            static_cast<__nv_bfloat16*>(out), M, q.N, r, r, 1);
        launches += 2;
    } else {
        if (r > 0) {
            if (M <= 16 && q.N % 8 == 0 && q.N <= 40960) {
                const cudaError_t e = dec::launch_pre<true>(a, l1, T, reinterpret_cast<int*>(ws), nullptr, 0, M, q.N, r, st);
                if (e != cudaSuccess) return e;
            } else {
                lowrank_pre_kernel<<<M, 256, 0, st>>>(a, l1, T, q.N, r, 1, r);
                ++launches;
            }
        }
        constexpr int MT = 2;
        dim3 grid(((q.K + 127) / 128 + 3) / 4, p.splits, (M + MT - 1) / MT);
        small_bwd_kernel<B, MT><<<grid, 128, 0, st>>>(q, a, P, M, p.per_split);
        const long long tot = static_cast<long long>(M) * q.K;
        finalize_kernel<<<static_cast<unsigned>((tot + 255) / 256), 256, 0, st>>>(P, p.splits, T, l2,
            static_cast<__nv_bfloat16*>(out), M, q.K, r, 1, q.K);
        launches += 2;
    }
    count_launch(launches);
    return cudaGetLastError();
}

}  // namespace lq
