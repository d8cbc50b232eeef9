// The low-rank plus quantized decomposition of Sec. 3.1 (Algorithm 2) with Factorize of Sec. 3.3 (Algorithm 4) on the
// GPU, in nn.Linear orientation:  W [N, K]  ~  deq(Q) [N, K] + L1 [N, r] L2 [r, K].
//
//   Q <- 0;  repeat:  L1, L2 <- Factorize(W - Q, F, r);  Q <- Quantize(W - L1 L2, c);  error;  until the error rises.
//
// Factorize uses a randomized SVD (the paper's footnote to Eq. (2)): range finder Y = A Omega with a caller-supplied
// Gaussian test matrix, a few power iterations with re-orthonormalization, B = Qb^T A, and the exact SVD of the
// small matrix B through the symmetric eigenproblem of B B^T.  The large products (everything that touches the N x K
// matrix) run in the fp32 kernels below, Quantize is the library's own encoder, the error is reduced on the device;
// the (r + p) x (r + p) factorizations (Cholesky for the orthonormalization, Jacobi for the eigenproblem) run on the
// host in fp64 between the launches.  This is preparation work, done once per matrix, not the layer's hot path: the
// call synchronizes the stream every step to read the error, as the stopping rule needs it.
#pragma once

#include <cmath>
#include <vector>

#include "codec.cuh"
#include "common.cuh"

namespace lq {
namespace lqd {

// ------------------------------------------------------------------------------------ kernels
// C[M x N] = alpha * op(A) op(B) + beta * C, row-major operands with leading dimensions; op = transpose when TA / TB.
// 64 x 64 tile per CTA, 16 x 16 threads with 4 x 4 outputs each, contraction in chunks of 16, fp32 throughout.
template <bool TA, bool TB>
__global__ void __launch_bounds__(256) sgemm_kernel(int M, int N, int Kc, float alpha, const float* __restrict__ A, int lda,
                                                    const float* __restrict__ B, int ldb, float beta, float* __restrict__ C, int ldc) {
    __shared__ float As[16][68], Bs[16][68];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * 64, n0 = blockIdx.x * 64;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
    for (int k0 = 0; k0 < Kc; k0 += 16) {
        if (!TA) {
            const int m = tid >> 2, kk = (tid & 3) * 4;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int gm = m0 + m, gk = k0 + kk + e;
                As[kk + e][m] = (gm < M && gk < Kc) ? A[static_cast<size_t>(gm) * lda + gk] : 0.0f;
            }
        } else {
            const int kk = tid >> 4, m = (tid & 15) * 4;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int gm = m0 + m + e, gk = k0 + kk;
                As[kk][m + e] = (gm < M && gk < Kc) ? A[static_cast<size_t>(gk) * lda + gm] : 0.0f;
            }
        }
        if (!TB) {
            const int kk = tid >> 4, n = (tid & 15) * 4;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int gn = n0 + n + e, gk = k0 + kk;
                Bs[kk][n + e] = (gn < N && gk < Kc) ? B[static_cast<size_t>(gk) * ldb + gn] : 0.0f;
            }
        } else {
            const int n = tid >> 2, kk = (tid & 3) * 4;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int gn = n0 + n, gk = k0 + kk + e;
                Bs[kk + e][n] = (gn < N && gk < Kc) ? B[static_cast<size_t>(gn) * ldb + gk] : 0.0f;
            }
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int gm = m0 + ty * 4 + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gn = n0 + tx * 4 + j;
            if (gn >= N) continue;
            float* c = C + static_cast<size_t>(gm) * ldc + gn;
            *c = (beta == 0.0f) ? alpha * acc[i][j] : fmaf(alpha, acc[i][j], beta * *c);
        }
    }
}

// out = (a - b) * drow[n] * dcol[k]   (b, drow, dcol optional)
__global__ void diff_scale_kernel(const float* __restrict__ a, const float* __restrict__ b, const float* __restrict__ drow,
                                  const float* __restrict__ dcol, float* __restrict__ out, long long total, int K) {
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
        float v = a[i] - (b ? b[i] : 0.0f);
        if (drow) v *= drow[i / K] * dcol[i % K];
        out[i] = v;
    }
}

// *acc += sum_i f_i (a_i - b_i)^2  in fp64 (f optional: Eq. (3))
__global__ void sqerr_kernel(const float* __restrict__ a, const float* __restrict__ b, const float* __restrict__ f, double* acc, long long total) {
    double s = 0.0;
    for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < total; i += static_cast<long long>(gridDim.x) * blockDim.x) {
        const double d = static_cast<double>(a[i]) - static_cast<double>(b[i]);
        s += (f ? static_cast<double>(f[i]) : 1.0) * d * d;
    }
    __shared__ double red[256];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (static_cast<int>(threadIdx.x) < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) atomicAdd(acc, red[0]);
}

// D_row[n] = mean_k sqrt(F[n][k])  (one CTA per row)  and  D_col[k] = mean_n sqrt(F[n][k])  (one thread per column)
__global__ void row_mean_sqrt_kernel(const float* __restrict__ F, float* __restrict__ drow, int K) {
    double s = 0.0;
    const float* row = F + static_cast<size_t>(blockIdx.x) * K;
    for (int k = threadIdx.x; k < K; k += blockDim.x) s += sqrt(static_cast<double>(row[k]));
    __shared__ double red[256];
    red[threadIdx.x] = s;
    __syncthreads();
    for (int o = 128; o > 0; o >>= 1) {
        if (static_cast<int>(threadIdx.x) < o) red[threadIdx.x] += red[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) drow[blockIdx.x] = static_cast<float>(red[0] / K);
}
__global__ void col_mean_sqrt_kernel(const float* __restrict__ F, float* __restrict__ dcol, int N, int K) {
    const int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= K) return;
    double s = 0.0;
    for (int n = 0; n < N; ++n) s += sqrt(static_cast<double>(F[static_cast<size_t>(n) * K + k]));
    dcol[k] = static_cast<float>(s / N);
}
// X[n][j] /= d[n]  (rows)   or   X[j][k] /= d[k]  (columns)
__global__ void div_rows_kernel(float* X, const float* __restrict__ d, int rows, int cols) {
    const long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (i < static_cast<long long>(rows) * cols) X[i] /= d[i / cols];
}
__global__ void div_cols_kernel(float* X, const float* __restrict__ d, int rows, int cols) {
    const long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (i < static_cast<long long>(rows) * cols) X[i] /= d[i % cols];
}
__global__ void to_bf16_kernel(const float* __restrict__ x, __nv_bfloat16* __restrict__ y, long long total) {
    const long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x;
    if (i < total) y[i] = __float2bfloat16_rn(x[i]);
}

// ------------------------------------------------------------------------------------ host: small dense factorizations (fp64)
// Upper-triangular R with R^T R = G (n x n, row major); returns false if G is not positive definite.
inline bool cholesky_upper(std::vector<double>& G, int n) {
    for (int j = 0; j < n; ++j) {
        double d = G[j * n + j];
        for (int k = 0; k < j; ++k) d -= G[k * n + j] * G[k * n + j];
        if (!(d > 0.0)) return false;
        d = std::sqrt(d);
        G[j * n + j] = d;
        for (int i = j + 1; i < n; ++i) {
            double s = G[j * n + i];
            for (int k = 0; k < j; ++k) s -= G[k * n + j] * G[k * n + i];
            G[j * n + i] = s / d;
        }
        for (int i = 0; i < j; ++i) G[j * n + i] = 0.0;
    }
    return true;
}
// inverse of an upper-triangular matrix (row major)
inline std::vector<double> invert_upper(const std::vector<double>& R, int n) {
    std::vector<double> X(static_cast<size_t>(n) * n, 0.0);
    for (int j = 0; j < n; ++j) {
        X[j * n + j] = 1.0 / R[j * n + j];
        for (int i = j - 1; i >= 0; --i) {
            double s = 0.0;
            for (int k = i + 1; k <= j; ++k) s += R[i * n + k] * X[k * n + j];
            X[i * n + j] = -s / R[i * n + i];
        }
    }
    return X;
}
// Cyclic Jacobi for a symmetric n x n matrix: on return G holds the eigenvalues on its diagonal and V the
// eigenvectors in its columns.
inline void jacobi_eigh(std::vector<double>& G, std::vector<double>& V, int n) {
    V.assign(static_cast<size_t>(n) * n, 0.0);
    for (int i = 0; i < n; ++i) V[i * n + i] = 1.0;
    for (int sweep = 0; sweep < 60; ++sweep) {
        double off = 0.0, diag = 0.0;
        for (int i = 0; i < n; ++i)
            for (int j = 0; j < n; ++j) (i == j ? diag : off) += G[i * n + j] * G[i * n + j];
        if (off <= 1e-30 * diag) break;
        for (int p = 0; p < n - 1; ++p)
            for (int q = p + 1; q < n; ++q) {
                const double apq = G[p * n + q];
                if (apq == 0.0) continue;
                const double theta = (G[q * n + q] - G[p * n + p]) / (2.0 * apq);
                const double t = (theta >= 0.0 ? 1.0 : -1.0) / (std::fabs(theta) + std::sqrt(theta * theta + 1.0));
                const double c = 1.0 / std::sqrt(t * t + 1.0), s = t * c;
                for (int k = 0; k < n; ++k) {
                    const double gkp = G[k * n + p], gkq = G[k * n + q];
                    G[k * n + p] = c * gkp - s * gkq;
                    G[k * n + q] = s * gkp + c * gkq;
                }
                for (int k = 0; k < n; ++k) {
                    const double gpk = G[p * n + k], gqk = G[q * n + k];
                    G[p * n + k] = c * gpk - s * gqk;
                    G[q * n + k] = s * gpk + c * gqk;
                }
                for (int k = 0; k < n; ++k) {
                    const double vkp = V[k * n + p], vkq = V[k * n + q];
                    V[k * n + p] = c * vkp - s * vkq;
                    V[k * n + q] = s * vkp + c * vkq;
                }
            }
    }
}

// ------------------------------------------------------------------------------------ host: the algorithm
struct Buffers {
    float* buf0;      // [N][K]  A = W - Q (scaled), then R = W - L1 L2
    float* buf1;      // [N][K]  dequantized candidate Q
    float* Y;         // [N][l]
    float* Y2;        // [N][l]
    float* Z;         // [K][l]
    float* Z2;        // [K][l]
    float* Bm;        // [l][K]
    float* small;     // [l][l] device scratch for the small matrices (Gram in / factor out)
    float* L1c;       // [N][r] candidate factors
    float* L2c;       // [r][K]
    float* drow;      // [N]
    float* dcol;      // [K]
    double* err;      // one fp64 accumulator
    float* absmax;    // encoder scratch
    void* q_codes;    // candidate quantized matrix
    uint8_t* q_sc;
    float* q_v;
};

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

inline size_t workspace_bytes(int64_t N, int64_t K, const lqlora_config* cfg, int r, int p) {
    const int64_t l = r + p;
    size_t cb = 0, sb = 0, s2 = 0, ew = 0;
    lqlora_packed_sizes(N, K, cfg, &cb, &sb, &s2, &ew);
    size_t t = 0;
    t += 2 * align256(static_cast<size_t>(N) * K * 4);
    t += 2 * align256(static_cast<size_t>(N) * l * 4) + 2 * align256(static_cast<size_t>(K) * l * 4) + align256(static_cast<size_t>(l) * K * 4);
    t += align256(static_cast<size_t>(l) * l * 4);
    t += align256(static_cast<size_t>(N) * r * 4) + align256(static_cast<size_t>(r) * K * 4);
    t += align256(static_cast<size_t>(N) * 4) + align256(static_cast<size_t>(K) * 4) + 256;
    t += align256(ew) + align256(cb) + align256(sb) + align256(s2);
    return t;
}

template <bool TA, bool TB>
inline void gemm(int M, int N, int Kc, float alpha, const float* A, int lda, const float* B, int ldb, float beta, float* C, int ldc,
                 cudaStream_t st) {
    dim3 grid((N + 63) / 64, (M + 63) / 64);
    sgemm_kernel<TA, TB><<<grid, 256, 0, st>>>(M, N, Kc, alpha, A, lda, B, ldb, beta, C, ldc);
    count_launch(1);
}

// X [rows x l] <- X R^-1 with R^T R = X^T X (Cholesky QR), twice; `tmp` receives the result of the first pass and the
// final result is left in X.  Returns false on a CUDA error or a Gram matrix that is not positive definite.
inline bool orthonormalize(float* X, float* tmp, int rows, int l, float* small_dev, cudaStream_t st) {
    std::vector<float> gh(static_cast<size_t>(l) * l);
    std::vector<double> G(static_cast<size_t>(l) * l);
    float* src = X;
    float* dst = tmp;
    for (int pass = 0; pass < 2; ++pass) {
        gemm<true, false>(l, l, rows, 1.0f, src, l, src, l, 0.0f, small_dev, l, st);
        if (cudaMemcpyAsync(gh.data(), small_dev, gh.size() * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) return false;
        for (size_t i = 0; i < G.size(); ++i) G[i] = gh[i];
        // a tiny ridge keeps the factorization alive when the test matrix hits a deficient range
        double tr = 0.0;
        for (int i = 0; i < l; ++i) tr += G[i * l + i];
        for (int i = 0; i < l; ++i) G[i * l + i] += 1e-12 * tr / l;
        if (!cholesky_upper(G, l)) return false;
        const std::vector<double> Ri = invert_upper(G, l);
        for (size_t i = 0; i < gh.size(); ++i) gh[i] = static_cast<float>(Ri[i]);
        if (cudaMemcpyAsync(small_dev, gh.data(), gh.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return false;
        gemm<false, false>(rows, l, l, 1.0f, src, l, small_dev, l, 0.0f, dst, l, st);
        if (cudaStreamSynchronize(st) != cudaSuccess) return false;      // gh is reused by the next pass
        float* t = src; src = dst; dst = t;
    }
    // two passes: the result is back in X (src == X)
    return src == X;
}

// One Factorize(A, F, r) with A in b.buf0 (already scaled by D_row, D_col when F is given): candidate factors into
// b.L1c, b.L2c.
inline int factorize(const Buffers& b, int N, int K, int r, int l, const float* omega, int power_iters, bool fisher, cudaStream_t st) {
    const float* A = b.buf0;
    gemm<false, false>(N, l, K, 1.0f, A, K, omega, l, 0.0f, b.Y, l, st);               // Y = A Omega
    for (int it = 0; it < power_iters; ++it) {
        if (!orthonormalize(b.Y, b.Y2, N, l, b.small, st)) return LQLORA_ERR_CUDA;
        gemm<true, false>(K, l, N, 1.0f, A, K, b.Y, l, 0.0f, b.Z, l, st);              // Z = A^T Y
        if (!orthonormalize(b.Z, b.Z2, K, l, b.small, st)) return LQLORA_ERR_CUDA;
        gemm<false, false>(N, l, K, 1.0f, A, K, b.Z, l, 0.0f, b.Y, l, st);             // Y = A Z
    }
    if (!orthonormalize(b.Y, b.Y2, N, l, b.small, st)) return LQLORA_ERR_CUDA;         // Qb
    gemm<true, false>(l, K, N, 1.0f, b.Y, l, A, K, 0.0f, b.Bm, K, st);                  // B = Qb^T A
    gemm<false, true>(l, l, K, 1.0f, b.Bm, K, b.Bm, K, 0.0f, b.small, l, st);           // B B^T
    std::vector<float> gh(static_cast<size_t>(l) * l);
    if (cudaMemcpyAsync(gh.data(), b.small, gh.size() * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
        return LQLORA_ERR_CUDA;
    std::vector<double> G(gh.begin(), gh.end()), V;
    for (int i = 0; i < l; ++i)
        for (int j = i + 1; j < l; ++j) { const double s = 0.5 * (G[i * l + j] + G[j * l + i]); G[i * l + j] = G[j * l + i] = s; }
    jacobi_eigh(G, V, l);
    std::vector<int> order(l);
    for (int i = 0; i < l; ++i) order[i] = i;
    for (int i = 0; i < l; ++i)
        for (int j = i + 1; j < l; ++j)
            if (G[order[j] * l + order[j]] > G[order[i] * l + order[i]]) { const int t = order[i]; order[i] = order[j]; order[j] = t; }
    // M1 [l x r] = Ub_r sqrt(S_r),  M2 [r x l] = S_r^-1/2 Ub_r^T   (S = sqrt(eigenvalue))
    std::vector<float> M1(static_cast<size_t>(l) * r), M2(static_cast<size_t>(r) * l);
    for (int j = 0; j < r; ++j) {
        const double lam = G[order[j] * l + order[j]];
        const double sig = lam > 0.0 ? std::sqrt(lam) : 0.0;
        const double rs = std::sqrt(sig), irs = sig > 0.0 ? 1.0 / rs : 0.0;
        for (int i = 0; i < l; ++i) {
            M1[static_cast<size_t>(i) * r + j] = static_cast<float>(V[i * l + order[j]] * rs);
            M2[static_cast<size_t>(j) * l + i] = static_cast<float>(V[i * l + order[j]] * irs);
        }
    }
    // the two small operands go through the device scratch one after the other
    if (cudaMemcpyAsync(b.small, M1.data(), M1.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return LQLORA_ERR_CUDA;
    gemm<false, false>(N, r, l, 1.0f, b.Y, l, b.small, r, 0.0f, b.L1c, r, st);          // L1 = Qb M1
    if (cudaStreamSynchronize(st) != cudaSuccess) return LQLORA_ERR_CUDA;
    if (cudaMemcpyAsync(b.small, M2.data(), M2.size() * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return LQLORA_ERR_CUDA;
    gemm<false, false>(r, K, l, 1.0f, b.small, l, b.Bm, K, 0.0f, b.L2c, K, st);         // L2 = M2 B
    if (cudaStreamSynchronize(st) != cudaSuccess) return LQLORA_ERR_CUDA;
    if (fisher) {
        div_rows_kernel<<<static_cast<unsigned>((static_cast<long long>(N) * r + 255) / 256), 256, 0, st>>>(b.L1c, b.drow, N, r);
        div_cols_kernel<<<static_cast<unsigned>((static_cast<long long>(r) * K + 255) / 256), 256, 0, st>>>(b.L2c, b.dcol, r, K);
        count_launch(2);
    }
    return LQLORA_OK;
}

template <int B>
inline int run(const float* W, const float* F, lqlora_qmatrix* out, float* L1, float* L2, int r, int max_steps, const float* omega,
               int p, int power_iters, double* errors_host, int* steps_taken, char* ws, cudaStream_t st) {
    const int N = static_cast<int>(out->N), K = static_cast<int>(out->K), l = r + p;
    const long long total = static_cast<long long>(N) * K;
    size_t cb = 0, sb = 0, s2 = 0, ew = 0;
    lqlora_packed_sizes(N, K, &out->cfg, &cb, &sb, &s2, &ew);
    Buffers b;
    char* w = ws;
    auto take = [&](size_t bytes) { char* ptr = w; w += align256(bytes); return ptr; };
    b.buf0 = reinterpret_cast<float*>(take(static_cast<size_t>(total) * 4));
    b.buf1 = reinterpret_cast<float*>(take(static_cast<size_t>(total) * 4));
    b.Y = reinterpret_cast<float*>(take(static_cast<size_t>(N) * l * 4));
    b.Y2 = reinterpret_cast<float*>(take(static_cast<size_t>(N) * l * 4));
    b.Z = reinterpret_cast<float*>(take(static_cast<size_t>(K) * l * 4));
    b.Z2 = reinterpret_cast<float*>(take(static_cast<size_t>(K) * l * 4));
    b.Bm = reinterpret_cast<float*>(take(static_cast<size_t>(l) * K * 4));
    b.small = reinterpret_cast<float*>(take(static_cast<size_t>(l) * l * 4));
    b.L1c = reinterpret_cast<float*>(take(static_cast<size_t>(N) * r * 4));
    b.L2c = reinterpret_cast<float*>(take(static_cast<size_t>(r) * K * 4));
    b.drow = reinterpret_cast<float*>(take(static_cast<size_t>(N) * 4));
    b.dcol = reinterpret_cast<float*>(take(static_cast<size_t>(K) * 4));
    b.err = reinterpret_cast<double*>(take(256));
    b.absmax = reinterpret_cast<float*>(take(ew));
    b.q_codes = take(cb);
    b.q_sc = reinterpret_cast<uint8_t*>(take(sb));
    b.q_v = reinterpret_cast<float*>(take(s2));

    lqlora_qmatrix cand = *out;
    cand.codes = b.q_codes; cand.scale_codes = b.q_sc; cand.scale2 = b.q_v;
    const QView cv = make_view(&cand);
    const bool fisher = F != nullptr;
    const unsigned ew_grid = 148 * 8;
    if (fisher) {
        row_mean_sqrt_kernel<<<N, 256, 0, st>>>(F, b.drow, K);
        col_mean_sqrt_kernel<<<(K + 255) / 256, 256, 0, st>>>(F, b.dcol, N, K);
        count_launch(2);
    }
    double prev = INFINITY;
    int steps = 0;
    bool have_q = false;
    for (int t = 0; t < max_steps; ++t) {
        // A = W - Q  (Q = 0 at the start; buf1 holds the dequantized accepted Q afterwards), scaled for the weighted SVD
        diff_scale_kernel<<<ew_grid, 256, 0, st>>>(W, have_q ? b.buf1 : nullptr, fisher ? b.drow : nullptr, b.dcol, b.buf0, total, K);
        count_launch(1);
        int rc = factorize(b, N, K, r, l, omega, power_iters, fisher, st);
        if (rc != LQLORA_OK) return rc;
        // R = W - L1 L2
        if (cudaMemcpyAsync(b.buf0, W, static_cast<size_t>(total) * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return LQLORA_ERR_CUDA;
        gemm<false, false>(N, K, r, -1.0f, b.L1c, r, b.L2c, K, 1.0f, b.buf0, K, st);
        // Q = Quantize(R, c) into the candidate arrays
        if (launch_encode<B>(b.buf0, &cand, b.absmax, st) != cudaSuccess) return LQLORA_ERR_CUDA;
        // error = || R - deq(Q) || (weighted by F when given).  The candidate's dequantized value overwrites that of the
        // accepted Q in buf1: the old one is needed again only if this step is accepted too (and then it is the new one).
        if (launch_export<B>(cv, nullptr, b.buf1, nullptr, st) != cudaSuccess) return LQLORA_ERR_CUDA;
        if (cudaMemsetAsync(b.err, 0, sizeof(double), st) != cudaSuccess) return LQLORA_ERR_CUDA;
        sqerr_kernel<<<ew_grid, 256, 0, st>>>(b.buf0, b.buf1, F, b.err, total);
        count_launch(1);
        double e2 = 0.0;
        if (cudaMemcpyAsync(&e2, b.err, sizeof(double), cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
            return LQLORA_ERR_CUDA;
        const double err = std::sqrt(e2);
        errors_host[steps++] = err;
        if (err > prev) break;                     // the error rose: the accepted iterate stays
        prev = err;
        have_q = true;
        // accept: candidate -> outputs
        if (cudaMemcpyAsync(out->codes, b.q_codes, cb, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(out->scale_codes, b.q_sc, sb, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(out->scale2, b.q_v, s2, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(L1, b.L1c, static_cast<size_t>(N) * r * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
            cudaMemcpyAsync(L2, b.L2c, static_cast<size_t>(r) * K * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return LQLORA_ERR_CUDA;
    }
    *steps_taken = steps;
    if (cudaStreamSynchronize(st) != cudaSuccess) return LQLORA_ERR_CUDA;
    return LQLORA_OK;
}

}  // namespace lqd
}  // namespace lq
