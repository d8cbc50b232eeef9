// CPU oracle for the LQ-LoRA quantized-plus-low-rank linear layer (arXiv 2311.12023).
//
// THIS IS TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  It is a plain, slow, obviously
// correct restatement of what the paper defines, written so that it can be checked
// against the paper by eye.  It shares no code, table or constant with the CUDA
// library; only tests, the smoke check and the benchmark's CPU-baseline leg call it.
//
// Orientation: the paper writes the layer as X(W + L1 L2) with W in R^{d x k} (Sec. 2.1).
// Here matrices are stored like nn.Linear weights: W and Q are [N = out, K = in] row
// major (the paper's W transposed), L1 is [N, r], L2 is [r, K], X is [M, K]:
//     Y  = X deq(Q)^T + (X L2^T) L1^T          dX = dY deq(Q) + (dY L1) L2
//
// Arithmetic: every fp32 operation below is a single IEEE-754 binary32 operation with
// round-to-nearest-even (x86-64 SSE scalar code, no fast-math, no contraction: build
// with -O2 -ffp-contract=off).  The layer products are fp64 throughout.
//
// Parity pins (tests/test_oracle_*.py): every function here is pinned -- none is
// "parity unpinned".
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// Number of positive integer levels of the b1-bit round-to-nearest quantizer of Sec. 2.2:
// 2^(b1-1) - 1.  The footnote of Sec. 3.2 is read as using the RTN scaling factor
// absmax / (2^(b1-1) - 1) of Sec. 2.2.
inline int rtn_levels(int b1) { return (1 << (b1 - 1)) - 1; }

// Phi(x): standard normal CDF.
inline double normal_cdf(double x) { return 0.5 * std::erfc(-x / std::sqrt(2.0)); }

// Phi^{-1}(p) by bisection on the CDF (slow and plain on purpose).
double normal_quantile(double p) {
    if (p == 0.5) return 0.0;
    double lo = -40.0, hi = 40.0;
    for (int it = 0; it < 200; ++it) {
        double mid = 0.5 * (lo + hi);
        if (mid == lo || mid == hi) break;
        if (normal_cdf(mid) < p) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

inline double bf16_to_double(uint16_t b) {
    uint32_t u = static_cast<uint32_t>(b) << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return static_cast<double>(f);
}

// fp32 -> bf16, round to nearest, ties to even (finite inputs).
inline uint16_t f32_to_bf16_rne(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    return static_cast<uint16_t>(u >> 16);
}

// fp32 -> IEEE binary16 -> fp32, round to nearest, ties to even, written from the format's definition: 5 exponent bits
// (bias 15), 10 fraction bits, subnormals down to 2^-24, overflow to infinity beyond 65504 + half an ulp.
inline float round_through_fp16(float f) {
    if (std::isnan(f) || std::isinf(f) || f == 0.0f) return f;
    const double a = std::fabs(static_cast<double>(f));
    int e;
    std::frexp(a, &e);                    // a = m * 2^e, 0.5 <= m < 1  ->  a in [2^(e-1), 2^e)
    int ex = e - 1;                       // binade exponent
    if (ex < -14) ex = -14;               // subnormal range shares the spacing of the lowest binade
    const double ulp = std::ldexp(1.0, ex - 10);
    double qd = a / ulp;                  // exact (power-of-two scaling)
    double fl = std::floor(qd);
    const double frac = qd - fl;
    if (frac > 0.5 || (frac == 0.5 && std::fmod(fl, 2.0) == 1.0)) fl += 1.0;
    double r = fl * ulp;
    if (r > 65504.0) r = INFINITY;
    return static_cast<float>(f < 0 ? -r : r);
}

}  // namespace

extern "C" {

// ----------------------------------------------------------------------------------
// cast(v, b2) of Sec. 3.2 for the second-level scales: kind 32 = fp32 (identity), 16 = IEEE fp16, -16 = bfloat16;
// round to nearest even, result returned as the fp32 value the stored number decodes to.
// ----------------------------------------------------------------------------------
int oracle_cast_scale2(const float* v, int64_t n, int kind, float* out) {
    if (kind != 32 && kind != 16 && kind != -16) return -1;
    for (int64_t i = 0; i < n; ++i) {
        if (kind == 32) out[i] = v[i];
        else if (kind == 16) out[i] = round_through_fp16(v[i]);
        else out[i] = static_cast<float>(bf16_to_double(f32_to_bf16_rne(v[i])));
    }
    return 0;
}

// ----------------------------------------------------------------------------------
// NF codebook, Sec. 2.2: 2^(b-1) evenly spaced probabilities on [delta, 1/2] and
// 2^(b-1)+1 on [1/2, 1-delta], delta = (1/30 + 1/32)/2; the shared 1/2 is kept once so
// that 2^b values remain; q_i = Phi^{-1}(p_i); q~_i = q_i / q_{2^b}.  Built in fp64,
// returned as fp32.  Returns 0 on success.
// ----------------------------------------------------------------------------------
int oracle_nf_codebook(int b, float* out) {
    if (b < 1 || b > 8) return -1;
    const int half = 1 << (b - 1);
    const double delta = 0.5 * (1.0 / 30.0 + 1.0 / 32.0);
    std::vector<double> p;
    for (int i = 0; i < half; ++i) {            // [delta, 1/2], 2^(b-1) values
        double t = (half == 1) ? 1.0 : static_cast<double>(i) / (half - 1);
        p.push_back(delta + (0.5 - delta) * t);
    }
    p.back() = 0.5;
    for (int i = 1; i <= half; ++i) {           // (1/2, 1-delta], the 1/2 already present
        double t = static_cast<double>(i) / half;
        p.push_back(0.5 + (0.5 - delta) * t);
    }
    const int n = 1 << b;
    std::vector<double> q(n);
    for (int i = 0; i < n; ++i) q[i] = normal_quantile(p[i]);
    for (int i = 0; i < n; ++i) out[i] = static_cast<float>(q[i] / q[n - 1]);
    return 0;
}

// ----------------------------------------------------------------------------------
// Storage cost in bits per parameter, Eq. (2) of Sec. 3.2: b0 + b1/B0 + b2/(B0 B1).
// ----------------------------------------------------------------------------------
double oracle_storage_bits_per_param(int b0, int b1, int b2, int B0, int B1) {
    return static_cast<double>(b0) + static_cast<double>(b1) / B0 +
           static_cast<double>(b2) / (static_cast<double>(B0) * B1);
}

// ----------------------------------------------------------------------------------
// Quantize(A, c), Sec. 2.2 and Sec. 3.2.
//   A [N, K] row major fp32, flattened row by row and cut into blocks of B0 (K % B0 == 0,
//   so every block lies inside one row, along K).
//   Quantize-NF:  s_i = max|u_j| over the block; c_j = argmin_i |q~_i - u_j / s_i|,
//                 the smallest index on a tie; an all-zero block takes the code of 0.
//   Quantize-INT: blocks are grouped B1 at a time in flattened order (the last group may
//                 be short); v_g = max s_i; sigma_g = v_g / (2^(b1-1)-1);
//                 s^_i = clamp(round_half_even(s_i / sigma_g), 0, 2^(b1-1)-1).
//   cast(v, fp32) is the identity.
// Outputs: codes [N*K] uint8 (one code per byte), absmax [nblk] fp32 (optional, may be
// null), scale_codes [nblk] uint8, scale2 [ngrp] fp32.  Returns 0 on success.
// ----------------------------------------------------------------------------------
int oracle_encode(const float* A, int64_t N, int64_t K, int b0, int B0, int b1, int B1,
                  uint8_t* codes, float* absmax, uint8_t* scale_codes, float* scale2) {
    if (N <= 0 || K <= 0 || B0 <= 0 || B1 <= 0 || K % B0 != 0 || b1 < 2 || b1 > 8) return -1;
    float cb[256];
    if (oracle_nf_codebook(b0, cb) != 0) return -1;
    const int ncode = 1 << b0;
    const int zero_code = (1 << (b0 - 1)) - 1;
    const int64_t nblk = N * K / B0;
    const int64_t ngrp = (nblk + B1 - 1) / B1;
    std::vector<float> s(nblk);

#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < nblk; ++i) {
        const float* u = A + i * B0;
        float m = 0.0f;
        for (int j = 0; j < B0; ++j) m = std::fmax(m, std::fabs(u[j]));
        s[i] = m;
        for (int j = 0; j < B0; ++j) {
            int best = zero_code;
            if (m != 0.0f) {
                const float x = u[j] / m;                       // one fp32 division
                double bestd = INFINITY;
                for (int c = 0; c < ncode; ++c) {
                    // the difference of two fp32 numbers is exact in fp64
                    double d = std::fabs(static_cast<double>(cb[c]) - static_cast<double>(x));
                    if (d < bestd) { bestd = d; best = c; }     // strict: lower index wins ties
                }
            }
            codes[i * B0 + j] = static_cast<uint8_t>(best);
        }
    }
    if (absmax) std::memcpy(absmax, s.data(), sizeof(float) * nblk);

    const int levels = rtn_levels(b1);
    for (int64_t g = 0; g < ngrp; ++g) {
        const int64_t lo = g * B1, hi = (lo + B1 < nblk) ? lo + B1 : nblk;
        float v = 0.0f;
        for (int64_t i = lo; i < hi; ++i) v = std::fmax(v, s[i]);
        scale2[g] = v;
        const float sigma = v / static_cast<float>(levels);     // one fp32 division
        for (int64_t i = lo; i < hi; ++i) {
            float code = 0.0f;
            if (v != 0.0f) {
                code = std::nearbyintf(s[i] / sigma);           // ties to even
                if (code < 0.0f) code = 0.0f;
                if (code > static_cast<float>(levels)) code = static_cast<float>(levels);
            }
            scale_codes[i] = static_cast<uint8_t>(code);
        }
    }
    return 0;
}

// ----------------------------------------------------------------------------------
// Dequantize: the inverse of the steps above, applied in reverse order (Sec. 3.2).
//   sigma_g = v_g / (2^(b1-1)-1);  s~_i = float(s^_i) * sigma_g;  w~_j = q~[c_j] * s~_i
//   deq32 = w~ (fp32); deq16 = w~ rounded to bf16 (the cast for bf16 training, App. A).
// Either output may be null.
// ----------------------------------------------------------------------------------
int oracle_dequant(const uint8_t* codes, const uint8_t* scale_codes, const float* scale2,
                   int64_t N, int64_t K, int b0, int B0, int b1, int B1,
                   float* deq32, uint16_t* deq16) {
    if (N <= 0 || K <= 0 || K % B0 != 0) return -1;
    float cb[256];
    if (oracle_nf_codebook(b0, cb) != 0) return -1;
    const int64_t nblk = N * K / B0;
    const int levels = rtn_levels(b1);
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < nblk; ++i) {
        const float sigma = scale2[i / B1] / static_cast<float>(levels);
        const float st = static_cast<float>(scale_codes[i]) * sigma;
        for (int j = 0; j < B0; ++j) {
            const float w = cb[codes[i * B0 + j]] * st;
            if (deq32) deq32[i * B0 + j] = w;
            if (deq16) deq16[i * B0 + j] = f32_to_bf16_rne(w);
        }
    }
    return 0;
}

// ----------------------------------------------------------------------------------
// Forward of the layer (Sec. 2.1, Sec. 3.1):  Y = X (Q + L1 L2) in the paper's
// orientation, i.e. Y[m, n] = sum_k X[m,k] w~[n,k] + sum_j (sum_k X[m,k] L2[j,k]) L1[n,j].
// fp64 throughout, no intermediate rounding.  Only the rows listed in `rows` (nrows of
// them, indices into X) are computed; Y is [nrows, N] fp64.
// bf16 inputs are passed as raw 16-bit patterns.
// ----------------------------------------------------------------------------------
int oracle_linear_fwd(const float* W /*[N,K] deq32*/, const uint16_t* L1 /*[N,r]*/,
                      const uint16_t* L2 /*[r,K]*/, int r, const uint16_t* X /*[M,K]*/,
                      int64_t M, int64_t N, int64_t K, const int64_t* rows, int64_t nrows,
                      double* Y) {
    for (int64_t i = 0; i < nrows; ++i) if (rows[i] < 0 || rows[i] >= M) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < nrows; ++i) {
        const uint16_t* x = X + rows[i] * K;
        std::vector<double> xd(K), t(r > 0 ? r : 1, 0.0);
        for (int64_t k = 0; k < K; ++k) xd[k] = bf16_to_double(x[k]);
        for (int j = 0; j < r; ++j) {                 // t = x L2^T
            double acc = 0.0;
            for (int64_t k = 0; k < K; ++k) acc += xd[k] * bf16_to_double(L2[j * K + k]);
            t[j] = acc;
        }
        for (int64_t n = 0; n < N; ++n) {
            double acc = 0.0;
            const float* w = W + n * K;
            for (int64_t k = 0; k < K; ++k) acc += xd[k] * static_cast<double>(w[k]);
            double lr = 0.0;
            for (int j = 0; j < r; ++j) lr += t[j] * bf16_to_double(L1[n * r + j]);
            Y[i * N + n] = acc + lr;
        }
    }
    return 0;
}

// ----------------------------------------------------------------------------------
// Input gradient of the same layer:  dX = dY (Q + L1 L2)^T in the paper's orientation,
// i.e. dX[m, k] = sum_n dY[m,n] w~[n,k] + sum_j (sum_n dY[m,n] L1[n,j]) L2[j,k].
// fp64 throughout.  Q receives no gradient (only the low-rank part is trained, Sec. 1).
// ----------------------------------------------------------------------------------
int oracle_linear_bwd_input(const float* W /*[N,K] deq32*/, const uint16_t* L1, const uint16_t* L2,
                            int r, const uint16_t* dY /*[M,N]*/, int64_t M, int64_t N, int64_t K,
                            const int64_t* rows, int64_t nrows, double* dX) {
    for (int64_t i = 0; i < nrows; ++i) if (rows[i] < 0 || rows[i] >= M) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t i = 0; i < nrows; ++i) {
        const uint16_t* g = dY + rows[i] * N;
        double* out = dX + i * K;
        std::vector<double> t(r > 0 ? r : 1, 0.0);
        for (int64_t k = 0; k < K; ++k) out[k] = 0.0;
        for (int64_t n = 0; n < N; ++n) {             // sum over n in ascending order
            const double gd = bf16_to_double(g[n]);
            const float* w = W + n * K;
            for (int64_t k = 0; k < K; ++k) out[k] += gd * static_cast<double>(w[k]);
            for (int j = 0; j < r; ++j) t[j] += gd * bf16_to_double(L1[n * r + j]);
        }
        for (int64_t k = 0; k < K; ++k) {
            double lr = 0.0;
            for (int j = 0; j < r; ++j) lr += t[j] * bf16_to_double(L2[j * K + k]);
            out[k] += lr;
        }
    }
    return 0;
}

// ----------------------------------------------------------------------------------
// Gradients of the low-rank factors of the same layer (the trained parameters, Sec. 1 and
// Sec. 2.1).  Y = X W~^T + (X L2^T) L1^T is linear in L1 and in L2, so by the chain rule
//     dL1[n, j] = sum_m dY[m, n] (sum_k X[m, k] L2[j, k])
//     dL2[j, k] = sum_m (sum_n dY[m, n] L1[n, j]) X[m, k]
// fp64 throughout, sums in ascending index order.  The quantized matrix does not enter.
// ----------------------------------------------------------------------------------
int oracle_lora_grads(const uint16_t* L1 /*[N,r]*/, const uint16_t* L2 /*[r,K]*/, int r, const uint16_t* X /*[M,K]*/,
                      const uint16_t* dY /*[M,N]*/, int64_t M, int64_t N, int64_t K, double* dL1 /*[N,r]*/,
                      double* dL2 /*[r,K]*/) {
    if (r <= 0 || M <= 0 || N <= 0 || K <= 0) return -1;
    std::vector<double> T(static_cast<size_t>(M) * r), Tp(static_cast<size_t>(M) * r);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m) {
        for (int j = 0; j < r; ++j) {
            double t = 0.0;
            for (int64_t k = 0; k < K; ++k) t += bf16_to_double(X[m * K + k]) * bf16_to_double(L2[j * K + k]);
            T[m * r + j] = t;
            double tp = 0.0;
            for (int64_t n = 0; n < N; ++n) tp += bf16_to_double(dY[m * N + n]) * bf16_to_double(L1[n * r + j]);
            Tp[m * r + j] = tp;
        }
    }
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
        for (int j = 0; j < r; ++j) {
            double g = 0.0;
            for (int64_t m = 0; m < M; ++m) g += bf16_to_double(dY[m * N + n]) * T[m * r + j];
            dL1[n * r + j] = g;
        }
#pragma omp parallel for schedule(static)
    for (int64_t k = 0; k < K; ++k)
        for (int j = 0; j < r; ++j) {
            double g = 0.0;
            for (int64_t m = 0; m < M; ++m) g += Tp[m * r + j] * bf16_to_double(X[m * K + k]);
            dL2[j * K + k] = g;
        }
    return 0;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // extern "C"
