// NormalFloat code book (Sec. 2.2) built on the host in fp64 and uploaded to constant memory,
// plus host-only helpers of the C ABI (storage formula, sizes, status strings).
#pragma once

#include <atomic>
#include <cmath>
#include <mutex>

#include "common.cuh"

namespace lq {

namespace detail {

// Gaussian quantile by Newton's method on Phi(x) - p, started from a closed-form guess.
inline double gauss_quantile(double p) {
    if (p == 0.5) return 0.0;
    const bool upper = p > 0.5;
    const double pp = upper ? 1.0 - p : p;                 // lower tail probability
    const double t = std::sqrt(-2.0 * std::log(pp));
    double x = -(t - (2.30753 + 0.27061 * t) / (1.0 + t * (0.99229 + 0.04481 * t)));  // rough start
    const double inv_sqrt_2pi = 0.3989422804014326779;
    for (int it = 0; it < 60; ++it) {
        const double cdf = 0.5 * std::erfc(-x / std::sqrt(2.0));
        const double pdf = inv_sqrt_2pi * std::exp(-0.5 * x * x);
        const double step = (cdf - pp) / pdf;
        x -= step;
        if (std::fabs(step) < 1e-17 * std::fmax(1.0, std::fabs(x))) break;
    }
    return upper ? -x : x;
}

struct HostTables {
    float codebook[4][256];
    float threshold[4][256];
    BinEntry bins[4][kMaxBins + 1];
    int nbins[4];
    float satbias[2][8];
    // Bin count for `n - 1` thresholds: the candidate with the largest distance between any threshold and any
    // bin edge among those with at most one threshold per bin.
    void build_bins(int t, int n) {
        const int lo = (n <= 16) ? 48 : 1000, hi = (n <= 16) ? 96 : kMaxBins;
        int best_nb = 0;
        double best_clear = -1.0;
        for (int nb = lo; nb <= hi; ++nb) {
            double clear = 1e9;
            bool ok = true;
            int prev_bin = -1;
            for (int i = 0; i + 1 < n && ok; ++i) {
                const double pos = (static_cast<double>(threshold[t][i]) + 1.0) * 0.5 * nb;
                const int b = static_cast<int>(std::floor(pos));
                if (b == prev_bin) ok = false;
                prev_bin = b;
                const double d = std::fmin(pos - std::floor(pos), std::ceil(pos) - pos) * 2.0 / nb;
                clear = std::fmin(clear, d);
            }
            if (ok && clear > best_clear) { best_clear = clear; best_nb = nb; }
        }
        nbins[t] = best_nb;
        for (int k = 0; k <= kMaxBins; ++k) { bins[t][k].thr = INFINITY; bins[t][k].base = n - 1; }
        int below = 0;
        for (int k = 0; k < best_nb; ++k) {
            bins[t][k].base = below;
            bins[t][k].thr = INFINITY;
            while (below + 1 < n) {
                const double pos = (static_cast<double>(threshold[t][below]) + 1.0) * 0.5 * best_nb;
                if (static_cast<int>(std::floor(pos)) != k) break;
                bins[t][k].thr = threshold[t][below];
                ++below;
            }
        }
        bin_clearance[t] = best_clear;
    }
    double bin_clearance[4];
    HostTables() {
        const int bits[4] = {2, 3, 4, 8};
        const double delta = 0.5 * (1.0 / 30.0 + 1.0 / 32.0);
        for (int t = 0; t < 4; ++t) {
            const int b = bits[t], n = 1 << b, half = n >> 1;
            double q[256];
            // upper side first: probabilities 1/2 + (1/2 - delta) i / 2^(b-1), i = 1 .. 2^(b-1)
            for (int i = 1; i <= half; ++i)
                q[half - 1 + i] = gauss_quantile(0.5 + (0.5 - delta) * static_cast<double>(i) / half);
            q[half - 1] = 0.0;                              // probability exactly 1/2
            // lower side: delta + (1/2 - delta) i / (2^(b-1) - 1), i = 0 .. 2^(b-1) - 2
            for (int i = 0; i + 1 < half; ++i)
                q[i] = gauss_quantile(delta + (0.5 - delta) * static_cast<double>(i) / (half - 1));
            const double top = q[n - 1];
            for (int i = 0; i < 256; ++i) { codebook[t][i] = 0.0f; threshold[t][i] = INFINITY; }
            for (int i = 0; i < n; ++i) codebook[t][i] = static_cast<float>(q[i] / top);
            for (int i = 0; i + 1 < n; ++i) {
                const double mid = 0.5 * (static_cast<double>(codebook[t][i]) + static_cast<double>(codebook[t][i + 1]));
                float th = static_cast<float>(mid);
                if (static_cast<double>(th) > mid) th = std::nextafterf(th, -INFINITY);
                threshold[t][i] = th;                       // largest fp32 <= midpoint
            }
            build_bins(t, n);
        }
        for (int t = 0; t < 2; ++t)
            for (int i = 0; i < 8; ++i)
                satbias[t][i] = (i + 1 < (4 << t)) ? static_cast<float>(0.5 - static_cast<double>(threshold[t][i]) * static_cast<double>(kSatScale)) : 0.0f;
    }
};

inline const HostTables& host_tables() {
    static const HostTables t;
    return t;
}

}  // namespace detail

const float* host_codebook(int b0) { return detail::host_tables().codebook[bits_index(b0)]; }

int ensure_tables() {
    static std::mutex mu;
    static bool done[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return LQLORA_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(mu);
    if (done[dev]) return LQLORA_OK;
    const detail::HostTables& t = detail::host_tables();
    if (cudaMemcpyToSymbol(c_codebook, t.codebook, sizeof(t.codebook)) != cudaSuccess ||
        cudaMemcpyToSymbol(c_threshold, t.threshold, sizeof(t.threshold)) != cudaSuccess ||
        cudaMemcpyToSymbol(c_satbias, t.satbias, sizeof(t.satbias)) != cudaSuccess ||
        cudaMemcpyToSymbol(g_bins, t.bins, sizeof(t.bins)) != cudaSuccess ||
        cudaMemcpyToSymbol(c_nbins, t.nbins, sizeof(t.nbins)) != cudaSuccess) {
        cudaGetLastError();
        return LQLORA_ERR_CUDA;
    }
    done[dev] = true;
    return LQLORA_OK;
}

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

}  // namespace lq

extern "C" {

double lqlora_storage_bits_per_param(const lqlora_config* cfg) {
    if (lq::check_config(cfg) != LQLORA_OK) return -1.0;
    const int b2 = cfg->b2 < 0 ? -cfg->b2 : cfg->b2;
    return static_cast<double>(cfg->b0) + static_cast<double>(cfg->b1) / cfg->B0 +
           static_cast<double>(b2) / (static_cast<double>(cfg->B0) * cfg->B1);
}

int lqlora_packed_sizes(int64_t N, int64_t K, const lqlora_config* cfg, size_t* code_bytes,
                        size_t* scale_bytes, size_t* scale2_bytes, size_t* encode_workspace_bytes) {
    int rc = lq::check_config(cfg);
    if (rc != LQLORA_OK) return rc;
    rc = lq::check_shape(N, K, cfg);
    if (rc != LQLORA_OK) return rc;
    const int64_t Np = (N + lq::kTileRows - 1) / lq::kTileRows * lq::kTileRows;
    const int64_t nblk = N * K / cfg->B0;
    const int64_t ngrp = (nblk + cfg->B1 - 1) / cfg->B1;
    if (code_bytes) *code_bytes = static_cast<size_t>(Np) * K * cfg->b0 / 8;
    // scale codes: a bit stream of b1 bits each (eight codes take b1 bytes); second-level scales: 4 or 2 bytes each
    if (scale_bytes) *scale_bytes = (cfg->b1 == 8) ? static_cast<size_t>(nblk) : static_cast<size_t>((nblk + 7) / 8) * cfg->b1;
    if (scale2_bytes) *scale2_bytes = static_cast<size_t>(ngrp) * (cfg->b2 == lq::kB2Fp32 ? 4 : 2);
    // encoder scratch: the block absmax values, plus byte codes and fp32 scales before packing
    if (encode_workspace_bytes)
        *encode_workspace_bytes = (static_cast<size_t>(nblk) * sizeof(float) + 255) / 256 * 256 +
                                  (lq::packed_scales(cfg) ? (static_cast<size_t>(nblk) + 255) / 256 * 256 + static_cast<size_t>(ngrp) * 4 : 0);
    return LQLORA_OK;
}

int lqlora_nf_codebook(int b0, float* out_host) {
    if (!out_host) return LQLORA_ERR_NULL_POINTER;
    if (!(b0 == 2 || b0 == 3 || b0 == 4 || b0 == 8)) return LQLORA_ERR_INVALID_CONFIG;
    const float* cb = lq::host_codebook(b0);
    for (int i = 0; i < (1 << b0); ++i) out_host[i] = cb[i];
    return LQLORA_OK;
}

double lqlora_encode_search_clearance(int b0) {
    if (!(b0 == 2 || b0 == 3 || b0 == 4 || b0 == 8)) return -1.0;
    return lq::detail::host_tables().bin_clearance[lq::bits_index(b0)];
}

int64_t lqlora_launch_count(void) { return lq::g_launches.load(std::memory_order_relaxed); }

const char* lqlora_status_string(int status) {
    switch (status) {
        case LQLORA_OK: return "ok";
        case LQLORA_ERR_INVALID_CONFIG: return "invalid quantization configuration";
        case LQLORA_ERR_INVALID_SHAPE: return "invalid shape";
        case LQLORA_ERR_NULL_POINTER: return "null pointer";
        case LQLORA_ERR_MISALIGNED: return "pointer not 16-byte aligned";
        case LQLORA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
        case LQLORA_ERR_CUDA: return "CUDA error";
        case LQLORA_ERR_TIMEOUT: return "device-side wait timed out";
        case LQLORA_ERR_UNSUPPORTED: return "unsupported arguments";
        default: return "unknown status";
    }
}

}  // extern "C"
