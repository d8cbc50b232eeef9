// C ABI of the LQ-LoRA library: argument validation, dispatch, launches.
// Single translation unit: the kernels live in the headers included below.
#include "../../include/lqlora.h"

#include "common.cuh"
#include "tables.cuh"
#include "codec.cuh"
#include "linear_decode.cuh"
#include "linear_small.cuh"
#include "linear_tc.cuh"
#include "lora_grad.cuh"
#include "lq_decompose.cuh"
#include "config_search.cuh"

namespace lq {

static int check_qmatrix(const lqlora_qmatrix* q) {
    if (!q) return LQLORA_ERR_NULL_POINTER;
    int rc = check_config(&q->cfg);
    if (rc != LQLORA_OK) return rc;
    rc = check_shape(q->N, q->K, &q->cfg);
    if (rc != LQLORA_OK) return rc;
    if (!q->codes || !q->scale_codes || !q->scale2) return LQLORA_ERR_NULL_POINTER;
    if (!aligned16(q->codes) || !aligned16(q->scale_codes) || !aligned16(q->scale2)) return LQLORA_ERR_MISALIGNED;
    return LQLORA_OK;
}

static int cuda_rc(cudaError_t e) {
    if (e == cudaSuccess) return LQLORA_OK;
    cudaGetLastError();
    return LQLORA_ERR_CUDA;
}

// Scratch bytes one direction of the linear needs for M rows, for the kernel family it dispatches to.
static size_t linear_need_base(const QView& v, int r, int64_t M, bool backward) {
    if (tc_supported(v, r, M, backward)) return tc_workspace_bytes(v.N, v.K, r, M, backward);
    if (backward ? dec::bwd_supported(v, M) : dec::supported(v, M)) return dec::workspace_bytes(v, r, static_cast<int>(M), backward);
    const SmallPlan p = small_plan(v.N, v.K, r, M, backward);
    return kStatusBytes + p.t_bytes + p.p_bytes;
}
// ... plus, for matrices whose scales are stored packed (b1 < 8) or in 16 bits, room for their expanded copy
static size_t linear_need(const lqlora_qmatrix* q, int r, int64_t M, bool backward) {
    const size_t base = (linear_need_base(make_view(q), r, M, backward) + 255) / 256 * 256;
    return base + expanded_scale_bytes(q->N, q->K, &q->cfg);
}

static int check_linear(const lqlora_qmatrix* q, const void* L1, const void* L2, int r, const void* A, int64_t M,
                        void* out, void* ws, size_t ws_bytes, bool backward) {
    int rc = check_qmatrix(q);
    if (rc != LQLORA_OK) return rc;
    if (M <= 0 || M > (int64_t(1) << 24)) return LQLORA_ERR_INVALID_SHAPE;
    if (r < 0 || r > 128 || (r % 16) != 0) return LQLORA_ERR_INVALID_SHAPE;
    if (!A || !out || !ws) return LQLORA_ERR_NULL_POINTER;
    if (r > 0 && (!L1 || !L2)) return LQLORA_ERR_NULL_POINTER;
    if (!aligned16(A) || !aligned16(out) || !aligned16(ws) || !aligned16(L1) || !aligned16(L2)) return LQLORA_ERR_MISALIGNED;
    if ((backward ? q->N : q->K) % 8 != 0 || (backward ? q->K : q->N) % 8 != 0) {
        // rows of X / Y must start on 16-byte boundaries for the vector loads and TMA
        if (M > 1) return LQLORA_ERR_INVALID_SHAPE;
    }
    if (ws_bytes < linear_need(q, r, M, backward)) return LQLORA_ERR_WORKSPACE_TOO_SMALL;
    return LQLORA_OK;
}

static int run_linear(const lqlora_qmatrix* q, const void* L1, const void* L2, int r, const void* A, int64_t M,
                      void* out, void* ws, size_t ws_bytes, void* stream, bool backward) {
    int rc = check_linear(q, L1, L2, r, A, M, out, ws, ws_bytes, backward);
    if (rc != LQLORA_OK) return rc;
    rc = ensure_tables();
    if (rc != LQLORA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    QView v = make_view(q);
    if (packed_scales(&q->cfg)) {
        // scales stored packed or in 16 bits: the kernels read an expanded copy behind the call's own scratch
        const size_t base = (linear_need_base(v, r, M, backward) + 255) / 256 * 256;
        if (expand_scales(q, &v, static_cast<char*>(ws) + base, st) != cudaSuccess) return cuda_rc(cudaGetLastError());
    }
    const bool use_tc = tc_supported(v, r, M, backward);
    const bool use_decode = !use_tc && (backward ? dec::bwd_supported(v, M) : dec::supported(v, M));
    // With a rank-r term the first kernel of the call (the pre-product) clears what has to start at zero (the status
    // word, and the arrival counters of the weight-streaming kernels); otherwise a memset does.
    const bool first_kernel_clears = r > 0 && (use_decode || use_tc);
    if (!first_kernel_clears) {
        const size_t n = use_decode ? dec::clear_bytes(v, backward) : static_cast<size_t>(kStatusBytes);
        if (cudaMemsetAsync(ws, 0, n, st) != cudaSuccess) return cuda_rc(cudaGetLastError());
    }
    cudaError_t e = cudaSuccess;
    if (use_tc) {
        return tc_launch(v, L1, L2, r, A, static_cast<int>(M), out, static_cast<char*>(ws), backward, st);
    }
    if (use_decode) {
        char* w = static_cast<char*>(ws);
        const int m = static_cast<int>(M);
        if (!backward) {
            switch (v.b0) {
                case 2: e = dec::launch_fwd<2>(v, L1, L2, r, A, m, out, w, st); break;
                case 3: e = dec::launch_fwd<3>(v, L1, L2, r, A, m, out, w, st); break;
                case 4: e = dec::launch_fwd<4>(v, L1, L2, r, A, m, out, w, st); break;
                default: e = dec::launch_fwd<8>(v, L1, L2, r, A, m, out, w, st); break;
            }
        } else {
            switch (v.b0) {
                case 2: e = dec::launch_bwd<2>(v, L1, L2, r, A, m, out, w, st); break;
                case 3: e = dec::launch_bwd<3>(v, L1, L2, r, A, m, out, w, st); break;
                case 4: e = dec::launch_bwd<4>(v, L1, L2, r, A, m, out, w, st); break;
                default: e = dec::launch_bwd<8>(v, L1, L2, r, A, m, out, w, st); break;
            }
        }
        return cuda_rc(e);
    }
    switch (v.b0) {
        case 2: e = launch_small<2>(v, L1, L2, r, A, static_cast<int>(M), out, static_cast<char*>(ws), backward, st); break;
        case 3: e = launch_small<3>(v, L1, L2, r, A, static_cast<int>(M), out, static_cast<char*>(ws), backward, st); break;
        case 4: e = launch_small<4>(v, L1, L2, r, A, static_cast<int>(M), out, static_cast<char*>(ws), backward, st); break;
        default: e = launch_small<8>(v, L1, L2, r, A, static_cast<int>(M), out, static_cast<char*>(ws), backward, st); break;
    }
    return cuda_rc(e);
}


// ---------------------------------------------------------------------------------------
// Built-in scratch for lqlora_linear_fwd_static.  The array lives in every device's copy of
// the module from the moment the library is loaded there until the process exits.
// In host code the name `g_static_scratch` is only a handle for the symbol, not a device
// address; the address is looked up once per device (with that device current) below.
// ---------------------------------------------------------------------------------------
constexpr size_t kStaticScratchBytes = size_t(8) << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

static int static_scratch_ptr(void** out) {
    static std::mutex mu;
    static void* ptrs[64] = {};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return LQLORA_ERR_CUDA; }
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return LQLORA_ERR_CUDA; }
        ptrs[dev] = p;
    }
    *out = ptrs[dev];
    return LQLORA_OK;
}

// Self-test of the bounded waits: a CTA arms an mbarrier for bytes that nobody delivers and waits on it with the same
// helper (and the same status word) as the linear kernels, holding a tensor-memory allocation meanwhile; when the
// budget runs out the wait is abandoned, the status word is set, tensor memory is freed and the kernel returns.
__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(int* status, long long budget) {
    __shared__ uint64_t bar;
    __shared__ uint32_t tmem_slot;
    __shared__ int abort_s;
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        dev::mbar_init(dev::smem_u32(&bar), 1);
        abort_s = 0;
        dev::fence_barrier_init();
    }
    if (warp == 1) { tc::tmem_alloc(dev::smem_u32(&tmem_slot), 32); tc::tmem_relinquish(); }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = tmem_slot;
    if (threadIdx.x == 0) {
        dev::Ctl ctl{&abort_s, status, budget};
        dev::mbar_expect_tx(dev::smem_u32(&bar), 128);           // 128 bytes that never arrive
        dev::wait(dev::smem_u32(&bar), 0, ctl, 99);
    }
    tc::tc_fence_before();
    __syncthreads();
    if (warp == 1) tc::tmem_dealloc(tmem, 32);
}

}  // namespace lq

extern "C" {

int lqlora_selftest_bounded_wait(void* workspace_dev, int64_t budget_cycles, void* stream) {
    if (!workspace_dev) return LQLORA_ERR_NULL_POINTER;
    if (budget_cycles < 1000 || budget_cycles > 2000000000LL) return LQLORA_ERR_INVALID_SHAPE;     // at most about a second
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace_dev, 0, lq::kStatusBytes, st) != cudaSuccess) return lq::cuda_rc(cudaGetLastError());
    lq::bounded_wait_selftest_kernel<<<1, 64, 0, st>>>(static_cast<int*>(workspace_dev), budget_cycles);
    lq::count_launch(1);
    return lq::cuda_rc(cudaGetLastError());
}

int lqlora_encode(const float* W_dev, lqlora_qmatrix* out, void* workspace_dev, size_t workspace_bytes, void* stream) {
    using namespace lq;
    if (!W_dev || !workspace_dev) return LQLORA_ERR_NULL_POINTER;
    int rc = check_qmatrix(out);
    if (rc != LQLORA_OK) return rc;
    if (!aligned16(W_dev) || !aligned16(workspace_dev)) return LQLORA_ERR_MISALIGNED;
    size_t need = 0;
    lqlora_packed_sizes(out->N, out->K, &out->cfg, nullptr, nullptr, nullptr, &need);
    if (workspace_bytes < need) return LQLORA_ERR_WORKSPACE_TOO_SMALL;
    rc = ensure_tables();
    if (rc != LQLORA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    float* absmax = static_cast<float*>(workspace_dev);
    cudaError_t e;
    switch (out->cfg.b0) {
        case 2: e = launch_encode<2>(W_dev, out, absmax, st); break;
        case 3: e = launch_encode<3>(W_dev, out, absmax, st); break;
        case 4: e = launch_encode<4>(W_dev, out, absmax, st); break;
        default: e = launch_encode<8>(W_dev, out, absmax, st); break;
    }
    return cuda_rc(e);
}

int lqlora_unpack(const lqlora_qmatrix* q, uint8_t* codes_dev, void* stream) {
    using namespace lq;
    int rc = check_qmatrix(q);
    if (rc != LQLORA_OK) return rc;
    if (!codes_dev) return LQLORA_ERR_NULL_POINTER;
    rc = ensure_tables();
    if (rc != LQLORA_OK) return rc;
    const QView v = make_view(q);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    switch (v.b0) {
        case 2: e = launch_export<2>(v, codes_dev, nullptr, nullptr, st); break;
        case 3: e = launch_export<3>(v, codes_dev, nullptr, nullptr, st); break;
        case 4: e = launch_export<4>(v, codes_dev, nullptr, nullptr, st); break;
        default: e = launch_export<8>(v, codes_dev, nullptr, nullptr, st); break;
    }
    return cuda_rc(e);
}

int lqlora_dequant(const lqlora_qmatrix* q, float* deq32_dev, void* deq16_dev, void* stream) {
    using namespace lq;
    int rc = check_qmatrix(q);
    if (rc != LQLORA_OK) return rc;
    if (!deq32_dev && !deq16_dev) return LQLORA_ERR_NULL_POINTER;
    rc = ensure_tables();
    if (rc != LQLORA_OK) return rc;
    const QView v = make_view(q);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaError_t e;
    switch (v.b0) {
        case 2: e = launch_export<2>(v, nullptr, deq32_dev, deq16_dev, st); break;
        case 3: e = launch_export<3>(v, nullptr, deq32_dev, deq16_dev, st); break;
        case 4: e = launch_export<4>(v, nullptr, deq32_dev, deq16_dev, st); break;
        default: e = launch_export<8>(v, nullptr, deq32_dev, deq16_dev, st); break;
    }
    return cuda_rc(e);
}

int lqlora_unpack_scales(const lqlora_qmatrix* q, uint8_t* scale_codes_dev, float* scale2_dev, void* stream) {
    using namespace lq;
    int rc = check_qmatrix(q);
    if (rc != LQLORA_OK) return rc;
    if (!scale_codes_dev || !scale2_dev) return LQLORA_ERR_NULL_POINTER;
    const long long nblk = static_cast<long long>(q->N) * q->K / q->cfg.B0, ngrp = (nblk + q->cfg.B1 - 1) / q->cfg.B1;
    const long long threads = (nblk + 7) / 8 > ngrp ? (nblk + 7) / 8 : ngrp;
    expand_scales_kernel<<<static_cast<unsigned>((threads + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        q->scale_codes, q->scale2, scale_codes_dev, scale2_dev, nblk, ngrp, q->cfg.b1, q->cfg.b2);
    count_launch(1);
    return cuda_rc(cudaGetLastError());
}

// Layer with quantized factors (the compression setting of Sec. 4.2: L1, L2 stored in NF-8 after training): the two
// factors are dequantized to bf16 into the tail of the workspace, then the ordinary path runs.
static int run_linear_qfactors(const lqlora_qmatrix* q, const lqlora_qmatrix* qL1, const lqlora_qmatrix* qL2, const void* A,
                               int64_t M, void* out, void* ws, size_t ws_bytes, void* stream, bool backward) {
    using namespace lq;
    int rc = check_qmatrix(q);
    if (rc == LQLORA_OK) rc = check_qmatrix(qL1);
    if (rc == LQLORA_OK) rc = check_qmatrix(qL2);
    if (rc != LQLORA_OK) return rc;
    const int64_t r = qL1->K;
    if (qL1->N != q->N || qL2->N != r || qL2->K != q->K || r > 128 || r % 16 != 0) return LQLORA_ERR_INVALID_SHAPE;
    if (!ws || !aligned16(ws)) return ws ? LQLORA_ERR_MISALIGNED : LQLORA_ERR_NULL_POINTER;
    if (M <= 0 || M > (int64_t(1) << 24)) return LQLORA_ERR_INVALID_SHAPE;
    const size_t base = (linear_need(q, static_cast<int>(r), M, backward) + 255) / 256 * 256;
    const size_t l1_bytes = (static_cast<size_t>(q->N) * r * 2 + 255) / 256 * 256, l2_bytes = (static_cast<size_t>(r) * q->K * 2 + 255) / 256 * 256;
    if (ws_bytes < base + l1_bytes + l2_bytes) return LQLORA_ERR_WORKSPACE_TOO_SMALL;
    rc = ensure_tables();
    if (rc != LQLORA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* w = static_cast<char*>(ws);
    void* L1 = w + base;
    void* L2 = w + base + l1_bytes;
    const lqlora_qmatrix* fs[2] = {qL1, qL2};
    void* dst[2] = {L1, L2};
    for (int i = 0; i < 2; ++i) {
        const QView v = make_view(fs[i]);
        cudaError_t e;
        switch (v.b0) {
            case 2: e = launch_export<2>(v, nullptr, nullptr, dst[i], st); break;
            case 3: e = launch_export<3>(v, nullptr, nullptr, dst[i], st); break;
            case 4: e = launch_export<4>(v, nullptr, nullptr, dst[i], st); break;
            default: e = launch_export<8>(v, nullptr, nullptr, dst[i], st); break;
        }
        if (e != cudaSuccess) return cuda_rc(e);
    }
    return run_linear(q, L1, L2, static_cast<int>(r), A, M, out, ws, base, stream, backward);
}

int lqlora_linear_qfactors_workspace_bytes(int64_t N, int64_t K, const lqlora_config* cfg, int r, int64_t M, size_t* bytes) {
    size_t base = 0;
    const int rc = lqlora_linear_workspace_bytes(N, K, cfg, r, M, &base);
    if (rc != LQLORA_OK) return rc;
    *bytes = (base + 255) / 256 * 256 + (static_cast<size_t>(N) * r * 2 + 255) / 256 * 256 + (static_cast<size_t>(r) * K * 2 + 255) / 256 * 256;
    return LQLORA_OK;
}

int lqlora_linear_fwd_qfactors(const lqlora_qmatrix* q, const lqlora_qmatrix* qL1, const lqlora_qmatrix* qL2, const void* X_dev,
                               int64_t M, void* Y_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
    return run_linear_qfactors(q, qL1, qL2, X_dev, M, Y_dev, workspace_dev, workspace_bytes, stream, false);
}

int lqlora_linear_bwd_input_qfactors(const lqlora_qmatrix* q, const lqlora_qmatrix* qL1, const lqlora_qmatrix* qL2, const void* dY_dev,
                                     int64_t M, void* dX_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
    return run_linear_qfactors(q, qL1, qL2, dY_dev, M, dX_dev, workspace_dev, workspace_bytes, stream, true);
}

int lqlora_linear_workspace_bytes(int64_t N, int64_t K, const lqlora_config* cfg, int r, int64_t M, size_t* bytes) {
    using namespace lq;
    int rc = check_config(cfg);
    if (rc != LQLORA_OK) return rc;
    rc = check_shape(N, K, cfg);
    if (rc != LQLORA_OK) return rc;
    if (M <= 0 || r < 0 || r > 128 || r % 16) return LQLORA_ERR_INVALID_SHAPE;
    if (!bytes) return LQLORA_ERR_NULL_POINTER;
    // the same workspace must serve the forward and the input gradient
    lqlora_qmatrix q{};
    q.N = N; q.K = K; q.cfg = *cfg;
    const size_t f = linear_need(&q, r, M, false), b = linear_need(&q, r, M, true);
    const size_t need = f > b ? f : b;
    *bytes = need;
    return LQLORA_OK;
}

int lqlora_linear_fwd(const lqlora_qmatrix* q, const void* L1_dev, const void* L2_dev, int r, const void* X_dev,
                      int64_t M, void* Y_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
    return lq::run_linear(q, L1_dev, L2_dev, r, X_dev, M, Y_dev, workspace_dev, workspace_bytes, stream, false);
}

int lqlora_linear_bwd_input(const lqlora_qmatrix* q, const void* L1_dev, const void* L2_dev, int r, const void* dY_dev,
                            int64_t M, void* dX_dev, void* workspace_dev, size_t workspace_bytes, void* stream) {
    return lq::run_linear(q, L1_dev, L2_dev, r, dY_dev, M, dX_dev, workspace_dev, workspace_bytes, stream, true);
}

size_t lqlora_static_scratch_bytes(void) { return lq::kStaticScratchBytes; }

int lqlora_linear_fwd_static(const lqlora_qmatrix* q, const void* L1_dev, const void* L2_dev, int r, const void* X_dev,
                             int64_t M, void* Y_dev, void* stream) {
    using namespace lq;
    // size check first: nothing is looked up or enqueued for a problem that cannot fit
    int rc = check_qmatrix(q);
    if (rc != LQLORA_OK) return rc;
    if (M <= 0 || M > (int64_t(1) << 24) || r < 0 || r > 128 || (r % 16) != 0) return LQLORA_ERR_INVALID_SHAPE;
    if (linear_need(q, r, M, false) > kStaticScratchBytes) return LQLORA_ERR_WORKSPACE_TOO_SMALL;
    void* scratch = nullptr;
    rc = static_scratch_ptr(&scratch);
    if (rc != LQLORA_OK) return rc;
    // the first kernel of the call (or run_linear's memset) clears the status word at the head of the scratch;
    // nothing else of what the previous call left behind is read before it is overwritten
    return run_linear(q, L1_dev, L2_dev, r, X_dev, M, Y_dev, scratch, kStaticScratchBytes, stream, false);
}

int lqlora_static_scratch_status(void* stream) {
    void* scratch = nullptr;
    const int rc = lq::static_scratch_ptr(&scratch);
    if (rc != LQLORA_OK) return rc;
    return lqlora_workspace_status(scratch, stream);
}

static int check_lora_grads(int64_t N, int64_t K, int r, int64_t M) {
    if (N <= 0 || K <= 0 || N > (int64_t(1) << 30) || K > (int64_t(1) << 30) || (N % 8) != 0 || (K % 8) != 0) return LQLORA_ERR_INVALID_SHAPE;
    if (M <= 0 || M > (int64_t(1) << 24)) return LQLORA_ERR_INVALID_SHAPE;
    if (r < 16 || r > 128 || (r % 16) != 0) return LQLORA_ERR_INVALID_SHAPE;
    return LQLORA_OK;
}

int lqlora_lora_grads_workspace_bytes(int64_t N, int64_t K, int r, int64_t M, size_t* bytes) {
    if (!bytes) return LQLORA_ERR_NULL_POINTER;
    const int rc = check_lora_grads(N, K, r, M);
    if (rc != LQLORA_OK) return rc;
    *bytes = lq::tc::lora_grads_workspace(N, K, r, M);
    return LQLORA_OK;
}

int lqlora_lora_grads(const void* L1_dev, const void* L2_dev, int r, int64_t N, int64_t K, const void* X_dev,
                      const void* dY_dev, int64_t M, float* dL1_dev, float* dL2_dev, void* workspace_dev,
                      size_t workspace_bytes, void* stream) {
    using namespace lq;
    const int rc = check_lora_grads(N, K, r, M);
    if (rc != LQLORA_OK) return rc;
    if (!L1_dev || !L2_dev || !X_dev || !dY_dev || !dL1_dev || !dL2_dev || !workspace_dev) return LQLORA_ERR_NULL_POINTER;
    if (!aligned16(L1_dev) || !aligned16(L2_dev) || !aligned16(X_dev) || !aligned16(dY_dev) || !aligned16(dL1_dev) ||
        !aligned16(dL2_dev) || !aligned16(workspace_dev))
        return LQLORA_ERR_MISALIGNED;
    if (workspace_bytes < tc::lora_grads_workspace(N, K, r, M)) return LQLORA_ERR_WORKSPACE_TOO_SMALL;
    return tc::lora_grads_launch(L1_dev, L2_dev, r, N, K, X_dev, dY_dev, M, dL1_dev, dL2_dev, static_cast<char*>(workspace_dev),
                                 static_cast<cudaStream_t>(stream));
}

int lqlora_linear_intermediate_offset(int64_t N, int64_t K, const lqlora_config* cfg, int r, int64_t M, int backward, size_t* offset) {
    using namespace lq;
    if (!offset) return LQLORA_ERR_NULL_POINTER;
    if (check_config(cfg) != LQLORA_OK || check_shape(N, K, cfg) != LQLORA_OK) return LQLORA_ERR_INVALID_CONFIG;
    if (M <= 0 || r <= 0 || r > 128 || r % 16) return LQLORA_ERR_INVALID_SHAPE;
    lqlora_qmatrix q{};
    q.N = N; q.K = K; q.cfg = *cfg;
    const QView v = make_view(&q);
    const bool bwd = backward != 0;
    // the tensor-core and the plain kernels keep [status][T]; the weight-streaming kernels [status][arrival counters][T]
    size_t off = kStatusBytes;
    if (!tc_supported(v, r, M, bwd) && (bwd ? dec::bwd_supported(v, M) : dec::supported(v, M))) off = dec::clear_bytes(v, bwd);
    *offset = off;
    return LQLORA_OK;
}

int lqlora_lora_grads_from(const void* T_dev, const void* Tp_dev, int r, int64_t N, int64_t K, const void* X_dev,
                           const void* dY_dev, int64_t M, float* dL1_dev, float* dL2_dev, void* workspace_dev,
                           size_t workspace_bytes, void* stream) {
    using namespace lq;
    const int rc = check_lora_grads(N, K, r, M);
    if (rc != LQLORA_OK) return rc;
    if (!T_dev || !Tp_dev || !X_dev || !dY_dev || !dL1_dev || !dL2_dev || !workspace_dev) return LQLORA_ERR_NULL_POINTER;
    if (!aligned16(T_dev) || !aligned16(Tp_dev) || !aligned16(X_dev) || !aligned16(dY_dev) || !aligned16(dL1_dev) ||
        !aligned16(dL2_dev) || !aligned16(workspace_dev))
        return LQLORA_ERR_MISALIGNED;
    if (workspace_bytes < static_cast<size_t>(kStatusBytes)) return LQLORA_ERR_WORKSPACE_TOO_SMALL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(workspace_dev, 0, kStatusBytes, st) != cudaSuccess) return cuda_rc(cudaGetLastError());
    return tc::launch_wgrad(dY_dev, X_dev, M, N, K, T_dev, Tp_dev, r, dL1_dev, dL2_dev, static_cast<int*>(workspace_dev), st);
}

int lqlora_lq_workspace_bytes(int64_t N, int64_t K, const lqlora_config* cfg, int r, int oversample, size_t* bytes) {
    using namespace lq;
    int rc = check_config(cfg);
    if (rc != LQLORA_OK) return rc;
    rc = check_shape(N, K, cfg);
    if (rc != LQLORA_OK) return rc;
    if (r < 1 || r > 128 || oversample < 0 || oversample > 64 || r + oversample > N || r + oversample > K) return LQLORA_ERR_INVALID_SHAPE;
    if (!bytes) return LQLORA_ERR_NULL_POINTER;
    *bytes = lqd::workspace_bytes(N, K, cfg, r, oversample);
    return LQLORA_OK;
}

int lqlora_lq_decompose(const float* W_dev, const float* F_dev, lqlora_qmatrix* out, float* L1_dev, float* L2_dev, int r,
                        int max_steps, const float* omega_dev, int oversample, int power_iters, double* errors_host,
                        int* steps_taken, void* workspace_dev, size_t workspace_bytes, void* stream) {
    using namespace lq;
    if (!W_dev || !L1_dev || !L2_dev || !omega_dev || !errors_host || !steps_taken || !workspace_dev) return LQLORA_ERR_NULL_POINTER;
    int rc = check_qmatrix(out);
    if (rc != LQLORA_OK) return rc;
    if (r < 1 || r > 128 || oversample < 0 || oversample > 64 || r + oversample > out->N || r + oversample > out->K) return LQLORA_ERR_INVALID_SHAPE;
    if (max_steps < 1 || max_steps > 1000 || power_iters < 0 || power_iters > 16) return LQLORA_ERR_INVALID_SHAPE;
    if (!aligned16(W_dev) || !aligned16(L1_dev) || !aligned16(L2_dev) || !aligned16(omega_dev) || !aligned16(workspace_dev) ||
        (F_dev && !aligned16(F_dev)))
        return LQLORA_ERR_MISALIGNED;
    if (workspace_bytes < lqd::workspace_bytes(out->N, out->K, &out->cfg, r, oversample)) return LQLORA_ERR_WORKSPACE_TOO_SMALL;
    rc = ensure_tables();
    if (rc != LQLORA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    char* ws = static_cast<char*>(workspace_dev);
    *steps_taken = 0;
    switch (out->cfg.b0) {
        case 2: return lqd::run<2>(W_dev, F_dev, out, L1_dev, L2_dev, r, max_steps, omega_dev, oversample, power_iters, errors_host, steps_taken, ws, st);
        case 3: return lqd::run<3>(W_dev, F_dev, out, L1_dev, L2_dev, r, max_steps, omega_dev, oversample, power_iters, errors_host, steps_taken, ws, st);
        case 4: return lqd::run<4>(W_dev, F_dev, out, L1_dev, L2_dev, r, max_steps, omega_dev, oversample, power_iters, errors_host, steps_taken, ws, st);
        default: return lqd::run<8>(W_dev, F_dev, out, L1_dev, L2_dev, r, max_steps, omega_dev, oversample, power_iters, errors_host, steps_taken, ws, st);
    }
}

int lqlora_to_bf16(const float* x_dev, void* y_dev, int64_t n, void* stream) {
    if (!x_dev || !y_dev) return LQLORA_ERR_NULL_POINTER;
    if (n <= 0) return LQLORA_ERR_INVALID_SHAPE;
    lq::lqd::to_bf16_kernel<<<static_cast<unsigned>((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(stream)>>>(
        x_dev, static_cast<__nv_bfloat16*>(y_dev), n);
    lq::count_launch(1);
    return lq::cuda_rc(cudaGetLastError());
}

int lqlora_assign_configs(const double* errors, const double* storage, int n_matrices, int n_configs, double budget,
                          int* assignment, double* total_error, double* total_storage) {
    if (!errors || !storage || !assignment) return LQLORA_ERR_NULL_POINTER;
    if (n_matrices < 1 || n_configs < 1) return LQLORA_ERR_INVALID_SHAPE;
    return lq::cfgsearch::assign(errors, storage, n_matrices, n_configs, budget, assignment, total_error, total_storage) == 0
               ? LQLORA_OK : LQLORA_ERR_UNSUPPORTED;
}

int lqlora_encode_host(const float* W_host, float* W_stage_dev, lqlora_qmatrix* out, void* workspace_dev,
                       size_t workspace_bytes, void* stream) {
    if (!W_host || !W_stage_dev || !out) return LQLORA_ERR_NULL_POINTER;
    int rc = lq::check_qmatrix(out);
    if (rc != LQLORA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(W_stage_dev, W_host, sizeof(float) * out->N * out->K, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return lq::cuda_rc(cudaGetLastError());
    return lqlora_encode(W_stage_dev, out, workspace_dev, workspace_bytes, stream);
}

static int linear_host(const lqlora_qmatrix* q, const void* L1, const void* L2, int r, const void* A_host, int64_t M,
                       void* out_host, void* A_stage, void* out_stage, void* ws, size_t ws_bytes, void* stream, bool backward) {
    if (!A_host || !out_host) return LQLORA_ERR_NULL_POINTER;
    int rc = lq::check_linear(q, L1, L2, r, A_stage, M, out_stage, ws, ws_bytes, backward);
    if (rc != LQLORA_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t in_bytes = static_cast<size_t>(M) * (backward ? q->N : q->K) * 2;
    const size_t out_bytes = static_cast<size_t>(M) * (backward ? q->K : q->N) * 2;
    if (cudaMemcpyAsync(A_stage, A_host, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return lq::cuda_rc(cudaGetLastError());
    rc = lq::run_linear(q, L1, L2, r, A_stage, M, out_stage, ws, ws_bytes, stream, backward);
    if (rc != LQLORA_OK) return rc;
    if (cudaMemcpyAsync(out_host, out_stage, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) return lq::cuda_rc(cudaGetLastError());
    return LQLORA_OK;
}

int lqlora_linear_fwd_host(const lqlora_qmatrix* q, const void* L1_dev, const void* L2_dev, int r, const void* X_host,
                           int64_t M, void* Y_host, void* X_stage_dev, void* Y_stage_dev, void* workspace_dev,
                           size_t workspace_bytes, void* stream) {
    return linear_host(q, L1_dev, L2_dev, r, X_host, M, Y_host, X_stage_dev, Y_stage_dev, workspace_dev, workspace_bytes, stream, false);
}

int lqlora_linear_bwd_input_host(const lqlora_qmatrix* q, const void* L1_dev, const void* L2_dev, int r, const void* dY_host,
                                 int64_t M, void* dX_host, void* dY_stage_dev, void* dX_stage_dev, void* workspace_dev,
                                 size_t workspace_bytes, void* stream) {
    return linear_host(q, L1_dev, L2_dev, r, dY_host, M, dX_host, dY_stage_dev, dX_stage_dev, workspace_dev, workspace_bytes, stream, true);
}

int lqlora_workspace_status(const void* workspace_dev, void* stream) {
    if (!workspace_dev) return LQLORA_ERR_NULL_POINTER;
    int word = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(&word, workspace_dev, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) {
        cudaGetLastError();
        return LQLORA_ERR_CUDA;
    }
    return word == 0 ? LQLORA_OK : LQLORA_ERR_TIMEOUT;
}

int lqlora_linear_path(int64_t N, int64_t K, const lqlora_config* cfg, int r, int64_t M, int backward, int* splits) {
    using namespace lq;
    if (check_config(cfg) != LQLORA_OK || check_shape(N, K, cfg) != LQLORA_OK) return LQLORA_ERR_INVALID_CONFIG;
    if (M <= 0 || r < 0 || r > 128 || r % 16) return LQLORA_ERR_INVALID_SHAPE;
    lqlora_qmatrix q{};
    q.N = N; q.K = K; q.cfg = *cfg;
    const QView v = make_view(&q);
    const bool bwd = backward != 0;
    int kernel = LQLORA_PATH_PLAIN, ks = 1;
    if (tc_supported(v, r, M, bwd)) {
        const int64_t out_cols = bwd ? K : N;
        const int steps_q = static_cast<int>(((bwd ? N : K) + tc::BK - 1) / tc::BK);
        if (tc::tc_use_pair(M, out_cols, tc::sm_count())) kernel = LQLORA_PATH_TC_PAIR;
        else { kernel = LQLORA_PATH_TC_ONE; ks = tc::tc_ksplit(M, out_cols, steps_q, tc::sm_count()); }
    } else if (bwd ? dec::bwd_supported(v, M) : dec::supported(v, M)) {
        kernel = LQLORA_PATH_STREAM;
        ks = bwd ? dec::bwd_splits(v, static_cast<int>(M)) : dec::fwd_splits(v, static_cast<int>(M));
    }
    if (splits) *splits = ks;
    return kernel;
}

}  // extern "C"
