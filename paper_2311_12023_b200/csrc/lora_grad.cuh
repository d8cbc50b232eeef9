// Gradients of the low-rank factors of the layer Y = X (Q + L1 L2) (Sec. 2.1, Sec. 3.1; nn.Linear orientation:
// Y = X deq(Q)^T + (X L2^T) L1^T).  By the chain rule
//     dL1 [N, r] = dY^T (X L2^T) = dY^T T,        dL2 [r, K] = (dY L1)^T X = T'^T X,
// with T = X L2^T and T' = dY L1 the same rank-r intermediates the forward pass and the input gradient use (bf16,
// from tc_lowrank_kernel).  Q takes no part: only the low-rank factors are trained.
//
// Both products have the shape  G [P, r] = sum_m A[m, P]^T T[m, r]  (A = dY, P = N  or  A = X, P = K): a long
// contraction over the tokens and a narrow output, bound by reading A once from HBM.  tc_wgrad_kernel: one CTA per
// 128 rows of G and slice of the tokens; A and T tiles come by TMA (boxes of 64 token rows x 64 columns, 128-byte
// swizzle) and enter tcgen05.mma as MN-major operands (the contraction index is the slow index of both), fp32
// accumulators in tensor memory.  The token slices of a tile form a cluster; their accumulators are sent to the CTA
// that owns the column through distributed shared memory, added there in a fixed order and written (fp32),
// transposed for dL2.
// Every wait on an mbarrier is bounded (status word LQLORA_ERR_TIMEOUT, as in the linear kernels).
#pragma once

#include "linear_tc.cuh"

namespace lq {
namespace tc {

struct WgradParams {
    float* out;            // TRANS ? [r][P] : [P][r]
    int* status;
    int M, P, r, rp;       // rp = r rounded up to 64 (MMA N)
    int steps;             // token steps of 64 in total
    int steps_per_split;
    int stages;
};

// Body for the CTA (row tile `ptile` of G, token slice `split` of `nsplit` = cluster size); tensor maps are kernel parameters.
template <bool TRANS>
__device__ __forceinline__ void wgrad_body(const CUtensorMap& tmA, const CUtensorMap& tmT, const WgradParams& p, int ptile, int split,
                                           int nsplit) {
    constexpr int A_BYTES = 16384;                 // 64 token rows x 128 columns of A
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int b_bytes = p.rp * 128;                // 64 token rows x rp columns of T
    const int stage_bytes = A_BYTES + b_bytes;
    // receive buffer of the cluster reduction: its own region (other CTAs write to it while this one may still be in
    // its main loop), rp x 128 fp32
    float* recv = reinterpret_cast<float*>(base + static_cast<size_t>(p.stages) * stage_bytes);
    uint8_t* tail = reinterpret_cast<uint8_t*>(recv) + static_cast<size_t>(p.rp) * 512;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);      // full[8], empty[8], acc_full, drain
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 160);
    volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int p0 = ptile * 128;
    const int s_lo = min(p.steps, split * p.steps_per_split);
    const int s_hi = min(p.steps, s_lo + p.steps_per_split);
    const int total = s_hi - s_lo;
    const Ctl ctl{abort_s, p.status};
    const uint32_t tmem_cols = (p.rp <= 64) ? 64u : 128u;

    auto full = [&](int s) { return smem_u32(bars + s); };
    auto empty = [&](int s) { return smem_u32(bars + 8 + s); };
    const uint32_t acc_full = smem_u32(bars + 16), drain = smem_u32(bars + 17);

    // first phase of the cluster barrier: every CTA of the cluster runs before its shared memory is written remotely
    if (nsplit > 1) dec::cluster_arrive_relaxed();
    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(full(s), 1); mbar_init(empty(s), 1); }
        mbar_init(acc_full, 1);
        mbar_init(drain, 1);
        *abort_s = 0;
        fence_barrier_init();
    }
    if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), tmem_cols); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    bool acc_ok = false;

    if (warp == 0) {
        if (lane == 0) {
            // The kernel that writes T may still be running (programmatic dependent launch): the tiles of A of the
            // first ring pass are requested at once, the tiles of T only after that kernel has finished.
            const int first = min(total, p.stages);
            for (int i = 0; i < first; ++i) {
                const uint32_t a_dst = smem_u32(base + static_cast<size_t>(i) * stage_bytes);
                const int m = (s_lo + i) * BK;               // first token row of the step (rows past M read as zero)
                mbar_expect_tx(full(i), A_BYTES + b_bytes);
                for (int t = 0; t < 2; ++t) tma_load_2d(a_dst + t * 8192, &tmA, p0 + t * 64, m, full(i));
            }
            pdl_wait();
            fence_proxy_async_all();
            for (int i = 0; i < first; ++i) {
                const uint32_t b_dst = smem_u32(base + static_cast<size_t>(i) * stage_bytes) + A_BYTES;
                const int m = (s_lo + i) * BK;
                for (int t = 0; t < p.rp / 64; ++t) tma_load_2d(b_dst + t * 8192, &tmT, t * 64, m, full(i));
            }
            for (int i = first; i < total; ++i) {
                const int s = i % p.stages;
                const uint32_t ph = (i / p.stages) & 1;
                if (!wait(empty(s), ph ^ 1, ctl, 61)) break;
                const uint32_t a_dst = smem_u32(base + static_cast<size_t>(s) * stage_bytes), b_dst = a_dst + A_BYTES;
                const int m = (s_lo + i) * BK;
                mbar_expect_tx(full(s), A_BYTES + b_bytes);
                for (int t = 0; t < 2; ++t) tma_load_2d(a_dst + t * 8192, &tmA, p0 + t * 64, m, full(s));
                for (int t = 0; t < p.rp / 64; ++t) tma_load_2d(b_dst + t * 8192, &tmT, t * 64, m, full(s));
            }
            if (*abort_s) {
                // let copies that are still in flight land before the CTA exits (bounded)
                for (int s = 0; s < p.stages; ++s) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(full(s), 0) && !mbar_try_wait(full(s), 1) && clock64() - t0 < 20000000LL) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            // fp32 accumulators, bf16 operands, both MN-major (bits 15 and 16), N = rp, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                                   (static_cast<uint32_t>(p.rp >> 3) << 17) | (static_cast<uint32_t>(128 >> 4) << 24);
            bool ok = true;
            for (int i = 0; i < total && ok; ++i) {
                const int s = i % p.stages;
                const uint32_t ph = (i / p.stages) & 1;
                ok = wait(full(s), ph, ctl, 62);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_src = smem_u32(base + static_cast<size_t>(s) * stage_bytes), b_src = a_src + A_BYTES;
#pragma unroll
                for (int k16 = 0; k16 < 4; ++k16) {
                    // 16 token rows = 2048 bytes down the tile; groups of 64 columns are 8192 bytes apart
                    const uint64_t adesc = make_desc(a_src + k16 * 2048, 8192, 1024);
                    const uint64_t bdesc = make_desc(b_src + k16 * 2048, 8192, 1024);
                    tc_mma(tmem, adesc, bdesc, idesc, (i > 0 || k16 > 0) ? 1u : 0u);
                }
                tc_commit(empty(s));
            }
            if (ok) tc_commit(acc_full);
            else {
                tc_commit(drain);
                const long long t0 = clock64();
                while (!mbar_try_wait(drain, 0) && clock64() - t0 < 20000000LL) {}
            }
        }
        __syncwarp();
    } else {
        acc_ok = (total > 0) ? wait(acc_full, 0, ctl, 63) : true;
    }
    // ---------------------------------------------------------------------- sum over the token slices
    // CTA `o` of the cluster owns columns [o * rp / nsplit, (o + 1) * rp / nsplit) of the tile.  Every CTA sends its
    // accumulators straight from tensor memory to the owners' receive buffers (remote shared-memory stores, no round
    // trip): recv[(src * cols_share + local column) * 128 + row].  After one cluster barrier every
    // CTA adds what it received, in rank order, and stores its columns.  The barriers are executed by all threads of
    // all CTAs whatever happened before.
    __syncthreads();
    if (nsplit > 1) dec::cluster_wait();                    // every CTA of the cluster has started (arrival at kernel entry)
    const uint32_t recv_addr = smem_u32(recv);
    const int cols_share = p.rp / nsplit;                   // nsplit divides 64
    if (warp >= 2 && acc_ok) {
        tc_fence_after();
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        for (int col = 0; col < p.rp; col += 32) {
            uint32_t v[32];
            if (total > 0) { tmem_ld32(tmem + (static_cast<uint32_t>(quarter * 32) << 16) + col, v); tmem_ld_wait(); }
            else {
#pragma unroll
                for (int i = 0; i < 32; ++i) v[i] = 0u;
            }
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int c = col + i;
                const int owner = c / cols_share, cl = c - owner * cols_share;
                const uint32_t off = static_cast<uint32_t>((split * cols_share + cl) * 128 + row) * 4u;
                if (nsplit > 1) dec::st_dsmem_f32(recv_addr + off, static_cast<uint32_t>(owner), __uint_as_float(v[i]));
                else recv[(cl) * 128 + row] = __uint_as_float(v[i]);
            }
        }
    }
    __syncthreads();
    if (nsplit > 1) dec::cluster_sync_all();                // everything has arrived; only local shared memory is read below
    for (int item = threadIdx.x; item < 128 * cols_share; item += 192) {
        const int row = item & 127, cl = item >> 7;
        float sum = 0.0f;
        for (int src = 0; src < nsplit; ++src) sum += recv[(src * cols_share + cl) * 128 + row];
        const int pr = p0 + row, col = split * cols_share + cl;
        if (pr < p.P && col < p.r) {
            if (TRANS) p.out[static_cast<size_t>(col) * p.P + pr] = sum;
            else p.out[static_cast<size_t>(pr) * p.r + col] = sum;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, tmem_cols);
}

// Both weight gradients of a layer in one launch: grid.z = 0 computes dL1 = dY^T T, grid.z = 1 computes dL2 = T'^T X;
// grid.x covers the larger number of row tiles (whole clusters beyond a product's own number leave at once), grid.y =
// token slices = cluster size.
__global__ void __launch_bounds__(192, 1)
tc_wgrad_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmT0, const WgradParams p0,
                const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmT1, const WgradParams p1) {
    if (blockIdx.z == 0) {
        if (static_cast<int>(blockIdx.x) * 128 < p0.P) wgrad_body<false>(tmA0, tmT0, p0, blockIdx.x, blockIdx.y, gridDim.y);
    } else {
        if (static_cast<int>(blockIdx.x) * 128 < p1.P) wgrad_body<true>(tmA1, tmT1, p1, blockIdx.x, blockIdx.y, gridDim.y);
    }
}

// Token slices of the weight-gradient kernel: as many as keep all CTAs resident in one wave, each with at least
// four steps; a power of two (it divides the 64 columns of the accumulator), at most eight.
inline int wgrad_splits(int ptiles, int steps) {
    int ns = 1;
    while (ns < 8 && static_cast<long long>(ptiles) * (2 * ns) <= sm_count() && steps / (2 * ns) >= 4) ns *= 2;
    if (ns == 8 && ptiles > 15) ns = 4;      // a cluster lives in one GPC: fewer clusters of eight fit than SMs / 8
    return ns;
}

// dL1 [N, r] = dY^T T and dL2 [r, K] = T'^T X in one launch.
inline int launch_wgrad(const void* dY, const void* X, int64_t M, int64_t N, int64_t K, const void* T, const void* Tp, int r,
                        float* dL1, float* dL2, int* status, cudaStream_t st) {
    WgradParams p0, p1;
    p0.out = dL1; p0.status = status; p0.M = static_cast<int>(M); p0.P = static_cast<int>(N); p0.r = r; p0.rp = (r <= 64) ? 64 : 128;
    p0.steps = static_cast<int>((M + BK - 1) / BK);
    const int pt0 = static_cast<int>((N + 127) / 128), pt1 = static_cast<int>((K + 127) / 128);
    const int ns = wgrad_splits(pt0 + pt1, p0.steps);
    p0.steps_per_split = (p0.steps + ns - 1) / ns;
    const int stage = 16384 + p0.rp * 128;
    const int recv_bytes = p0.rp * 512;
    int stages = (kSmemLimit - 1024 - 256 - recv_bytes) / stage;
    if (stages > 8) stages = 8;
    p0.stages = stages;
    const int smem = 1024 + stages * stage + recv_bytes + 256;
    p1 = p0;
    p1.out = dL2; p1.P = static_cast<int>(K);
    CUtensorMap tA0, tT0, tA1, tT1;
    if (!make_map(&tA0, dY, M, N, 64) || !make_map(&tT0, T, M, r, 64) || !make_map(&tA1, X, M, K, 64) || !make_map(&tT1, Tp, M, r, 64))
        return LQLORA_ERR_CUDA;
    auto kern = tc_wgrad_kernel;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess) {
            cudaGetLastError();
            return LQLORA_ERR_CUDA;
        }
        attr_done = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(pt0 > pt1 ? pt0 : pt1, ns, 2);
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = ns; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;      // overlaps the end of the pre-product kernel
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tA0, tT0, p0, tA1, tT1, p1);
    count_launch(1);
    if (e != cudaSuccess) { cudaGetLastError(); return LQLORA_ERR_CUDA; }
    return LQLORA_OK;
}

// Both pre-products in one launch (tc_lowrank_both_kernel); `nsplit` splits of the contraction = cluster size.
inline int launch_pre_both(const CUtensorMap& tA0, const CUtensorMap& tB0, PreParams p0, const CUtensorMap& tA1, const CUtensorMap& tB1,
                           PreParams p1, int nsplit, int mtiles, cudaStream_t st) {
    const int stage = 16384 + p0.rp * 128;
    const int recv_bytes = p0.rp * 512;
    int stages = (kSmemLimit - 1024 - 256 - recv_bytes) / stage;
    if (stages > 8) stages = 8;
    p0.stages = stages; p1.stages = stages;
    const int smem = 1024 + stages * stage + recv_bytes + 256;
    auto kern = tc_lowrank_both_kernel;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess) {
            cudaGetLastError();
            return LQLORA_ERR_CUDA;
        }
        attr_done = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(mtiles, nsplit, 2);
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = nsplit; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tA0, tB0, p0, tA1, tB1, p1);
    count_launch(1);
    if (e != cudaSuccess) { cudaGetLastError(); return LQLORA_ERR_CUDA; }
    return LQLORA_OK;
}

// Plan of the two rank-r pre-products of a weight-gradient call (they have the GPU to themselves).
struct GradPlan {
    int mtiles, rp, steps_x, steps_y, nsplit, sps_x, sps_y;
    size_t t_bytes;
};

inline GradPlan grad_plan(int64_t N, int64_t K, int r, int64_t M) {
    GradPlan g;
    g.mtiles = static_cast<int>((M + 127) / 128);
    g.rp = (r <= 64) ? 64 : 128;
    g.steps_x = static_cast<int>((K + BK - 1) / BK);
    g.steps_y = static_cast<int>((N + BK - 1) / BK);
    // splits of the contraction = cluster size, the same for both products: a power of two up to eight that keeps all
    // CTAs of both products resident at once and leaves every CTA at least two steps
    const int steps_min = g.steps_x < g.steps_y ? g.steps_x : g.steps_y;
    int ns = 1;
    while (ns < 8 && 2LL * g.mtiles * (2 * ns) <= sm_count() && steps_min / (2 * ns) >= 2) ns *= 2;
    if (ns == 8 && 2 * g.mtiles > 15) ns = 4;          // fewer clusters of eight fit than SMs / 8
    g.nsplit = ns;
    g.sps_x = (g.steps_x + ns - 1) / ns;
    g.sps_y = (g.steps_y + ns - 1) / ns;
    g.t_bytes = round_up(static_cast<size_t>(M) * r * 2, 256);
    return g;
}

inline size_t lora_grads_workspace(int64_t N, int64_t K, int r, int64_t M) {
    const GradPlan g = grad_plan(N, K, r, M);
    return kStatusBytes + 2 * g.t_bytes;
}

// ws: [status][T bf16][T' bf16]
inline int lora_grads_launch(const void* L1, const void* L2, int r, int64_t N, int64_t K, const void* X, const void* dY, int64_t M,
                             float* dL1, float* dL2, char* ws, cudaStream_t st) {
    const GradPlan g = grad_plan(N, K, r, M);
    int* status = reinterpret_cast<int*>(ws);          // cleared by the first kernel of the call
    __nv_bfloat16* T = reinterpret_cast<__nv_bfloat16*>(ws + kStatusBytes);
    __nv_bfloat16* Tp = reinterpret_cast<__nv_bfloat16*>(ws + kStatusBytes + g.t_bytes);
    CUtensorMap tA0, tB0, tA1, tB1;
    if (!make_map(&tA0, X, M, K, 128) || !make_map(&tB0, L2, r, K, g.rp)) return LQLORA_ERR_CUDA;        // T = X L2^T
    if (!make_map(&tA1, dY, M, N, 128) || !make_map(&tB1, L1, N, r, 64)) return LQLORA_ERR_CUDA;         // T' = dY L1
    PreParams p0, p1;
    p0.T = T; p0.status = status;
    p0.M = static_cast<int>(M); p0.r = r; p0.rp = g.rp; p0.steps = g.steps_x; p0.steps_per_split = g.sps_x; p0.stages = 0; p0.clear_status = 1;
    p1 = p0;
    p1.T = Tp; p1.steps = g.steps_y; p1.steps_per_split = g.sps_y; p1.clear_status = 0;
    const int rc = launch_pre_both(tA0, tB0, p0, tA1, tB1, p1, g.nsplit, g.mtiles, st);
    if (rc != LQLORA_OK) return rc;
    return launch_wgrad(dY, X, M, N, K, T, Tp, r, dL1, dL2, status, st);
}

}  // namespace tc
}  // namespace lq
