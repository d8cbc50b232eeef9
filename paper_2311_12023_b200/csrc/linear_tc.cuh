// Tensor-core path for many rows of X (training-sized M) on sm_100a.
//
// One CTA computes a [MH*128, 256] tile of the output.  Per pipeline step of 64 contraction
// elements:
//   - a producer thread issues a TMA tile load of the bf16 activations (128-byte swizzle) and
//     bulk copies of the packed code slabs into shared memory;
//   - eight dequantization warps unpack the codes, multiply by the block scale in fp32, round to
//     bf16 and write the weight tile into shared memory in the 128-byte-swizzled layout that the
//     tensor core reads (one thread = one weight row);
//   - one thread issues tcgen05.mma (M = 128, N = 256, K = 16) with fp32 accumulators in tensor
//     memory and commits the stage back to the producer.
// The rank-r term is folded in as extra contraction steps whose two operands come by TMA
// (forward: [X L2^T | L1]; backward: [dY L1 | L2]).  The epilogue reads the accumulators with
// tcgen05.ld, rounds to bf16 and stores.
//
// The same shared-memory weight tile ([rows of Q] x 64 columns, 128 bytes per row, swizzled)
// serves both passes: the forward reads it as a K-major B operand (contraction along the row),
// the input gradient as an MN-major B operand (contraction across rows).
//
// Every wait on an mbarrier is bounded; when a wait expires the kernel records it in the status
// word of the workspace, stops issuing work, lets its copies land, frees its tensor memory and
// returns (lqlora_workspace_status then reports LQLORA_ERR_TIMEOUT).
#pragma once

#include <cuda.h>   // CUtensorMap and enums only; cuTensorMapEncodeTiled is resolved at run time

#include "common.cuh"
#include "linear_small.cuh"

namespace lq {
namespace tc {

constexpr int BK = 64;
constexpr int BN = 256;
constexpr int kDeqWarps = 8;
constexpr int kThreads = (2 + kDeqWarps) * 32;
constexpr int kBBytes = BN * 128;            // bf16 weight tile of one step
constexpr long long kWaitCycles = 4000000000LL;   // about two seconds

struct Params {
    QView q;
    __nv_bfloat16* out;
    int* status;
    int M;
    int out_cols;      // N (forward) or K (backward)
    int steps_q;       // steps whose weights are dequantized
    int steps_d;       // steps of the rank-r term
    int stages;
};

// ------------------------------------------------------------------------------------ PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((saddr & 0x3FFFFu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= static_cast<uint64_t>((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

// Bounded wait.  Returns false when the wait was abandoned (another thread aborted, or time ran out).
struct Ctl {
    volatile int* abort_s;
    int* status_g;
};
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, const Ctl& c, int where) {
    const long long t0 = clock64();
    for (int it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63) == 63) {
            if (*c.abort_s) return false;
            if (clock64() - t0 > kWaitCycles) {
                *c.abort_s = 1;
                atomicCAS(c.status_g, 0, where);
                return false;
            }
        }
    }
}
__device__ __forceinline__ bool wait(uint32_t bar, uint32_t parity, const Ctl& c, int where) {
    if (mbar_try_wait(bar, parity)) return true;
    return wait_slow(bar, parity, c, where);
}

// ------------------------------------------------------------------------------------ dequantization
// One thread dequantizes 64 consecutive weights of one row (two groups of 32 codes) and writes
// them as eight 16-byte chunks of a 128-byte row, chunk index XOR (row % 8).
template <int B>
__device__ __forceinline__ void dequant_row(const uint32_t* __restrict__ slab, int lane, const float* __restrict__ cb,
                                            const float (&scale)[4], uint8_t* __restrict__ out_row, int row_in_8) {
#pragma unroll
    for (int g = 0; g < 2; ++g) {
        uint32_t w[B + 1];
#pragma unroll
        for (int i = 0; i < B; ++i) w[i] = slab[(g * B + i) * 32 + lane];
        w[B] = 0u;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t packed[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int j = c * 8 + e * 2;
                const uint32_t c0 = extract_code<B>(w, j), c1 = extract_code<B>(w, j + 1);
                float q0, q1;
                if constexpr (B <= 4) { q0 = cb[c0 * 32 + lane]; q1 = cb[c1 * 32 + lane]; }
                else { q0 = cb[c0]; q1 = cb[c1]; }
                const float s = scale[g * 2 + (c >> 1)];
                const __nv_bfloat162 h = __floats2bfloat162_rn(__fmul_rn(q0, s), __fmul_rn(q1, s));
                packed[e] = *reinterpret_cast<const uint32_t*>(&h);
            }
            const int chunk = (g * 4 + c) ^ row_in_8;
            *reinterpret_cast<uint4*>(out_row + chunk * 16) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
        }
    }
}

// Block scales s~ of the four 16-column quarters of (row, columns k .. k+63).
__device__ __forceinline__ void load_scales(const QView& q, int row, int k, float (&scale)[4]) {
    if (row >= q.N || k >= q.K) { scale[0] = scale[1] = scale[2] = scale[3] = 0.0f; return; }
    const long long blk = static_cast<long long>(row) * q.KB + (k >> q.logB0);
    if (q.B0 >= 64) {
        const float s = block_scale(q.sc[blk], q.v[blk >> q.logB1]);
        scale[0] = scale[1] = scale[2] = scale[3] = s;
    } else if (q.B0 == 32) {
        const float s0 = block_scale(q.sc[blk], q.v[blk >> q.logB1]);
        const float s1 = block_scale(q.sc[blk + 1], q.v[(blk + 1) >> q.logB1]);
        scale[0] = scale[1] = s0; scale[2] = scale[3] = s1;
    } else {
#pragma unroll
        for (int i = 0; i < 4; ++i) scale[i] = block_scale(q.sc[blk + i], q.v[(blk + i) >> q.logB1]);
    }
}

// ------------------------------------------------------------------------------------ kernel
template <int B, bool BWD, int MH>
__global__ void __launch_bounds__(kThreads, 1)
tc_linear_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA2,
                 const __grid_constant__ CUtensorMap tmB2, const Params p) {
    constexpr int A_BYTES = MH * 128 * 128;
    constexpr int P_BYTES = 2048 * B;
    constexpr int STAGE = A_BYTES + kBBytes + P_BYTES;
    constexpr int CB_FLOATS = (B <= 4) ? (1 << B) * 32 : 256;
    constexpr uint32_t TMEM_COLS = MH * BN;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* tail = base + static_cast<size_t>(p.stages) * STAGE;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);            // full_tma[8], full_b[8], empty[8], acc_full, drain
    float* cb = reinterpret_cast<float*>(tail + 256);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 256 + CB_FLOATS * 4);
    volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * (MH * 128);
    const int c0 = blockIdx.y * BN;          // first output column: n0 (forward) or k0 (backward)
    const int total = p.steps_q + p.steps_d;
    const Ctl ctl{abort_s, p.status};

    auto full_tma = [&](int s) { return smem_u32(bars + s); };
    auto full_b = [&](int s) { return smem_u32(bars + 8 + s); };
    auto empty = [&](int s) { return smem_u32(bars + 16 + s); };
    const uint32_t acc_full = smem_u32(bars + 24), drain = smem_u32(bars + 25);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(full_tma(s), 1); mbar_init(full_b(s), kDeqWarps); mbar_init(empty(s), 1); }
        mbar_init(acc_full, 1);
        mbar_init(drain, 1);
        *abort_s = 0;
        fence_barrier_init();
    }
    for (int i = threadIdx.x; i < CB_FLOATS; i += kThreads)
        cb[i] = (B <= 4) ? c_codebook[bits_index(B)][i >> 5] : c_codebook[3][i];
    if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer
        if (lane == 0) {
            for (int step = 0; step < total; ++step) {
                const int s = step % p.stages;
                const uint32_t ph = (step / p.stages) & 1;
                if (!wait(empty(s), ph ^ 1, ctl, 1)) break;
                uint8_t* st = base + static_cast<size_t>(s) * STAGE;
                const uint32_t a_dst = smem_u32(st), b_dst = a_dst + A_BYTES, p_dst = b_dst + kBBytes;
                if (step < p.steps_q) {
                    const uint8_t* codes = reinterpret_cast<const uint8_t*>(p.q.codes);
                    uint32_t bytes = A_BYTES;
                    if (!BWD) {
                        int nt_have = 0;
                        for (int t = 0; t < 2; ++t) if ((c0 >> 7) + t < p.q.ntiles) ++nt_have;
                        bytes += nt_have * 1024 * B;
                        mbar_expect_tx(full_tma(s), bytes);
                        tma_load_2d(a_dst, &tmA, step * BK, m0, full_tma(s));
                        for (int t = 0; t < nt_have; ++t) {
                            const size_t tile = static_cast<size_t>((c0 >> 7) + t) * p.q.ktiles + step;
                            bulk_load(p_dst + t * 1024 * B, codes + tile * (1024 * B), 1024 * B, full_tma(s));
                        }
                    } else {
                        const int nn0 = step * BK;
                        int kt_have = 0;
                        for (int t = 0; t < 4; ++t) if ((c0 >> 6) + t < p.q.ktiles) ++kt_have;
                        bytes += kt_have * 512 * B;
                        mbar_expect_tx(full_tma(s), bytes);
                        tma_load_2d(a_dst, &tmA, nn0, m0, full_tma(s));
                        for (int t = 0; t < kt_have; ++t) {
                            const size_t tile = static_cast<size_t>(nn0 >> 7) * p.q.ktiles + (c0 >> 6) + t;
                            bulk_load(p_dst + t * 512 * B, codes + tile * (1024 * B) + ((nn0 >> 6) & 1) * (512 * B), 512 * B,
                                      full_tma(s));
                        }
                    }
                } else {
                    const int d = step - p.steps_q;
                    if (!BWD) {
                        mbar_expect_tx(full_tma(s), A_BYTES + kBBytes);
                        tma_load_2d(a_dst, &tmA2, d * BK, m0, full_tma(s));
                        tma_load_2d(b_dst, &tmB2, d * BK, c0, full_tma(s));
                    } else {
                        int kt_have = 0;
                        for (int t = 0; t < 4; ++t) if (c0 + t * 64 < p.out_cols) ++kt_have;
                        mbar_expect_tx(full_tma(s), A_BYTES + kt_have * 8192);
                        tma_load_2d(a_dst, &tmA2, d * BK, m0, full_tma(s));
                        for (int t = 0; t < kt_have; ++t) tma_load_2d(b_dst + t * 8192, &tmB2, c0 + t * 64, d * BK, full_tma(s));
                    }
                }
            }
            if (*abort_s) {
                // let copies that are still in flight land before the CTA exits (bounded)
                for (int s = 0; s < p.stages; ++s) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(full_tma(s), 0) && !mbar_try_wait(full_tma(s), 1) && clock64() - t0 < 20000000LL) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((BWD ? 1u : 0u) << 16) |
                                       (static_cast<uint32_t>(BN >> 3) << 17) | (static_cast<uint32_t>(128 >> 4) << 24);
            bool ok = true;
            for (int step = 0; step < total && ok; ++step) {
                const int s = step % p.stages;
                const uint32_t ph = (step / p.stages) & 1;
                ok = wait(full_tma(s), ph, ctl, 2) && wait(full_b(s), ph, ctl, 3);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_src = smem_u32(base + static_cast<size_t>(s) * STAGE), b_src = a_src + A_BYTES;
#pragma unroll
                for (int h = 0; h < MH; ++h) {
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16) {
                        const uint64_t adesc = make_desc(a_src + h * 16384 + k16 * 32, 16, 1024);
                        const uint64_t bdesc = BWD ? make_desc(b_src + k16 * 2048, 8192, 1024)
                                                   : make_desc(b_src + k16 * 32, 16, 1024);
                        tc_mma(tmem + h * BN, adesc, bdesc, idesc, (step > 0 || k16 > 0) ? 1u : 0u);
                    }
                }
                tc_commit(empty(s));
            }
            if (ok) {
                tc_commit(acc_full);
            } else {
                tc_commit(drain);      // wait (bounded) for issued MMAs before tensor memory is freed
                const long long t0 = clock64();
                while (!mbar_try_wait(drain, 0) && clock64() - t0 < 20000000LL) {}
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ dequantization warps, then epilogue
        const int dw = warp - 2;
        const uint32_t* slab_off = nullptr;
        int row_local, row_sub;   // row inside the B tile / inside its 128-byte-row sub-tile
        uint32_t b_off;           // byte offset of this thread's row inside the B tile
        if (!BWD) { row_local = dw * 32 + lane; row_sub = row_local; b_off = row_local * 128; }
        else { row_local = (dw & 1) * 32 + lane; row_sub = row_local; b_off = (dw >> 1) * 8192 + row_local * 128; }
        (void)slab_off;
        float scale[4];
        if (p.steps_q > 0) {
            if (!BWD) load_scales(p.q, c0 + row_local, 0, scale);
            else load_scales(p.q, row_local, c0 + (dw >> 1) * 64, scale);
        }
        bool ok = true;
        for (int step = 0; step < total && ok; ++step) {
            const int s = step % p.stages;
            const uint32_t ph = (step / p.stages) & 1;
            ok = wait(full_tma(s), ph, ctl, 4);
            if (!ok) break;
            if (step < p.steps_q) {
                uint8_t* st = base + static_cast<size_t>(s) * STAGE;
                const uint32_t* slab = reinterpret_cast<const uint32_t*>(st + A_BYTES + kBBytes) + dw * (64 * B);
                float next[4];
                if (step + 1 < p.steps_q) {     // prefetch the next step's scales before the ALU work
                    if (!BWD) load_scales(p.q, c0 + row_local, (step + 1) * BK, next);
                    else load_scales(p.q, (step + 1) * BK + row_local, c0 + (dw >> 1) * 64, next);
                }
                dequant_row<B>(slab, lane, cb, scale, st + A_BYTES + b_off, row_sub & 7);
                if (step + 1 < p.steps_q) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) scale[i] = next[i];
                }
                fence_proxy_async();            // make the generic-proxy stores visible to the tensor core
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(full_b(s));
        }
        // epilogue: warp reads its quarter of the 128 accumulator lanes, half of the 256 columns
        if (ok && wait(acc_full, 0, ctl, 5)) {
            tc_fence_after();
            const int quarter = warp & 3, colhalf = dw >> 2;
#pragma unroll 1
            for (int h = 0; h < MH; ++h) {
                const int m = m0 + h * 128 + quarter * 32 + lane;
#pragma unroll 1
                for (int cc = 0; cc < 4; ++cc) {
                    const int col = colhalf * 128 + cc * 32;
                    uint32_t v[32];
                    tmem_ld32(tmem + (static_cast<uint32_t>(quarter * 32) << 16) + h * BN + col, v);
                    tmem_ld_wait();
                    if (m < p.M) {
                        __nv_bfloat16* dst = p.out + static_cast<size_t>(m) * p.out_cols + c0 + col;
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            if (c0 + col + i * 8 < p.out_cols) {
                                uint32_t w[4];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(v[i * 8 + 2 * e]),
                                                                                   __uint_as_float(v[i * 8 + 2 * e + 1]));
                                    w[e] = *reinterpret_cast<const uint32_t*>(&hh);
                                }
                                *reinterpret_cast<uint4*>(dst + i * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                            }
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

// ------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            f = nullptr;
        }
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// bf16 row-major [rows, cols] matrix, box of 64 columns x box_rows rows, 128-byte swizzle, zero fill.
inline bool make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

constexpr int kSmemLimit = 232448;   // 227 KB of dynamic shared memory per CTA

template <int B, int MH>
constexpr int stage_bytes() { return MH * 16384 + kBBytes + 2048 * B; }
template <int B>
constexpr int tail_bytes() { return 256 + ((B <= 4) ? (1 << B) * 32 : 256) * 4 + 64; }

template <int B, bool BWD, int MH>
inline int launch_one(const CUtensorMap& tA, const CUtensorMap& tA2, const CUtensorMap& tB2, Params p, cudaStream_t st) {
    int stages = (kSmemLimit - 1024 - tail_bytes<B>()) / stage_bytes<B, MH>();
    if (stages > 8) stages = 8;
    if (stages < 2) return LQLORA_ERR_UNSUPPORTED;
    p.stages = stages;
    const int smem = 1024 + stages * stage_bytes<B, MH>() + tail_bytes<B>();
    auto kern = tc_linear_kernel<B, BWD, MH>;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess) {
            cudaGetLastError();
            return LQLORA_ERR_CUDA;
        }
        attr_done = true;
    }
    dim3 grid((p.M + MH * 128 - 1) / (MH * 128), (p.out_cols + BN - 1) / BN);
    kern<<<grid, kThreads, smem, st>>>(tA, tA2, tB2, p);
    count_launch(1);
    if (cudaGetLastError() != cudaSuccess) return LQLORA_ERR_CUDA;
    return LQLORA_OK;
}

template <int B>
inline int launch_b(const CUtensorMap& tA, const CUtensorMap& tA2, const CUtensorMap& tB2, const Params& p, bool bwd, int mh,
                    cudaStream_t st) {
    if (!bwd) return mh == 2 ? launch_one<B, false, 2>(tA, tA2, tB2, p, st) : launch_one<B, false, 1>(tA, tA2, tB2, p, st);
    return mh == 2 ? launch_one<B, true, 2>(tA, tA2, tB2, p, st) : launch_one<B, true, 1>(tA, tA2, tB2, p, st);
}

}  // namespace tc

constexpr int kTcMinRows = 33;   // fewer rows go to the weight-streaming kernels

inline bool tc_supported(const QView& q, int r, int64_t M, bool backward) {
    (void)r;
    if (M < kTcMinRows) return false;
    if (q.N % 8 != 0 || q.K % 8 != 0) return false;
    (void)backward;
    return true;
}

inline size_t tc_workspace_bytes(int64_t N, int64_t K, int r, int64_t M, bool backward) {
    (void)N; (void)K; (void)backward;
    return kStatusBytes + round_up(static_cast<size_t>(M) * (r > 0 ? r : 1) * 2, 256);
}

inline int tc_launch(const QView& q, const void* L1, const void* L2, int r, const void* A, int M, void* out, char* ws,
                     bool backward, cudaStream_t st) {
    using namespace tc;
    __nv_bfloat16* T = reinterpret_cast<__nv_bfloat16*>(ws + kStatusBytes);
    const __nv_bfloat16* a = static_cast<const __nv_bfloat16*>(A);
    const int C = backward ? q.N : q.K;              // contraction length
    if (r > 0) {
        if (!backward) lowrank_pre_kernel<<<M, 256, 0, st>>>(a, static_cast<const __nv_bfloat16*>(L2), T, q.K, r, q.K, 1);
        else lowrank_pre_kernel<<<M, 256, 0, st>>>(a, static_cast<const __nv_bfloat16*>(L1), T, q.N, r, 1, r);
        count_launch(1);
    }
    const int mh = (M > 128) ? 2 : 1;
    CUtensorMap tA, tA2, tB2;
    if (!make_map(&tA, A, M, C, mh * 128)) return LQLORA_ERR_CUDA;
    if (r > 0) {
        if (!make_map(&tA2, T, M, r, mh * 128)) return LQLORA_ERR_CUDA;
        const bool okb = backward ? make_map(&tB2, L2, r, q.K, 64) : make_map(&tB2, L1, q.N, r, 256);
        if (!okb) return LQLORA_ERR_CUDA;
    } else {
        tA2 = tA; tB2 = tA;
    }
    Params p;
    p.q = q;
    p.out = static_cast<__nv_bfloat16*>(out);
    p.status = reinterpret_cast<int*>(ws);
    p.M = M;
    p.out_cols = backward ? q.K : q.N;
    p.steps_q = (C + BK - 1) / BK;
    p.steps_d = (r + BK - 1) / BK;
    p.stages = 0;
    switch (q.b0) {
        case 2: return launch_b<2>(tA, tA2, tB2, p, backward, mh, st);
        case 3: return launch_b<3>(tA, tA2, tB2, p, backward, mh, st);
        case 4: return launch_b<4>(tA, tA2, tB2, p, backward, mh, st);
        default: return launch_b<8>(tA, tA2, tB2, p, backward, mh, st);
    }
}

}  // namespace lq
