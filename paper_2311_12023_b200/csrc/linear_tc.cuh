// Tensor-core path for many rows of X (training-sized M) on sm_100a.
//
// One CTA computes a [MH*128, 256] tile of the output.  Per pipeline step of 64 contraction
// elements:
//   - a producer thread issues a TMA tile load of the bf16 activations (128-byte swizzle) and
//     bulk copies of the packed code slabs into shared memory;
//   - sixteen dequantization warps unpack the codes, multiply by the block scale in fp32, round to
//     bf16 and write the weight tile into shared memory in the 128-byte-swizzled layout that the
//     tensor core reads (one thread = 32 weights of one row);
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
#include "device_util.cuh"
#include "linear_small.cuh"

namespace lq {
namespace tc {
using namespace dev;

constexpr int BK = 64;
constexpr int BN = 256;
constexpr int kDeqWarps = 16;
constexpr int kThreads = (2 + kDeqWarps) * 32;
constexpr int kBBytes = BN * 128;            // bf16 weight tile of one step

struct Params {
    QView q;
    __nv_bfloat16* out;
    int* status;
    int M;
    int out_cols;      // N (forward) or K (backward)
    int steps_q;       // steps whose weights are dequantized
    int steps_d;       // steps of the rank-r term
    int stages;
    int c_base;        // first output column of this launch (a call may be split over two launches by output columns)
    int c_tiles;       // number of 256-column output tiles of this launch
};

// ------------------------------------------------------------------------------------ PTX (tensor memory, tcgen05)
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

// ------------------------------------------------------------------------------------ dequantization
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ void sts_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}
// One thread dequantizes the 32 consecutive weights of one (row, group) -- b0 words of the slab,
// `words` pointing at the thread's first word, the others 32 words apart -- and writes them as four
// 16-byte chunks of the row's 128 bytes; `dst` is the row start, `goff` the byte offset of the group
// in the row (0 or 64), `xr` is (row % 8) * 16; a chunk at byte offset o of the row lives at o ^ xr.
// 8-bit codes read the code book from shared memory.  REP: the table is stored once per bank, entry c of the copy
// of lane l at lut8[c * 32 + l], and `lut8` already points at the lane's copy, so no look-up meets a bank conflict.
template <int B, bool REP = false>
__device__ __forceinline__ void dequant_group(uint32_t words, float s_lo, float s_hi, bool two_scales,
                                              uint32_t dst, uint32_t goff, uint32_t xr, const float* __restrict__ lut8) {
    // `words` and `dst` are 32-bit shared-memory addresses (explicit shared-space loads and stores)
    uint32_t w[B];
#pragma unroll
    for (int i = 0; i < B; ++i) w[i] = lds_u32(words + i * 128);
    const uint32_t x = dst + (goff ^ xr);    // chunk c sits at this address with bits 4, 5 flipped by c
    if constexpr (B == 8) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float s = (c < 2) ? s_lo : s_hi;
            uint32_t packed[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t ww = w[2 * c + (e >> 1)] >> (16 * (e & 1));
                const float q0 = REP ? lut8[(ww & 255u) << 5] : lut8[ww & 255u];
                const float q1 = REP ? lut8[((ww >> 8) & 255u) << 5] : lut8[(ww >> 8) & 255u];
                const __nv_bfloat162 h = __floats2bfloat162_rn(__fmul_rn(q0, s), __fmul_rn(q1, s));
                packed[e] = *reinterpret_cast<const uint32_t*>(&h);
            }
            sts_v4(x ^ (c << 4), packed[0], packed[1], packed[2], packed[3]);
        }
    } else {
        BlockTable<B> tab;
        tab.build(s_lo);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (c == 2 && two_scales) tab.build(s_hi);
            const uint32_t sel = chunk_selector<B>(w, c);
            uint32_t selA = sel, selB = 0u;
            if constexpr (B == 4) { selA = sel & 0x77777777u; selB = ((sel >> 1) & 0x44444444u) | 0x32103210u; }
            uint32_t o[4];
            tab.lookup4(selA, selB, o[0], o[1]);
            tab.lookup4(selA >> 16, selB >> 16, o[2], o[3]);
            sts_v4(x ^ (c << 4), o[0], o[1], o[2], o[3]);
        }
    }
}

// Raw scale data of the 32 weights (row, k .. k+31): the one or two 8-bit scale codes and the
// second-level scale of their group (B1 >= 16 blocks, so both codes share it).
struct RawScale { uint32_t sc; float v; };
// s~ = fl32(float(s^) * fl32(v / 127)); the quotient is recomputed only when v changes.
__device__ __forceinline__ void make_scales(const QView& q, const RawScale& r, float& v_cached, float& sigma, float& s_lo, float& s_hi) {
    if (r.v != v_cached) { v_cached = r.v; sigma = __fdiv_rn(r.v, q.levels); }
    s_lo = __fmul_rn(static_cast<float>(r.sc & 0xFFu), sigma);
    s_hi = (q.B0 == 16) ? __fmul_rn(static_cast<float>(r.sc >> 8), sigma) : s_lo;
}

// Forward pass: the scale codes a thread needs in consecutive steps are consecutive bytes of its row, so it keeps a
// window of 16 of them (one 128-bit load, with the second-level scale of the window: 16 aligned blocks share their
// group since B1 >= 16) and the next window, requested one window period ahead.  `base` = block offset of the
// window inside the row (a multiple of 16); rows need KB % 16 == 0 for the alignment.
struct ScaleWindow { uint4 w; float v; };
__device__ __forceinline__ ScaleWindow load_scale_window(const QView& q, uint32_t row_blk0, int base, bool row_ok) {
    ScaleWindow s{make_uint4(0u, 0u, 0u, 0u), 0.0f};
    if (row_ok && base < q.KB) {
        s.w = __ldg(reinterpret_cast<const uint4*>(q.sc + row_blk0 + base));
        s.v = __ldg(q.v + ((row_blk0 + base) >> q.logB1));
    }
    return s;
}
// scale code(s) of block offset b (and b + 1 when two blocks of 16 columns make up the thread's 32 columns)
__device__ __forceinline__ RawScale window_scale(const ScaleWindow& s, int b, bool two) {
    const int i = b & 15;
    const uint32_t word = (i < 8) ? ((i < 4) ? s.w.x : s.w.y) : ((i < 12) ? s.w.z : s.w.w);
    const uint32_t sh = word >> ((i & 3) * 8);
    return RawScale{two ? (sh & 0xFFFFu) : (sh & 0xFFu), s.v};
}

// ------------------------------------------------------------------------------------ kernel
// Shared memory: [activation ring: SA x A_BYTES][weight ring: 2 x 32 KB][packed ring: SA x 2048*b0]
// [barriers][8-bit look-up table].  The activation / packed-code ring runs several steps ahead of
// the tensor core (it hides the latency of global memory); the dequantized weight ring needs two
// stages only (one being read by the tensor core, one being written).
constexpr int kSmemLimit = 232448;   // 227 KB of dynamic shared memory per CTA
// stages of the dequantized weight ring: three, so that the dequantization of a step may start two
// tensor-core steps before its result is needed (two for 8-bit codes, whose packed data leave less room)
template <int B, int MH>
__host__ __device__ constexpr int b_stages() { return (B == 8 && MH == 2) ? 2 : 3; }

template <int B, int MH>
__host__ __device__ constexpr int stage_bytes() { return MH * 16384 + 2048 * B; }        // one stage of the activation + packed-code ring
template <int B>
__host__ __device__ constexpr int tail_bytes() { return 256 + (B == 8 ? 1024 : 0) + 64; }
template <int B, int MH>
__host__ __device__ constexpr int fixed_bytes() { return 1024 + b_stages<B, MH>() * kBBytes; }   // alignment slack + weight ring
template <int B, int MH>
__host__ __device__ constexpr int ring_stages() {
    const int s = (kSmemLimit - fixed_bytes<B, MH>() - tail_bytes<B>()) / stage_bytes<B, MH>();
    return s > 6 ? 6 : s;
}

// Ring position that advances without divisions: stage index and the parity of the current pass.
template <int S> struct RingPos {
    int s = 0;
    uint32_t ph = 0;
    __device__ __forceinline__ void advance() { if (++s == S) { s = 0; ph ^= 1u; } }
};

template <int B, bool BWD, int MH>
__global__ void __launch_bounds__(kThreads, 1)
tc_linear_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA2,
                 const __grid_constant__ CUtensorMap tmB2, const Params p) {
    constexpr int A_BYTES = MH * 128 * 128;
    constexpr int P_BYTES = 2048 * B;
    constexpr uint32_t TMEM_COLS = MH * BN;
    constexpr int SA = ring_stages<B, MH>();
    constexpr int kBStages = b_stages<B, MH>();

    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* a_ring = base;
    uint8_t* b_ring = a_ring + static_cast<size_t>(SA) * A_BYTES;
    uint8_t* p_ring = b_ring + kBStages * kBBytes;
    uint8_t* tail = p_ring + static_cast<size_t>(SA) * P_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);   // full_a[8], empty_a[8], full_b[4], empty_b[4], acc_full, drain
    float* lut8 = reinterpret_cast<float*>(tail + 256);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 256 + (B == 8 ? 1024 : 0));
    volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * (MH * 128);
    const int c0 = p.c_base + blockIdx.y * BN;          // first output column: n0 (forward) or k0 (backward)
    // split of the contraction over the CTAs of a cluster (gridDim.z of them); the rank-r steps go to split 0
    const int nsplit = gridDim.z, split = blockIdx.z;
    const int per_split = (p.steps_q + nsplit - 1) / nsplit;
    const int q_lo = min(p.steps_q, split * per_split);
    const int nq = min(p.steps_q, q_lo + per_split) - q_lo;       // dequantized steps of this CTA
    const int total = nq + (split == 0 ? p.steps_d : 0);
    const Ctl ctl{abort_s, p.status};

    auto full_a = [&](int s) { return smem_u32(bars + s); };
    auto empty_a = [&](int s) { return smem_u32(bars + 8 + s); };
    auto full_b = [&](int s) { return smem_u32(bars + 16 + s); };
    auto empty_b = [&](int s) { return smem_u32(bars + 20 + s); };
    const uint32_t acc_full = smem_u32(bars + 24), drain = smem_u32(bars + 25);

    if (threadIdx.x == 0) {
        for (int s = 0; s < SA; ++s) { mbar_init(full_a(s), 1); mbar_init(empty_a(s), 1); }
        for (int s = 0; s < kBStages; ++s) { mbar_init(full_b(s), kDeqWarps); mbar_init(empty_b(s), 1); }
        mbar_init(acc_full, 1);
        mbar_init(drain, 1);
        *abort_s = 0;
        fence_barrier_init();
    }
    if constexpr (B == 8) {
        for (int i = threadIdx.x; i < 256; i += kThreads) lut8[i] = c_codebook[3][i];
    }
    if (warp == 1) { tmem_alloc(smem_u32(tmem_slot), TMEM_COLS); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    bool acc_ok = false;          // this thread saw the accumulators complete (dequantization warps only)

    if (warp == 0) {
        // ------------------------------------------------------------------ producer: activations + packed codes
        if (lane == 0) {
            const uint8_t* codes = reinterpret_cast<const uint8_t*>(p.q.codes);
            RingPos<SA> ra;
            for (int step = 0; step < total; ++step, ra.advance()) {
                const int s = ra.s;
                if (!wait(empty_a(s), ra.ph ^ 1, ctl, 1)) break;
                const uint32_t a_dst = smem_u32(a_ring) + s * A_BYTES;
                const uint32_t p_dst = smem_u32(p_ring) + s * P_BYTES;
                if (step < nq) {
                    const int qs = q_lo + step;                  // step index in the whole contraction
                    if (!BWD) {
                        int nt_have = 0;
                        for (int t = 0; t < 2; ++t) if ((c0 >> 7) + t < p.q.ntiles) ++nt_have;
                        mbar_expect_tx(full_a(s), A_BYTES + nt_have * 1024 * B);
                        tma_load_2d(a_dst, &tmA, qs * BK, m0, full_a(s));
                        for (int t = 0; t < nt_have; ++t) {
                            const size_t tile = static_cast<size_t>((c0 >> 7) + t) * p.q.ktiles + qs;
                            bulk_load(p_dst + t * 1024 * B, codes + tile * (1024 * B), 1024 * B, full_a(s));
                        }
                    } else {
                        const int nn0 = qs * BK;
                        int kt_have = 0;
                        for (int t = 0; t < 4; ++t) if ((c0 >> 6) + t < p.q.ktiles) ++kt_have;
                        mbar_expect_tx(full_a(s), A_BYTES + kt_have * 512 * B);
                        tma_load_2d(a_dst, &tmA, nn0, m0, full_a(s));
                        for (int t = 0; t < kt_have; ++t) {
                            const size_t tile = static_cast<size_t>(nn0 >> 7) * p.q.ktiles + (c0 >> 6) + t;
                            bulk_load(p_dst + t * 512 * B, codes + tile * (1024 * B) + ((nn0 >> 6) & 1) * (512 * B), 512 * B,
                                      full_a(s));
                        }
                    }
                } else {
                    if (step == nq) {
                        // the rank-r intermediate is written by the preceding kernel, which may still be
                        // running (programmatic dependent launch): wait for it, then order this thread's
                        // bulk-copy reads after what it wrote
                        pdl_wait();
                        fence_proxy_async_all();
                    }
                    mbar_expect_tx(full_a(s), A_BYTES);
                    tma_load_2d(a_dst, &tmA2, (step - nq) * BK, m0, full_a(s));
                }
            }
            if (*abort_s) {
                // let copies that are still in flight land before the CTA exits (bounded)
                for (int s = 0; s < SA; ++s) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(full_a(s), 0) && !mbar_try_wait(full_a(s), 1) && clock64() - t0 < 20000000LL) {}
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
            RingPos<SA> ra;
            RingPos<kBStages> rb;
            for (int step = 0; step < total && ok; ++step, ra.advance(), rb.advance()) {
                const int sa = ra.s, sb = rb.s;
                ok = wait(full_a(sa), ra.ph, ctl, 2) && wait(full_b(sb), rb.ph, ctl, 3);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_src = smem_u32(a_ring) + sa * A_BYTES;
                const uint32_t b_src = smem_u32(b_ring) + sb * kBBytes;
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
                tc_commit(empty_a(sa));
                tc_commit(empty_b(sb));
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
        // warp dw handles slab (dw / 2) of the step's packed data and the 32-column group (dw % 2);
        // one thread = one row of that slab.
        const int dw = warp - 2;
        const int slab_i = dw >> 1, g = dw & 1;
        int row_local;            // row inside the 128-byte-row (sub-)tile of the B operand
        uint32_t b_off;           // byte offset of this thread's row inside the B tile
        if (!BWD) { row_local = slab_i * 32 + lane; b_off = row_local * 128; }
        else { row_local = (slab_i & 1) * 32 + lane; b_off = (slab_i >> 1) * 8192 + row_local * 128; }
        const uint32_t xr = (row_local & 7) << 4;
        const bool two_scales = (p.q.B0 == 16);
        // block index of the scale of step `st` (32-bit: the host checks that N*K/B0 fits):
        //   forward  (row c0 + row_local, columns st*64 + 32 g ..), backward (row st*64 + row_local, columns c0 + 64*(slab_i/2) + 32 g ..)
        const int my_row = BWD ? row_local : c0 + row_local;
        const int my_col = BWD ? c0 + (slab_i >> 1) * 64 + g * 32 : g * 32;
        const bool col_ok = my_col < p.q.K;
        const uint32_t blk0 = static_cast<uint32_t>(my_row) * p.q.KB + (BWD ? (my_col >> p.q.logB0) : 0);
        const uint32_t row_stride = static_cast<uint32_t>(BK) * p.q.KB;
        const uint8_t* __restrict__ scp = p.q.sc;
        const float* __restrict__ vp = p.q.v;
        const int logB0 = p.q.logB0, logB1 = p.q.logB1;
        auto fetch = [&](int st) {
            RawScale r{0u, 0.0f};
            const int row = BWD ? st * BK + my_row : my_row;
            if (row < p.q.N && col_ok) {
                const uint32_t blk = BWD ? blk0 + st * row_stride : blk0 + ((st * BK + my_col) >> logB0);
                r.sc = two_scales ? static_cast<uint32_t>(__ldg(reinterpret_cast<const uint16_t*>(scp + blk))) : static_cast<uint32_t>(__ldg(scp + blk));
                r.v = __ldg(vp + (blk >> logB1));
            }
            return r;
        };
        // The raw scale data of step s + 4 are requested right after those of step s have been used,
        // into the same slot; the loop is unrolled by four so that the slots are fixed registers and
        // no instruction touches a slot while its load is in flight.
        float v_cached = -1.0f, sigma = 0.0f, s_lo = 0.0f, s_hi = 0.0f;
        RawScale slot[4];
        // forward, rows aligned to 16 blocks: windows of 16 scale codes instead of one load per step
        const bool use_win = !BWD && (p.q.KB % 16 == 0);
        const bool win_row_ok = !BWD && my_row < p.q.N;
        ScaleWindow cur{make_uint4(0u, 0u, 0u, 0u), 0.0f}, nxt = cur;
        int cur_base = 0;
        if (use_win) {
            cur_base = ((q_lo * BK + my_col) >> logB0) & ~15;
            cur = load_scale_window(p.q, blk0, cur_base, win_row_ok);
            nxt = load_scale_window(p.q, blk0, cur_base + 16, win_row_ok);
        } else {
#pragma unroll
            for (int u = 0; u < 4; ++u) slot[u] = (u < nq) ? fetch(q_lo + u) : RawScale{0u, 0.0f};
        }
        // word plane slot of this thread's row: rotated by 8 g + 16 (tile column % 2), see slab_row_slot();
        // forward: the tile column is the step index, backward: it is fixed per thread
        const uint32_t slab_base = smem_u32(p_ring) + (slab_i * (64 * B) + g * (B * 32)) * 4;      // byte address in shared memory
        const int slot_even = slab_row_slot(lane, g, BWD ? ((c0 >> 6) + (slab_i >> 1)) : 0);
        const int slot_odd = BWD ? slot_even : slab_row_slot(lane, g, 1);
        const uint32_t my_b = smem_u32(b_ring) + b_off;
        bool ok = true;
        RingPos<SA> ra;
        RingPos<kBStages> rb;
        for (int step4 = 0; step4 < total && ok; step4 += 4) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int step = step4 + u;
                if (step >= total || !ok) break;
                const int sa = ra.s, sb = rb.s;
                ok = wait(empty_b(sb), rb.ph ^ 1, ctl, 6);
                if (!ok) break;
                if (step < nq) {
                    if (use_win) {
                        const int b = ((q_lo + step) * BK + my_col) >> logB0;
                        if ((b & ~15) != cur_base) {
                            cur = nxt;
                            cur_base += 16;
                            nxt = load_scale_window(p.q, blk0, cur_base + 16, win_row_ok);
                        }
                        make_scales(p.q, window_scale(cur, b, two_scales), v_cached, sigma, s_lo, s_hi);
                    } else {
                        make_scales(p.q, slot[u], v_cached, sigma, s_lo, s_hi);
                        if (step + 4 < nq) slot[u] = fetch(q_lo + step + 4);
                    }
                    ok = wait(full_a(sa), ra.ph, ctl, 4);
                    if (!ok) break;
                    dequant_group<B>(slab_base + sa * P_BYTES + (((q_lo + step) & 1) ? slot_odd : slot_even) * 4, s_lo, s_hi, two_scales, my_b + sb * kBBytes, g << 6, xr, lut8);
                    fence_proxy_async();            // make the generic-proxy stores visible to the tensor core
                    __syncwarp();
                    if (lane == 0) mbar_arrive(full_b(sb));
                } else if (dw == 0) {
                    // rank-r step: the second operand ([L1 | ..] rows or L2 rows) comes by TMA into the weight ring
                    if (lane == 0) {
                        const int d = step - nq;
                        const uint32_t dst = smem_u32(b_ring) + sb * kBBytes;
                        if (!BWD) {
                            mbar_expect_tx(full_b(sb), kBBytes);
                            tma_load_2d(dst, &tmB2, d * BK, c0, full_b(sb));
                        } else {
                            int kt_have = 0;
                            for (int t = 0; t < 4; ++t) if (c0 + t * 64 < p.out_cols) ++kt_have;
                            mbar_expect_tx(full_b(sb), kt_have * 8192);
                            for (int t = 0; t < kt_have; ++t) tma_load_2d(dst + t * 8192, &tmB2, c0 + t * 64, d * BK, full_b(sb));
                        }
                    }
                    __syncwarp();
                } else {
                    if (lane == 0) mbar_arrive(full_b(sb));
                }
                ra.advance();
                rb.advance();
            }
        }
        // epilogue: warp reads its quarter of the 128 accumulator lanes and 64 of the 256 columns
        acc_ok = ok && wait(acc_full, 0, ctl, 5);
        if (acc_ok && nsplit == 1) {
            tc_fence_after();
            const int quarter = warp & 3, colq = dw >> 2;
#pragma unroll 1
            for (int h = 0; h < MH; ++h) {
                const int m = m0 + h * 128 + quarter * 32 + lane;
#pragma unroll 1
                for (int cc = 0; cc < 2; ++cc) {
                    const int col = colq * 64 + cc * 32;
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
    if (nsplit > 1) {
        // ------------------------------------------------------------------ sum over the splits of the contraction
        // Every CTA of the cluster writes its accumulator tile (fp32, [256 columns][128 rows]) over the idle
        // rings; CTA `split` then adds the 256 / nsplit columns it owns from all CTAs through distributed
        // shared memory, rounds to bf16 and stores.  The barriers are executed by all threads of all CTAs,
        // whatever happened before (a CTA that gave up on a wait still takes part; its output is undefined
        // and the status word says so).
        float* accbuf = reinterpret_cast<float*>(base);
        const uint32_t accbuf_addr = smem_u32(accbuf);
        // CTA `split` owns the groups of eight columns [split * 32 / nsplit, (split + 1) * 32 / nsplit) (any cluster size)
        const int g_lo = split * (BN / 8) / nsplit, g_hi = (split + 1) * (BN / 8) / nsplit;
#pragma unroll 1
        for (int h = 0; h < MH; ++h) {
            if (warp >= 2 && acc_ok) {
                tc_fence_after();
                const int dw = warp - 2, quarter = warp & 3, colq = dw >> 2;
#pragma unroll 1
                for (int cc = 0; cc < 2; ++cc) {
                    const int col = colq * 64 + cc * 32;
                    uint32_t v[32];
                    tmem_ld32(tmem + (static_cast<uint32_t>(quarter * 32) << 16) + h * BN + col, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 32; ++i) accbuf[(col + i) * 128 + quarter * 32 + lane] = __uint_as_float(v[i]);
                }
            }
            __syncthreads();
            dec::cluster_sync_all();
            for (int item = threadIdx.x; item < 128 * (g_hi - g_lo); item += kThreads) {
                const int row = item & 127, cg = item >> 7;
                const int m = m0 + h * 128 + row;
                const int col = (g_lo + cg) * 8;
                // all remote loads are requested before the first is used (a round trip costs about two thousand clocks)
                float part[8][8];
#pragma unroll
                for (int rk = 0; rk < 8; ++rk)
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        part[rk][i] = (rk < nsplit) ? dec::ld_dsmem_f32(accbuf_addr + static_cast<uint32_t>((col + i) * 128 + row) * 4u, static_cast<uint32_t>(rk)) : 0.0f;
                float sum[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    sum[i] = 0.0f;
#pragma unroll
                    for (int rk = 0; rk < 8; ++rk) sum[i] += part[rk][i];
                }
                if (m < p.M && c0 + col < p.out_cols) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const __nv_bfloat162 hh = __floats2bfloat162_rn(sum[2 * e], sum[2 * e + 1]);
                        w[e] = *reinterpret_cast<const uint32_t*>(&hh);
                    }
                    *reinterpret_cast<uint4*>(p.out + static_cast<size_t>(m) * p.out_cols + c0 + col) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
            __syncthreads();
            dec::cluster_sync_all();           // the buffers may be overwritten (next half) or released (exit) only now
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}


// ------------------------------------------------------------------------------------ rank-r pre-product
// T = bf16(A F) with a short output width (r <= 128):  forward  T = X L2^T  (F = L2 [r, K], K-major B operand),
// backward T = dY L1 (F = L1 [N, r], MN-major B operand).  Grid = (row tiles of 128, splits of the
// contraction).  Each CTA accumulates its part in tensor memory; with one split it rounds its tile to bf16 and
// stores it, with several the splits of a tile form a cluster (see CL below).
struct PreParams {
    __nv_bfloat16* T;      // [M][r]
    int* status;
    int M, r, rp;          // rp = r rounded up to 64 (MMA N)
    int steps;             // contraction steps of 64 in total
    int steps_per_split;
    int stages;
    int clear_status;      // 1: this kernel is the first of a call and clears the status word (no memset in front of it)
};

// Body of the kernel for the CTA (row tile `tile`, split `split` of `nsplit`); the tensor maps are kernel parameters.
// CL: the splits of a tile are the CTAs of a cluster (nsplit = cluster size <= 8, a divisor of 64); their accumulators
// go to the CTA that owns the column through distributed shared memory (own receive buffer behind the ring, rp x 128
// fp32), are added there in rank order and stored as bf16 -- no partial tiles in global memory, no counters.
template <bool BWD, bool CL = false>
__device__ __forceinline__ void lowrank_body(const CUtensorMap& tmA, const CUtensorMap& tmB, const PreParams& p, int tile, int split,
                                             int nsplit) {
    constexpr int A_BYTES = 16384;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    const int b_bytes = p.rp * 128;
    const int stage_bytes = A_BYTES + b_bytes;
    float* recv = reinterpret_cast<float*>(base + static_cast<size_t>(p.stages) * stage_bytes);
    uint8_t* tail = reinterpret_cast<uint8_t*>(recv) + (CL ? static_cast<size_t>(p.rp) * 512 : 0);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);      // full[8], empty[8], acc_full, drain
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 160);
    volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_slot + 1);

    // The CTAs of a cluster write into each other's shared memory at the end; that is allowed once every CTA of the
    // cluster runs, which the first phase of the cluster barrier establishes: arrive here, wait before the first store.
    if (CL && nsplit > 1) dec::cluster_arrive_relaxed();
    // cleared before this CTA lets the dependent kernel start: that kernel is launched once all CTAs have passed here
    if (p.clear_status && tile == 0 && split == 0 && threadIdx.x == 0) *p.status = 0;
    pdl_launch_dependents();      // the linear kernel behind this one needs T only in its last steps
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = tile * 128;
    const int s_lo = split * p.steps_per_split;
    const int s_hi = min(p.steps, s_lo + p.steps_per_split);
    const int total = s_hi - s_lo;
    const Ctl ctl{abort_s, p.status};
    const uint32_t tmem_cols = (p.rp <= 64) ? 64u : 128u;

    auto full = [&](int s) { return smem_u32(bars + s); };
    auto empty = [&](int s) { return smem_u32(bars + 8 + s); };
    const uint32_t acc_full = smem_u32(bars + 16), drain = smem_u32(bars + 17);

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
    bool cl_ok = false;          // CL: this thread saw the accumulators complete (epilogue warps)

    if (warp == 0) {
        if (lane == 0) {
            for (int i = 0; i < total; ++i) {
                const int s = i % p.stages;
                const uint32_t ph = (i / p.stages) & 1;
                if (!wait(empty(s), ph ^ 1, ctl, 11)) break;
                const uint32_t a_dst = smem_u32(base + static_cast<size_t>(s) * stage_bytes), b_dst = a_dst + A_BYTES;
                const int c = (s_lo + i) * BK;
                mbar_expect_tx(full(s), A_BYTES + b_bytes);
                tma_load_2d(a_dst, &tmA, c, m0, full(s));
                if (!BWD) tma_load_2d(b_dst, &tmB, c, 0, full(s));                       // [rp rows of L2] x 64 columns
                else for (int t = 0; t < p.rp / 64; ++t) tma_load_2d(b_dst + t * 8192, &tmB, t * 64, c, full(s));  // 64 rows of L1
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((BWD ? 1u : 0u) << 16) |
                                   (static_cast<uint32_t>(p.rp >> 3) << 17) | (static_cast<uint32_t>(128 >> 4) << 24);
            bool ok = true;
            for (int i = 0; i < total && ok; ++i) {
                const int s = i % p.stages;
                const uint32_t ph = (i / p.stages) & 1;
                ok = wait(full(s), ph, ctl, 12);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_src = smem_u32(base + static_cast<size_t>(s) * stage_bytes), b_src = a_src + A_BYTES;
#pragma unroll
                for (int k16 = 0; k16 < 4; ++k16) {
                    const uint64_t adesc = make_desc(a_src + k16 * 32, 16, 1024);
                    const uint64_t bdesc = BWD ? make_desc(b_src + k16 * 2048, 8192, 1024) : make_desc(b_src + k16 * 32, 16, 1024);
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
        // epilogue warps 2..5: TMEM lane quarter = warp % 4
        const int quarter = warp & 3;
        const int m = m0 + quarter * 32 + lane;
        const bool ok = (total > 0) ? wait(acc_full, 0, ctl, 13) : true;
        cl_ok = ok;
        if (ok && !CL) {
            // one split: the accumulator row of this thread goes straight to T as bf16 (r is a multiple of 16, so a
            // run of eight columns lies inside or outside of it as a whole)
            tc_fence_after();
            for (int col = 0; col < p.rp; col += 32) {
                uint32_t v[32];
                if (total > 0) { tmem_ld32(tmem + (static_cast<uint32_t>(quarter * 32) << 16) + col, v); tmem_ld_wait(); }
                else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) v[i] = 0u;
                }
                if (m < p.M) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (col + 8 * i < p.r) {
                            uint32_t w[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(v[8 * i + 2 * e]), __uint_as_float(v[8 * i + 2 * e + 1]));
                                w[e] = *reinterpret_cast<const uint32_t*>(&h);
                            }
                            *reinterpret_cast<uint4*>(p.T + static_cast<size_t>(m) * p.r + col + 8 * i) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                }
            }
        }
    }
    if constexpr (CL) {
        // all threads of all CTAs of the cluster pass here, whatever happened before
        __syncthreads();
        if (nsplit > 1) dec::cluster_wait();           // every CTA of the cluster has started
        const uint32_t recv_addr = smem_u32(recv);
        const int cols_share = p.rp / nsplit;
        if (warp >= 2 && cl_ok) {
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
                    else recv[cl * 128 + row] = __uint_as_float(v[i]);
                }
            }
        }
        __syncthreads();
        if (nsplit > 1) dec::cluster_sync_all();
        for (int item = threadIdx.x; item < 128 * cols_share; item += 192) {
            const int row = item & 127, cl = item >> 7;
            float sum = 0.0f;
            for (int src = 0; src < nsplit; ++src) sum += recv[(src * cols_share + cl) * 128 + row];
            const int m = m0 + row, col = split * cols_share + cl;
            if (m < p.M && col < p.r) p.T[static_cast<size_t>(m) * p.r + col] = __float2bfloat16_rn(sum);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, tmem_cols);
}

template <bool BWD>
__global__ void __launch_bounds__(192, 1)
tc_lowrank_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const PreParams p) {
    lowrank_body<BWD>(tmA, tmB, p, blockIdx.x, blockIdx.y, gridDim.y);
}

// The same with the splits of a tile as the CTAs of a cluster (grid.y = cluster size, a power of two up to eight).
template <bool BWD>
__global__ void __launch_bounds__(192, 1)
tc_lowrank_cl_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, const PreParams p) {
    lowrank_body<BWD, true>(tmA, tmB, p, blockIdx.x, blockIdx.y, gridDim.y);
}

// Both pre-products of one layer in one launch (the weight-gradient path, which has the GPU to itself): grid.z = 0
// computes T = X L2^T with (tmA0, tmB0, p0), grid.z = 1 computes T' = dY L1 with (tmA1, tmB1, p1); grid.y = splits of
// the contraction = cluster size (the same for both), reduced through distributed shared memory.
__global__ void __launch_bounds__(192, 1)
tc_lowrank_both_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0, const PreParams p0,
                       const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1, const PreParams p1) {
    if (blockIdx.z == 0) lowrank_body<false, true>(tmA0, tmB0, p0, blockIdx.x, blockIdx.y, gridDim.y);
    else lowrank_body<true, true>(tmA1, tmB1, p1, blockIdx.x, blockIdx.y, gridDim.y);
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
// A descriptor depends only on (pointer, rows, columns, box rows); a training step issues the same few over and over, so
// the last ones built by this thread are kept (a call needs four to six of them).
inline bool make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    struct Entry { const void* ptr; uint64_t rows, cols; uint32_t box_rows; bool valid; CUtensorMap map; };
    constexpr int kEntries = 64;
    thread_local Entry cache[kEntries] = {};
    uint64_t h = reinterpret_cast<uintptr_t>(ptr) >> 4;
    h = (h ^ (h >> 17)) * 0x9E3779B97F4A7C15ull + rows * 31u + cols * 131u + box_rows;
    Entry& e = cache[(h >> 20) % kEntries];
    if (e.valid && e.ptr == ptr && e.rows == rows && e.cols == cols && e.box_rows == box_rows) { *map = e.map; return true; }
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    if (fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    e.ptr = ptr; e.rows = rows; e.cols = cols; e.box_rows = box_rows; e.map = *map; e.valid = true;
    return true;
}

template <int B, bool BWD, int MH>
inline int launch_one(const CUtensorMap& tA, const CUtensorMap& tA2, const CUtensorMap& tB2, Params p, int ksplit, cudaStream_t st,
                      bool after_pre = true) {
    constexpr int stages = ring_stages<B, MH>();
    static_assert(stages >= 2, "activation ring too shallow");
    p.stages = stages;
    constexpr int smem = fixed_bytes<B, MH>() + stages * stage_bytes<B, MH>() + tail_bytes<B>();
    static_assert(smem <= kSmemLimit, "shared memory budget exceeded");
    auto kern = tc_linear_kernel<B, BWD, MH>;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess) {
            cudaGetLastError();
            return LQLORA_ERR_CUDA;
        }
        attr_done = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((p.M + MH * 128 - 1) / (MH * 128), p.c_tiles, ksplit);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;      // the splits of the contraction of one tile form a cluster
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = ksplit;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (p.steps_d > 0 && after_pre) ? 2 : 1;      // overlap with the rank-r pre-product kernel in front of it
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tA, tA2, tB2, p);
    count_launch(1);
    if (e != cudaSuccess) { cudaGetLastError(); return LQLORA_ERR_CUDA; }
    return LQLORA_OK;
}


// Clusters of `ks` CTAs of the one-CTA kernel (one CTA per SM, all of its shared memory) that can be resident at the
// same time.  A cluster lives inside one GPC, so fewer fit than SMs / ks: 15 clusters of eight on a B200, not 18.
// Asked once per cluster size; the figures measured on a B200 stand in when there is no device to ask.
inline int tc_max_clusters(int ks) {
    static int cached[8] = {-1, -1, -1, -1, -1, -1, -1, -1};       // ks = 1 .. 8
    const int idx = (ks < 1 ? 1 : ks > 8 ? 8 : ks) - 1;
    if (cached[idx] >= 0) return cached[idx];
    const int fallback[8] = {148, 74, 48, 36, 28, 24, 16, 15};
    int n = 0;
    auto kern = tc_linear_kernel<3, false, 1>;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1, 1, ks);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = kSmemLimit;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = ks;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess ||
        cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        n = fallback[idx];
    }
    cached[idx] = n;
    return n;
}

// Splits of the contraction for the one-CTA kernel: few output tiles would leave most SMs idle, so
// the contraction of a tile is divided over a cluster of up to eight CTAs (any size: each keeps at least 8 steps, 16 beyond four CTAs, and
// all clusters must be resident at once: a second wave costs more than the finer split saves).
// CTA pairs on [512, 256] tiles take over once their tiles fill more than half of the SMs; below that the one-CTA
// kernel with its split of the contraction puts at least twice as many SMs to work (4096 x 4096 at 512 rows: 32 CTAs
// as pairs, 128 as single CTAs in clusters of four).
inline bool tc_use_pair(int64_t M, int64_t out_cols, int sms) {
    if (M <= 256) return false;
    const long long pair_ctas = 2 * ((M + 511) / 512) * ((out_cols + BN - 1) / BN);
    return 2 * pair_ctas > sms;
}

inline int tc_ksplit_tiles(long long tiles, int steps_q, int sms) {
    for (int ks = 8; ks > 1; --ks)
        if (tiles * ks <= sms && steps_q / ks >= (ks > 4 ? 16 : 8) && tiles <= tc_max_clusters(ks)) return ks;   // the reduction grows with ks
    return 1;
}
inline int tc_ksplit(int64_t M, int64_t out_cols, int steps_q, int sms) {
    if (tc_use_pair(M, out_cols, sms)) return 1;
    const int mh = (M > 128) ? 2 : 1;
    return tc_ksplit_tiles(((M + mh * 128 - 1) / (mh * 128)) * ((out_cols + BN - 1) / BN), steps_q, sms);
}

struct PrePlan {
    int mtiles, nsplit, steps, steps_per_split, rp;
    size_t t_bytes;
};

// Number of SMs of the current device (148 on B200; also the answer when no device is present).
inline int sm_count() {
    static const int n = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) {
            cudaGetLastError();
            v = 148;
        }
        return v;
    }();
    return n;
}

// C = contraction length, out_cols = width of the output of the linear kernel that follows.
inline PrePlan pre_plan(int64_t C, int r, int64_t M, int64_t out_cols) {
    PrePlan pl;
    pl.mtiles = static_cast<int>((M + 127) / 128);
    pl.steps = static_cast<int>((C + BK - 1) / BK);
    // The pre-product runs beside the linear kernel that follows it (programmatic dependent launch):
    // give it the SMs that the last wave of that kernel leaves idle, and at least one CTA per row tile.
    const int mh = (M > 128) ? 2 : 1;
    const int sms = sm_count();
    const long long main_ctas = ((M + mh * 128 - 1) / (mh * 128)) * ((out_cols + BN - 1) / BN) * tc_ksplit(M, out_cols, pl.steps, sms);
    const int idle = static_cast<int>((sms - main_ctas % sms) % sms);
    int want = idle / pl.mtiles;
    if (want > pl.steps / 2) want = pl.steps / 2;
    if (want > 8) want = 8;          // splits of a tile form a cluster (and more than eight made the sum the critical path)
    if (idle < 48) {
        // beside a nearly full linear kernel (itself made of clusters) large pre-product clusters took a cluster's place
        // from it: at most four pre-product CTAs in all
        const int cap = (4 / pl.mtiles > 1) ? 4 / pl.mtiles : 1;
        if (want > cap) want = cap;
    }
    if (want < 1) want = 1;
    while (want & (want - 1)) want &= want - 1;          // a power of two: it divides the 64 columns of the accumulator
    pl.steps_per_split = (pl.steps + want - 1) / want;
    pl.nsplit = want;
    pl.rp = (r <= 64) ? 64 : 128;
    pl.t_bytes = round_up(static_cast<size_t>(M) * (r > 0 ? r : 1) * 2, 256);
    return pl;
}

template <bool BWD>
inline int launch_pre(const CUtensorMap& tA, const CUtensorMap& tB, PreParams p, int mtiles, int nsplit, cudaStream_t st) {
    const int stage = 16384 + p.rp * 128;
    const bool cl = nsplit > 1;            // several splits: reduced inside a cluster
    const int recv_bytes = cl ? p.rp * 512 : 0;
    int stages = (kSmemLimit - 1024 - 256 - recv_bytes) / stage;
    if (stages > 8) stages = 8;
    p.stages = stages;
    const int smem = 1024 + stages * stage + recv_bytes + 256;
    void (*kern)(const CUtensorMap, const CUtensorMap, const PreParams) = cl ? tc_lowrank_cl_kernel<BWD> : tc_lowrank_kernel<BWD>;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(tc_lowrank_kernel<BWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess ||
            cudaFuncSetAttribute(tc_lowrank_cl_kernel<BWD>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess) {
            cudaGetLastError();
            return LQLORA_ERR_CUDA;
        }
        attr_done = true;
    }
    // One split: launched as clusters of two row tiles where possible (the CTAs then fill whole TPCs, and the CTA pairs
    // of the linear kernel that runs beside this one find as many free TPCs as the SM count suggests).
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(mtiles, nsplit);
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (!cl && mtiles % 2 == 0) ? 2 : 1; attr[0].val.clusterDim.y = cl ? nsplit : 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tA, tB, p);
    count_launch(1);
    if (e != cudaSuccess) { cudaGetLastError(); return LQLORA_ERR_CUDA; }
    return LQLORA_OK;
}

template <int B>
inline int launch_b(const CUtensorMap& tA, const CUtensorMap& tA2, const CUtensorMap& tB2, const Params& p, bool bwd, int mh,
                    int ksplit, cudaStream_t st, bool after_pre = true) {
    if (!bwd) return mh == 2 ? launch_one<B, false, 2>(tA, tA2, tB2, p, ksplit, st, after_pre) : launch_one<B, false, 1>(tA, tA2, tB2, p, ksplit, st, after_pre);
    return mh == 2 ? launch_one<B, true, 2>(tA, tA2, tB2, p, ksplit, st, after_pre) : launch_one<B, true, 1>(tA, tA2, tB2, p, ksplit, st, after_pre);
}

}  // namespace tc
}  // namespace lq

#include "linear_tc2.cuh"

namespace lq {

constexpr int kTcMinRows = 17;   // up to 16 rows go to the weight-streaming kernels
constexpr int kTcMinRowsBwd = 9;  // input gradient of matrices with at least 2048 rows: up to 8 rows

inline bool tc_supported(const QView& q, int r, int64_t M, bool backward) {
    (void)r;
    // The input gradient of 9..16 rows is faster here than in the weight-streaming kernel (which then runs one CTA of
    // eight warps per SM) unless the matrix has few rows: 8192 x 8192 at 16 rows 49 -> 41 us, 8192 x 28672 162 -> 100 us.
    const int min_rows = (backward && q.N >= 2048) ? kTcMinRowsBwd : kTcMinRows;
    if (M < min_rows) return false;
    if (q.N % 8 != 0 || q.K % 8 != 0) return false;
    if (static_cast<long long>(q.N) * q.KB >= (1LL << 31)) return false;   // block indices are 32-bit in the kernel
    return true;
}

inline size_t tc_workspace_bytes(int64_t N, int64_t K, int r, int64_t M, bool backward) {
    const tc::PrePlan pl = tc::pre_plan(backward ? N : K, r, M, backward ? K : N);
    return kStatusBytes + pl.t_bytes;
}

inline int tc_launch(const QView& q, const void* L1, const void* L2, int r, const void* A, int M, void* out, char* ws,
                     bool backward, cudaStream_t st) {
    using namespace tc;
    const int C = backward ? q.N : q.K;              // contraction length
    const PrePlan pl = pre_plan(C, r, M, backward ? q.K : q.N);
    // workspace: [status word][T bf16]; the status word is cleared by the first kernel of the call (or the caller's memset)
    __nv_bfloat16* T = reinterpret_cast<__nv_bfloat16*>(ws + kStatusBytes);
    const int mh = (M > 128) ? 2 : 1;
    const bool pair = tc_use_pair(M, backward ? q.K : q.N, sm_count());      // CTA pairs (cta_group::2) on [512, 256] tiles; boxes of 128 rows
    CUtensorMap tA, tA2, tB2;
    if (!make_map(&tA, A, M, C, pair ? 128 : mh * 128)) return LQLORA_ERR_CUDA;
    if (r > 0) {
        // rank-r pre-product on the tensor cores: T = X L2^T (forward) or dY L1 (backward)
        CUtensorMap tPA, tPB;
        if (!make_map(&tPA, A, M, C, 128)) return LQLORA_ERR_CUDA;
        const bool okp = backward ? make_map(&tPB, L1, q.N, r, 64) : make_map(&tPB, L2, r, q.K, pl.rp);
        if (!okp) return LQLORA_ERR_CUDA;
        PreParams pp;
        pp.T = T; pp.status = reinterpret_cast<int*>(ws);
        pp.M = M; pp.r = r; pp.rp = pl.rp; pp.steps = pl.steps; pp.steps_per_split = pl.steps_per_split; pp.stages = 0;
        pp.clear_status = 1;           // first kernel of the call (run_linear issues no memset when there is a rank-r term)
        const int rc = backward ? launch_pre<true>(tPA, tPB, pp, pl.mtiles, pl.nsplit, st)
                                : launch_pre<false>(tPA, tPB, pp, pl.mtiles, pl.nsplit, st);
        if (rc != LQLORA_OK) return rc;
        if (!make_map(&tA2, T, M, r, pair ? 128 : mh * 128)) return LQLORA_ERR_CUDA;
        const bool okb = backward ? make_map(&tB2, L2, r, q.K, 64) : make_map(&tB2, L1, q.N, r, pair ? 128 : 256);
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
    p.c_base = 0;
    p.c_tiles = static_cast<int>((p.out_cols + BN - 1) / BN);
    if (pair) {
        // Wave quantisation: the pair tiles run in waves of sms / 2 clusters.  When the last wave would hold only a few
        // tiles (at most a quarter of a wave), the output columns it would cover are peeled off and computed by the
        // one-CTA kernel with the contraction split over clusters, which spreads that small remainder over many SMs
        // (28672 x 8192 at 2048 rows: 448 pair tiles = 6 waves + 4 tiles, 817 -> 740 us).  Larger remainders stay with
        // the pairs: the one-CTA kernel needs about 1.6 pair-tile times for three quarters of a wave (measured).
        const int mt = (M + 511) / 512, pairs = sm_count() / 2;
        const int tiles = mt * p.c_tiles, rem = tiles % pairs;
        int peel = 0;
        if (tiles > pairs && rem > 0 && 4 * rem <= pairs) peel = (rem + mt - 1) / mt;
        if (peel >= p.c_tiles) peel = 0;
        CUtensorMap tOut;         // output as boxes of 32 rows x 64 columns
        if (!make_map(&tOut, out, M, p.out_cols, 32)) return LQLORA_ERR_CUDA;
        p.c_tiles -= peel;
        int rc;
        switch (q.b0) {
            case 2: rc = backward ? launch_pair<2, true>(tA, tA2, tB2, tOut, p, st) : launch_pair<2, false>(tA, tA2, tB2, tOut, p, st); break;
            case 3: rc = backward ? launch_pair<3, true>(tA, tA2, tB2, tOut, p, st) : launch_pair<3, false>(tA, tA2, tB2, tOut, p, st); break;
            case 4: rc = backward ? launch_pair<4, true>(tA, tA2, tB2, tOut, p, st) : launch_pair<4, false>(tA, tA2, tB2, tOut, p, st); break;
            default: rc = backward ? launch_pair<8, true>(tA, tA2, tB2, tOut, p, st) : launch_pair<8, false>(tA, tA2, tB2, tOut, p, st); break;
        }
        if (rc != LQLORA_OK || peel == 0) return rc;
        // the peeled columns: boxes of 256 rows for the one-CTA kernel; it runs behind the pair kernel (which has waited
        // for the rank-r intermediate), so it needs no programmatic dependency of its own
        CUtensorMap uA, uA2, uB2;
        if (!make_map(&uA, A, M, C, 256)) return LQLORA_ERR_CUDA;
        if (r > 0) {
            if (!make_map(&uA2, T, M, r, 256)) return LQLORA_ERR_CUDA;
            const bool okb = backward ? make_map(&uB2, L2, r, q.K, 64) : make_map(&uB2, L1, q.N, r, 256);
            if (!okb) return LQLORA_ERR_CUDA;
        } else {
            uA2 = uA; uB2 = uA;
        }
        Params p2 = p;
        p2.c_base = p.c_tiles * BN;
        p2.c_tiles = peel;
        const int ks2 = tc_ksplit_tiles(static_cast<long long>(peel) * ((M + 255) / 256), p.steps_q, sm_count());
        switch (q.b0) {
            case 2: return launch_b<2>(uA, uA2, uB2, p2, backward, 2, ks2, st, false);
            case 3: return launch_b<3>(uA, uA2, uB2, p2, backward, 2, ks2, st, false);
            case 4: return launch_b<4>(uA, uA2, uB2, p2, backward, 2, ks2, st, false);
            default: return launch_b<8>(uA, uA2, uB2, p2, backward, 2, ks2, st, false);
        }
    }
    const int ksplit = tc_ksplit(M, p.out_cols, p.steps_q, sm_count());
    switch (q.b0) {
        case 2: return launch_b<2>(tA, tA2, tB2, p, backward, mh, ksplit, st);
        case 3: return launch_b<3>(tA, tA2, tB2, p, backward, mh, ksplit, st);
        case 4: return launch_b<4>(tA, tA2, tB2, p, backward, mh, ksplit, st);
        default: return launch_b<8>(tA, tA2, tB2, p, backward, mh, ksplit, st);
    }
}

}  // namespace lq
