// Tensor-core linear on CTA pairs (tcgen05 cta_group::2) for many rows of X (M > 256 and tiles on more than half of the SMs).
//
// A pair of CTAs (a cluster of two, on one TPC) computes a [512, 256] tile of the output: each CTA holds
// 2 x 128 rows of the activations (two accumulators of 128 lanes x 256 fp32 columns in its tensor memory)
// and HALF of the weight tile of a step (128 of the 256 output columns).  One thread of the leader CTA issues
// tcgen05.mma with M = 256: the tensor cores of both CTAs read the two halves of the weight tile from both
// shared memories.  Compared with the single-CTA kernel each CTA dequantizes half as many weights per MMA
// flop and its shared memory serves half of the weight-operand traffic.
//
// Per CTA: warp 0 lane 0 loads activations (TMA) and packed codes (bulk copies) into a ring; sixteen
// dequantization warps, eight per step (even / odd steps), write the CTA's half of the weight tile into a
// second ring and arrive on the LEADER's barrier (remote arrive for the second CTA); the leader's MMA
// thread waits for the sixteen arrivals of a step, issues the MMAs and commits the ring stages back to both
// CTAs (multicast commit).  Forward and input gradient share the code (K-major / MN-major weight operand)
// as in the single-CTA kernel; the rank-r term is one more step whose operands come by TMA; the output
// leaves through shared memory and TMA stores.
// Every wait is bounded; both CTAs meet at a cluster barrier before tensor memory is freed.
#pragma once

namespace lq {
namespace tc {

// ------------------------------------------------------------------------------------ PTX, cta_group::2
__device__ __forceinline__ void tmem_alloc2(uint32_t slot_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc2(uint32_t addr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_mma2(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// Arrives (once all earlier MMAs of this thread have completed) on the barrier at the same shared-memory
// offset in both CTAs of the pair.
__device__ __forceinline__ void tc_commit_both(uint32_t bar) {
    const uint16_t mask = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"(mask) : "memory");
}
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on the barrier at local address `bar` of CTA `rank` of the cluster (release at cluster scope).
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar, uint32_t rank) {
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(bar), "r"(rank));
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(ra) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait_acq_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __noinline__ bool wait_cluster(uint32_t bar, uint32_t parity, const Ctl& c, int where) {
    const long long t0 = clock64();
    for (int it = 0;; ++it) {
        if (mbar_try_wait_acq_cluster(bar, parity)) return true;
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

constexpr int kPairBBytes = 128 * 128;        // this CTA's half of the bf16 weight tile of one step
constexpr int kPairABytes = 2 * 128 * 128;    // two activation tiles of 128 rows x 64 columns
constexpr int kPairBStages = 4;
template <int B> __host__ __device__ constexpr int pair_a_stages() { return (B == 8) ? 3 : 4; }
template <int B> __host__ __device__ constexpr int pair_smem_bytes() {
    return 1024 + pair_a_stages<B>() * (kPairABytes + 1024 * B) + kPairBStages * kPairBBytes + 512 + (B == 8 ? 32768 : 0);   // 8-bit: code book once per bank
}

template <int B, bool BWD>
__global__ void __launch_bounds__(kThreads, 1)
tc_pair_linear_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmA2,
                      const __grid_constant__ CUtensorMap tmB2, const __grid_constant__ CUtensorMap tmOut, const Params p) {
    constexpr int SA = pair_a_stages<B>();
    constexpr int SB = kPairBStages;
    constexpr int P_BYTES = 1024 * B;
    constexpr uint32_t TMEM_COLS = 512;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* a_ring = base;
    uint8_t* b_ring = a_ring + SA * kPairABytes;
    uint8_t* p_ring = b_ring + SB * kPairBBytes;
    uint8_t* tail = p_ring + SA * P_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);   // full_a[4], empty_a[4], full_b[4], empty_b[4], dbar[4], acc_full, drain
    float* lut8 = reinterpret_cast<float*>(tail + 256);
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 256 + (B == 8 ? 32768 : 0));
    volatile int* abort_s = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_rank();                 // 0 = leader
    const int m0 = (blockIdx.x >> 1) * 512;               // first token row of the pair
    const int c0 = p.c_base + blockIdx.y * BN;            // first output column of the pair
    const int total = p.steps_q + p.steps_d;
    const Ctl ctl{abort_s, p.status};

    auto full_a = [&](int s) { return smem_u32(bars + s); };
    auto empty_a = [&](int s) { return smem_u32(bars + 4 + s); };
    auto full_b = [&](int s) { return smem_u32(bars + 8 + s); };
    auto empty_b = [&](int s) { return smem_u32(bars + 12 + s); };
    auto dbar = [&](int s) { return smem_u32(bars + 16 + s); };
    const uint32_t acc_full = smem_u32(bars + 20), drain = smem_u32(bars + 21);

    if (threadIdx.x == 0) {
        for (int s = 0; s < SA; ++s) { mbar_init(full_a(s), 1); mbar_init(empty_a(s), 1); }
        for (int s = 0; s < SB; ++s) { mbar_init(full_b(s), 16); mbar_init(empty_b(s), 1); mbar_init(dbar(s), 1); }
        mbar_init(acc_full, 1);
        mbar_init(drain, 1);
        *abort_s = 0;
        fence_barrier_init();
    }
    if constexpr (B == 8) {
        for (int i = threadIdx.x; i < 256 * 32; i += kThreads) lut8[i] = c_codebook[3][i >> 5];     // entry c of lane l's copy at c * 32 + l
    }
    if (warp == 1) { tmem_alloc2(smem_u32(tmem_slot), TMEM_COLS); tmem_relinquish2(); }
    tc_fence_before();
    __syncthreads();
    cluster_barrier();                                    // barriers of both CTAs are initialised before any remote arrive
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ producer: activations + packed codes of this CTA
        if (lane == 0) {
            const uint8_t* codes = reinterpret_cast<const uint8_t*>(p.q.codes);
            RingPos<SA> ra;
            for (int step = 0; step < total; ++step, ra.advance()) {
                const int s = ra.s;
                if (!wait(empty_a(s), ra.ph ^ 1, ctl, 41)) break;
                const uint32_t a_dst = smem_u32(a_ring) + s * kPairABytes;
                const uint32_t p_dst = smem_u32(p_ring) + s * P_BYTES;
                const int my_m = m0 + static_cast<int>(rank) * 128;
                if (step < p.steps_q) {
                    if (!BWD) {
                        const int tile_row = (c0 >> 7) + static_cast<int>(rank);
                        const bool have = tile_row < p.q.ntiles;
                        mbar_expect_tx(full_a(s), kPairABytes + (have ? 1024 * B : 0));
                        tma_load_2d(a_dst, &tmA, step * BK, my_m, full_a(s));
                        tma_load_2d(a_dst + 16384, &tmA, step * BK, my_m + 256, full_a(s));
                        if (have) bulk_load(p_dst, codes + (static_cast<size_t>(tile_row) * p.q.ktiles + step) * (1024 * B), 1024 * B, full_a(s));
                    } else {
                        const int nn0 = step * BK;
                        const int kt_base = (c0 >> 6) + static_cast<int>(rank) * 2;
                        int have = 0;
                        for (int t = 0; t < 2; ++t) if (kt_base + t < p.q.ktiles) ++have;
                        mbar_expect_tx(full_a(s), kPairABytes + have * 512 * B);
                        tma_load_2d(a_dst, &tmA, nn0, my_m, full_a(s));
                        tma_load_2d(a_dst + 16384, &tmA, nn0, my_m + 256, full_a(s));
                        for (int t = 0; t < have; ++t) {
                            const size_t tile = static_cast<size_t>(nn0 >> 7) * p.q.ktiles + kt_base + t;
                            bulk_load(p_dst + t * 512 * B, codes + tile * (1024 * B) + ((nn0 >> 6) & 1) * (512 * B), 512 * B, full_a(s));
                        }
                    }
                } else {
                    if (step == p.steps_q) {
                        pdl_wait();                       // the rank-r intermediate comes from the kernel in front
                        fence_proxy_async_all();
                    }
                    const int d = step - p.steps_q;
                    mbar_expect_tx(full_a(s), kPairABytes);
                    tma_load_2d(a_dst, &tmA2, d * BK, my_m, full_a(s));
                    tma_load_2d(a_dst + 16384, &tmA2, d * BK, my_m + 256, full_a(s));
                }
            }
            if (*abort_s) {
                for (int s = 0; s < SA; ++s) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(full_a(s), 0) && !mbar_try_wait(full_a(s), 1) && clock64() - t0 < 20000000LL) {}
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((BWD ? 1u : 0u) << 16) |
                                       (static_cast<uint32_t>(BN >> 3) << 17) | (static_cast<uint32_t>(256 >> 4) << 24);
            bool ok = true;
            RingPos<SA> ra;
            RingPos<SB> rb;
            for (int step = 0; step < total && ok; ++step, ra.advance(), rb.advance()) {
                const int sa = ra.s, sb = rb.s;
                // sixteen arrivals: the eight warps of this step in each CTA, each after its CTA's copies have landed
                ok = mbar_try_wait_acq_cluster(full_b(sb), rb.ph) || wait_cluster(full_b(sb), rb.ph, ctl, 42);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_src = smem_u32(a_ring) + sa * kPairABytes;
                const uint32_t b_src = smem_u32(b_ring) + sb * kPairBBytes;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
#pragma unroll
                    for (int k16 = 0; k16 < 4; ++k16) {
                        const uint64_t adesc = make_desc(a_src + h * 16384 + k16 * 32, 16, 1024);
                        const uint64_t bdesc = BWD ? make_desc(b_src + k16 * 2048, 8192, 1024)
                                                   : make_desc(b_src + k16 * 32, 16, 1024);
                        tc_mma2(tmem + h * BN, adesc, bdesc, idesc, (step > 0 || k16 > 0) ? 1u : 0u);
                    }
                }
                tc_commit_both(empty_a(sa));
                tc_commit_both(empty_b(sb));
            }
            if (ok) {
                tc_commit_both(acc_full);
            } else {
                tc_commit_both(drain);
                const long long t0 = clock64();
                while (!mbar_try_wait(drain, 0) && clock64() - t0 < 20000000LL) {}
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ dequantization warps, then epilogue
        const int dw = warp - 2;
        const int task = dw & 7, par = dw >> 3;           // this warp works on the steps with step % 2 == par
        int row_local, slab_words_off, my_col, my_row, tile_col;
        uint32_t b_off;
        int g;
        if (!BWD) {
            const int slab_i = task >> 1;
            g = task & 1;
            row_local = slab_i * 32 + lane;               // 0..127: row of this CTA's half of the weight tile
            b_off = row_local * 128;
            slab_words_off = slab_i * (64 * B) + g * (B * 32);
            my_row = c0 + static_cast<int>(rank) * 128 + row_local;
            my_col = g * 32;
            tile_col = 0;                                 // forward: the tile column is the step index
        } else {
            const int sub = task >> 2, slab2 = (task >> 1) & 1;
            g = task & 1;
            row_local = slab2 * 32 + lane;                // 0..63: contraction row of the step
            b_off = sub * 8192 + row_local * 128;
            slab_words_off = sub * (128 * B) + slab2 * (64 * B) + g * (B * 32);
            my_row = row_local;
            my_col = c0 + static_cast<int>(rank) * 128 + sub * 64 + g * 32;
            tile_col = (c0 >> 6) + static_cast<int>(rank) * 2 + sub;
        }
        const uint32_t xr = (row_local & 7) << 4;
        const bool two_scales = (p.q.B0 == 16);
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
        const uint32_t slab_base = smem_u32(p_ring) + slab_words_off * 4;        // byte address in shared memory
        const int slot_even = slab_row_slot(lane, g, tile_col);
        const int slot_odd = BWD ? slot_even : slab_row_slot(lane, g, 1);
        const uint32_t my_b = smem_u32(b_ring) + b_off;
        float v_cached = -1.0f, sigma = 0.0f, s_lo = 0.0f, s_hi = 0.0f;
        RawScale slot[4];
        // forward, rows aligned to 16 blocks: windows of 16 scale codes instead of one load per step
        const bool use_win = !BWD && (p.q.KB % 16 == 0);
        const bool win_row_ok = !BWD && my_row < p.q.N;
        ScaleWindow cur{make_uint4(0u, 0u, 0u, 0u), 0.0f}, nxt = cur;
        int cur_base = 0;
        if (use_win) {
            cur_base = ((par * BK + my_col) >> logB0) & ~15;
            cur = load_scale_window(p.q, blk0, cur_base, win_row_ok);
            nxt = load_scale_window(p.q, blk0, cur_base + 16, win_row_ok);
        } else {
#pragma unroll
            for (int u = 0; u < 4; ++u) slot[u] = (par + 2 * u < p.steps_q) ? fetch(par + 2 * u) : RawScale{0u, 0.0f};
        }
        bool ok = true;
        RingPos<SA> ra;
        RingPos<SB> rb;
        if (par) { ra.advance(); rb.advance(); }
        for (int step4 = par; step4 < total && ok; step4 += 8) {
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int step = step4 + 2 * u;
                if (step >= total || !ok) break;
                const int sa = ra.s, sb = rb.s;
                ok = wait(empty_b(sb), rb.ph ^ 1, ctl, 46);
                if (!ok) break;
                if (step < p.steps_q) {
                    if (use_win) {
                        const int b = (step * BK + my_col) >> logB0;
                        if ((b & ~15) != cur_base) {
                            cur = nxt;
                            cur_base += 16;
                            nxt = load_scale_window(p.q, blk0, cur_base + 16, win_row_ok);
                        }
                        make_scales(p.q, window_scale(cur, b, two_scales), v_cached, sigma, s_lo, s_hi);
                    } else {
                        make_scales(p.q, slot[u], v_cached, sigma, s_lo, s_hi);
                        if (step + 8 < p.steps_q) slot[u] = fetch(step + 8);
                    }
                    ok = wait(full_a(sa), ra.ph, ctl, 44);
                    if (!ok) break;
                    dequant_group<B, true>(slab_base + sa * P_BYTES + ((step & 1) ? slot_odd : slot_even) * 4, s_lo, s_hi, two_scales,
                                           my_b + sb * kPairBBytes, g << 6, xr, lut8 + lane);
                    fence_proxy_async();
                } else {
                    // rank-r step: the weight-side operand of this CTA's half comes by TMA
                    if (task == 0) {
                        if (lane == 0) {
                            const int d = step - p.steps_q;
                            const uint32_t dst = smem_u32(b_ring) + sb * kPairBBytes;
                            if (!BWD) {
                                mbar_expect_tx(dbar(sb), kPairBBytes);
                                tma_load_2d(dst, &tmB2, d * BK, c0 + static_cast<int>(rank) * 128, dbar(sb));
                            } else {
                                int have = 0;
                                for (int t = 0; t < 2; ++t) if (c0 + static_cast<int>(rank) * 128 + t * 64 < p.out_cols) ++have;
                                mbar_expect_tx(dbar(sb), have * 8192);
                                for (int t = 0; t < have; ++t)
                                    tma_load_2d(dst + t * 8192, &tmB2, c0 + static_cast<int>(rank) * 128 + t * 64, d * BK, dbar(sb));
                            }
                        }
                        ok = wait(dbar(sb), ((step - p.steps_q) / SB) & 1, ctl, 47) && wait(full_a(sa), ra.ph, ctl, 48);
                        if (!ok) break;
                    }
                }
                __syncwarp();
                if (lane == 0) {
                    if (rank == 0) mbar_arrive(full_b(sb));
                    else mbar_arrive_cluster(full_b(sb), 0);
                }
                ra.advance(); ra.advance();
                rb.advance(); rb.advance();
            }
        }
        // epilogue: a warp owns 32 accumulator lanes (rows) x 64 columns of both accumulators.  It rounds them to
        // bf16 into a private 4 KB tile of the (now idle) activation ring, in the 128-byte-swizzled layout of a
        // TMA box of 32 rows x 64 columns, and one lane stores the box with a bulk tensor copy, which clips at the
        // edges of the output.
        if (ok && wait(acc_full, 0, ctl, 45)) {
            tc_fence_after();
            const int quarter = warp & 3, colq = dw >> 2;
            const uint32_t xs = static_cast<uint32_t>(lane & 7);
            bool stored = false;
#pragma unroll 1
            for (int h = 0; h < 2; ++h) {
                uint8_t* stage = a_ring + (dw * 2 + h) * 4096;
                uint8_t* row = stage + lane * 128;
#pragma unroll 1
                for (int cc = 0; cc < 2; ++cc) {
                    uint32_t v[32];
                    tmem_ld32(tmem + (static_cast<uint32_t>(quarter * 32) << 16) + h * BN + colq * 64 + cc * 32, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(v[i * 8 + 2 * e]),
                                                                           __uint_as_float(v[i * 8 + 2 * e + 1]));
                            w[e] = *reinterpret_cast<const uint32_t*>(&hh);
                        }
                        *reinterpret_cast<uint4*>(row + (((cc * 4 + i) ^ xs) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
                fence_proxy_async();
                __syncwarp();
                const int x = c0 + colq * 64, y = m0 + h * 256 + static_cast<int>(rank) * 128 + quarter * 32;
                if (lane == 0 && x < p.out_cols && y < p.M) {
                    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];"
                                 ::"l"(reinterpret_cast<uint64_t>(&tmOut)), "r"(x), "r"(y), "r"(smem_u32(stage)) : "memory");
                    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    stored = true;
                }
            }
            if (stored) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
            __syncwarp();
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_barrier();            // neither CTA frees tensor memory or exits while the other may still use its shared memory
    if (warp == 1) tmem_dealloc2(tmem, TMEM_COLS);
}

template <int B, bool BWD>
inline int launch_pair(const CUtensorMap& tA, const CUtensorMap& tA2, const CUtensorMap& tB2, const CUtensorMap& tOut, Params p, cudaStream_t st) {
    constexpr int smem = pair_smem_bytes<B>();
    static_assert(smem <= kSmemLimit, "shared memory budget exceeded");
    auto kern = tc_pair_linear_kernel<B, BWD>;
    static bool attr_done = false;
    if (!attr_done) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit) != cudaSuccess) {
            cudaGetLastError();
            return LQLORA_ERR_CUDA;
        }
        attr_done = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * ((p.M + 511) / 512), p.c_tiles);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (p.steps_d > 0) ? 2 : 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tA, tA2, tB2, tOut, p);
    count_launch(1);
    if (e != cudaSuccess) { cudaGetLastError(); return LQLORA_ERR_CUDA; }
    return LQLORA_OK;
}

}  // namespace tc
}  // namespace lq
