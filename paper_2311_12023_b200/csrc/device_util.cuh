// Device-side helpers shared by the linear kernels: mbarrier / bulk-copy / programmatic-launch PTX
// wrappers and the register byte-table dequantization.
#pragma once

#include <cuda.h>   // CUtensorMap

#include "common.cuh"

namespace lq {
namespace dev {

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
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar) : "memory");
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may
// start while its predecessor in the stream still runs; pdl_wait() blocks until that predecessor
// has completed and its memory is visible, pdl_launch_dependents() lets the successor start early.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

constexpr long long kWaitCycles = 4000000000LL;   // about two seconds

// Bounded wait.  Returns false when the wait was abandoned (another thread aborted, or time ran out).
struct Ctl {
    volatile int* abort_s;
    int* status_g;
    long long budget = kWaitCycles;      // clock cycles a wait may take before it is abandoned
};
__device__ __noinline__ bool wait_slow(uint32_t bar, uint32_t parity, const Ctl& c, int where) {
    const long long t0 = clock64();
    for (int it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 63) == 63) {
            if (*c.abort_s) return false;
            if (clock64() - t0 > c.budget) {
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

// ------------------------------------------------------------------------------------ dequantization tables
// The 2^b0 products fl32(q~[c] * s~) of one block, rounded to bf16, are kept in registers as a
// byte table: lo[] holds the low bytes, hi[] the high bytes, four entries per register.  One
// byte-permute with a selector word (four 4-bit table indices) then fetches four low bytes, a
// second one the four high bytes, and two more interleave them into two bf16 pairs.  The results
// are the same bits as rounding each fp32 product on its own.
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
    uint32_t d;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
    return d;
}

template <int B> struct BlockTable {
    static constexpr int kRegs = (B == 2) ? 1 : (B == 3) ? 2 : 4;
    uint32_t lo[kRegs], hi[kRegs];
    __device__ __forceinline__ void build(float s) {
        const float* cb = c_codebook[bits_index(B)];
        uint32_t e[(1 << B) / 2];
#pragma unroll
        for (int i = 0; i < (1 << B) / 2; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(__fmul_rn(cb[2 * i], s), __fmul_rn(cb[2 * i + 1], s));
            e[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
#pragma unroll
        for (int j = 0; j < kRegs; ++j) {
            lo[j] = prmt(e[2 * j], e[2 * j + 1], 0x6420u);
            hi[j] = prmt(e[2 * j], e[2 * j + 1], 0x7531u);
        }
    }
    // four weights from the four indices in the low 16 bits of `sel` (sel2: second-level selector, 4-bit codes only)
    __device__ __forceinline__ void lookup4(uint32_t sel, uint32_t sel2, uint32_t& out0, uint32_t& out1) const {
        uint32_t l, h;
        if constexpr (B == 2) { l = prmt(lo[0], 0u, sel); h = prmt(hi[0], 0u, sel); }
        else if constexpr (B == 3) { l = prmt(lo[0], lo[1], sel); h = prmt(hi[0], hi[1], sel); }
        else {
            l = prmt(prmt(lo[0], lo[1], sel), prmt(lo[2], lo[3], sel), sel2);
            h = prmt(prmt(hi[0], hi[1], sel), prmt(hi[2], hi[3], sel), sel2);
        }
        out0 = prmt(l, h, 0x5140u);
        out1 = prmt(l, h, 0x7362u);
    }
};

// Selector word (eight 4-bit indices) of chunk c (columns 8c .. 8c+7 of the group) from the group's words.
template <int B>
__device__ __forceinline__ uint32_t chunk_selector(const uint32_t (&w)[B], int c) {
    if constexpr (B == 4) return w[c];
    else if constexpr (B == 2) return (c & 1) ? ((w[c >> 1] >> 2) & 0x33333333u) : (w[c >> 1] & 0x33333333u);
    else {
        if (c < 3) return w[c] & 0x77777777u;
        return ((w[0] >> 3) & 0x11111111u) | ((w[1] >> 2) & 0x22222222u) | ((w[2] >> 1) & 0x44444444u);
    }
}

}  // namespace dev
}  // namespace lq
