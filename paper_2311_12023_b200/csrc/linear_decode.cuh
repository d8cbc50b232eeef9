// Forward pass and input gradient for decode-sized inputs (M <= 16 rows): the packed matrix is streamed once.
//
//   - Forward: one CTA owns a tile row of Q (128 rows) and a slice of K.  The packed tiles of the CTA (they are
//     contiguous in memory) and the matching activations are streamed into a shared-memory ring with bulk copies: warp 0
//     fills the ring once, afterwards the warp that finishes a stage last refills its slot (no producer warp).  Eight
//     warps dequantize in registers with the byte-table method (bf16 bits identical to the exported dequantized
//     weights) and feed mma.sync m16n8k16 (weights = the 16-row operand, tokens = the 8-column operand, fp32
//     accumulators).  The contraction index is permuted so that a thread supplies 4 consecutive weights of one row per
//     MMA and reads the matching 4 activations with one 128-bit load per 8 columns.
//   - Block scales of the CTA's rows and columns are staged once in shared memory: as fp32 s~, or, where the slices
//     are uniform, as the 8-bit codes plus fl(v / 127) per 16 block columns (a quarter of the size; s~ is formed at use).
//   - The rank-r intermediate T = X L2^T comes from a small kernel launched in front; the two overlap (programmatic
//     dependent launch) and T L1^T is added on the tensor cores as a few more contraction steps after the main loop.
//   - The K slices of a tile row are added through global memory: every CTA stores its fp32 sums in its own slot of
//     the workspace and counts itself on the tile row's arrival counter; the CTA that arrives last adds the slots in
//     slice order (the same bits on every run) and writes the bf16 output.  No clusters: the CTAs spread over all SMs,
//     leave as soon as their sums are stored, and any number of slices is possible.  The counters are cleared by the
//     first kernel of the call (the pre-product, or the caller's memset when there is no rank-r term).
//   - The input gradient has the same structure with a CTA per window of 256 columns and slices of the rows.
#pragma once

#include "common.cuh"
#include "device_util.cuh"

namespace lq {
namespace dec {
using namespace dev;

constexpr int kConsumerWarps = 8;
constexpr int kThreads = kConsumerWarps * 32;
constexpr int kStageTiles = 4;              // 64-column tiles per ring stage of the forward kernel (two windows of 128 columns)
constexpr int kSmemLimit = 232448;
constexpr int kStabStride = 136;            // floats per block column of the scale table (128 rows + padding against bank conflicts)
constexpr int kStab8Stride = 148;           // bytes per block column of the compact scale table (8-bit codes; one sigma per 16 block columns)

constexpr int kXRowBytes = kStageTiles * kTileCols * 2 + 16;   // one token's activations of a stage, padded
// A ring stage: the packed tiles, then the activations of the stage's 512 columns for 8 NT token rows.
// NT = number of 8-token groups (1: M <= 8, two CTAs per SM; 2: M <= 16, one CTA per SM)
template <int B, int NT> __host__ __device__ constexpr int stage_bytes() { return kStageTiles * 1024 * B + 8 * NT * kXRowBytes; }
// CTAs per SM the forward kernel is compiled for: two (128 registers per thread), except for 8-bit codes with 16 tokens
template <int B, int NT> __host__ __device__ constexpr int fwd_ctas_per_sm() { return (B == 8 && NT == 2) ? 1 : 2; }
// Ring depth: what fits into about 84 KB per CTA (two CTAs per SM) or twice that, between two and eight stages
template <int B, int NT> __host__ __device__ constexpr int num_stages() {
    constexpr int budget = (fwd_ctas_per_sm<B, NT>() == 2 ? 84 : 168) * 1024;
    constexpr int n = budget / stage_bytes<B, NT>();
    return n < 2 ? 2 : n > 8 ? 8 : n;
}

struct Params {
    QView q;
    const __nv_bfloat16* X;    // [M][K]
    const __nv_bfloat16* T;    // [M][r], written by the kernel in front of this one (r > 0)
    const __nv_bfloat16* L1;   // [N][r]
    __nv_bfloat16* Y;          // [M][N]
    float* partial;            // [S][M][ntiles * 128] sums of the K slices (S > 1)
    int* counters;             // [ntiles] arrival counters, zero when the kernel starts (S > 1)
    int* status;
    int M, r;
    int S;                     // K slices per tile row
    int tiles_per_split;       // 64-column tiles per CTA (even)
    int nkb_cap;               // capacity of the scale table in blocks
    int stab8;                 // 1: compact scale table (codes as bytes + fl(v / 127) per 16 block columns), 0: fp32 table
};

__device__ __forceinline__ void mma16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Split cluster barrier: arrive early, wait where the guarantee is needed.
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.aligned;" ::: "memory"); }
__device__ __forceinline__ float ld_dsmem_f32(uint32_t local_addr, uint32_t rank) {
    uint32_t ra;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
    return v;
}

// Stores v at the shared-memory offset `local_addr` of CTA `rank` of the cluster.
__device__ __forceinline__ void st_dsmem_f32(uint32_t local_addr, uint32_t rank, float v) {
    uint32_t ra;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra), "f"(v) : "memory");
}

// Counts a warp as done with a ring slot; orders the warp's reads of the slot before the count and, for the warp
// that sees the last count, the other warps' reads before what it does next (the refill of the slot).
__device__ __forceinline__ uint32_t slot_done(uint32_t counter_smem) {
    uint32_t old;
    asm volatile("atom.acq_rel.cta.shared.add.u32 %0, [%1], 1;" : "=r"(old) : "r"(counter_smem) : "memory");
    return old;
}

__device__ __forceinline__ uint32_t pick(const uint4& v, int i) { return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w; }
__device__ __forceinline__ float pickf(const float4& v, int i) { return i == 0 ? v.x : i == 1 ? v.y : i == 2 ? v.z : v.w; }

// Chunk c (columns 8c .. 8c+7) of one (row, group) as four bf16 pairs: o[e] holds columns 8c + 2e, 8c + 2e + 1.
template <int B>
__device__ __forceinline__ void dequant_chunk(const uint32_t (&w)[B], int c, const BlockTable<B>& tab, float s,
                                              uint32_t (&o)[4], const float* __restrict__ lut8) {
    if constexpr (B == 8) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const uint32_t ww = w[2 * c + (e >> 1)] >> (16 * (e & 1));
            const float q0 = lut8[ww & 255u], q1 = lut8[(ww >> 8) & 255u];
            const __nv_bfloat162 h = __floats2bfloat162_rn(__fmul_rn(q0, s), __fmul_rn(q1, s));
            o[e] = *reinterpret_cast<const uint32_t*>(&h);
        }
    } else {
        const uint32_t sel = chunk_selector<B>(w, c);
        uint32_t selA = sel, selB = 0u;
        if constexpr (B == 4) { selA = sel & 0x77777777u; selB = ((sel >> 1) & 0x44444444u) | 0x32103210u; }
        tab.lookup4(selA, selB, o[0], o[1]);
        tab.lookup4(selA >> 16, selB >> 16, o[2], o[3]);
    }
}

// Loads VW consecutive scale codes (VW = 16, 8, 4: one vector load; 1: one byte) as four words.
template <int VW>
__device__ __forceinline__ uint4 load_scale_codes(const uint8_t* src) {
    uint4 w = make_uint4(0u, 0u, 0u, 0u);
    if constexpr (VW == 16) w = __ldg(reinterpret_cast<const uint4*>(src));
    else if constexpr (VW == 8) { const uint2 t2 = __ldg(reinterpret_cast<const uint2*>(src)); w.x = t2.x; w.y = t2.y; }
    else if constexpr (VW == 4) w.x = __ldg(reinterpret_cast<const uint32_t*>(src));
    else w.x = __ldg(src);
    return w;
}

// fp32 scale table of a forward CTA: stab[kb * kStabStride + row] = s~ of block column kb_first + kb of row
// tile_row * 128 + row (0 for rows past N), VW codes per load (the caller has checked alignment and divisibility).
// Two loads per thread are in flight; `after_first_loads` runs once, after the first loads have been issued.
template <int VW, typename F>
__device__ __forceinline__ void build_scale_table(const QView& q, int tile_row, int kb_first, int nkb, float* stab, F&& after_first_loads) {
    const int nvec = nkb / VW;
    const int total = nvec * 128;
    for (int e0 = threadIdx.x; e0 < total; e0 += 2 * kThreads) {
        uint4 sc[2];
        float v0[2], v1[2];
        int rowv[2], kbv[2];
        uint32_t blkv[2];
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int e = e0 + u * kThreads;
            sc[u] = make_uint4(0u, 0u, 0u, 0u); v0[u] = v1[u] = 0.0f; rowv[u] = -1; kbv[u] = 0; blkv[u] = 0u;
            if (e < total) {
                const int row = e / nvec, kv = e - row * nvec;
                const int grow = tile_row * 128 + row;
                rowv[u] = row; kbv[u] = kv * VW;
                if (grow < q.N) {
                    const uint32_t blk = static_cast<uint32_t>(grow) * q.KB + kb_first + kv * VW;
                    blkv[u] = blk;
                    sc[u] = load_scale_codes<VW>(q.sc + blk);
                    v0[u] = __ldg(q.v + (blk >> q.logB1));
                    v1[u] = __ldg(q.v + ((blk + VW - 1) >> q.logB1));          // B1 >= 16 >= VW: at most two groups
                }
            }
        }
        after_first_loads();
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            if (rowv[u] < 0) continue;
            const uint32_t g0 = blkv[u] >> q.logB1;
            const uint32_t words[4] = {sc[u].x, sc[u].y, sc[u].z, sc[u].w};
#pragma unroll
            for (int i = 0; i < VW; ++i) {
                const uint32_t code = (words[i >> 2] >> (8 * (i & 3))) & 255u;
                const float vv = (((blkv[u] + i) >> q.logB1) == g0) ? v0[u] : v1[u];
                stab[(kbv[u] + i) * kStabStride + rowv[u]] = block_scale(static_cast<uint8_t>(code), vv, q.levels);
            }
        }
    }
}

template <int B, int NT, bool TWO>
__global__ void __launch_bounds__(kThreads, fwd_ctas_per_sm<B, NT>())
decode_fwd_kernel(const Params p) {
    constexpr int NS = num_stages<B, NT>();
    constexpr int STAGE = stage_bytes<B, NT>();
    constexpr int XOFF = kStageTiles * 1024 * B;      // activations inside a stage
    constexpr int MT = 8 * NT;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
    uint8_t* ring = base;
    float* recv = reinterpret_cast<float*>(ring + NS * STAGE);        // [2 windows][MT][128 rows] sums of the two warps of a row
    float* lut8 = recv + 2 * 128 * MT;                                 // 256 floats (8-bit codes only)
    uint64_t* bars = reinterpret_cast<uint64_t*>(lut8 + (B == 8 ? 256 : 0));   // full[NS], then NS counters of warps done with a slot
    uint32_t* done = reinterpret_cast<uint32_t*>(bars + NS);
    volatile int* abort_s = reinterpret_cast<volatile int*>(bars + 2 * NS);
    volatile int* last_s = abort_s + 1;
    float* stab = reinterpret_cast<float*>(bars + 2 * NS + 2);         // [nkb][kStabStride] block scales s~ (fp32 table)
    // compact table: s^ as bytes [nkb][kStab8Stride], then sigma = fl(v / 127) as [nkb / 16][kStabStride] floats
    const uint8_t* stab8 = reinterpret_cast<const uint8_t*>(stab);
    const float* sig = reinterpret_cast<const float*>(stab8 + static_cast<size_t>(p.nkb_cap) * kStab8Stride);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int tile_row = blockIdx.x;
    const int split = blockIdx.y;
    const QView& q = p.q;
    const int kt0 = split * p.tiles_per_split;
    const int kt1 = min(q.ktiles, kt0 + p.tiles_per_split);
    const int ntiles_cta = max(0, kt1 - kt0);
    const int nstage_total = (ntiles_cta + kStageTiles - 1) / kStageTiles;
    const Ctl ctl{abort_s, p.status};

    auto full = [&](int s) { return smem_u32(bars + s); };

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(full(s), 1); done[s] = 0u; }
        *abort_s = 0;
        *last_s = 0;
        fence_barrier_init();
    }
    __syncthreads();

    const uint8_t* codes = reinterpret_cast<const uint8_t*>(q.codes) +
                           (static_cast<size_t>(tile_row) * q.ktiles + kt0) * (1024 * B);
    // One stage by one warp: lane 0 arms the barrier and requests the packed tiles (one contiguous run), lanes
    // 1 .. M each request one token row of the activations (a bulk copy costs its issuing thread about a hundred
    // clocks, so the copies of a stage are issued side by side).
    auto issue_stage = [&](int it, int ln) {
        const int s = it % NS;
        const int nt = min(kStageTiles, ntiles_cta - it * kStageTiles);
        const uint32_t dst = smem_u32(ring + s * STAGE);
        if (ln == 0) {
            mbar_expect_tx(full(s), nt * 1024 * B + p.M * nt * (kTileCols * 2));
            bulk_load(dst, codes + static_cast<size_t>(it) * (kStageTiles * 1024 * B), nt * 1024 * B, full(s));
        } else if (ln <= p.M) {
            const int m = ln - 1;
            const __nv_bfloat16* xsrc = p.X + static_cast<size_t>(kt0 + it * kStageTiles) * kTileCols + static_cast<size_t>(m) * q.K;
            bulk_load(dst + XOFF + m * kXRowBytes, xsrc, nt * (kTileCols * 2), full(s));
        }
    };
    // There is no producer warp: warp 0 fills the ring once, afterwards the warp that is last to finish a stage
    // refills its slot (nobody waits for a free slot, and the CTA has eight warps, two per scheduler).  The stages are
    // small (four tiles) so that the first one of every CTA arrives early and the dequantization, which is what
    // binds, starts while the rest of the ring is still on its way.  The first fill is issued right after the first
    // loads of the scale table below, which are few and should not queue behind the bulk copies.
    bool ring_filled = false;
    auto fill_ring = [&]() {
        if (!ring_filled && warp == 0) {
            for (int it = 0; it < NS && it < nstage_total; ++it) issue_stage(it, lane);
        }
        ring_filled = true;
    };

    // block scales of the CTA's rows and columns: s~ = fl32(float(s^) * fl32(v / 127)), 0 for rows past N
    const int kb_first = (kt0 * kTileCols) >> q.logB0;
    const int nkb = (ntiles_cta > 0) ? (((kt1 * kTileCols - 1) >> q.logB0) - kb_first + 1) : 0;
    if (p.stab8) {
        // the host chose this form only where every CTA meets the conditions of the 16-code loads; the 16 codes of a
        // load share their second-level group (aligned, B1 >= 16)
        uint8_t* st8 = reinterpret_cast<uint8_t*>(stab);
        float* sg = reinterpret_cast<float*>(st8 + static_cast<size_t>(p.nkb_cap) * kStab8Stride);
        const int nvec = nkb >> 4;
        for (int e0 = threadIdx.x; e0 < nvec * 128; e0 += 2 * kThreads) {
            uint4 sc16[2];
            float v0[2];
            int rowv[2], kvv[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int e = e0 + u * kThreads;
                sc16[u] = make_uint4(0u, 0u, 0u, 0u); v0[u] = 0.0f; rowv[u] = -1; kvv[u] = 0;
                if (e < nvec * 128) {
                    const int row = e / nvec, kv = e - row * nvec;
                    const int grow = tile_row * 128 + row;
                    rowv[u] = row; kvv[u] = kv;
                    if (grow < q.N) {
                        const uint32_t blk = static_cast<uint32_t>(grow) * q.KB + kb_first + kv * 16;
                        sc16[u] = __ldg(reinterpret_cast<const uint4*>(q.sc + blk));
                        v0[u] = __ldg(q.v + (blk >> q.logB1));
                    }
                }
            }
            fill_ring();
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if (rowv[u] < 0) continue;
                const uint32_t words[4] = {sc16[u].x, sc16[u].y, sc16[u].z, sc16[u].w};
#pragma unroll
                for (int i = 0; i < 16; ++i)
                    st8[(kvv[u] * 16 + i) * kStab8Stride + rowv[u]] = static_cast<uint8_t>((words[i >> 2] >> (8 * (i & 3))) & 255u);
                sg[kvv[u] * kStabStride + rowv[u]] = __fdiv_rn(v0[u], q.levels);
            }
        }
    } else {
        // as many codes per load as the alignment of the CTA's run of blocks allows
        const int al = q.KB | nkb | kb_first;
        if ((al & 15) == 0) build_scale_table<16>(q, tile_row, kb_first, nkb, stab, fill_ring);
        else if ((al & 7) == 0) build_scale_table<8>(q, tile_row, kb_first, nkb, stab, fill_ring);
        else if ((al & 3) == 0) build_scale_table<4>(q, tile_row, kb_first, nkb, stab, fill_ring);
        else build_scale_table<1>(q, tile_row, kb_first, nkb, stab, fill_ring);
    }
    fill_ring();          // (a CTA without blocks has not passed through the loops above)
    if constexpr (B == 8) {
        for (int i = threadIdx.x; i < 256; i += kThreads) lut8[i] = c_codebook[3][i];
    }
    __syncthreads();

    // acc[set][nt][e]: row 4 gid + 2 set + (e >> 1) of the warp's slab, token nt * 8 + 2 t + (e & 1)
    float acc[2][NT][4];
#pragma unroll
    for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int c = 0; c < NT; ++c)
#pragma unroll
            for (int d = 0; d < 4; ++d) acc[a][c][d] = 0.0f;

    // ------------------------------------------------------------------ main loop
    // A stage holds four tiles = two windows of 128 columns; warp w takes slab (w & 3) of window (w >> 2): lane
    // (gid, t) dequantizes rows 4 gid .. 4 gid + 3 of the 32-column group (t & 1) of tile 2 (w >> 2) + (t >> 1).
    const int gid = lane >> 2, t = lane & 3;
    const int slab = warp & 3, window = warp >> 2;
    {
        bool ok = true;
        for (int it = 0; it < nstage_total && ok; ++it) {
            const int s = it % NS;
            const int tiles_here = min(kStageTiles, ntiles_cta - it * kStageTiles);
            const bool active = 2 * window < tiles_here;
            const int tile_in_stage = 2 * window + (t >> 1);
            const bool kt_ok = tile_in_stage < tiles_here;
            const int col0 = (kt0 + it * kStageTiles + tile_in_stage) * kTileCols + (t & 1) * 32;
            ok = wait(full(s), (it / NS) & 1, ctl, 22);
            if (!ok) break;
            if (active) {
                const uint32_t* tile = reinterpret_cast<const uint32_t*>(ring + s * STAGE) + (kt_ok ? tile_in_stage : 0) * (256 * B);
                const int kb = kt_ok ? ((col0 >> q.logB0) - kb_first) : 0;
                // activations of this thread's 32 columns (token rows past M and missing tiles read as zero)
                const uint8_t* xbase = ring + s * STAGE + XOFF + (tile_in_stage * kTileCols + (t & 1) * 32) * 2;
                uint4 x0[4];
                {
                    const bool have = gid < p.M && kt_ok;
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        x0[c] = have ? reinterpret_cast<const uint4*>(xbase + gid * kXRowBytes)[c] : make_uint4(0u, 0u, 0u, 0u);
                }
                uint4 x1[NT == 2 ? 4 : 1];
                if constexpr (NT == 2) {
                    const bool have1 = gid + 8 < p.M && kt_ok;
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        x1[c] = have1 ? reinterpret_cast<const uint4*>(xbase + (gid + 8) * kXRowBytes)[c] : make_uint4(0u, 0u, 0u, 0u);
                }
                const uint32_t* sp = tile + slab * (64 * B) + (t & 1) * (B * 32) + slab_row_slot(4 * gid, t & 1, tile_in_stage);
                uint4 w4[B];
#pragma unroll
                for (int i = 0; i < B; ++i) w4[i] = *reinterpret_cast<const uint4*>(sp + i * 32);
                float4 sc_lo, sc_hi;
                if (p.stab8) {
                    // s~ = fl32(float(s^) * fl32(v / 127)) from the compact table
                    const float4 sg4 = *reinterpret_cast<const float4*>(sig + (kb >> 4) * kStabStride + slab * 32 + 4 * gid);
                    const uint32_t c_lo = *reinterpret_cast<const uint32_t*>(stab8 + kb * kStab8Stride + slab * 32 + 4 * gid);
                    sc_lo = make_float4(__fmul_rn(static_cast<float>(c_lo & 255u), sg4.x), __fmul_rn(static_cast<float>((c_lo >> 8) & 255u), sg4.y),
                                        __fmul_rn(static_cast<float>((c_lo >> 16) & 255u), sg4.z), __fmul_rn(static_cast<float>(c_lo >> 24), sg4.w));
                    sc_hi = sc_lo;
                    if (TWO) {
                        // kb is even here (two blocks of 16 columns per 32-column group), so kb + 1 has the same sigma
                        const uint32_t c_hi = *reinterpret_cast<const uint32_t*>(stab8 + (kb + 1) * kStab8Stride + slab * 32 + 4 * gid);
                        sc_hi = make_float4(__fmul_rn(static_cast<float>(c_hi & 255u), sg4.x), __fmul_rn(static_cast<float>((c_hi >> 8) & 255u), sg4.y),
                                            __fmul_rn(static_cast<float>((c_hi >> 16) & 255u), sg4.z), __fmul_rn(static_cast<float>(c_hi >> 24), sg4.w));
                    }
                } else {
                    sc_lo = *reinterpret_cast<const float4*>(stab + kb * kStabStride + slab * 32 + 4 * gid);
                    sc_hi = sc_lo;
                    if (TWO) sc_hi = *reinterpret_cast<const float4*>(stab + (kb + 1) * kStabStride + slab * 32 + 4 * gid);
                }
                if (!kt_ok) { sc_lo = make_float4(0.f, 0.f, 0.f, 0.f); sc_hi = sc_lo; }
#pragma unroll
                for (int set = 0; set < 2; ++set) {
                    // rows a = 2 set, b = 2 set + 1 of the thread's four; the two MMAs of a chunk are issued right
                    // after its eight weights are ready, so consecutive MMAs on one accumulator are spaced out
                    uint32_t wa[B], wb[B];
#pragma unroll
                    for (int i = 0; i < B; ++i) { wa[i] = pick(w4[i], 2 * set); wb[i] = pick(w4[i], 2 * set + 1); }
                    const float sa_lo = pickf(sc_lo, 2 * set), sb_lo = pickf(sc_lo, 2 * set + 1);
                    const float sa_hi = pickf(sc_hi, 2 * set), sb_hi = pickf(sc_hi, 2 * set + 1);
                    BlockTable<B> ta, tb;
                    if constexpr (B != 8) { ta.build(sa_lo); tb.build(sb_lo); }
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        if constexpr (B != 8) {
                            if (TWO && c == 2) { ta.build(sa_hi); tb.build(sb_hi); }
                        }
                        uint32_t oa[4], ob[4];
                        dequant_chunk<B>(wa, c, ta, (TWO && c >= 2) ? sa_hi : sa_lo, oa, lut8);
                        dequant_chunk<B>(wb, c, tb, (TWO && c >= 2) ? sb_hi : sb_lo, ob, lut8);
                        mma16816(acc[set][0], oa[0], ob[0], oa[1], ob[1], x0[c].x, x0[c].y);
                        mma16816(acc[set][0], oa[2], ob[2], oa[3], ob[3], x0[c].z, x0[c].w);
                        if constexpr (NT == 2) {
                            mma16816(acc[set][1], oa[0], ob[0], oa[1], ob[1], x1[c].x, x1[c].y);
                            mma16816(acc[set][1], oa[2], ob[2], oa[3], ob[3], x1[c].z, x1[c].w);
                        }
                    }
                }
            }
            __syncwarp();
            uint32_t last = 0u;
            if (lane == 0) last = (slot_done(smem_u32(done + s)) == kConsumerWarps - 1) ? 1u : 0u;
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                // this warp is the last one done with the slot: it refills it
                if (lane == 0) done[s] = 0u;
                if (it + NS < nstage_total && !*abort_s) issue_stage(it + NS, lane);
            }
        }
    }

    // ---------------------------------------------------------------------- rank-r term, reduction, output
    __syncthreads();
    if (*abort_s) {
        // a wait gave up: let copies that are still in flight land before the CTA exits (bounded)
        if (threadIdx.x == 0) {
            for (int s = 0; s < NS; ++s) {
                const long long t0 = clock64();
                while (!mbar_try_wait(full(s), 0) && !mbar_try_wait(full(s), 1) && clock64() - t0 < 20000000LL) {}
            }
        }
        __syncthreads();
    }
    // The kernel launched in front of this one has written T and cleared the arrival counters: wait for it here.
    if (p.r > 0) pdl_wait();
    // T L1^T on the tensor cores, as more contraction steps of the same accumulators (first K slice only): 16 columns
    // of the factors per MMA, lane t supplies columns 4 t .. 4 t + 3 of the rows a, b of its set and of the tokens
    // gid (gid + 8); the warps of window 0 take the even groups of 16 columns, those of window 1 the odd ones.
    if (p.r > 0 && split == 0) {
        const int n0 = tile_row * 128 + slab * 32 + 4 * gid;
        for (int ch = window; ch * 16 < p.r; ch += 2) {
            const int j = ch * 16 + 4 * t;
            uint2 tk0 = make_uint2(0u, 0u), tk1 = make_uint2(0u, 0u);
            if (gid < p.M) tk0 = __ldcg(reinterpret_cast<const uint2*>(p.T + static_cast<size_t>(gid) * p.r + j));
            if (NT == 2 && gid + 8 < p.M) tk1 = __ldcg(reinterpret_cast<const uint2*>(p.T + static_cast<size_t>(gid + 8) * p.r + j));
#pragma unroll
            for (int set = 0; set < 2; ++set) {
                const int na = n0 + 2 * set, nb = na + 1;
                uint2 la = make_uint2(0u, 0u), lb = make_uint2(0u, 0u);
                if (na < q.N) la = __ldg(reinterpret_cast<const uint2*>(p.L1 + static_cast<size_t>(na) * p.r + j));
                if (nb < q.N) lb = __ldg(reinterpret_cast<const uint2*>(p.L1 + static_cast<size_t>(nb) * p.r + j));
                mma16816(acc[set][0], la.x, lb.x, la.y, lb.y, tk0.x, tk0.y);
                if constexpr (NT == 2) mma16816(acc[set][1], la.x, lb.x, la.y, lb.y, tk1.x, tk1.y);
            }
        }
    }
    // the two warps that cover the same rows (windows 0 and 1) meet in shared memory: recv[(window * MT + m) * 128 + row]
#pragma unroll
    for (int set = 0; set < 2; ++set)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int row = slab * 32 + 4 * gid + 2 * set + (e >> 1);
                const int m = nt * 8 + 2 * t + (e & 1);
                if (m < p.M) recv[(window * MT + m) * 128 + row] = acc[set][nt][e];
            }
    __syncthreads();
    const int npad = q.ntiles * 128;
    if (p.S == 1) {
        for (int idx = threadIdx.x; idx < 128 * p.M; idx += kThreads) {
            const int m = idx >> 7, row = idx & 127;
            const int n = tile_row * 128 + row;
            if (n < q.N) p.Y[static_cast<size_t>(m) * q.N + n] = __float2bfloat16_rn(recv[m * 128 + row] + recv[(MT + m) * 128 + row]);
        }
        return;
    }
    // several K slices: store this CTA's sums in its slot, count it on the tile row's counter; the last one adds up
    for (int idx = threadIdx.x; idx < 128 * p.M; idx += kThreads) {
        const int m = idx >> 7, row = idx & 127;
        __stcg(p.partial + (static_cast<size_t>(split) * p.M + m) * npad + tile_row * 128 + row, recv[m * 128 + row] + recv[(MT + m) * 128 + row]);
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) *last_s = (atomicAdd(p.counters + tile_row, 1) == p.S - 1) ? 1 : 0;
    __syncthreads();
    if (!*last_s) return;
    __threadfence();
    for (int idx = threadIdx.x; idx < 128 * p.M; idx += kThreads) {
        const int m = idx >> 7, row = idx & 127;
        const int n = tile_row * 128 + row;
        const float* src = p.partial + static_cast<size_t>(m) * npad + n;
        float sum = 0.0f;
        for (int sp = 0; sp < p.S; ++sp) sum += __ldcg(src + static_cast<size_t>(sp) * p.M * npad);
        if (n < q.N) p.Y[static_cast<size_t>(m) * q.N + n] = __float2bfloat16_rn(sum);
    }
}

// ------------------------------------------------------------------------------------ input gradient for few rows
// dX[m][k] = sum_n dY[m][n] deq16(Q)[n][k] + sum_j T'[m][j] L2[j][k],  M <= 16.
// One CTA owns a window of 256 columns of Q (four 64-column tiles) and a slice of the rows; the row slices
// of a window form a cluster.  A ring stage holds two tile rows (256 rows x 256 columns of packed codes,
// two contiguous pieces) and the matching 256 entries of every dY row.  Work item of a warp: 16 rows x 256
// columns; lane (gid, t) holds rows 4t .. 4t+3 and the 32-column group gid.  The contraction runs over
// rows, so the tensor-core operand needs pairs (W[n][k], W[n+1][k]): the byte-table look-ups of two rows
// are merged by two more byte-permute stages (three permutes per two weights instead of two).
// mma.sync m16n8k16: 16 columns x 16 rows (weights) times 16 rows x 8 tokens (dY).
struct BwdParams {
    QView q;
    const __nv_bfloat16* dY;   // [M][N]
    const __nv_bfloat16* T;    // [M][r] = dY L1, written by the kernel in front of this one (r > 0)
    const __nv_bfloat16* L2;   // [r][K]
    __nv_bfloat16* dX;         // [M][K]
    float* partial;            // [S][M][nwin * 256] sums of the row slices (S > 1)
    int* counters;             // [nwin] arrival counters, zero when the kernel starts (S > 1)
    int* status;
    int M, r;
    int S;                     // row slices per column window
    int trows_per_split;       // tile rows (128 rows) per CTA, even
    int rows_stride;           // entries per block column of the scale table
    int stab8;                 // 1: compact scale table (codes as bytes [nkb][rows_stride] + fl(v / 127) per row), 0: fp32 table
    int nkb_cap;               // block columns of the table
};

constexpr int kBwdStageRows = 256;
constexpr int kBwdYRowBytes = kBwdStageRows * 2 + 16;
template <int B, int NT> __host__ __device__ constexpr int bwd_stage_bytes() { return 8 * 1024 * B + 8 * NT * kBwdYRowBytes; }
// CTAs per SM the input-gradient kernel is compiled for: two for up to 8 tokens and 2/3-bit codes
template <int B, int NT> __host__ __device__ constexpr int bwd_ctas_per_sm() { return (NT == 1 && B <= 3) ? 2 : 1; }
template <int B, int NT> __host__ __device__ constexpr int bwd_stages() { return (B == 8 || bwd_ctas_per_sm<B, NT>() == 2) ? 2 : 3; }

// C8: compact scale table (codes as bytes [nkb][rows_stride] + fl(v / 127) per row) instead of the fp32 table
template <int B, int NT, bool TWO, bool C8>
__global__ void __launch_bounds__(kThreads, bwd_ctas_per_sm<B, NT>())
decode_bwd_kernel(const BwdParams p) {
    constexpr int NS = bwd_stages<B, NT>();
    constexpr int STAGE = bwd_stage_bytes<B, NT>();
    constexpr int YOFF = 8 * 1024 * B;
    constexpr int KF = 64 * NT;            // accumulator registers per thread

    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
    uint8_t* ring = base;
    float* outs = reinterpret_cast<float*>(ring + NS * STAGE);        // [8 NT tokens][256 columns] sums of the CTA
    float* lut8 = outs + KF * 32;
    uint64_t* bars = reinterpret_cast<uint64_t*>(lut8 + (B == 8 ? 256 : 0));   // full[NS], then NS counters of warps done with a slot
    uint32_t* done = reinterpret_cast<uint32_t*>(bars + NS);
    volatile int* abort_s = reinterpret_cast<volatile int*>(bars + 2 * NS);
    volatile int* last_s = abort_s + 1;
    float* stab = reinterpret_cast<float*>(bars + 2 * NS + 2);         // [nkb][rows_stride] block scales s~

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const QView& q = p.q;
    const int cw = blockIdx.x, split = blockIdx.y;
    const int kt_first = 4 * cw;
    const int ncol_tiles = min(4, q.ktiles - kt_first);
    const int tr0 = split * p.trows_per_split;
    const int tr1 = min(q.ntiles, tr0 + p.trows_per_split);
    const int ntr_cta = max(0, tr1 - tr0);
    const int nstage_total = (ntr_cta + 1) >> 1;
    const Ctl ctl{abort_s, p.status};

    auto full = [&](int s) { return smem_u32(bars + s); };

    if (threadIdx.x == 0) {
        for (int s = 0; s < NS; ++s) { mbar_init(full(s), 1); done[s] = 0u; }
        *abort_s = 0;
        fence_barrier_init();
    }
    __syncthreads();

    const uint8_t* codes = reinterpret_cast<const uint8_t*>(q.codes);
    // One stage by one warp: lane 0 arms the barrier, lanes 0 and 1 request the two runs of packed tiles, lanes
    // 2 .. M + 1 one row of dY each (the copies of a stage are issued side by side).
    auto issue_stage = [&](int it, int ln) {
        const int s = it % NS;
        const int ntr = min(2, ntr_cta - 2 * it);
        const uint32_t dst = smem_u32(ring + s * STAGE);
        const int row0 = (tr0 + 2 * it) * 128;
        const int nrows = min(ntr * 128, q.N - row0);             // entries of dY that exist (a multiple of 8)
        if (ln == 0) mbar_expect_tx(full(s), ntr * ncol_tiles * 1024 * B + p.M * nrows * 2);
        if (ln < ntr)
            bulk_load(dst + ln * (4 * 1024 * B), codes + (static_cast<size_t>(tr0 + 2 * it + ln) * q.ktiles + kt_first) * (1024 * B),
                      ncol_tiles * 1024 * B, full(s));
        else if (ln >= 2 && ln < 2 + p.M) {
            const int m = ln - 2;
            bulk_load(dst + YOFF + m * kBwdYRowBytes, p.dY + static_cast<size_t>(m) * q.N + row0, nrows * 2, full(s));
        }
    };
    // warp 0 fills the ring once (after the first loads of the scale table below have been issued, so that they do
    // not queue behind the bulk copies); afterwards the warp that is last to finish a stage refills its slot
    bool ring_filled = false;
    auto fill_ring = [&]() {
        if (!ring_filled && warp == 0) {
            for (int it = 0; it < NS && it < nstage_total; ++it) issue_stage(it, lane);
        }
        ring_filled = true;
    };

    // block scales of the CTA's rows and its (at most 256) columns
    const int col_first = kt_first * kTileCols;
    const int kb_first = col_first >> q.logB0;
    const int nkb = (((col_first + ncol_tiles * kTileCols - 1) >> q.logB0) - kb_first) + 1;
    const int nrows_cta = ntr_cta * 128;
    // Fast path: the nkb scale codes of a row segment are contiguous, a power of two in number, aligned, and share
    // one second-level group (B1 >= 16 >= nkb, both powers of two) -> one vector load per row, four rows in flight.
    const bool seg_vec = ncol_tiles == 4 && nkb <= 16 && (nkb & (nkb - 1)) == 0 && (q.KB % nkb) == 0 && (kb_first % nkb) == 0 &&
                         (1 << q.logB1) >= nkb;
    // compact table (chosen by the host only where every CTA meets the conditions above): s^ as bytes, sigma per row
    uint8_t* st8 = reinterpret_cast<uint8_t*>(stab);
    float* sg = reinterpret_cast<float*>(st8 + static_cast<size_t>(p.nkb_cap) * p.rows_stride);
    if (seg_vec) {
        for (int r0 = threadIdx.x; r0 < nrows_cta; r0 += 4 * kThreads) {
            uint4 sc16[4];
            float v[4];
            int rowv[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int row = r0 + u * kThreads;
                sc16[u] = make_uint4(0u, 0u, 0u, 0u); v[u] = 0.0f; rowv[u] = -1;
                if (row < nrows_cta) {
                    rowv[u] = row;
                    const int grow = tr0 * 128 + row;
                    if (grow < q.N) {
                        const uint32_t blk = static_cast<uint32_t>(grow) * q.KB + kb_first;
                        const uint8_t* src = q.sc + blk;
                        if (nkb == 16) sc16[u] = __ldg(reinterpret_cast<const uint4*>(src));
                        else if (nkb == 8) { const uint2 t2 = __ldg(reinterpret_cast<const uint2*>(src)); sc16[u].x = t2.x; sc16[u].y = t2.y; }
                        else if (nkb == 4) sc16[u].x = __ldg(reinterpret_cast<const uint32_t*>(src));
                        else if (nkb == 2) sc16[u].x = __ldg(reinterpret_cast<const uint16_t*>(src));
                        else sc16[u].x = __ldg(src);
                        v[u] = __ldg(q.v + (blk >> q.logB1));
                    }
                }
            }
            fill_ring();
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (rowv[u] < 0) continue;
                const uint32_t words[4] = {sc16[u].x, sc16[u].y, sc16[u].z, sc16[u].w};
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    if (i < nkb) {
                        const uint32_t code = (words[i >> 2] >> (8 * (i & 3))) & 255u;
                        if constexpr (C8) st8[i * p.rows_stride + rowv[u]] = static_cast<uint8_t>(code);
                        else stab[i * p.rows_stride + rowv[u]] = block_scale(static_cast<uint8_t>(code), v[u], q.levels);
                    }
                }
                if constexpr (C8) sg[rowv[u]] = __fdiv_rn(v[u], q.levels);
            }
        }
    } else {
    for (int e0 = threadIdx.x; e0 < nkb * nrows_cta; e0 += 4 * kThreads) {
        uint32_t sc8[4];
        float v[4];
        int slot[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int e = e0 + u * kThreads;
            sc8[u] = 0u; v[u] = 0.0f; slot[u] = -1;
            if (e < nkb * nrows_cta) {
                const int row = e / nkb, kb = e - row * nkb;
                const int grow = tr0 * 128 + row;
                slot[u] = kb * p.rows_stride + row;
                if (grow < q.N) {
                    const uint32_t blk = static_cast<uint32_t>(grow) * q.KB + kb_first + kb;
                    sc8[u] = __ldg(q.sc + blk);
                    v[u] = __ldg(q.v + (blk >> q.logB1));
                }
            }
        }
        fill_ring();
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (slot[u] >= 0) stab[slot[u]] = block_scale(static_cast<uint8_t>(sc8[u]), v[u], q.levels);
    }
    }
    fill_ring();
    if constexpr (B == 8) {
        for (int i = threadIdx.x; i < 256; i += kThreads) lut8[i] = c_codebook[3][i];
    }
    __syncthreads();

    // acc[mm][nt][e]: mm = chunk * 4 + half * 2 + pair -> columns cA = 8 chunk + 4 half + 2 pair (e < 2) and cA + 1 (e >= 2)
    // of the thread's group; token nt * 8 + 2 t + (e & 1)
    float acc[16][NT][4];
#pragma unroll
    for (int a = 0; a < 16; ++a)
#pragma unroll
        for (int b = 0; b < NT; ++b)
#pragma unroll
            for (int d = 0; d < 4; ++d) acc[a][b][d] = 0.0f;

    {
        const int gid = lane >> 2, t = lane & 3;
        const int ctile = gid >> 1, grp = gid & 1;
        const bool col_ok = ctile < ncol_tiles;
        const int kb = col_ok ? (((col_first + ctile * kTileCols + grp * 32) >> q.logB0) - kb_first) : 0;
        bool ok = true;
        for (int it = 0; it < nstage_total && ok; ++it) {
            const int s = it % NS;
            const int ntr = min(2, ntr_cta - 2 * it);
            ok = wait(full(s), (it / NS) & 1, ctl, 32);
            if (!ok) break;
            const uint8_t* stage = ring + s * STAGE;
#pragma unroll 1
            for (int ii = 0; ii < 2; ++ii) {
                const int item = warp * 2 + ii;                 // 0..15: tile row j, half-slab hs
                const int j = item >> 3, hs = item & 7;
                if (j >= ntr) continue;
                const int slab = hs >> 1, row_in_tile = slab * 32 + (hs & 1) * 16 + 4 * t;
                const int row_local = (2 * it + j) * 128 + row_in_tile;       // within the CTA's rows
                const bool row_ok = tr0 * 128 + row_local < q.N;
                const uint32_t* sp = reinterpret_cast<const uint32_t*>(stage) + (j * 4 + (col_ok ? ctile : 0)) * (256 * B) + slab * (64 * B) +
                                     grp * (B * 32) + slab_row_slot((hs & 1) * 16 + 4 * t, grp, ctile);
                uint4 w4[B];
#pragma unroll
                for (int i = 0; i < B; ++i) w4[i] = *reinterpret_cast<const uint4*>(sp + i * 32);
                float4 sc_lo, sc_hi;
                if constexpr (C8) {
                    // s~ = fl32(float(s^) * fl32(v / 127)) from the compact table
                    const float4 sg4 = *reinterpret_cast<const float4*>(sg + row_local);
                    const uint32_t c_lo = *reinterpret_cast<const uint32_t*>(st8 + kb * p.rows_stride + row_local);
                    sc_lo = make_float4(__fmul_rn(static_cast<float>(c_lo & 255u), sg4.x), __fmul_rn(static_cast<float>((c_lo >> 8) & 255u), sg4.y),
                                        __fmul_rn(static_cast<float>((c_lo >> 16) & 255u), sg4.z), __fmul_rn(static_cast<float>(c_lo >> 24), sg4.w));
                    sc_hi = sc_lo;
                    if (TWO) {
                        const uint32_t c_hi = *reinterpret_cast<const uint32_t*>(st8 + (kb + 1) * p.rows_stride + row_local);
                        sc_hi = make_float4(__fmul_rn(static_cast<float>(c_hi & 255u), sg4.x), __fmul_rn(static_cast<float>((c_hi >> 8) & 255u), sg4.y),
                                            __fmul_rn(static_cast<float>((c_hi >> 16) & 255u), sg4.z), __fmul_rn(static_cast<float>(c_hi >> 24), sg4.w));
                    }
                } else {
                    sc_lo = *reinterpret_cast<const float4*>(stab + kb * p.rows_stride + row_local);
                    sc_hi = sc_lo;
                    if (TWO) sc_hi = *reinterpret_cast<const float4*>(stab + (kb + 1) * p.rows_stride + row_local);
                }
                if (!col_ok) { sc_lo = make_float4(0.f, 0.f, 0.f, 0.f); sc_hi = sc_lo; }
                // dY of the four rows for this lane's token(s)
                uint32_t y0[NT], y1[NT];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    const int m = nt * 8 + gid;
                    y0[nt] = 0u; y1[nt] = 0u;
                    if (m < p.M && row_ok) {
                        const uint2 yy = *reinterpret_cast<const uint2*>(stage + YOFF + m * kBwdYRowBytes + (j * 128 + row_in_tile) * 2);
                        y0[nt] = yy.x; y1[nt] = yy.y;
                    }
                }
                uint32_t w[4][B];
#pragma unroll
                for (int rr = 0; rr < 4; ++rr)
#pragma unroll
                    for (int i = 0; i < B; ++i) w[rr][i] = pick(w4[i], rr);
                BlockTable<B> tab[4];
                if constexpr (B != 8) {
#pragma unroll
                    for (int rr = 0; rr < 4; ++rr) tab[rr].build(pickf(sc_lo, rr));
                }
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    if constexpr (B != 8) {
                        if (TWO && c == 2) {
#pragma unroll
                            for (int rr = 0; rr < 4; ++rr) tab[rr].build(pickf(sc_hi, rr));
                        }
                    }
                    uint32_t o[4][4];      // o[row][e]: columns 8c + 2e, 8c + 2e + 1 of the row
#pragma unroll
                    for (int rr = 0; rr < 4; ++rr) dequant_chunk<B>(w[rr], c, tab[rr], pickf((TWO && c >= 2) ? sc_hi : sc_lo, rr), o[rr], lut8);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        // columns cA = 8c + 2e, cB = cA + 1: pairs along the rows
                        const uint32_t a0 = prmt(o[0][e], o[1][e], 0x5410u), a1 = prmt(o[0][e], o[1][e], 0x7632u);
                        const uint32_t a2 = prmt(o[2][e], o[3][e], 0x5410u), a3 = prmt(o[2][e], o[3][e], 0x7632u);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) mma16816(acc[c * 4 + e][nt], a0, a1, a2, a3, y0[nt], y1[nt]);
                    }
                }
            }
            __syncwarp();
            uint32_t last = 0u;
            if (lane == 0) last = (slot_done(smem_u32(done + s)) == kConsumerWarps - 1) ? 1u : 0u;
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                if (lane == 0) done[s] = 0u;
                if (it + NS < nstage_total && !*abort_s) issue_stage(it + NS, lane);
            }
        }
    }

    // ---------------------------------------------------------------------- sum over the eight warps (they all cover the same columns)
    // tree: the upper half of the active warps writes its accumulators to the idle ring, the lower half adds them
    float* red = reinterpret_cast<float*>(ring);
    static_assert(4 * KF * 32 * 4 <= NS * STAGE, "reduction buffer must fit into the ring");
    __syncthreads();
    if (*abort_s) {
        // a wait gave up: let copies that are still in flight land before the ring is reused (bounded)
        if (threadIdx.x == 0) {
            for (int s = 0; s < NS; ++s) {
                const long long t0 = clock64();
                while (!mbar_try_wait(full(s), 0) && !mbar_try_wait(full(s), 1) && clock64() - t0 < 20000000LL) {}
            }
        }
        __syncthreads();
    }
    for (int active = kConsumerWarps; active > 1; active >>= 1) {
        const int hw = active >> 1;
        if (warp >= hw && warp < active) {
#pragma unroll
            for (int mm = 0; mm < 16; ++mm)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) red[(((warp - hw) * 16 + mm) * NT + nt) * 128 + e * 32 + lane] = acc[mm][nt][e];
        }
        __syncthreads();
        if (warp < hw) {
#pragma unroll
            for (int mm = 0; mm < 16; ++mm)
#pragma unroll
                for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[mm][nt][e] += red[((warp * 16 + mm) * NT + nt) * 128 + e * 32 + lane];
        }
        __syncthreads();
    }
    // Warp 0 holds the CTA's sums of the quantized part, in fragment order: idx = ((mm * NT + nt) * 4 + e) * 32 + lane is
    // column 32 (lane / 4) + 8 (mm / 4) + 2 (mm % 4) + (e >> 1) of the window and token nt * 8 + 2 (lane % 4) + (e & 1).
    // They are laid out as out[m][column] in shared memory; the first row slice adds T' L2; then the slices of a window
    // meet in global memory (own slot per slice, arrival counter per window, the last CTA adds them in slice order).
    constexpr int MT = 8 * NT;
    if (warp == 0) {
#pragma unroll
        for (int mm = 0; mm < 16; ++mm)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int col_local = (lane >> 2) * 32 + (mm >> 2) * 8 + (mm & 3) * 2 + (e >> 1);
                    const int m = nt * 8 + 2 * (lane & 3) + (e & 1);
                    outs[m * 256 + col_local] = acc[mm][nt][e];
                }
    }
    // the kernel launched in front of this one has written T' and cleared the arrival counters
    if (p.r > 0) pdl_wait();
    __syncthreads();
    const int split_id = split;
    // thread = one column of the window; the rank-r term (first row slice only): sum_j T'[m][j] L2[j][col]
    {
        const int cl = threadIdx.x;              // kThreads == 256 columns
        const int kcol = col_first + cl;
        const bool col_live = kcol < q.K;
        float add[MT];
#pragma unroll
        for (int m = 0; m < MT; ++m) add[m] = 0.0f;
        if (p.r > 0 && split_id == 0 && col_live) {
            for (int j0 = 0; j0 < p.r; j0 += 8) {
                float f[8];
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) f[jj] = __bfloat162float(p.L2[static_cast<size_t>(j0 + jj) * q.K + kcol]);
#pragma unroll
                for (int m = 0; m < MT; ++m) {
                    if (m < p.M) {
                        const uint4 tv = __ldcg(reinterpret_cast<const uint4*>(p.T + static_cast<size_t>(m) * p.r + j0));
                        const uint32_t tw[4] = {tv.x, tv.y, tv.z, tv.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            add[m] = fmaf(__uint_as_float(tw[e] << 16), f[2 * e], add[m]);
                            add[m] = fmaf(__uint_as_float(tw[e] & 0xffff0000u), f[2 * e + 1], add[m]);
                        }
                    }
                }
            }
        }
        const int kpad = gridDim.x * 256;
        if (p.S == 1) {
#pragma unroll
            for (int m = 0; m < MT; ++m)
                if (m < p.M && col_live) p.dX[static_cast<size_t>(m) * q.K + kcol] = __float2bfloat16_rn(outs[m * 256 + cl] + add[m]);
            return;
        }
#pragma unroll
        for (int m = 0; m < MT; ++m)
            if (m < p.M) __stcg(p.partial + (static_cast<size_t>(split_id) * p.M + m) * kpad + cw * 256 + cl, outs[m * 256 + cl] + add[m]);
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) *last_s = (atomicAdd(p.counters + cw, 1) == p.S - 1) ? 1 : 0;
        __syncthreads();
        if (!*last_s) return;
        __threadfence();
#pragma unroll
        for (int m = 0; m < MT; ++m) {
            if (m < p.M && col_live) {
                const float* src = p.partial + static_cast<size_t>(m) * kpad + cw * 256 + cl;
                float sum = 0.0f;
                for (int sp = 0; sp < p.S; ++sp) sum += __ldcg(src + static_cast<size_t>(sp) * p.M * kpad);
                p.dX[static_cast<size_t>(m) * q.K + kcol] = __float2bfloat16_rn(sum);
            }
        }
    }
}

// ------------------------------------------------------------------------------------ rank-r pre-product for few rows
// T[m][j] = bf16( sum_c A[m][c] * F(j, c) ) for m < M <= 16, j < r <= 128:
//   forward  A = X [M][K],  F(j, c) = L2[j][c]   (T = X L2^T)
//   backward A = dY [M][N], F(j, c) = L1[c][j]   (T = dY L1)
// One cluster of CTAs; each CTA sums a slice of the contraction, the slices are added through
// distributed shared memory by rank 0.  Thread = (column j, one of four contraction phases).
struct PreParams {
    const __nv_bfloat16* A;
    const __nv_bfloat16* F;
    __nv_bfloat16* T;
    int* status;       // cleared here: this kernel is the first of a call
    int* counters;     // arrival counters of the linear kernel behind this one, cleared here too
    int ncounters;
    int M, C, r;
    int chunk;         // contraction elements per CTA (multiple of 8)
    int nranks;
};

constexpr int kPreThreads = 512;      // 8 columns j x 64 contraction phases
constexpr int kPreJ = 8;              // columns of T per CTA
constexpr int kPrePhases = kPreThreads / kPreJ;

// Grid (ranks, r / 8), cluster (ranks, 1, 1): a cluster computes 8 columns of T, each of its CTAs over a slice
// of the contraction.  Dynamic shared memory: [A slice: MP rows x chunk bf16][red: 64 x 16 x 8 fp32][part: 16 x 8 fp32]
// MP = M rounded up to a power of two (rows staged).
template <bool BWD, int MP>
__global__ void __launch_bounds__(kPreThreads) decode_pre_kernel(const PreParams p) {
    extern __shared__ uint8_t pre_smem[];
    __nv_bfloat16* as = reinterpret_cast<__nv_bfloat16*>(pre_smem);
    float* red = reinterpret_cast<float*>(pre_smem + static_cast<size_t>(MP) * p.chunk * 2);
    float* part = red + kPrePhases * 16 * kPreJ;
    pdl_launch_dependents();
    if (blockIdx.x == 0 && blockIdx.y == 0) {
        if (threadIdx.x == 0) *p.status = 0;
        for (int i = threadIdx.x; i < p.ncounters; i += kPreThreads) p.counters[i] = 0;
    }
    const int jl = threadIdx.x & (kPreJ - 1), ph = threadIdx.x / kPreJ;
    const int j = blockIdx.y * kPreJ + jl;
    const int c_lo = blockIdx.x * p.chunk;
    const int c_hi = min(p.C, c_lo + p.chunk);
    // stage the CTA's slice of A (rows past M and columns past the end read as zero)
    const int nvec = p.chunk >> 3;
    for (int i = threadIdx.x; i < MP * nvec; i += kPreThreads) {
        const int m = i / nvec, v = i - m * nvec;
        const int c = c_lo + v * 8;
        uint4 val = make_uint4(0u, 0u, 0u, 0u);
        if (m < p.M && c < c_hi) val = __ldg(reinterpret_cast<const uint4*>(p.A + static_cast<size_t>(m) * p.C + c));
        *reinterpret_cast<uint4*>(as + static_cast<size_t>(m) * p.chunk + v * 8) = val;
    }
#pragma unroll 1
    for (int m = 0; m < 16; ++m) red[(ph * 16 + m) * kPreJ + jl] = 0.0f;
    __syncthreads();
    if (j < p.r) {
        // vectors of eight contraction elements, phase ph takes vectors ph, ph + 64, ...; up to four are in flight at a time
#pragma unroll 1
        for (int v0 = ph; v0 < nvec; v0 += 4 * kPrePhases) {
            float f[4][8];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int v = v0 + u * kPrePhases;
                const int c = c_lo + v * 8;
                const bool in = (v < nvec) && (c < c_hi);
                if (!BWD) {
                    uint4 w = make_uint4(0u, 0u, 0u, 0u);
                    if (in) w = __ldg(reinterpret_cast<const uint4*>(p.F + static_cast<size_t>(j) * p.C + c));
                    const uint32_t vv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) { f[u][2 * e] = __uint_as_float(vv[e] << 16); f[u][2 * e + 1] = __uint_as_float(vv[e] & 0xffff0000u); }
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e) f[u][e] = in ? __bfloat162float(p.F[static_cast<size_t>(c + e) * p.r + j]) : 0.0f;
                }
            }
#pragma unroll 1
            for (int m = 0; m < p.M; ++m) {
                float acc = 0.0f;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int v = v0 + u * kPrePhases;
                    if (v >= nvec) break;
                    const uint4 w = *reinterpret_cast<const uint4*>(as + static_cast<size_t>(m) * p.chunk + v * 8);
                    const uint32_t vv[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        acc = fmaf(__uint_as_float(vv[e] << 16), f[u][2 * e], acc);
                        acc = fmaf(__uint_as_float(vv[e] & 0xffff0000u), f[u][2 * e + 1], acc);
                    }
                }
                red[(ph * 16 + m) * kPreJ + jl] += acc;
            }
        }
    }
    __syncthreads();
    if (threadIdx.x < 16 * kPreJ) {
        float sum = 0.0f;
#pragma unroll 8
        for (int q8 = 0; q8 < kPrePhases; ++q8) sum += red[q8 * 16 * kPreJ + threadIdx.x];
        part[threadIdx.x] = sum;          // part[m * kPreJ + jl]
    }
    cluster_sync_all();
    if (p.nranks == 1 || cluster_ctarank() == 0) {
        const uint32_t part_addr = smem_u32(part);
        if (threadIdx.x < 16 * kPreJ) {
            const int m = threadIdx.x / kPreJ, jj = blockIdx.y * kPreJ + (threadIdx.x & (kPreJ - 1));
            if (m < p.M && jj < p.r) {
                float v[8];
#pragma unroll
                for (int rk = 0; rk < 8; ++rk)
                    v[rk] = (rk < p.nranks) ? ld_dsmem_f32(part_addr + static_cast<uint32_t>(threadIdx.x) * 4u, static_cast<uint32_t>(rk)) : 0.0f;
                p.T[static_cast<size_t>(m) * p.r + jj] = __float2bfloat16_rn(((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7])));
            }
        }
    }
    cluster_sync_all();
}

// ------------------------------------------------------------------------------------ host side
inline size_t round_up_ws(size_t x) { return (x + 255) / 256 * 256; }

inline int sm_count_cached() {
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

// Workspace of a decode-sized call: [status word 256 B][arrival counters][T bf16 [M][r]][slots of the slices, fp32]
struct WsLayout {
    size_t counters_off, counters_bytes, t_off, partial_off, total;
};
inline WsLayout ws_layout(int ncounters, int M, int r, int S, int out_pad) {
    WsLayout w;
    w.counters_off = kStatusBytes;
    w.counters_bytes = round_up_ws(static_cast<size_t>(ncounters) * 4);
    w.t_off = w.counters_off + w.counters_bytes;
    w.partial_off = w.t_off + round_up_ws(static_cast<size_t>(M) * (r > 0 ? r : 1) * 2);
    w.total = w.partial_off + (S > 1 ? round_up_ws(static_cast<size_t>(S) * M * out_pad * 4) : 0);
    return w;
}

struct Plan {
    bool ok;
    int NT, S, tiles_per_split, nkb_cap, tile_rows, stab8;
    size_t smem;
};

template <int B, int NT>
inline size_t smem_bytes(int nkb_cap, bool stab8) {
    const size_t table = stab8 ? static_cast<size_t>(nkb_cap) * kStab8Stride + static_cast<size_t>((nkb_cap + 15) / 16) * (kStabStride * 4)
                               : static_cast<size_t>(nkb_cap) * (kStabStride * 4);
    return 128 + static_cast<size_t>(num_stages<B, NT>()) * stage_bytes<B, NT>() + 2 * 128 * 8 * NT * 4 + (B == 8 ? 1024 : 0) +
           (2 * num_stages<B, NT>() + 2) * 8 + table;
}

// Estimated time of a grid of `n` equal CTAs of `work` units each (a unit = one 128 x 64 tile of dequantization, which
// is what binds).  The grid runs in waves of sms * per_sm resident CTAs; CTAs that share an SM share its ALU pipe (a
// wave of pairs takes 2 * work), a lone CTA per SM reaches about 0.65 of the SM's rate.  The first bytes from HBM, the
// scale table and the reduction cost about `fixed` units once, and a little per further wave (the waves overlap).
inline double grid_cost(long n, double work, int per_sm, int sms, double fixed) {
    const long slots = static_cast<long>(sms) * per_sm;
    const long waves = n / slots, rem = n - waves * slots;
    const double full = (per_sm == 2) ? 2.0 * work : work / 0.65;
    double t = static_cast<double>(waves) * full;
    if (rem > 0) t += (per_sm == 2 && rem > sms) ? 2.0 * work : work / 0.65;
    const long nw = waves + (rem > 0 ? 1 : 0);
    return t + fixed + 0.25 * fixed * static_cast<double>(nw - 1);
}

template <int B>
inline Plan make_plan(const QView& q, int M) {
    Plan best{};
    best.ok = false;
    const int NT = (M <= 8) ? 1 : 2;
    const int per_sm = (NT == 1) ? fwd_ctas_per_sm<B, 1>() : fwd_ctas_per_sm<B, 2>();
    const int sms = sm_count_cached();
    double best_cost = 0.0;
    int last_tps = -1;
    // Number of K slices: the one with the smallest estimated time (any number up to 16; more slices mean more
    // slots to add up at the end, hence the small penalty per slice).
    for (int S = 1; S <= 16; ++S) {
        if (S > 1 && q.ktiles / S < 2) break;
        int tps = (q.ktiles + S - 1) / S;
        tps += tps & 1;
        if (tps == last_tps) continue;
        last_tps = tps;
        const int splits = (q.ktiles + tps - 1) / tps;
        // compact scale table where every CTA has the same, 16-aligned run of blocks per row
        const int cols = tps * kTileCols;
        const bool uniform = (q.ktiles % tps == 0) && (cols % q.B0 == 0) && (q.KB % 16 == 0) && ((cols >> q.logB0) % 16 == 0) &&
                             (1 << q.logB1) >= 16;
        const int nkb_cap = uniform ? (cols >> q.logB0) : ((cols >> q.logB0) + 2);
        const size_t smem = (NT == 1) ? smem_bytes<B, 1>(nkb_cap, uniform) : smem_bytes<B, 2>(nkb_cap, uniform);
        if (smem > static_cast<size_t>(kSmemLimit)) continue;
        const int c = (per_sm == 2 && smem <= 113 * 1024) ? 2 : 1;
        // (slices that are not whole stages, or that rule out the compact table, measured 20-40 % slower)
        const double cost = (grid_cost(static_cast<long>(q.ntiles) * splits, tps, c, sms, 12.0) + 0.1 * splits) *
                            ((tps % kStageTiles == 0 && q.ktiles % tps == 0) ? (uniform ? 1.0 : 1.05) : 1.3);
        if (!best.ok || cost < best_cost) {
            best.ok = true; best.NT = NT; best.tile_rows = q.ntiles; best.S = splits; best.tiles_per_split = tps; best.nkb_cap = nkb_cap;
            best.smem = smem; best.stab8 = uniform ? 1 : 0;
            best_cost = cost;
        }
    }
    return best;
}

template <int B>
inline size_t fwd_workspace(const QView& q, int r, int M) {
    const Plan pl = make_plan<B>(q, M);
    return ws_layout(q.ntiles, M, r, pl.ok ? pl.S : 1, q.ntiles * 128).total;
}

inline bool supported(const QView& q, int64_t M) {
    if (M > 16 || q.K % 8 != 0 || q.K > 40960) return false;   // the pre-product stages K / 8 columns of X per CTA
    if (static_cast<long long>(q.N) * q.KB >= (1LL << 31)) return false;
    switch (q.b0) {
        case 2: return make_plan<2>(q, static_cast<int>(M)).ok;
        case 3: return make_plan<3>(q, static_cast<int>(M)).ok;
        case 4: return make_plan<4>(q, static_cast<int>(M)).ok;
        default: return make_plan<8>(q, static_cast<int>(M)).ok;
    }
}

// Launches the pre-product kernel for few rows (both directions use it).  It is the first kernel of the call: it clears
// the status word and the arrival counters of the linear kernel behind it.
template <bool BWD>
inline cudaError_t launch_pre(const __nv_bfloat16* A, const __nv_bfloat16* F, __nv_bfloat16* T, int* status, int* counters,
                              int ncounters, int M, int C, int r, cudaStream_t st) {
    PreParams pp;
    pp.A = A; pp.F = F; pp.T = T; pp.status = status; pp.counters = counters; pp.ncounters = ncounters; pp.M = M; pp.C = C; pp.r = r;
    int nranks = 8;
    while (nranks > 1 && C / nranks < 512) nranks >>= 1;
    int chunk = (C + nranks - 1) / nranks;
    chunk = (chunk + 7) / 8 * 8;
    pp.chunk = chunk; pp.nranks = nranks;
    const int MP = M <= 1 ? 1 : M <= 2 ? 2 : M <= 4 ? 4 : M <= 8 ? 8 : 16;
    const size_t smem = static_cast<size_t>(MP) * chunk * 2 + (kPrePhases * 16 * kPreJ + 16 * kPreJ) * sizeof(float);
    if (smem > static_cast<size_t>(kSmemLimit)) return cudaErrorInvalidValue;
    void (*kern)(PreParams) = decode_pre_kernel<BWD, 16>;
    if (M <= 1) kern = decode_pre_kernel<BWD, 1>;
    else if (M <= 2) kern = decode_pre_kernel<BWD, 2>;
    else if (M <= 4) kern = decode_pre_kernel<BWD, 4>;
    else if (M <= 8) kern = decode_pre_kernel<BWD, 8>;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaSuccess;
        if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_pre_kernel<BWD, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_pre_kernel<BWD, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_pre_kernel<BWD, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_pre_kernel<BWD, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(decode_pre_kernel<BWD, 16>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(nranks, (r + kPreJ - 1) / kPreJ);
    cfg.blockDim = dim3(kPreThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = nranks; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    count_launch(1);
    return cudaLaunchKernelEx(&cfg, kern, pp);
}

// Launch of a linear kernel behind the pre-product: programmatic dependent launch lets the two overlap.
template <typename Kern, typename P>
inline cudaError_t launch_stream_kernel(Kern kern, const P& p, dim3 grid, size_t smem, bool after_pre, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = after_pre ? 1 : 0;
    count_launch(1);
    return cudaLaunchKernelEx(&cfg, kern, p);
}

template <int B, int NT, bool TWO>
inline cudaError_t launch_fwd_nt(const Params& p, const Plan& pl, bool after_pre, cudaStream_t st) {
    auto kern = decode_fwd_kernel<B, NT, TWO>;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    return launch_stream_kernel(kern, p, dim3(pl.tile_rows, pl.S), pl.smem, after_pre, st);
}

// Forward for M <= 16.  When r > 0 the pre-product kernel clears the status word and the arrival counters; otherwise the
// caller has cleared them (clear_bytes of the workspace).
template <int B>
inline cudaError_t launch_fwd(const QView& q, const void* L1, const void* L2, int r, const void* X, int M, void* Y, char* ws,
                              cudaStream_t st) {
    const Plan pl = make_plan<B>(q, M);
    const WsLayout w = ws_layout(q.ntiles, M, r, pl.S, q.ntiles * 128);
    Params p;
    p.q = q;
    p.X = static_cast<const __nv_bfloat16*>(X);
    p.T = reinterpret_cast<const __nv_bfloat16*>(ws + w.t_off);
    p.L1 = static_cast<const __nv_bfloat16*>(L1);
    p.Y = static_cast<__nv_bfloat16*>(Y);
    p.partial = reinterpret_cast<float*>(ws + w.partial_off);
    p.counters = reinterpret_cast<int*>(ws + w.counters_off);
    p.status = reinterpret_cast<int*>(ws);
    p.M = M; p.r = r; p.S = pl.S; p.tiles_per_split = pl.tiles_per_split; p.nkb_cap = pl.nkb_cap; p.stab8 = pl.stab8;
    if (r > 0) {
        cudaError_t e = launch_pre<false>(p.X, static_cast<const __nv_bfloat16*>(L2), reinterpret_cast<__nv_bfloat16*>(ws + w.t_off),
                                          p.status, p.counters, q.ntiles, M, q.K, r, st);
        if (e != cudaSuccess) return e;
    }
    if (q.B0 == 16) return (pl.NT == 1) ? launch_fwd_nt<B, 1, true>(p, pl, r > 0, st) : launch_fwd_nt<B, 2, true>(p, pl, r > 0, st);
    return (pl.NT == 1) ? launch_fwd_nt<B, 1, false>(p, pl, r > 0, st) : launch_fwd_nt<B, 2, false>(p, pl, r > 0, st);
}

struct BwdPlan {
    bool ok;
    int NT, S, trows_per_split, rows_stride, nwin, stab8, nkb_cap;
    size_t smem;
};

// Plan for `trps` tile rows per CTA; ok = false when the scale table does not fit.
template <int B>
inline BwdPlan make_bwd_plan_t(const QView& q, int M, int trps, bool allow_compact) {
    BwdPlan pl{};
    pl.NT = (M <= 8) ? 1 : 2;
    pl.nwin = (q.ktiles + 3) / 4;
    const int nkb_cap = (256 >> q.logB0) > 0 ? (256 >> q.logB0) : 1;      // a window is 256 aligned columns and B0 divides 256
    // compact scale table where every window is whole and its blocks of a row are aligned and share a second-level group
    const bool compact = allow_compact && (q.K % 256 == 0) && (q.KB % nkb_cap == 0) && (1 << q.logB1) >= nkb_cap;
    const int rows_stride = trps * 128 + (compact ? 16 : 8);
    const size_t stage = (pl.NT == 1) ? bwd_stage_bytes<B, 1>() : bwd_stage_bytes<B, 2>();
    const int ns = (pl.NT == 1) ? bwd_stages<B, 1>() : bwd_stages<B, 2>();
    const size_t smem = 128 + ns * stage + 64 * pl.NT * 32 * 4 + (B == 8 ? 1024 : 0) + (2 * ns + 2) * 8 +
                        (compact ? static_cast<size_t>(nkb_cap) * rows_stride + static_cast<size_t>(rows_stride) * 4
                                 : static_cast<size_t>(nkb_cap) * rows_stride * 4);
    pl.ok = smem <= static_cast<size_t>(kSmemLimit);
    pl.S = (q.ntiles + trps - 1) / trps;
    pl.trows_per_split = trps; pl.rows_stride = rows_stride; pl.smem = smem; pl.stab8 = compact ? 1 : 0; pl.nkb_cap = nkb_cap;
    return pl;
}

// Number of row slices and form of the scale table: the pair with the smallest estimated time (host arithmetic only).
// A unit of work is one tile row of the window (128 x 256 weights); the compact table costs a few conversions per use
// (about 4 %) and wins where the fp32 table would force more slices or a single CTA per SM.
template <int B>
inline BwdPlan make_bwd_plan(const QView& q, int M) {
    BwdPlan best{};
    double best_cost = 0.0;
    const int NT = (M <= 8) ? 1 : 2;
    const int per_sm = (NT == 1) ? bwd_ctas_per_sm<B, 1>() : bwd_ctas_per_sm<B, 2>();
    const int sms = sm_count_cached();
    for (int mode = 0; mode < 2; ++mode) {
        int last_trps = -1;
        for (int S = 1; S <= 32; ++S) {
            if (S > 1 && q.ntiles / S < 1) break;
            int trps = (q.ntiles + S - 1) / S;
            trps += trps & 1;
            if (trps == last_trps) continue;
            last_trps = trps;
            const BwdPlan c = make_bwd_plan_t<B>(q, M, trps, mode == 1);
            if (!c.ok || (mode == 1 && !c.stab8)) continue;
            const int on = (per_sm == 2 && c.smem <= 113 * 1024) ? 2 : 1;
            double cost = grid_cost(static_cast<long>(c.nwin) * c.S, 4.0 * trps, on, sms, 14.0) + 0.1 * c.S;
            if (q.ntiles % trps != 0) cost *= 1.15;              // uneven slices
            if (mode == 1) cost *= 1.04;
            if (!best.ok || cost < best_cost) { best = c; best_cost = cost; }
        }
    }
    return best;
}

template <int B>
inline size_t bwd_workspace(const QView& q, int r, int M) {
    const BwdPlan pl = make_bwd_plan<B>(q, M);
    const int nwin = (q.ktiles + 3) / 4;
    return ws_layout(nwin, M, r, pl.ok ? pl.S : 1, nwin * 256).total;
}

inline bool bwd_supported(const QView& q, int64_t M) {
    if (M > 16 || q.N % 8 != 0 || q.K % 8 != 0 || q.N > 40960) return false;
    if (static_cast<long long>(q.N) * q.KB >= (1LL << 31)) return false;
    switch (q.b0) {
        case 2: return make_bwd_plan<2>(q, static_cast<int>(M)).ok;
        case 3: return make_bwd_plan<3>(q, static_cast<int>(M)).ok;
        case 4: return make_bwd_plan<4>(q, static_cast<int>(M)).ok;
        default: return make_bwd_plan<8>(q, static_cast<int>(M)).ok;
    }
}

template <int B, int NT, bool TWO>
inline cudaError_t launch_bwd_nt(BwdParams p, const BwdPlan& pl, bool after_pre, cudaStream_t st) {
    void (*kerns[2])(BwdParams) = {decode_bwd_kernel<B, NT, TWO, false>, decode_bwd_kernel<B, NT, TWO, true>};
    static bool attr_done = false;
    if (!attr_done) {
        for (int i = 0; i < 2; ++i) {
            cudaError_t e = cudaFuncSetAttribute(kerns[i], cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
            if (e != cudaSuccess) return e;
        }
        attr_done = true;
    }
    p.S = pl.S; p.trows_per_split = pl.trows_per_split; p.rows_stride = pl.rows_stride; p.stab8 = pl.stab8; p.nkb_cap = pl.nkb_cap;
    return launch_stream_kernel(kerns[pl.stab8 ? 1 : 0], p, dim3(pl.nwin, pl.S), pl.smem, after_pre, st);
}

// Input gradient for M <= 16; same conventions as launch_fwd.
template <int B>
inline cudaError_t launch_bwd(const QView& q, const void* L1, const void* L2, int r, const void* dY, int M, void* dX, char* ws,
                              cudaStream_t st) {
    const BwdPlan pl = make_bwd_plan<B>(q, M);
    if (!pl.ok) return cudaErrorInvalidValue;
    const WsLayout w = ws_layout(pl.nwin, M, r, pl.S, pl.nwin * 256);
    BwdParams p;
    p.q = q;
    p.dY = static_cast<const __nv_bfloat16*>(dY);
    p.T = reinterpret_cast<const __nv_bfloat16*>(ws + w.t_off);
    p.L2 = static_cast<const __nv_bfloat16*>(L2);
    p.dX = static_cast<__nv_bfloat16*>(dX);
    p.partial = reinterpret_cast<float*>(ws + w.partial_off);
    p.counters = reinterpret_cast<int*>(ws + w.counters_off);
    p.status = reinterpret_cast<int*>(ws);
    p.M = M; p.r = r;
    if (r > 0) {
        cudaError_t e = launch_pre<true>(p.dY, static_cast<const __nv_bfloat16*>(L1), reinterpret_cast<__nv_bfloat16*>(ws + w.t_off),
                                         p.status, p.counters, pl.nwin, M, q.N, r, st);
        if (e != cudaSuccess) return e;
    }
    if (q.B0 == 16) return (pl.NT == 1) ? launch_bwd_nt<B, 1, true>(p, pl, r > 0, st) : launch_bwd_nt<B, 2, true>(p, pl, r > 0, st);
    return (pl.NT == 1) ? launch_bwd_nt<B, 1, false>(p, pl, r > 0, st) : launch_bwd_nt<B, 2, false>(p, pl, r > 0, st);
}

// Bytes at the head of the workspace that must be zero when the linear kernel starts (status word and arrival counters)
// and workspace need of a decode-sized call; slices per output tile (for lqlora_linear_path).
inline size_t clear_bytes(const QView& q, bool backward) {
    return kStatusBytes + round_up_ws(static_cast<size_t>(backward ? (q.ktiles + 3) / 4 : q.ntiles) * 4);
}
inline size_t workspace_bytes(const QView& q, int r, int M, bool backward) {
    switch (q.b0) {
        case 2: return backward ? bwd_workspace<2>(q, r, M) : fwd_workspace<2>(q, r, M);
        case 3: return backward ? bwd_workspace<3>(q, r, M) : fwd_workspace<3>(q, r, M);
        case 4: return backward ? bwd_workspace<4>(q, r, M) : fwd_workspace<4>(q, r, M);
        default: return backward ? bwd_workspace<8>(q, r, M) : fwd_workspace<8>(q, r, M);
    }
}
inline int fwd_splits(const QView& q, int M) {
    switch (q.b0) {
        case 2: return make_plan<2>(q, M).S;
        case 3: return make_plan<3>(q, M).S;
        case 4: return make_plan<4>(q, M).S;
        default: return make_plan<8>(q, M).S;
    }
}
inline int bwd_splits(const QView& q, int M) {
    switch (q.b0) {
        case 2: return make_bwd_plan<2>(q, M).S;
        case 3: return make_bwd_plan<3>(q, M).S;
        case 4: return make_bwd_plan<4>(q, M).S;
        default: return make_bwd_plan<8>(q, M).S;
    }
}

}  // namespace dec
}  // namespace lq
