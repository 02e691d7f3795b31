// Skeleton shared by the three tensor-core kernels (window scoring pass 1 and 2, matching).
//
// Each CTA is persistent (one per SM) and walks a list of items.  An item is up to two 128-row
// operand halves A_0, A_1 (loaded once per item) against a stream of up-to-256-row operand tiles
// B_0 .. B_{n-1}; every B tile is used by both halves, which halves the operand traffic per
// multiply-add, and yields one 128 x 256 fp32 accumulator per half in TMEM (half h owns TMEM
// columns [256 h, 256 h + 256)).
// Roles: warp 0 issues the TMA loads, warp 1 issues tcgen05.mma, warps 2-17 run the kernel's
// epilogue: a quad of warps (one per 32 TMEM lanes) per (A half, column half), i.e. four epilogue
// warps per SM sub-partition, so that TMEM reads, shared-memory reads and dependent arithmetic of
// one warp are covered by the other three.  The two quads of a half split each accumulator's
// 256 columns (0-127 / 128-255) and combine per-row results through shared memory.
// Shared-memory stages (one per A half, two for B) and the two accumulators are handed around
// with mbarriers; every wait is bounded.
#pragma once
#include "tc_common.cuh"

namespace flowmm {
namespace tcs {

constexpr int kRows = 128;                   // rows of an A half (UMMA M)
constexpr int kCols = 256;                   // rows of a B tile (UMMA N)
constexpr int kItemRows = 2 * kRows;         // rows of A an item covers
constexpr int kEpiWarps = 16;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr uint32_t kAHalf = kRows * 128 * 2;             // bytes of an A half: two 64-element K halves
constexpr uint32_t kBStage = kCols * 128 * 2;
constexpr uint32_t kSmemA = 0;
constexpr uint32_t kSmemB = 2 * kAHalf;
constexpr uint32_t kExtraBytes = 1024;                   // per-column fp32 constants that travel with a B tile
constexpr int kExtraSlots = 4;                           // ring: a slot is rewritten four B tiles later
constexpr uint32_t kSmemExtra = kSmemB + 2 * kBStage;
constexpr uint32_t kSmemEpi = kSmemExtra + kExtraSlots * kExtraBytes;   // epilogue scratch
constexpr uint32_t kEpiBytes = 16384;
constexpr uint32_t kSmemBar = kSmemEpi + kEpiBytes;
constexpr uint32_t kSmemBytes = kSmemBar + 256;
constexpr int kStatusAlign = 6;                          // FLOWMM_ERR_ALIGN

// Where an item's operands come from.  All tensor maps are 4-D: (K element, c1, c2, c3).
struct TilePlan {
    int a1, a2, a3;            // box origin of A half 0
    int h1, h2;                // origin advance of half 1 along c1 / c2
    int n_halves;              // 0: nothing to compute, every role skips the item
    int b1, b2, b3;            // B box origin of tile 0
    int step1, step2;          // B origin advance per tile along c1 / c2
    int n_tiles;               // 0: every role skips the item
    int cols_total;            // valid B rows over all tiles (tile t has min(256, cols_total - 256 t))
    const float *extra;        // nullptr, or 256 fp32 per-column constants per tile: tile t reads extra + 256 t
    __device__ __forceinline__ bool empty() const { return n_tiles == 0 || n_halves == 0; }
};

struct Ctx {
    uint32_t base, bars, tmem_base;
    uint8_t *gen;              // generic pointer to the base
    volatile int *abort_flag;
    int warp, lane;
    int group, quarter;        // epilogue warps: which A half they serve, which 32 TMEM lanes they read
    int colhalf;               // ... and which 128 columns of each accumulator
    bool ok;                   // false: shared memory was not 1024-byte aligned; nothing may run
    // barrier slots: 0-1 a_full[h], 2-3 a_empty[h], 4-5 b_full[s], 6-7 b_empty[s], 8-9 acc_full[h], 10-11 acc_empty[h],
    // 12-15 x_full[slot] (per-column constants landed)
    __device__ __forceinline__ uint32_t bar(int i) const { return bars + 8u * i; }
    // scratch of this warp's quad (a quarter of the epilogue scratch) / of its partner quad on the same rows
    __device__ __forceinline__ uint8_t *epi_scratch() const {
        return gen + kSmemEpi + (uint32_t)(group * 2 + colhalf) * (kEpiBytes / 4);
    }
    __device__ __forceinline__ uint8_t *partner_scratch() const {
        return gen + kSmemEpi + (uint32_t)(group * 2 + (colhalf ^ 1)) * (kEpiBytes / 4);
    }
    // shared address of the per-column constants of the bt-th B tile this CTA streams (valid from the tile's
    // extra_wait to its release)
    __device__ __forceinline__ uint32_t extra(int bt) const {
        return base + kSmemExtra + (uint32_t)(bt & (kExtraSlots - 1)) * kExtraBytes;
    }
    // shared addresses of the scratch of this warp's quad / of its partner quad
    __device__ __forceinline__ uint32_t epi_addr() const { return base + kSmemEpi + (uint32_t)(group * 2 + colhalf) * (kEpiBytes / 4); }
    __device__ __forceinline__ uint32_t partner_addr() const {
        return base + kSmemEpi + (uint32_t)(group * 2 + (colhalf ^ 1)) * (kEpiBytes / 4);
    }
};

// `a_readers`: epilogue warps per half that read the A stage themselves and release it with a_release().
__device__ __forceinline__ Ctx setup(uint8_t *smem_raw, const CUtensorMap *ma, const CUtensorMap *mb, int *status,
                                     int a_readers = 0) {
    Ctx c;
    c.base = tc::smem_u32(smem_raw);
    c.gen = smem_raw;
    c.bars = c.base + kSmemBar;
    c.warp = threadIdx.x >> 5;
    c.lane = threadIdx.x & 31;
    c.group = ((c.warp - 2) >> 2) & 1;
    c.quarter = c.warp & 3;
    c.colhalf = (c.warp - 2) >> 3;
    c.tmem_base = 0;
    c.abort_flag = reinterpret_cast<volatile int *>(c.gen + kSmemBar + 132);
    c.ok = (c.base & 1023u) == 0;              // the swizzled operand tiles need a 1024-byte aligned base
    if (!c.ok) {
        if (threadIdx.x == 0) atomicCAS(status, 0, kStatusAlign);
        return c;
    }
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(c.gen + kSmemBar + 128);
    if (threadIdx.x == 0) {
        for (int i = 0; i < 10; ++i) tc::mbar_init(c.bar(i), (i == 2 || i == 3) ? 1 + a_readers : 1);
        tc::mbar_init(c.bar(10), 8);           // one arrival per epilogue warp of the half
        tc::mbar_init(c.bar(11), 8);
        for (int i = 12; i < 16; ++i) tc::mbar_init(c.bar(i), 1);
        *c.abort_flag = 0;
        tc::mbar_init_fence();
        tc::tma_prefetch_desc(ma);
        tc::tma_prefetch_desc(mb);
    }
    if (c.warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), 512);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    c.tmem_base = *tmem_slot;
    return c;
}

__device__ __forceinline__ void teardown(const Ctx &c) {
    if (!c.ok) return;
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (c.warp == 1) tc::tmem_dealloc(c.tmem_base, 512);
}

// Call from one thread.  a_bytes / b_bytes: bytes one A-half / B box pair delivers (both K halves).
template <class PlanFn>
__device__ __forceinline__ void producer(const Ctx &c, const CUtensorMap *ma, const CUtensorMap *mb, int n_items,
                                         uint32_t a_bytes, uint32_t b_bytes, PlanFn plan, int *status) {
    int ia[2] = {0, 0}, bt = 0;
    bool ok = true;
    for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const TilePlan p = plan(item);
        if (p.empty()) continue;
        for (int t = 0; ok && t < p.n_tiles; ++t, ++bt) {
            const int sb = bt & 1;
            ok = tc::mbar_wait(c.bar(6 + sb), ((bt >> 1) & 1) ^ 1, c.abort_flag, status);
            if (!ok) break;
            if (p.extra) {       // slot reuse is safe: both epilogues released tile bt-4 before the MMAs of bt-2 began
                const int xs = bt & (kExtraSlots - 1);
                tc::mbar_expect_tx(c.bar(12 + xs), kExtraBytes);
                tc::bulk_load(c.base + kSmemExtra + (uint32_t)xs * kExtraBytes, p.extra + (size_t)t * kCols, kExtraBytes,
                              c.bar(12 + xs));
            }
            tc::mbar_expect_tx(c.bar(4 + sb), b_bytes);
            const uint32_t b_dst = c.base + kSmemB + sb * kBStage;
            tc::tma_load_4d(b_dst, mb, c.bar(4 + sb), 0, p.b1 + t * p.step1, p.b2 + t * p.step2, p.b3);
            tc::tma_load_4d(b_dst + kBStage / 2, mb, c.bar(4 + sb), 64, p.b1 + t * p.step1, p.b2 + t * p.step2, p.b3);
            if (t == 0) {                  // the item's A halves go out right after its first B tile
                for (int h = 0; ok && h < p.n_halves; ++h) {
                    ok = tc::mbar_wait(c.bar(2 + h), (ia[h] & 1) ^ 1, c.abort_flag, status);
                    if (!ok) break;
                    tc::mbar_expect_tx(c.bar(h), a_bytes);
                    const uint32_t a_dst = c.base + kSmemA + h * kAHalf;
                    tc::tma_load_4d(a_dst, ma, c.bar(h), 0, p.a1 + h * p.h1, p.a2 + h * p.h2, p.a3);
                    tc::tma_load_4d(a_dst + kAHalf / 2, ma, c.bar(h), 64, p.a1 + h * p.h1, p.a2 + h * p.h2, p.a3);
                    ++ia[h];
                }
            }
        }
    }
    if (!ok) {          // winding down after a timeout: give copies already issued a moment to land
        for (int i = 0; i < 2; ++i) {
            for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(c.bar(i), 0) && !tc::mbar_try_wait(c.bar(i), 1); ++s) {}
            for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(c.bar(4 + i), 0) && !tc::mbar_try_wait(c.bar(4 + i), 1); ++s) {}
        }
    }
}

// Call from one thread.
template <class PlanFn>
__device__ __forceinline__ void mma_issuer(const Ctx &c, int n_items, PlanFn plan, int *status) {
    int ia[2] = {0, 0}, ta[2] = {0, 0}, bt = 0;
    bool ok = true;
    for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const TilePlan p = plan(item);
        if (p.empty()) continue;
        for (int t = 0; ok && t < p.n_tiles; ++t, ++bt) {
            const int sb = bt & 1;
            ok = tc::mbar_wait(c.bar(4 + sb), (bt >> 1) & 1, c.abort_flag, status);
            if (!ok) break;
            const int ncols = min(kCols, p.cols_total - t * kCols);
            const uint32_t idesc = tc::idesc_bf16(kRows, (uint32_t)((ncols + 15) & ~15));
            const uint32_t b_base = c.base + kSmemB + sb * kBStage;
            for (int h = 0; ok && h < p.n_halves; ++h) {
                if (t == 0) ok = tc::mbar_wait(c.bar(h), ia[h] & 1, c.abort_flag, status);
                ok = ok && tc::mbar_wait(c.bar(10 + h), (ta[h] & 1) ^ 1, c.abort_flag, status);
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t a_base = c.base + kSmemA + h * kAHalf;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {                     // head_dim 128 = 8 K slices of 16
                    const uint32_t a_off = (ks >> 2) * (kAHalf / 2) + (ks & 3) * 32;
                    const uint32_t b_off = (ks >> 2) * (kBStage / 2) + (ks & 3) * 32;
                    tc::umma_bf16(c.tmem_base + h * kCols, tc::smem_desc_sw128(a_base, a_off),
                                  tc::smem_desc_sw128(b_base, b_off), idesc, ks > 0);
                }
                tc::umma_commit(c.bar(8 + h));                       // accumulator of this half ready
                ++ta[h];
                if (t == p.n_tiles - 1) {                            // that was the half's last use of its A stage
                    tc::umma_commit(c.bar(2 + h));
                    ++ia[h];
                }
            }
            if (!ok) break;
            tc::umma_commit(c.bar(6 + sb));                          // B stage free once both halves' MMAs finish
        }
    }
}

// Epilogue side.  `k` counts the accumulator tiles this warp's half has consumed.
__device__ __forceinline__ bool acc_wait(const Ctx &c, int k, int *status) {
    const bool ok = tc::mbar_wait(c.bar(8 + c.group), k & 1, c.abort_flag, status);
    tc::tc_fence_after();
    return ok;
}
// For kernels whose epilogue reads its A half from shared memory: wait until the half of the
// n-th item this group takes part in has landed / hand it back (one arrival per warp).
__device__ __forceinline__ bool a_wait(const Ctx &c, int n, int *status) {
    return tc::mbar_wait(c.bar(c.group), n & 1, c.abort_flag, status);
}
__device__ __forceinline__ void a_release(const Ctx &c) {
    __syncwarp();
    if (c.lane == 0) tc::mbar_arrive(c.bar(2 + c.group));
}
// Waits until the per-column constants of the bt-th B tile are in shared memory.
__device__ __forceinline__ bool extra_wait(const Ctx &c, int bt, int *status) {
    return tc::mbar_wait(c.bar(12 + (bt & (kExtraSlots - 1))), (bt >> 2) & 1, c.abort_flag, status);
}
__device__ __forceinline__ void acc_release(const Ctx &c) {
    tc::tc_fence_before();
    __syncwarp();
    if (c.lane == 0) tc::mbar_arrive(c.bar(10 + c.group));
}
// TMEM address of columns [32*chunk, 32*chunk+32) of this warp's half for its 32 lanes.
__device__ __forceinline__ uint32_t acc_addr(const Ctx &c, int chunk) {
    return c.tmem_base + c.group * kCols + chunk * 32 + ((uint32_t)(c.quarter * 32) << 16);
}

// Runs f(chunk, values) over this warp's 32-column chunks of the current accumulator: chunks
// 4*colhalf .. 4*colhalf+3, as far as they lie below n_chunks (the tile's chunk count).
template <class F>
__device__ __forceinline__ void for_each_chunk(const Ctx &c, int n_chunks, F &&f) {
    const int hi = min(n_chunks, 4 * c.colhalf + 4);
    for (int ch = 4 * c.colhalf; ch < hi; ++ch) {
        uint32_t a[32];
        tc::tmem_ld32(acc_addr(c, ch), a);
        tc::tmem_ld_wait(a);
        f(ch, a);
    }
}
// The same walk in blocks of 16 columns (for epilogues that are short of registers): f(block, values)
// for blocks 8*colhalf .. 8*colhalf+7 below n_blocks = ceil(columns of the tile / 16).
template <class F>
__device__ __forceinline__ void for_each_block16(const Ctx &c, int n_blocks, F &&f) {
    const int hi = min(n_blocks, 8 * c.colhalf + 8);
    for (int b = 8 * c.colhalf; b < hi; ++b) {
        uint32_t a[16];
        tc::tmem_ld16(c.tmem_base + c.group * kCols + b * 16 + ((uint32_t)(c.quarter * 32) << 16), a);
        tc::tmem_ld_wait(a);
        f(b, a);
    }
}
// Meeting point of the two warps that share rows (same half, same lanes, other columns).
__device__ __forceinline__ void pair_sync(const Ctx &c) {
    asm volatile("bar.sync %0, 64;" ::"r"(1 + c.group * 4 + c.quarter) : "memory");
}

}  // namespace tcs
}  // namespace flowmm
