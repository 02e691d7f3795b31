// Skeleton shared by the three tensor-core kernels (window scoring pass 1 and 2, matching).
//
// Each CTA is persistent and walks a list of items.  An item is one 128-row operand tile A
// (loaded once) against a stream of up-to-256-row operand tiles B_0 .. B_{n-1}; tile t yields a
// 128 x 256 fp32 accumulator in TMEM.  Warp 0 issues the TMA loads, warp 1 issues tcgen05.mma,
// warps 2-5 run the kernel's own epilogue on the accumulators; shared-memory stages (2 x A,
// 2 x B) and TMEM buffers (2 x 256 columns) are handed around with mbarriers.
#pragma once
#include "tc_common.cuh"

namespace flowmm {
namespace tcs {

constexpr int kRows = 128;                   // rows of A per item (UMMA M)
constexpr int kCols = 256;                   // rows of B per tile (UMMA N)
constexpr int kThreads = 192;
constexpr uint32_t kAStage = kRows * 128 * 2;            // bytes of an A stage: two 64-element K halves
constexpr uint32_t kBStage = kCols * 128 * 2;
constexpr uint32_t kSmemA = 0;
constexpr uint32_t kSmemB = 2 * kAStage;
constexpr uint32_t kSmemEpi = kSmemB + 2 * kBStage;      // epilogue scratch
constexpr uint32_t kEpiBytes = 20480;
constexpr uint32_t kSmemBar = kSmemEpi + kEpiBytes;
constexpr uint32_t kSmemBytes = kSmemBar + 256 + 1024;   // + slack to align the base to 1024 bytes

// Where an item's operands come from.  All tensor maps are 4-D: (K element, c1, c2, c3).
struct TilePlan {
    int a1, a2, a3;            // A box origin
    int b1, b2, b3;            // B box origin of tile 0
    int step1, step2;          // B origin advance per tile along c1 / c2
    int n_tiles;               // 0: nothing to compute, every role skips the item
    int cols_total;            // valid B rows over all tiles (tile t has min(256, cols_total - 256 t))
};

struct Ctx {
    uint32_t base, bars, tmem_base;
    uint8_t *gen;              // generic pointer to the aligned base
    volatile int *abort_flag;
    int warp, lane;
    // barrier slots: 0-1 a_full, 2-3 a_empty, 4-5 b_full, 6-7 b_empty, 8-9 acc_full, 10-11 acc_empty
    __device__ __forceinline__ uint32_t bar(int i) const { return bars + 8u * i; }
    __device__ __forceinline__ uint8_t *epi_scratch() const { return gen + kSmemEpi; }
};

__device__ __forceinline__ Ctx setup(uint8_t *smem_raw, const CUtensorMap *ma, const CUtensorMap *mb) {
    Ctx c;
    c.base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    c.gen = smem_raw + (c.base - tc::smem_u32(smem_raw));
    c.bars = c.base + kSmemBar;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(c.gen + kSmemBar + 128);
    c.abort_flag = reinterpret_cast<volatile int *>(c.gen + kSmemBar + 132);
    c.warp = threadIdx.x >> 5;
    c.lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < 10; ++i) tc::mbar_init(c.bar(i), 1);
        tc::mbar_init(c.bar(10), 4);           // one arrival per epilogue warp
        tc::mbar_init(c.bar(11), 4);
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
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (c.warp == 1) tc::tmem_dealloc(c.tmem_base, 512);
}

// Call from one thread.  a_bytes / b_bytes: bytes one A / B box pair delivers (both K halves).
template <class PlanFn>
__device__ __forceinline__ void producer(const Ctx &c, const CUtensorMap *ma, const CUtensorMap *mb, int n_items,
                                         uint32_t a_bytes, uint32_t b_bytes, PlanFn plan, int *status) {
    int it = 0, bt = 0;
    bool ok = true;
    for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const TilePlan p = plan(item);
        if (p.n_tiles == 0) continue;
        const int sa = it & 1;
        ok = tc::mbar_wait(c.bar(2 + sa), ((it >> 1) & 1) ^ 1, c.abort_flag, status);
        if (!ok) break;
        tc::mbar_expect_tx(c.bar(sa), a_bytes);
        const uint32_t a_dst = c.base + kSmemA + sa * kAStage;
        tc::tma_load_4d(a_dst, ma, c.bar(sa), 0, p.a1, p.a2, p.a3);
        tc::tma_load_4d(a_dst + kAStage / 2, ma, c.bar(sa), 64, p.a1, p.a2, p.a3);
        for (int t = 0; t < p.n_tiles; ++t, ++bt) {
            const int sb = bt & 1;
            ok = tc::mbar_wait(c.bar(6 + sb), ((bt >> 1) & 1) ^ 1, c.abort_flag, status);
            if (!ok) break;
            tc::mbar_expect_tx(c.bar(4 + sb), b_bytes);
            const uint32_t b_dst = c.base + kSmemB + sb * kBStage;
            tc::tma_load_4d(b_dst, mb, c.bar(4 + sb), 0, p.b1 + t * p.step1, p.b2 + t * p.step2, p.b3);
            tc::tma_load_4d(b_dst + kBStage / 2, mb, c.bar(4 + sb), 64, p.b1 + t * p.step1, p.b2 + t * p.step2, p.b3);
        }
        ++it;
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
    int it = 0, bt = 0, tt = 0;
    bool ok = true;
    for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
        const TilePlan p = plan(item);
        if (p.n_tiles == 0) continue;
        const int sa = it & 1;
        ok = tc::mbar_wait(c.bar(sa), (it >> 1) & 1, c.abort_flag, status);
        if (!ok) break;
        const uint32_t a_base = c.base + kSmemA + sa * kAStage;
        for (int t = 0; t < p.n_tiles; ++t, ++bt, ++tt) {
            const int sb = bt & 1, ta = tt & 1;
            ok = tc::mbar_wait(c.bar(4 + sb), (bt >> 1) & 1, c.abort_flag, status) &&
                 tc::mbar_wait(c.bar(10 + ta), ((tt >> 1) & 1) ^ 1, c.abort_flag, status);
            if (!ok) break;
            tc::tc_fence_after();
            const int ncols = min(kCols, p.cols_total - t * kCols);
            const uint32_t idesc = tc::idesc_bf16(kRows, (uint32_t)((ncols + 15) & ~15));
            const uint32_t b_base = c.base + kSmemB + sb * kBStage;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {                         // head_dim 128 = 8 K slices of 16
                const uint32_t a_off = (ks >> 2) * (kAStage / 2) + (ks & 3) * 32;
                const uint32_t b_off = (ks >> 2) * (kBStage / 2) + (ks & 3) * 32;
                tc::umma_bf16(c.tmem_base + ta * kCols, tc::smem_desc_sw128(a_base, a_off),
                              tc::smem_desc_sw128(b_base, b_off), idesc, ks > 0);
            }
            tc::umma_commit(c.bar(6 + sb));                          // B stage free once these MMAs finish
            tc::umma_commit(c.bar(8 + ta));                          // accumulator ready
        }
        if (!ok) break;
        tc::umma_commit(c.bar(2 + sa));                              // A stage free
        ++it;
    }
}

// Epilogue side (warps 2-5).  `tt` counts accumulator tiles this CTA has consumed.
__device__ __forceinline__ bool acc_wait(const Ctx &c, int tt, int *status) {
    const bool ok = tc::mbar_wait(c.bar(8 + (tt & 1)), (tt >> 1) & 1, c.abort_flag, status);
    tc::tc_fence_after();
    return ok;
}
__device__ __forceinline__ void acc_release(const Ctx &c, int tt) {
    tc::tc_fence_before();
    __syncwarp();
    if (c.lane == 0) tc::mbar_arrive(c.bar(10 + (tt & 1)));
}
// TMEM address of columns [32*chunk, 32*chunk+32) of accumulator tt for this warp's 32 lanes.
__device__ __forceinline__ uint32_t acc_addr(const Ctx &c, int tt, int chunk) {
    return c.tmem_base + (tt & 1) * kCols + chunk * 32 + ((uint32_t)((c.warp & 3) * 32) << 16);
}

}  // namespace tcs
}  // namespace flowmm
