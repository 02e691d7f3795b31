// Skeleton shared by the three tensor-core kernels (window scoring pass 1 and 2, matching).
//
// Each CTA is persistent (one per SM) and walks a list of items.  An item is up to two 128-row
// operand halves A_0, A_1 (loaded once per item) against a stream of operand tiles B_0 .. B_{n-1}
// of up to NB rows; every B tile is used by both halves, which halves the operand traffic per
// multiply-add, and yields one 128 x NB fp32 accumulator per half in TMEM (half h owns TMEM
// columns [NB h, NB h + NB)).
// Roles: warp 0 issues the TMA loads, warp 1 issues tcgen05.mma, warps 2-17 run the kernel's
// epilogue: a quad of warps (one per 32 TMEM lanes) per (A half, column half), i.e. four epilogue
// warps per SM sub-partition, so that TMEM reads, shared-memory reads and dependent arithmetic of
// one warp are covered by the other three.  The two quads of a half split each accumulator's
// columns in two and combine per-row results through shared memory.
// Shared-memory stages (AST per A half, two for B) and the two accumulators are handed around
// with mbarriers; every wait is bounded.
//
// Two shapes are instantiated: Skel<256, 1> for long B streams (one A stage per half, 64 KB B
// stages) and Skel<128, 2> for problems whose items have few B columns, where the A operand is
// the stream: two A stages per half let the next item's rows load while this item is computed.
#pragma once
#include "tc_common.cuh"

namespace flowmm {
namespace tcs {

constexpr int kRows = 128;                   // rows of an A half (UMMA M)
constexpr int kItemRows = 2 * kRows;         // rows of A an item covers
constexpr int kEpiWarps = 16;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr uint32_t kAHalf = kRows * 128 * 2; // bytes of an A half: two 64-element K halves
constexpr int kExtraSlots = 4;               // ring of per-column constants: a slot is rewritten four B tiles later
constexpr uint32_t kEpiBytes = 16384;
constexpr int kStatusAlign = 6;              // FLOWMM_ERR_ALIGN

// Where an item's operands come from.  All tensor maps are 4-D: (K element, c1, c2, c3).
struct TilePlan {
    int a1, a2, a3;            // box origin of A half 0
    int h1, h2;                // origin advance of half 1 along c1 / c2
    int n_halves;              // 0: nothing to compute, every role skips the item
    int b1, b2, b3;            // B box origin of tile 0
    int step1, step2;          // B origin advance per tile along c1 / c2
    int n_tiles;               // 0: every role skips the item
    int cols_total;            // valid B rows over all tiles (tile t has min(NB, cols_total - NB t))
    const float *extra;        // nullptr, or NB fp32 per-column constants per tile: tile t reads extra + NB t
    __device__ __forceinline__ bool empty() const { return n_tiles == 0 || n_halves == 0; }
};

template <int NB, int AST>
struct Skel {
    static constexpr int kCols = NB;                         // rows of a B tile (UMMA N)
    static constexpr int kAStages = AST;
    static constexpr uint32_t kBStage = NB * 128 * 2;
    static constexpr uint32_t kExtraBytes = NB * 4;          // per-column fp32 constants that travel with a B tile
    static constexpr uint32_t kSmemA = 0;                    // [stage][half]
    static constexpr uint32_t kSmemB = 2 * AST * kAHalf;
    static constexpr uint32_t kSmemExtra = kSmemB + 2 * kBStage;
    static constexpr uint32_t kSmemEpi = kSmemExtra + kExtraSlots * kExtraBytes;   // epilogue scratch
    static constexpr uint32_t kSmemBar = kSmemEpi + kEpiBytes;
    static constexpr uint32_t kSmemBytes = kSmemBar + 256;
    // barrier slots
    static constexpr int kBarAFull = 0, kBarAEmpty = 2 * AST, kBarBFull = 4 * AST, kBarBEmpty = kBarBFull + 2,
                         kBarAccFull = kBarBEmpty + 2, kBarAccEmpty = kBarAccFull + 2, kBarXFull = kBarAccEmpty + 2,
                         kNumBars = kBarXFull + kExtraSlots;
    static_assert(8 * kNumBars + 8 <= 256, "barrier block too small");
    static_assert(kSmemBytes <= 232448, "shared memory budget");

    struct Ctx {
        uint32_t base, bars, tmem_base;
        volatile int *abort_flag;
        int warp, lane;
        int group, quarter;        // epilogue warps: which A half they serve, which 32 TMEM lanes they read
        int colhalf;               // ... and which half of each accumulator's columns
        bool ok;                   // false: shared memory was not 1024-byte aligned; nothing may run
        __device__ __forceinline__ uint32_t bar(int i) const { return bars + 8u * i; }
        // shared address of the per-column constants of the bt-th B tile this CTA streams (valid from the tile's
        // extra_wait to its release)
        __device__ __forceinline__ uint32_t extra(int bt) const {
            return base + kSmemExtra + (uint32_t)(bt & (kExtraSlots - 1)) * kExtraBytes;
        }
        // shared addresses of the scratch of this warp's quad / of its partner quad on the same rows
        __device__ __forceinline__ uint32_t epi_addr() const { return base + kSmemEpi + (uint32_t)(group * 2 + colhalf) * (kEpiBytes / 4); }
        __device__ __forceinline__ uint32_t partner_addr() const {
            return base + kSmemEpi + (uint32_t)(group * 2 + (colhalf ^ 1)) * (kEpiBytes / 4);
        }
        // shared address of A half `group` of the n-th item this group takes part in
        __device__ __forceinline__ uint32_t a_addr(int n) const {
            return base + kSmemA + (uint32_t)((n % AST) * 2 + group) * kAHalf;
        }
    };

    // `a_readers`: epilogue warps per half that read the A stage themselves and release it with a_release().
    static __device__ __forceinline__ Ctx setup(uint8_t *smem_raw, const CUtensorMap *ma, const CUtensorMap *mb,
                                                int *status, int a_readers = 0, int acc_arrivals = 8) {
        Ctx c;
        c.base = tc::smem_u32(smem_raw);
        c.bars = c.base + kSmemBar;
        c.warp = threadIdx.x >> 5;
        c.lane = threadIdx.x & 31;
        c.group = ((c.warp - 2) >> 2) & 1;
        c.quarter = c.warp & 3;
        c.colhalf = (c.warp - 2) >> 3;
        c.tmem_base = 0;
        c.abort_flag = reinterpret_cast<volatile int *>(smem_raw + kSmemBar + 8 * kNumBars + 4);
        c.ok = (c.base & 1023u) == 0;              // the swizzled operand tiles need a 1024-byte aligned base
        if (!c.ok) {
            if (threadIdx.x == 0) atomicCAS(status, 0, kStatusAlign);
            return c;
        }
        uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem_raw + kSmemBar + 8 * kNumBars);
        if (threadIdx.x == 0) {
            for (int i = 0; i < kNumBars; ++i) {
                int count = 1;
                if (i >= kBarAEmpty && i < kBarBFull) count = 1 + a_readers;
                if (i >= kBarAccEmpty && i < kBarXFull) count = acc_arrivals;   // one arrival per epilogue warp that reads the half
                tc::mbar_init(c.bar(i), count);
            }
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

    static __device__ __forceinline__ void teardown(const Ctx &c) {
        if (!c.ok) return;
        tc::tc_fence_before();
        __syncthreads();
        tc::tc_fence_after();
        if (c.warp == 1) tc::tmem_dealloc(c.tmem_base, 512);
    }

    // Call from one thread.  a_bytes / b_bytes: bytes one A-half / B box pair delivers (both K halves).
    template <class PlanFn>
    static __device__ __forceinline__ void producer(const Ctx &c, const CUtensorMap *ma, const CUtensorMap *mb, int n_items,
                                                    uint32_t a_bytes, uint32_t b_bytes, PlanFn plan, int *status) {
        int ia[2] = {0, 0}, bt = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
            const TilePlan p = plan(item);
            if (p.empty()) continue;
            for (int t = 0; ok && t < p.n_tiles; ++t, ++bt) {
                const int sb = bt & 1;
                ok = tc::mbar_wait(c.bar(kBarBEmpty + sb), ((bt >> 1) & 1) ^ 1, c.abort_flag, status);
                if (!ok) break;
                if (p.extra) {       // slot reuse is safe: both epilogues released tile bt-4 before the MMAs of bt-2 began
                    const int xs = bt & (kExtraSlots - 1);
                    tc::mbar_expect_tx(c.bar(kBarXFull + xs), kExtraBytes);
                    tc::bulk_load(c.base + kSmemExtra + (uint32_t)xs * kExtraBytes, p.extra + (size_t)t * NB, kExtraBytes,
                                  c.bar(kBarXFull + xs));
                }
                tc::mbar_expect_tx(c.bar(kBarBFull + sb), b_bytes);
                const uint32_t b_dst = c.base + kSmemB + sb * kBStage;
                tc::tma_load_4d(b_dst, mb, c.bar(kBarBFull + sb), 0, p.b1 + t * p.step1, p.b2 + t * p.step2, p.b3);
                tc::tma_load_4d(b_dst + kBStage / 2, mb, c.bar(kBarBFull + sb), 64, p.b1 + t * p.step1, p.b2 + t * p.step2, p.b3);
                if (t == 0) {                  // the item's A halves go out right after its first B tile
                    for (int h = 0; ok && h < p.n_halves; ++h) {
                        const int st = ia[h] % AST, full = kBarAFull + st * 2 + h;
                        ok = tc::mbar_wait(c.bar(kBarAEmpty + st * 2 + h), ((ia[h] / AST) & 1) ^ 1, c.abort_flag, status);
                        if (!ok) break;
                        tc::mbar_expect_tx(c.bar(full), a_bytes);
                        const uint32_t a_dst = c.base + kSmemA + (uint32_t)(st * 2 + h) * kAHalf;
                        tc::tma_load_4d(a_dst, ma, c.bar(full), 0, p.a1 + h * p.h1, p.a2 + h * p.h2, p.a3);
                        tc::tma_load_4d(a_dst + kAHalf / 2, ma, c.bar(full), 64, p.a1 + h * p.h1, p.a2 + h * p.h2, p.a3);
                        ++ia[h];
                    }
                }
            }
        }
        if (!ok) {          // winding down after a timeout: give copies already issued a moment to land
            for (int i = 0; i < 2 * AST; ++i)
                for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(c.bar(kBarAFull + i), 0) && !tc::mbar_try_wait(c.bar(kBarAFull + i), 1); ++s) {}
            for (int i = 0; i < 2; ++i)
                for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(c.bar(kBarBFull + i), 0) && !tc::mbar_try_wait(c.bar(kBarBFull + i), 1); ++s) {}
        }
    }

    // Call from one thread.
    template <class PlanFn>
    static __device__ __forceinline__ void mma_issuer(const Ctx &c, int n_items, PlanFn plan, int *status) {
        int ia[2] = {0, 0}, ta[2] = {0, 0}, bt = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < n_items; item += gridDim.x) {
            const TilePlan p = plan(item);
            if (p.empty()) continue;
            for (int t = 0; ok && t < p.n_tiles; ++t, ++bt) {
                const int sb = bt & 1;
                ok = tc::mbar_wait(c.bar(kBarBFull + sb), (bt >> 1) & 1, c.abort_flag, status);
                if (!ok) break;
                const int ncols = min(NB, p.cols_total - t * NB);
                const uint32_t idesc = tc::idesc_bf16(kRows, (uint32_t)((ncols + 15) & ~15));
                const uint32_t b_base = c.base + kSmemB + sb * kBStage;
                for (int h = 0; ok && h < p.n_halves; ++h) {
                    const int st = ia[h] % AST;
                    if (t == 0) ok = tc::mbar_wait(c.bar(kBarAFull + st * 2 + h), (ia[h] / AST) & 1, c.abort_flag, status);
                    ok = ok && tc::mbar_wait(c.bar(kBarAccEmpty + h), (ta[h] & 1) ^ 1, c.abort_flag, status);
                    if (!ok) break;
                    tc::tc_fence_after();
                    const uint32_t a_base = c.base + kSmemA + (uint32_t)(st * 2 + h) * kAHalf;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {                     // head_dim 128 = 8 K slices of 16
                        const uint32_t a_off = (ks >> 2) * (kAHalf / 2) + (ks & 3) * 32;
                        const uint32_t b_off = (ks >> 2) * (kBStage / 2) + (ks & 3) * 32;
                        tc::umma_bf16(c.tmem_base + h * NB, tc::smem_desc_sw128(a_base, a_off),
                                      tc::smem_desc_sw128(b_base, b_off), idesc, ks > 0);
                    }
                    tc::umma_commit(c.bar(kBarAccFull + h));             // accumulator of this half ready
                    ++ta[h];
                    if (t == p.n_tiles - 1) {                            // that was the half's last use of its A stage
                        tc::umma_commit(c.bar(kBarAEmpty + st * 2 + h));
                        ++ia[h];
                    }
                }
                if (!ok) break;
                tc::umma_commit(c.bar(kBarBEmpty + sb));                 // B stage free once both halves' MMAs finish
            }
        }
    }

    // Epilogue side.  `k` counts the accumulator tiles this warp's half has consumed.
    static __device__ __forceinline__ bool acc_wait(const Ctx &c, int k, int *status) {
        const bool ok = tc::mbar_wait(c.bar(kBarAccFull + c.group), k & 1, c.abort_flag, status);
        tc::tc_fence_after();
        return ok;
    }
    // For kernels whose epilogue reads its A half from shared memory: wait until the half of the
    // n-th item this group takes part in has landed (at Ctx::a_addr(n)) / hand it back (one arrival per warp).
    static __device__ __forceinline__ bool a_wait(const Ctx &c, int n, int *status) {
        return tc::mbar_wait(c.bar(kBarAFull + (n % AST) * 2 + c.group), (n / AST) & 1, c.abort_flag, status);
    }
    static __device__ __forceinline__ void a_release(const Ctx &c, int n) {
        __syncwarp();
        if (c.lane == 0) tc::mbar_arrive(c.bar(kBarAEmpty + (n % AST) * 2 + c.group));
    }
    // Waits until the per-column constants of the bt-th B tile are in shared memory.
    static __device__ __forceinline__ bool extra_wait(const Ctx &c, int bt, int *status) {
        return tc::mbar_wait(c.bar(kBarXFull + (bt & (kExtraSlots - 1))), (bt / kExtraSlots) & 1, c.abort_flag, status);
    }
    static __device__ __forceinline__ void acc_release(const Ctx &c) {
        tc::tc_fence_before();
        __syncwarp();
        if (c.lane == 0) tc::mbar_arrive(c.bar(kBarAccEmpty + c.group));
    }
    // TMEM address of columns [32*chunk, 32*chunk+32) of this warp's half for its 32 lanes.
    static __device__ __forceinline__ uint32_t acc_addr(const Ctx &c, int chunk) {
        return c.tmem_base + c.group * NB + chunk * 32 + ((uint32_t)(c.quarter * 32) << 16);
    }

    // Runs f(chunk, values) over this warp's 32-column chunks of the current accumulator: the chunks of
    // its column half, as far as they lie below n_chunks (the tile's chunk count).
    template <class F>
    static __device__ __forceinline__ void for_each_chunk(const Ctx &c, int n_chunks, F &&f) {
        constexpr int kPer = NB / 64;
        const int hi = min(n_chunks, kPer * c.colhalf + kPer);
        for (int ch = kPer * c.colhalf; ch < hi; ++ch) {
            uint32_t a[32];
            tc::tmem_ld32(acc_addr(c, ch), a);
            tc::tmem_ld_wait(a);
            f(ch, a);
        }
    }
    // The same walk in blocks of 16 columns (for epilogues that are short of registers): f(block, values)
    // for the blocks of this warp's column half below n_blocks = ceil(columns of the tile / 16).
    template <class F>
    static __device__ __forceinline__ void for_each_block16(const Ctx &c, int n_blocks, F &&f) {
        constexpr int kPer = NB / 32;
        const int hi = min(n_blocks, kPer * c.colhalf + kPer);
        for (int b = kPer * c.colhalf; b < hi; ++b) {
            uint32_t a[16];
            tc::tmem_ld16(c.tmem_base + c.group * NB + b * 16 + ((uint32_t)(c.quarter * 32) << 16), a);
            tc::tmem_ld_wait(a);
            f(b, a);
        }
    }
    // The same for epilogues in which all sixteen warps drain one accumulator at a time (warp = 32 lanes x
    // a quarter of the columns, both halves in turn): explicit half index, `k` = tiles of that half so far.
    static __device__ __forceinline__ bool acc_wait_h(const Ctx &c, int h, int k, int *status) {
        const bool ok = tc::mbar_wait(c.bar(kBarAccFull + h), k & 1, c.abort_flag, status);
        tc::tc_fence_after();
        return ok;
    }
    static __device__ __forceinline__ void acc_release_h(const Ctx &c, int h) {
        tc::tc_fence_before();
        __syncwarp();
        if (c.lane == 0) tc::mbar_arrive(c.bar(kBarAccEmpty + h));
    }
    template <class F>
    static __device__ __forceinline__ void for_each_chunk_q(const Ctx &c, int h, int colq, int n_chunks, F &&f) {
        constexpr int kPer = NB / 128;
        const int hi = min(n_chunks, kPer * colq + kPer);
        for (int ch = kPer * colq; ch < hi; ++ch) {
            uint32_t a[32];
            tc::tmem_ld32(c.tmem_base + h * NB + ch * 32 + ((uint32_t)(c.quarter * 32) << 16), a);
            tc::tmem_ld_wait(a);
            f(ch, a);
        }
    }
    // The same meeting point with a vote: returns whether either warp has given up on a wait, so that both leave
    // the item loop together and neither is left alone at the next meeting.
    static __device__ __forceinline__ bool pair_meet(const Ctx &c, bool gave_up) {
        uint32_t any;
        asm volatile(
            "{\n\t.reg .pred p, q;\n\t"
            "setp.ne.u32 q, %1, 0;\n\t"
            "barrier.cta.red.or.pred p, %2, 64, q;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(any)
            : "r"((uint32_t)gave_up), "r"(1 + c.group * 4 + c.quarter)
            : "memory");
        return any != 0;
    }
    // Meeting point of the two warps that share rows (same half, same lanes, other columns).
    static __device__ __forceinline__ void pair_sync(const Ctx &c) {
        asm volatile("bar.sync %0, 64;" ::"r"(1 + c.group * 4 + c.quarter) : "memory");
    }
};

using Big = Skel<256, 1>;       // long B streams
using Small = Skel<128, 2>;     // few B columns per item: the A operand is the stream

}  // namespace tcs
}  // namespace flowmm
