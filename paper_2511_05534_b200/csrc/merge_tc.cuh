// Weighted merge (Eq. 5) + compaction on the tensor cores, for budgets of up to 240 pivots per head
// (bf16, head_dim 128).
//
// Eq. 5 is out = W X with X the head's L rows of K (or V) and W a B x L matrix with one non-zero per
// column: W[s, t] = w_t if token t is merged into slot s, 1 for the pivot itself.  With few slots that
// product is cheap on the tensor cores and turns the gather into two linear streams (K and V, each row
// read from HBM once, by TMA) with no sort of the match beforehand:
//   merge_map_kernel   scatters (slot, weight) of every token into a per-position table;
//   merge_tc_kernel    persistent CTAs, one (unit, KV head) at a time, 128 tokens per step:
//       builder threads (one per token of the step) write the step's W^T slice into shared memory as a
//       K-major bf16 operand and add the same bf16-rounded weight to its slot's sum (fixed point in
//       shared memory: integer additions commute, so the sum does not depend on their order);
//       out^T[dim, slot] += X_step^T W_step^T as tcgen05.mma with M = 128 dims, N = slots, contraction
//       over the step's tokens; the X tile is the swizzled TMA tile read as an MN-major operand, for K
//       and for V against the same W slice;
//       after the last step four reader warps take out^T from TMEM, scale by 1 / (1 + sum of weights)
//       and store bf16 rows, while the next head's steps already run into a second set of sums and (up to
//       128 slots) a second set of accumulators.
// The weights enter rounded to bf16 (relative error <= 2^-9) in numerator and denominator alike, so every
// output row is still a weighted mean of its members with weights within 0.2 % of Eq. 5's; the change of
// the result is below the bf16 rounding of the output itself.
// Products of bf16 inputs are exact in fp32 and the accumulation order is the hardware's, fixed for a
// given shape, so results are bit-reproducible.  A non-finite K or V entry would reach every slot of its
// head through 0 x inf; the gather kernels confine it to its own slot.
#pragma once
#include "common.cuh"
#include "decode_tc.cuh"
#include "tc_common.cuh"

namespace flowmm {
namespace mtc {

constexpr int kTile = 128;                       // tokens per step
constexpr int kMaxSlots = 240;                   // N <= 240: two 60 KB weight slices and three tile stages fit in shared memory
constexpr int kThreads = 320;                    // TMA warp, MMA warp, four builder warps, four reader warps
constexpr int kPivotFlag = 1 << 30;              // in the table's slot word: the token is the slot's pivot
constexpr uint32_t kStageBytes = kTile * 128 * 2, kPanel = kStageBytes / 2;
constexpr int kMaxStages = 4;
constexpr int kBarFull = 0, kBarEmpty = kMaxStages, kBarWFull = 2 * kMaxStages, kBarWEmpty = kBarWFull + 2,
              kBarOutFull = kBarWEmpty + 2, kBarSumFull = kBarOutFull + 2, kBarOutEmpty = kBarSumFull + 2,
              kNumBars = kBarOutEmpty + 2;               // from kBarSumFull on: 128 arrivals each
constexpr uint32_t kTailData = 2 * kMaxSlots * 4 + kMaxSlots * 4;     // weight sums of two heads, reciprocal normalisers
constexpr float kSumScale = 65536.f;             // weights in [2^-3, 1] rounded to bf16 are whole multiples of 2^-10

struct Args {
    const int2 *tokmap;          // [UH, L] (slot | pivot flag, or -1; weight bits)
    void *k_out, *v_out;
    int *status;
    int Hkv, L, B, n_items, n_stages;
    int64_t kos[3], vos[3];
};

__host__ __device__ inline int slots16(int B) { return (B + 15) & ~15; }
__host__ __device__ inline uint32_t w_bytes(int B) { return (uint32_t)slots16(B) * 256u; }      // two 64-token panels of N rows
__host__ __device__ inline uint32_t smem_bytes(int B, int n_stages) {
    return (uint32_t)n_stages * kStageBytes + 2 * w_bytes(B) + kTailData + 8 * kNumBars + 16;
}

__device__ __forceinline__ void reader_sync() { asm volatile("bar.sync 2, 128;" ::: "memory"); }

struct MapArgs {
    const int *retained, *evicted, *match;
    const float *match_sim;
    int2 *tokmap;
    int L, B, E, merge_mode;
};

// grid = (UH, ceil(max(E, B) / 256))
__global__ void __launch_bounds__(256) merge_map_kernel(const MapArgs A) {
    const int uh = blockIdx.x, i = blockIdx.y * 256 + threadIdx.x;
    int2 *map = A.tokmap + (int64_t)uh * A.L;
    if (i < A.E) {
        const int tok = A.evicted[(int64_t)uh * A.E + i];
        const float w = A.merge_mode == 1 ? 1.f : __expf(A.match_sim[(int64_t)uh * A.E + i] - 1.f);
        if (tok >= 0 && tok < A.L) map[tok] = make_int2(A.match[(int64_t)uh * A.E + i], __float_as_int(w));
    }
    if (i < A.B) {
        const int tok = A.retained[(int64_t)uh * A.B + i];
        if (tok >= 0 && tok < A.L) map[tok] = make_int2(i | kPivotFlag, __float_as_int(1.f));
    }
}

__global__ void __launch_bounds__(kThreads, 1)
merge_tc_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap, const Args A) {
    extern __shared__ __align__(1024) uint8_t mtc_smem[];
    const uint32_t base = tc::smem_u32(mtc_smem);
    const int N = slots16(A.B);
    // accumulator sets in TMEM: up to 128 slots two sets (K at column 0, V at column 128 of a set), else one (V at 256)
    const int n_sets = N <= 128 ? 2 : 1;
    const uint32_t set_cols = 256u, v_col = N <= 128 ? 128u : 256u;
    const uint32_t wsize = w_bytes(A.B), wpanel = (uint32_t)N * 128u;
    const uint32_t w0 = base + (uint32_t)A.n_stages * kStageBytes;
    uint8_t *tail = mtc_smem + (size_t)A.n_stages * kStageBytes + 2 * (size_t)wsize;
    unsigned *wsum = reinterpret_cast<unsigned *>(tail);                                  // [2][kMaxSlots], units of 1 / kSumScale
    float *inv_s = reinterpret_cast<float *>(tail + 2 * kMaxSlots * 4);                   // [kMaxSlots]
    const uint32_t bars = tc::smem_u32(tail + kTailData);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(tail + kTailData + 8 * kNumBars);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tail + kTailData + 8 * kNumBars + 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((base & 1023u) != 0) {
        if (threadIdx.x == 0) atomicCAS(A.status, 0, 6);
        return;
    }
    auto bar = [&](int i) { return bars + 8u * i; };
    if (threadIdx.x == 0) {
        for (int i = 0; i < kNumBars; ++i)
            tc::mbar_init(bar(i), (i >= kBarWFull && i < kBarWFull + 2) || i >= kBarSumFull ? 128 : 1);
        *abort_flag = 0;
        tc::mbar_init_fence();
        tc::tma_prefetch_desc(&kmap);
        tc::tma_prefetch_desc(&vmap);
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), 512);
    for (uint32_t o = threadIdx.x * 16; o < 2 * wsize; o += kThreads * 16) dtc::sts128u(w0 + o, make_uint4(0, 0, 0, 0));
    for (int i = threadIdx.x; i < 2 * kMaxSlots; i += kThreads) wsum[i] = 0u;
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int n_chunk = (A.L + kTile - 1) / kTile;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int i = 0;
            for (int item = blockIdx.x; ok && item < A.n_items; item += gridDim.x) {
                const int u = item / A.Hkv, h = item % A.Hkv;
                for (int c = 0; ok && c < 2 * n_chunk; ++c, ++i) {   // per step the K tile, then the V tile
                    const int st = i % A.n_stages;
                    ok = tc::mbar_wait(bar(kBarEmpty + st), ((i / A.n_stages) & 1) ^ 1, abort_flag, A.status);
                    if (!ok) break;
                    const CUtensorMap *m = (c & 1) ? &vmap : &kmap;
                    const uint32_t dst = base + st * kStageBytes;
                    tc::mbar_expect_tx(bar(kBarFull + st), kStageBytes);
                    tc::tma_load_4d(dst, m, bar(kBarFull + st), 0, (c >> 1) * kTile, h, u);
                    tc::tma_load_4d(dst + kPanel, m, bar(kBarFull + st), 64, (c >> 1) * kTile, h, u);
                }
            }
            if (!ok)         // winding down after a timeout: give copies already issued a moment to land
                for (int s = 0; s < A.n_stages; ++s)
                    for (int n = 0; n < (1 << 16) && !tc::mbar_try_wait(bar(kBarFull + s), 0) && !tc::mbar_try_wait(bar(kBarFull + s), 1); ++n) {}
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_bf16(128, (uint32_t)N) | (1u << 15);       // A operand MN-major
            bool ok = true;
            int i = 0, j = 0, it = 0;
            for (int item = blockIdx.x; ok && item < A.n_items; item += gridDim.x, ++it) {
                const int set = it % n_sets, use = it / n_sets;
                ok = tc::mbar_wait(bar(kBarOutEmpty + set), (use & 1) ^ 1, abort_flag, A.status);   // the set's previous head is read out
                tc::tc_fence_after();
                for (int c = 0; ok && c < n_chunk; ++c, ++j) {
                    const int wb = j & 1;
                    ok = tc::mbar_wait(bar(kBarWFull + wb), (j >> 1) & 1, abort_flag, A.status);
                    const uint32_t w = w0 + wb * wsize;
                    for (int t = 0; ok && t < 2; ++t, ++i) {
                        const int st = i % A.n_stages;
                        ok = tc::mbar_wait(bar(kBarFull + st), (i / A.n_stages) & 1, abort_flag, A.status);
                        if (!ok) break;
                        tc::tc_fence_after();
                        const uint32_t a = base + st * kStageBytes;
#pragma unroll
                        for (int q = 0; q < 8; ++q)
                            tc::umma_bf16(tmem + set * set_cols + t * v_col, dtc::smem_desc_sw128_mn(a, q * 2048),
                                          tc::smem_desc_sw128(w + (q >> 2) * wpanel, (q & 3) * 32), idesc, (c | q) != 0);
                        tc::umma_commit(bar(kBarEmpty + st));
                    }
                    if (ok) tc::umma_commit(bar(kBarWEmpty + wb));
                }
                if (ok) tc::umma_commit(bar(kBarOutFull + set));
            }
        }
    } else if (warp < 6) {
        // builders: thread = token of a step
        const int e = threadIdx.x - 64;
        uint32_t wr0 = 0, wr1 = 0;                                   // where this thread's last entry of each W buffer sits
        bool ok = true;
        int j = 0, it = 0;
        // position of this thread's token inside a W panel row: 64 tokens per 128-byte row, 16-byte groups swizzled by row
        const uint32_t tok_off = (uint32_t)(e >> 6) * wpanel + (uint32_t)((e & 7) << 1);
        const int tok_grp = (e & 63) >> 3;
        int2 first = (int)blockIdx.x < A.n_items && e < A.L ? A.tokmap[(int64_t)blockIdx.x * A.L + e] : make_int2(-1, 0);
        for (int item = blockIdx.x; item < A.n_items; item += gridDim.x, ++it) {
            const int2 *map = A.tokmap + (int64_t)item * A.L;
            const int set = it % n_sets, use = it / n_sets;
            unsigned *sums = wsum + set * kMaxSlots;
            // the set's sums are zero again once its previous head has been read out
            ok = ok && tc::mbar_wait(bar(kBarOutEmpty + set), (use & 1) ^ 1, abort_flag, A.status);
            int2 nxt = first;
            for (int c = 0; c < n_chunk; ++c, ++j) {
                const int2 cur = nxt;
                const int t_next = (c + 1) * kTile + e;
                if (c + 1 < n_chunk) nxt = t_next < A.L ? map[t_next] : make_int2(-1, 0);
                else first = item + (int)gridDim.x < A.n_items && e < A.L ? map[(int64_t)gridDim.x * A.L + e] : make_int2(-1, 0);
                const int wb = j & 1;
                ok = ok && tc::mbar_wait(bar(kBarWEmpty + wb), ((j >> 1) & 1) ^ 1, abort_flag, A.status);
                const uint32_t w = w0 + wb * wsize;
                const uint32_t prev = wb ? wr1 : wr0;
                uint32_t mine = 0;
                if (prev) dtc::sts16(prev, 0);                       // take back what this thread wrote two steps ago
                const int slot = cur.x & ~kPivotFlag;
                if (cur.x >= 0 && slot < A.B) {
                    const __nv_bfloat16 wt = __float2bfloat16_rn(__int_as_float(cur.y));
                    const uint32_t at = w + tok_off + (uint32_t)slot * 128u + (uint32_t)((tok_grp ^ (slot & 7)) << 4);
                    dtc::sts16(at, __bfloat16_as_ushort(wt));
                    mine = at;
                    if (!(cur.x & kPivotFlag)) atomicAdd(sums + slot, (unsigned)(__bfloat162float(wt) * kSumScale + 0.5f));
                }
                if (wb) wr1 = mine; else wr0 = mine;
                dtc::fence_proxy_async();
                tc::mbar_arrive(bar(kBarWFull + wb));
            }
            tc::mbar_arrive(bar(kBarSumFull + set));                 // this head's weight sums are complete
        }
    } else {
        // readers: thread = output dim; columns = slots
        const int e = threadIdx.x - 192;
        const int row = 32 * (warp & 3) + lane;
        const uint32_t trow = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
        bool ok = true;
        int it = 0;
        for (int item = blockIdx.x; item < A.n_items; item += gridDim.x, ++it) {
            const int u = item / A.Hkv, h = item % A.Hkv;
            const int set = it % n_sets, use = it / n_sets;
            unsigned *sums = wsum + set * kMaxSlots;
            ok = ok && tc::mbar_wait(bar(kBarSumFull + set), use & 1, abort_flag, A.status);
            for (int sl = e; sl < N; sl += 128) {
                inv_s[sl] = 1.f / (1.f + (float)sums[sl] * (1.f / kSumScale));
                sums[sl] = 0u;
            }
            reader_sync();
            ok = ok && tc::mbar_wait(bar(kBarOutFull + set), use & 1, abort_flag, A.status);
            tc::tc_fence_after();
            if (*abort_flag == 0) {
#pragma unroll 1
                for (int t = 0; t < 2; ++t) {
                    __nv_bfloat16 *out = static_cast<__nv_bfloat16 *>(t ? A.v_out : A.k_out) +
                                         (t ? u * A.vos[0] + h * A.vos[1] : u * A.kos[0] + h * A.kos[1]) + row;
                    const int64_t stride = t ? A.vos[2] : A.kos[2];
                    const uint32_t tcol = trow + set * set_cols + t * v_col;
#pragma unroll 1
                    for (int s0 = 0; s0 < A.B; s0 += 16) {
                        uint32_t acc[16];
                        tc::tmem_ld16(tcol + s0, acc);
                        tc::tmem_ld_wait(acc);
#pragma unroll
                        for (int q = 0; q < 16; ++q)
                            if (s0 + q < A.B)
                                out[(int64_t)(s0 + q) * stride] = __float2bfloat16_rn(__uint_as_float(acc[q]) * inv_s[s0 + q]);
                    }
                }
            }
            tc::tc_fence_before();
            reader_sync();                                           // inv_s may be rewritten, the set reused
            tc::mbar_arrive(bar(kBarOutEmpty + set));
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (warp == 1) tc::tmem_dealloc(tmem, 512);
}

}  // namespace mtc
}  // namespace flowmm
