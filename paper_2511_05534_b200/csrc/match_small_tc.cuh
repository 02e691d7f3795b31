// Matching step (Eq. 9 and Eq. 10) on the tensor cores for short candidate lists (at most 256 columns
// per head, i.e. budgets of up to 224 pivots): the whole candidate matrix of a head is one operand tile.
//
// Same preparation as match_tc.cuh (match_prepare_kernel: admissible pivots gathered into a dense matrix,
// text group first, visual group from the next multiple of 32, NaN scales where there is no candidate).
// CTAs are persistent (one per SM) and take whole heads: warp 0 lane 0 loads the head's candidate tile,
// its reciprocal norms and slots (double-buffered by head up to 128 columns) and streams the head's
// 128-token tiles through a TMA ring; warp 1 lane 0 issues S = K_tile C^T (tcgen05.mma, M = 128 tokens,
// N = candidates) into one of four (two above 128 columns) TMEM accumulators; four teams of four warps
// take the tiles in turn: a thread owns a token,
// reads its key row from the A stage for the norm, walks its admissible candidate blocks (an intra-modal
// layer: only the blocks of the token's own modality), keeps the running maximum per group of 8 columns
// and recovers the exact column at the end.  Nothing is handed between warps.
#pragma once
#include "common.cuh"
#include "match_tc.cuh"
#include "tc_common.cuh"

namespace flowmm {
namespace mst {

constexpr int kTile = 128;
constexpr int kStages = 4;
constexpr int kMaxCols = 256;
constexpr int kMaxSets = 4;                   // TMEM accumulators: four of 128 columns or two of 256
constexpr int kTeams = 4;
constexpr int kThreads = 64 + kTeams * 128;
constexpr uint32_t kStageBytes = kTile * 128 * 2, kPanel = kStageBytes / 2;
constexpr uint32_t kBRegion = kMaxCols * 256;                      // candidate tiles (two panels of N rows each): two of up to 128 rows or one
constexpr uint32_t kSmemB = kStages * kStageBytes;
constexpr uint32_t kSmemMeta = kSmemB + kBRegion;                  // per candidate buffer: float scale[N], int slot[N]
constexpr uint32_t kSmemStash = kSmemMeta + 4096;                  // per team: 8 floats per row
constexpr uint32_t kSmemBar = kSmemStash + kTeams * 4096;
constexpr int kBarFull = 0, kBarEmpty = kStages, kBarBFull = 2 * kStages, kBarBEmpty = kBarBFull + 2,
              kBarAccFull = kBarBEmpty + 2, kBarSetFree = kBarAccFull + kMaxSets, kNumBars = kBarSetFree + kMaxSets;
constexpr uint32_t kSmemBytes = kSmemBar + 8 * kNumBars + 16;
static_assert(kSmemBytes <= 232448, "shared memory budget");

struct Args {
    const int *cand_count, *cand_slot, *rank, *strategy;
    const float *cand_scale;
    const uint8_t *modality;
    int *match;
    float *match_sim;
    int2 *tokmap;          // nullptr, or [UH, L]: the (slot, weight) table of the tensor-core merge, written here instead of by merge_map_kernel
    int *status;
    int Hkv, L, E, Ctot, n_heads, merge_mode;
};

__global__ void __launch_bounds__(kThreads, 1)
match_small_tc_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap cand_map, const Args A) {
    extern __shared__ __align__(1024) uint8_t mst_smem[];
    const uint32_t base = tc::smem_u32(mst_smem), bars = base + kSmemBar;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(mst_smem + kSmemBar + 8 * kNumBars + 4);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(mst_smem + kSmemBar + 8 * kNumBars);
    if ((base & 1023u) != 0) {
        if (threadIdx.x == 0) atomicCAS(A.status, 0, 6);
        return;
    }
    const int nt = (A.L + kTile - 1) / kTile, N = A.Ctot;
    const uint32_t b_bytes = (uint32_t)N * 256u, b_panel = (uint32_t)N * 128u;
    const int n_sets = N <= 128 ? 4 : 2, n_bbuf = N <= 128 ? 2 : 1;
    const uint32_t set_cols = N <= 128 ? 128u : 256u, b_stride = kBRegion / 2, m_stride = 2048, slot_off = 4u * (uint32_t)N;
    auto bar = [&](int i) { return bars + 8u * i; };
    if (threadIdx.x == 0) {
        for (int i = 0; i < kNumBars; ++i) {
            int count = 1;
            if (i >= kBarEmpty && i < kBarBFull) count = 1 + 4;          // the MMAs and the four warps that read the norm
            if (i >= kBarBEmpty && i < kBarAccFull) count = 1 + 4 * nt;  // the MMAs and every warp that used scales and slots
            if (i >= kBarSetFree) count = 4;
            tc::mbar_init(bar(i), count);
        }
        *abort_flag = 0;
        tc::mbar_init_fence();
        tc::tma_prefetch_desc(&k_map);
        tc::tma_prefetch_desc(&cand_map);
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), 512);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int i = 0, hc = 0;
            for (int uh = blockIdx.x; ok && uh < A.n_heads; uh += gridDim.x, ++hc) {
                const int u = uh / A.Hkv, h = uh % A.Hkv, hp = hc % n_bbuf;
                ok = tc::mbar_wait(bar(kBarBEmpty + hp), ((hc / n_bbuf) & 1) ^ 1, abort_flag, A.status);
                if (!ok) break;
                const uint32_t bd = base + kSmemB + hp * b_stride, md = base + kSmemMeta + hp * m_stride;
                tc::mbar_expect_tx(bar(kBarBFull + hp), b_bytes + 8u * (uint32_t)N);
                tc::tma_load_4d(bd, &cand_map, bar(kBarBFull + hp), 0, 0, uh, 0);
                tc::tma_load_4d(bd + b_panel, &cand_map, bar(kBarBFull + hp), 64, 0, uh, 0);
                tc::bulk_load(md, A.cand_scale + (int64_t)uh * N, 4u * (uint32_t)N, bar(kBarBFull + hp));
                tc::bulk_load(md + slot_off, A.cand_slot + (int64_t)uh * N, 4u * (uint32_t)N, bar(kBarBFull + hp));
                for (int t = 0; ok && t < nt; ++t, ++i) {
                    const int st = i % kStages;
                    ok = tc::mbar_wait(bar(kBarEmpty + st), ((i / kStages) & 1) ^ 1, abort_flag, A.status);
                    if (!ok) break;
                    const uint32_t dst = base + st * kStageBytes;
                    tc::mbar_expect_tx(bar(kBarFull + st), kStageBytes);
                    tc::tma_load_4d(dst, &k_map, bar(kBarFull + st), 0, t * kTile, h, u);
                    tc::tma_load_4d(dst + kPanel, &k_map, bar(kBarFull + st), 64, t * kTile, h, u);
                }
            }
            if (!ok) {       // winding down after a timeout: give copies already issued a moment to land
                for (int b = 0; b < kStages; ++b)
                    for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(bar(kBarFull + b), 0) && !tc::mbar_try_wait(bar(kBarFull + b), 1); ++s) {}
                for (int b = 0; b < 2; ++b)
                    for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(bar(kBarBFull + b), 0) && !tc::mbar_try_wait(bar(kBarBFull + b), 1); ++s) {}
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = tc::idesc_bf16(kTile, (uint32_t)N);
            bool ok = true;
            int i = 0, hc = 0;
            for (int uh = blockIdx.x; ok && uh < A.n_heads; uh += gridDim.x, ++hc) {
                const int hp = hc % n_bbuf;
                ok = tc::mbar_wait(bar(kBarBFull + hp), (hc / n_bbuf) & 1, abort_flag, A.status);
                const uint32_t bd = base + kSmemB + hp * b_stride;
                for (int t = 0; ok && t < nt; ++t, ++i) {
                    const int st = i % kStages, set = i % n_sets;
                    // Barriers go by team (tile i belongs to team i mod 4), accumulators by i mod n_sets: the accumulator
                    // of tile i was last used by tile i - n_sets, whose team signals on its own barrier.  (One barrier per
                    // accumulator would be waited on by two teams two phases apart, which a parity cannot tell apart.)
                    ok = tc::mbar_wait(bar(kBarFull + st), (i / kStages) & 1, abort_flag, A.status);
                    if (ok && i >= n_sets) {
                        const int j = i - n_sets;
                        ok = tc::mbar_wait(bar(kBarSetFree + (j & 3)), (j >> 2) & 1, abort_flag, A.status);
                    }
                    if (!ok) break;
                    tc::tc_fence_after();
                    const uint32_t a = base + st * kStageBytes;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        tc::umma_bf16(tmem + set_cols * set, tc::smem_desc_sw128(a + (j >> 2) * kPanel, (j & 3) * 32),
                                      tc::smem_desc_sw128(bd + (j >> 2) * b_panel, (j & 3) * 32), idesc, j > 0);
                    tc::umma_commit(bar(kBarEmpty + st));
                    tc::umma_commit(bar(kBarAccFull + (i & 3)));
                }
                if (ok) tc::umma_commit(bar(kBarBEmpty + hp));
            }
        }
    } else {
        const int team = (warp - 2) >> 2, wq = warp & 3;
        const int row = 32 * wq + lane;                              // TMEM lane = token of the tile
        const uint32_t tlane = tmem + ((uint32_t)(32 * wq) << 16);
        const uint32_t wrow = base + kSmemStash + team * 4096 + row * 32;
        bool ok = true;
        int hc = 0;
        for (int uh = blockIdx.x; uh < A.n_heads; uh += gridDim.x, ++hc) {
            const int u = uh / A.Hkv, hp = hc % n_bbuf;
            const uint32_t md = base + kSmemMeta + hp * m_stride;
            const int n_text = A.cand_count[2 * uh], n_vis = A.cand_count[2 * uh + 1];
            const bool intra = A.strategy[u] == 0;
            const int t0 = (n_text + 31) & ~31;
            const int end_all = n_vis > 0 ? t0 + n_vis : n_text;
            const int nb_all = (end_all + 15) >> 4;                  // blocks of 16 columns that hold candidates
            bool b_ready = false;
            for (int t = 0; t < nt; ++t) {                           // tile number i of this CTA's sequence goes to team i mod 4
                const int i = hc * nt + t, st = i % kStages, set = i % n_sets;
                if ((i & (kTeams - 1)) != team) continue;
                const uint32_t trow = tlane + set_cols * set;
                const int token = t * kTile + row;
                const bool in_range = token < A.L;
                const int my_mod = in_range ? A.modality[(int64_t)u * A.L + token] : 0;
                const int my_rank = in_range ? A.rank[(int64_t)uh * A.L + token] : -1;
                // the blocks this token may take: all of them in a cross-modal layer, else its own modality's group
                int blo = 0, bhi = nb_all;
                if (intra) {
                    if (my_mod == 0) bhi = (n_text + 15) >> 4;
                    else { blo = t0 >> 4; bhi = n_vis > 0 ? nb_all : blo; }
                }
                // the token's key row sits in the A stage (128-byte rows, 16-byte units XOR-swizzled by the row index)
                ok = ok && tc::mbar_wait(bar(kBarFull + st), (i / kStages) & 1, abort_flag, A.status);
                float ssq = 0.f;
                {
                    const uint32_t a_row = base + st * kStageBytes + row * 128;
#pragma unroll
                    for (int kh = 0; kh < 2; ++kh) {
#pragma unroll
                        for (int un = 0; un < 8; ++un) {
                            const float4 rawf = tc::lds128(a_row + kh * kPanel + ((un ^ (row & 7)) << 4));
                            const uint4 raw = make_uint4(__float_as_uint(rawf.x), __float_as_uint(rawf.y), __float_as_uint(rawf.z),
                                                         __float_as_uint(rawf.w));
                            float x[8];
                            Elem<__nv_bfloat16>::unpack(raw, x);
#pragma unroll
                            for (int e = 0; e < 8; ++e) ssq = fmaf(x[e], x[e], ssq);
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(bar(kBarEmpty + st));
                if (!b_ready) {                                      // scales and slots of this head have landed
                    ok = ok && tc::mbar_wait(bar(kBarBFull + hp), (hc / n_bbuf) & 1, abort_flag, A.status);
                    b_ready = true;
                }
                ok = ok && tc::mbar_wait(bar(kBarAccFull + team), (i >> 2) & 1, abort_flag, A.status);
                tc::tc_fence_after();
                // Running winner among the columns walked so far; candidates are laid out text group first, each group by
                // ascending slot, so the first maximum of a group is its lowest slot.  A token of a cross-modal layer sees
                // both groups: the text group's winner is set aside at the first visual block and the two meet by
                // (similarity, slot), so that equal similarities go to the lower slot.
                float best = -INFINITY, val_a = -INFINITY;
                int best_cc = -1, slot_a = -1;
                auto resolve = [&]() -> int {                        // slot of the running winner: lowest column of its group that holds the maximum
                    if (best_cc < 0) return -1;
                    int idx = 0;
#pragma unroll
                    for (int q4 = 1; q4 >= 0; --q4) {
                        const float4 w = tc::lds128(wrow + q4 * 16);
                        if (w.w == best) idx = 4 * q4 + 3;
                        if (w.z == best) idx = 4 * q4 + 2;
                        if (w.y == best) idx = 4 * q4 + 1;
                        if (w.x == best) idx = 4 * q4;
                    }
                    return index_ok(best_cc + idx, N, A.status) ? __float_as_int(tc::lds32(md + slot_off + (best_cc + idx) * 4)) : -1;
                };
                const int park_blk = intra ? -1 : (t0 >> 4);
                for (int blk = 0; blk < nb_all; ++blk) {
                    uint32_t acc[16];
                    tc::tmem_ld16(trow + blk * 16, acc);
                    tc::tmem_ld_wait(acc);
                    if (blk == park_blk) {
                        slot_a = resolve();
                        val_a = best;
                        best = -INFINITY;
                        best_cc = -1;
                    }
                    if (blk >= blo && blk < bhi) {
                        float v[16];
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {             // a column that is no candidate has scale NaN and never wins
                            const float4 s4 = tc::lds128(md + (blk * 4 + q4) * 16);
                            v[4 * q4 + 0] = __uint_as_float(acc[4 * q4 + 0]) * s4.x;
                            v[4 * q4 + 1] = __uint_as_float(acc[4 * q4 + 1]) * s4.y;
                            v[4 * q4 + 2] = __uint_as_float(acc[4 * q4 + 2]) * s4.z;
                            v[4 * q4 + 3] = __uint_as_float(acc[4 * q4 + 3]) * s4.w;
                        }
#pragma unroll
                        for (int g = 0; g < 2; ++g) {                // two groups of 8 columns, in column order
                            const float q8 = tc::max3(tc::max3(v[8 * g], v[8 * g + 1], v[8 * g + 2]),
                                                      tc::max3(v[8 * g + 3], v[8 * g + 4], v[8 * g + 5]),
                                                      fmaxf(v[8 * g + 6], v[8 * g + 7]));
                            if (q8 > best) {                         // strict: an earlier group keeps a tie (false for NaN)
                                best = q8;
                                best_cc = blk * 16 + 8 * g;
                                tc::sts128(wrow, v[8 * g], v[8 * g + 1], v[8 * g + 2], v[8 * g + 3]);
                                tc::sts128(wrow + 16, v[8 * g + 4], v[8 * g + 5], v[8 * g + 6], v[8 * g + 7]);
                            }
                        }
                    }
                }
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(bar(kBarSetFree + team));   // this warp has read the accumulator
                int slot = resolve();
                if (match_better(val_a, slot_a, best, slot)) { best = val_a; slot = slot_a; }
                if (in_range && my_rank >= 0 && ok && index_ok(my_rank, A.E, A.status)) {   // a non-pivot: report its match
                    float sim = 0.f;
                    if (slot >= 0 && ssq > 0.f) sim = best * rsqrtf(ssq);
                    A.match[(int64_t)uh * A.E + my_rank] = slot;
                    A.match_sim[(int64_t)uh * A.E + my_rank] = sim;
                    if (A.tokmap)                                    // same entry as merge_map_kernel would write
                        A.tokmap[(int64_t)uh * A.L + token] = make_int2(slot, __float_as_int(A.merge_mode == 1 ? 1.f : __expf(sim - 1.f)));
                } else if (in_range && ok && A.tokmap) {             // a pivot: its own slot with weight 1
                    A.tokmap[(int64_t)uh * A.L + token] = make_int2((-my_rank - 2) | (1 << 30), __float_as_int(1.f));
                }
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(bar(kBarBEmpty + hp));      // done with this head's scales and slots for this tile
            }
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (warp == 1) tc::tmem_dealloc(tmem, 512);
}

}  // namespace mst
}  // namespace flowmm
