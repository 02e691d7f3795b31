// Tensor-core path of the matching step (Eq. 9 and Eq. 10) for bf16 keys with head_dim 128.
//
// Per (unit, KV head) the admissible pivots (importance <= tau) are gathered into a dense
// candidate matrix, text candidates first and visual candidates from the next multiple of 32.
// The similarity contraction then runs as  S[128 tokens x 256 candidates] = K_tile . C_tile^T
// on tcgen05 with the token rows taken straight from the caller's K by TMA (every token of the
// head in prompt order; rows that are pivots are computed and dropped), fp32 accumulators in
// TMEM, and an epilogue that scales each column by the candidate's reciprocal norm and keeps a
// running row maximum.  Raw bf16 keys feed the MMA (their products are exact in fp32); the
// norms enter in fp32 afterwards, so no precision is lost before the argmax.
// An intra-modal layer visits only the candidate group of the row tile's modality.
#pragma once
#include "common.cuh"
#include "tc_common.cuh"

namespace flowmm {

constexpr int kMtRows = 128;                 // tokens per row tile (UMMA M)
constexpr int kMtCols = 256;                 // candidates per column tile (UMMA N)
constexpr int kMtThreads = 192;              // warp 0: TMA, warp 1: MMA, warps 2-5: epilogue
constexpr uint32_t kMtABytes = kMtRows * 128 * 2;     // one row tile, both K halves
constexpr uint32_t kMtBBytes = kMtCols * 128 * 2;
constexpr uint32_t kMtSmemA = 0;
constexpr uint32_t kMtSmemB = 2 * kMtABytes;
constexpr uint32_t kMtSmemWin = kMtSmemB + 2 * kMtBBytes;
constexpr uint32_t kMtSmemBar = kMtSmemWin + kMtRows * 32 * 4;
constexpr uint32_t kMtSmemBytes = kMtSmemBar + 256 + 1024;   // + slack to align the base to 1024

struct MatchPrepArgs {
    const void *k;
    const float *importance, *rn;
    const uint8_t *modality;
    const int *retained, *evicted;
    __nv_bfloat16 *cand_k;       // [UH, Ctot, 128]
    float *cand_scale;           // [UH, Ctot]
    int *cand_slot;              // [UH, Ctot]
    int *cand_count;             // [UH, 2]  admissible text / visual pivots
    int *rank;                   // [UH, L]  position in the non-pivot list, or -1 for a pivot
    uint8_t *tile_mod;           // [U, n_rt] bit 0: tile holds text tokens, bit 1: visual tokens
    int Hkv, L, B, E, Ctot, n_rt;
    float tau_eff;
    int64_t ks[3];
};

// grid = U*Hkv, block = 256.
__global__ void __launch_bounds__(256) match_prepare_kernel(const MatchPrepArgs A) {
    __shared__ int scratch[33];
    __shared__ int s_ntext;
    const int tid = threadIdx.x, uh = blockIdx.x, u = uh / A.Hkv, h = uh % A.Hkv;
    const int *ret = A.retained + (int64_t)uh * A.B;
    const int *evi = A.evicted + (int64_t)uh * A.E;
    const float *imp = A.importance + (int64_t)uh * A.L;
    const float *rn = A.rn + (int64_t)uh * A.L;
    const uint8_t *mod = A.modality + (int64_t)u * A.L;
    int *rank = A.rank + (int64_t)uh * A.L;
    int *slot_out = A.cand_slot + (int64_t)uh * A.Ctot;
    float *scale_out = A.cand_scale + (int64_t)uh * A.Ctot;

    for (int i = tid; i < A.Ctot; i += blockDim.x) { slot_out[i] = -1; scale_out[i] = 0.f; }
    for (int s = tid; s < A.B; s += blockDim.x) rank[ret[s]] = -1;
    for (int j = tid; j < A.E; j += blockDim.x) rank[evi[j]] = j;
    if (h == 0) {
        for (int t = tid; t < A.n_rt; t += blockDim.x) {
            int bits = 0;
            const int hi = min(A.L, (t + 1) * kMtRows);
            for (int i = t * kMtRows; i < hi; ++i) bits |= mod[i] ? 2 : 1;
            A.tile_mod[(int64_t)u * A.n_rt + t] = (uint8_t)bits;
        }
    }
    // admissible text pivots first: count them to know where the visual group starts
    int n_text = 0;
    for (int s = tid; s < A.B; s += blockDim.x) {
        const int r = ret[s];
        n_text += (imp[r] <= A.tau_eff && mod[r] == 0) ? 1 : 0;
    }
    int total;
    block_exclusive_scan(n_text, scratch, total);
    if (tid == 0) s_ntext = total;
    __syncthreads();
    const int t0 = (s_ntext + 31) & ~31;
    int seen_t = 0, seen_v = 0;
    for (int base = 0; base < A.B; base += blockDim.x) {
        const int s = base + tid;
        int ft = 0, fv = 0, r = 0;
        if (s < A.B) {
            r = ret[s];
            const bool adm = imp[r] <= A.tau_eff;              // Eq. 10: pivots above tau are kept out of merging
            ft = adm && mod[r] == 0;
            fv = adm && mod[r] != 0;
        }
        int tot_t, tot_v;
        const int pt = seen_t + block_exclusive_scan(ft, scratch, tot_t);
        const int pv = seen_v + block_exclusive_scan(fv, scratch, tot_v);
        if (ft) { slot_out[pt] = s; scale_out[pt] = rn[r]; }
        if (fv) { slot_out[t0 + pv] = s; scale_out[t0 + pv] = rn[r]; }
        seen_t += tot_t;
        seen_v += tot_v;
    }
    if (tid == 0) { A.cand_count[2 * uh] = seen_t; A.cand_count[2 * uh + 1] = seen_v; }
    __syncthreads();
    // copy the candidate key rows (256 bytes each): 16 lanes per row
    const __nv_bfloat16 *kb = static_cast<const __nv_bfloat16 *>(A.k) + u * A.ks[0] + h * A.ks[1];
    uint4 *dst = reinterpret_cast<uint4 *>(A.cand_k + (int64_t)uh * A.Ctot * 128);
    const int sub = tid & 15;
    for (int pos = tid >> 4; pos < A.Ctot; pos += blockDim.x >> 4) {
        const int s = slot_out[pos];
        uint4 val = make_uint4(0, 0, 0, 0);
        if (s >= 0) val = *reinterpret_cast<const uint4 *>(kb + (int64_t)ret[s] * A.ks[2] + sub * 8);
        dst[(int64_t)pos * 16 + sub] = val;
    }
}

struct MatchTcArgs {
    const int *cand_count, *cand_slot, *rank, *strategy;
    const float *cand_scale, *rn;
    const uint8_t *modality, *tile_mod;
    int *match;
    float *match_sim;
    int *status;
    int Hkv, L, E, Ctot, n_rt, n_items;
};

struct MatchItem {
    int u, h, uh, rt, lo, hi, n_tiles, n_text, t0, n_vis;
    bool intra;
};

__device__ __forceinline__ MatchItem match_plan(const MatchTcArgs &A, int item) {
    MatchItem p;
    p.uh = item / A.n_rt; p.rt = item % A.n_rt;
    p.u = p.uh / A.Hkv; p.h = p.uh % A.Hkv;
    p.n_text = A.cand_count[2 * p.uh]; p.n_vis = A.cand_count[2 * p.uh + 1];
    p.t0 = (p.n_text + 31) & ~31;
    p.intra = A.strategy[p.u] == 0;
    const int tm = A.tile_mod[(int64_t)p.u * A.n_rt + p.rt];
    const int end_all = p.n_vis > 0 ? p.t0 + p.n_vis : p.n_text;
    if (!p.intra || tm == 3) { p.lo = 0; p.hi = end_all; }
    else if (tm == 1) { p.lo = 0; p.hi = p.n_text; }
    else { p.lo = p.t0; p.hi = p.t0 + p.n_vis; }
    p.n_tiles = p.hi > p.lo ? (p.hi - p.lo + kMtCols - 1) / kMtCols : 0;
    return p;
}

// Persistent kernel: CTA b handles row-tile items b, b + gridDim.x, ...  One CTA per SM.
__global__ void __launch_bounds__(kMtThreads, 1)
match_tc_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap cand_map,
                const MatchTcArgs A) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t *gen = smem_raw + (base - tc::smem_u32(smem_raw));
    float *win = reinterpret_cast<float *>(gen + kMtSmemWin);
    const uint32_t bars = base + kMtSmemBar;
    // barrier slots: 0-1 a_full, 2-3 a_empty, 4-5 b_full, 6-7 b_empty, 8-9 t_full, 10-11 t_empty
    auto bar = [&](int i) { return bars + 8u * i; };
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(gen + kMtSmemBar + 128);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(gen + kMtSmemBar + 132);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < 10; ++i) tc::mbar_init(bar(i), 1);
        tc::mbar_init(bar(10), 4);
        tc::mbar_init(bar(11), 4);
        *abort_flag = 0;
        tc::mbar_init_fence();
        tc::tma_prefetch_desc(&k_map);
        tc::tma_prefetch_desc(&cand_map);
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), 512);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {                                             // ---- TMA producer
            int it = 0, bt = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < A.n_items; item += gridDim.x) {
                const MatchItem p = match_plan(A, item);
                if (p.n_tiles == 0) continue;
                const int sa = it & 1;
                ok = tc::mbar_wait(bar(2 + sa), ((it >> 1) & 1) ^ 1, abort_flag, A.status);
                if (!ok) break;
                tc::mbar_expect_tx(bar(sa), kMtABytes);
                const uint32_t a_dst = base + kMtSmemA + sa * kMtABytes;
                tc::tma_load_4d(a_dst, &k_map, bar(sa), 0, p.rt * kMtRows, p.h, p.u);
                tc::tma_load_4d(a_dst + kMtABytes / 2, &k_map, bar(sa), 64, p.rt * kMtRows, p.h, p.u);
                for (int t = 0; t < p.n_tiles; ++t, ++bt) {
                    const int sb = bt & 1;
                    ok = tc::mbar_wait(bar(6 + sb), ((bt >> 1) & 1) ^ 1, abort_flag, A.status);
                    if (!ok) break;
                    tc::mbar_expect_tx(bar(4 + sb), kMtBBytes);
                    const uint32_t b_dst = base + kMtSmemB + sb * kMtBBytes;
                    tc::tma_load_3d(b_dst, &cand_map, bar(4 + sb), 0, p.lo + t * kMtCols, p.uh);
                    tc::tma_load_3d(b_dst + kMtBBytes / 2, &cand_map, bar(4 + sb), 64, p.lo + t * kMtCols, p.uh);
                }
                ++it;
            }
            if (!ok) {                                               // let copies already issued land
                for (int i = 0; i < 2; ++i) {
                    for (int spin = 0; spin < (1 << 16) && !tc::mbar_try_wait(bar(i), 0) && !tc::mbar_try_wait(bar(i), 1); ++spin) {}
                    for (int spin = 0; spin < (1 << 16) && !tc::mbar_try_wait(bar(4 + i), 0) && !tc::mbar_try_wait(bar(4 + i), 1); ++spin) {}
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {                                             // ---- MMA issuer
            int it = 0, bt = 0, tt = 0;
            bool ok = true;
            for (int item = blockIdx.x; ok && item < A.n_items; item += gridDim.x) {
                const MatchItem p = match_plan(A, item);
                if (p.n_tiles == 0) continue;
                const int sa = it & 1;
                ok = tc::mbar_wait(bar(sa), (it >> 1) & 1, abort_flag, A.status);
                if (!ok) break;
                const uint32_t a_base = base + kMtSmemA + sa * kMtABytes;
                for (int t = 0; t < p.n_tiles; ++t, ++bt, ++tt) {
                    const int sb = bt & 1, ta = tt & 1;
                    ok = tc::mbar_wait(bar(4 + sb), (bt >> 1) & 1, abort_flag, A.status) &&
                         tc::mbar_wait(bar(10 + ta), ((tt >> 1) & 1) ^ 1, abort_flag, A.status);
                    if (!ok) break;
                    tc::tc_fence_after();
                    const int ncols = min(kMtCols, p.hi - (p.lo + t * kMtCols));
                    const uint32_t idesc = tc::idesc_bf16(kMtRows, (uint32_t)((ncols + 15) & ~15));
                    const uint32_t b_base = base + kMtSmemB + sb * kMtBBytes;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {                 // 8 K slices of 16 elements
                        const uint32_t a_off = (ks >> 2) * (kMtABytes / 2) + (ks & 3) * 32;
                        const uint32_t b_off = (ks >> 2) * (kMtBBytes / 2) + (ks & 3) * 32;
                        tc::umma_bf16(tmem_base + ta * kMtCols, tc::smem_desc_sw128(a_base, a_off),
                                      tc::smem_desc_sw128(b_base, b_off), idesc, ks > 0);
                    }
                    tc::umma_commit(bar(6 + sb));                    // B stage free once these MMAs are done
                    tc::umma_commit(bar(8 + ta));                    // accumulator ready
                }
                if (!ok) break;
                tc::umma_commit(bar(2 + sa));                        // A stage free
                ++it;
            }
        }
    } else {                                                         // ---- epilogue warps
        const int quarter = warp & 3;                                // TMEM lanes this warp may read
        const int row = quarter * 32 + lane;
        float4 *wrow = reinterpret_cast<float4 *>(win + row * 32);
        int tt = 0;
        bool ok = true;
        for (int item = blockIdx.x; ok && item < A.n_items; item += gridDim.x) {
            const MatchItem p = match_plan(A, item);
            const int token = p.rt * kMtRows + row;
            const bool in_range = token < A.L;
            const int my_mod = in_range ? A.modality[(int64_t)p.u * A.L + token] : 0;
            int r1hi = p.n_text, r2lo = p.t0, r2hi = p.t0 + p.n_vis;     // this row's admissible columns
            if (p.intra) { if (my_mod == 0) r2hi = r2lo; else r1hi = 0; }
            if (!in_range) { r1hi = 0; r2hi = r2lo; }
            float best = -INFINITY;
            int best_cc = -1;
            const float *scale = A.cand_scale + (int64_t)p.uh * A.Ctot;
            for (int t = 0; ok && t < p.n_tiles; ++t, ++tt) {
                const int ta = tt & 1;
                ok = tc::mbar_wait(bar(8 + ta), (tt >> 1) & 1, abort_flag, A.status);
                if (!ok) break;
                tc::tc_fence_after();
                const int col0 = p.lo + t * kMtCols;
                const int ncols = min(kMtCols, p.hi - col0);
                for (int c = 0; c * 32 < ncols; ++c) {
                    const int cc = col0 + c * 32;
                    const bool full = (cc + 32 <= r1hi) || (cc >= r2lo && cc + 32 <= r2hi);
                    const bool none = !((cc < r1hi) || (cc + 32 > r2lo && cc < r2hi));
                    if (__all_sync(0xFFFFFFFFu, none)) continue;
                    uint32_t acc[32];
                    tc::tmem_ld32(tmem_base + ta * kMtCols + c * 32 + ((uint32_t)(quarter * 32) << 16), acc);
                    const float4 *sp = reinterpret_cast<const float4 *>(scale + cc);
                    float4 s4[8];
#pragma unroll
                    for (int q4 = 0; q4 < 8; ++q4) s4[q4] = __ldg(sp + q4);
                    tc::tmem_ld_wait();
                    float v[32];
#pragma unroll
                    for (int q4 = 0; q4 < 8; ++q4) {
                        v[4 * q4 + 0] = __uint_as_float(acc[4 * q4 + 0]) * s4[q4].x;
                        v[4 * q4 + 1] = __uint_as_float(acc[4 * q4 + 1]) * s4[q4].y;
                        v[4 * q4 + 2] = __uint_as_float(acc[4 * q4 + 2]) * s4[q4].z;
                        v[4 * q4 + 3] = __uint_as_float(acc[4 * q4 + 3]) * s4[q4].w;
                    }
                    if (!__all_sync(0xFFFFFFFFu, full)) {            // ragged group edge or mixed-modality tile
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int col = cc + j;
                            const bool valid = (col < r1hi) || (col >= r2lo && col < r2hi);
                            v[j] = valid ? v[j] : -INFINITY;
                        }
                    }
                    float m12[12];
#pragma unroll
                    for (int i = 0; i < 10; ++i) m12[i] = tc::max3(v[3 * i], v[3 * i + 1], v[3 * i + 2]);
                    m12[10] = v[30]; m12[11] = v[31];
                    const float a0 = tc::max3(m12[0], m12[1], m12[2]), a1 = tc::max3(m12[3], m12[4], m12[5]);
                    const float a2 = tc::max3(m12[6], m12[7], m12[8]), a3 = tc::max3(m12[9], m12[10], m12[11]);
                    const float cmax = fmaxf(tc::max3(a0, a1, a2), a3);
                    if (cmax > best) {                               // strict: an earlier chunk keeps a tie
                        best = cmax;
                        best_cc = cc;
#pragma unroll
                        for (int q4 = 0; q4 < 8; ++q4)               // keep the chunk to find the column later
                            wrow[q4 ^ (row & 7)] = make_float4(v[4 * q4], v[4 * q4 + 1], v[4 * q4 + 2], v[4 * q4 + 3]);
                    }
                }
                tc::tc_fence_before();
                __syncwarp();
                if (lane == 0) tc::mbar_arrive(bar(10 + ta));
            }
            if (!ok) break;
            if (in_range) {
                const int j = A.rank[(int64_t)p.uh * A.L + token];
                if (j >= 0) {                                        // a non-pivot: report its match
                    int slot = -1;
                    float sim = 0.f;
                    if (best_cc >= 0) {
                        int idx = 0;
#pragma unroll
                        for (int q4 = 7; q4 >= 0; --q4) {
                            const float4 w = wrow[q4 ^ (row & 7)];
                            if (w.w == best) idx = 4 * q4 + 3;
                            if (w.z == best) idx = 4 * q4 + 2;
                            if (w.y == best) idx = 4 * q4 + 1;
                            if (w.x == best) idx = 4 * q4;
                        }
                        slot = A.cand_slot[(int64_t)p.uh * A.Ctot + best_cc + idx];
                        sim = best * A.rn[(int64_t)p.uh * A.L + token];
                    }
                    A.match[(int64_t)p.uh * A.E + j] = slot;
                    A.match_sim[(int64_t)p.uh * A.E + j] = sim;
                }
            }
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (warp == 1) tc::tmem_dealloc(tmem_base, 512);
}

}  // namespace flowmm
