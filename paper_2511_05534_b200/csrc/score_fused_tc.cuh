// Window scoring (Eq. 8 with the softmax of Eq. 4, and the masses of Eq. 7) in one pass over K, for
// short contexts with few proxy rows per KV head (bf16, head_dim 128).
//
// The two-pass kernels of score_tc.cuh read K twice because a column sum needs every row's final
// normaliser first.  When all logits of a head fit in TMEM - ceil(L / 128) tiles x (G W) columns <= 512 -
// one CTA per (unit, KV head) computes S_t = K_t Q^T once per 128-key tile (tcgen05.mma, keys as M,
// proxy rows as N), keeps every tile in TMEM, and then sweeps TMEM three times:
//   A  per proxy row the maximum over all keys (running while the K tiles still stream),
//   B  per proxy row the sum of exponentials, in total and over the keys of the other modality (Eq. 7),
//   C  per key the sum over proxy rows of exp / row sum: the importance (group mean over the G heads).
// Lanes are keys, so the per-row reductions of A and B cross lanes (shuffles, then shared memory across
// the warps) once per head; everything else is per thread.  K is read from HBM exactly once.
// Roles: warp 0 lane 0 TMA, warp 1 lane 0 MMA, warps 2-9 the sweeps (two warps per 32 TMEM lanes, each
// with half of the proxy rows; their partial importances meet in shared memory).
#pragma once
#include "common.cuh"
#include "decode_tc.cuh"
#include "tc_common.cuh"

namespace flowmm {
namespace sft {

constexpr int kTile = 128;
constexpr int kStages = 3;
constexpr int kMaxRows = 64;                    // proxy rows per KV head (G W): 32 or 64
constexpr int kMaxTiles = 16;
constexpr int kThreads = 320;                   // TMA warp, MMA warp, eight sweep warps
constexpr uint32_t kStageBytes = kTile * 128 * 2, kPanel = kStageBytes / 2;
constexpr uint32_t kSmemQ = kStages * kStageBytes;                 // Q operand: two panels of GW rows
constexpr int kBarFull = 0, kBarEmpty = kStages, kBarQ = 2 * kStages, kBarS = kBarQ + 1, kNumBars = kBarS + kMaxTiles;
// after the stages: the Q operand (two panels of GW rows), float [3][4 warps][kMaxRows] + int [kMaxRows] mask limits, barriers
template <int GW> struct Smem {
    static constexpr uint32_t kRed = kSmemQ + 2 * GW * 128;
    static constexpr uint32_t kBar = kRed + 13 * kMaxRows * 4;
    static constexpr uint32_t bytes(int n_tiles) { return kBar + 8 * kNumBars + 16 + (uint32_t)n_tiles * kTile * 4; }   // + partial importances
};

struct Args {
    const uint8_t *modality;    // [U, L]
    float *importance;          // [UH, L]
    float *cross_mass;          // [U, Hq]
    int *status;
    int Hq, Hkv, G, W, L, GW, tmem_cols;
    float scale_log2;
};

__device__ __forceinline__ void sweep_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

template <int GW>
__global__ void __launch_bounds__(kThreads, GW <= 32 ? 2 : 1)
score_fused_tc_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap, const Args A) {
    extern __shared__ __align__(1024) uint8_t sft_smem[];
    constexpr uint32_t kSmemRed = Smem<GW>::kRed, kSmemBar = Smem<GW>::kBar;
    const uint32_t base = tc::smem_u32(sft_smem), bars = base + kSmemBar;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(sft_smem + kSmemBar + 8 * kNumBars + 4);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(sft_smem + kSmemBar + 8 * kNumBars);
    if ((base & 1023u) != 0) {
        if (threadIdx.x == 0) atomicCAS(A.status, 0, 6);
        return;
    }
    auto bar = [&](int i) { return bars + 8u * i; };
    if (threadIdx.x == 0) {
        for (int i = 0; i < kNumBars; ++i) tc::mbar_init(bar(i), 1);
        *abort_flag = 0;
        tc::mbar_init_fence();
        tc::tma_prefetch_desc(&qmap);
        tc::tma_prefetch_desc(&kmap);
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), (uint32_t)A.tmem_cols);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int uh = blockIdx.x, u = uh / A.Hkv, h = uh % A.Hkv;
    const int nt = (A.L + kTile - 1) / kTile;

    if (warp == 0) {
        if (lane == 0) {
            tc::mbar_expect_tx(bar(kBarQ), GW * 256);
            tc::tma_load_4d(base + kSmemQ, &qmap, bar(kBarQ), 0, 0, h * A.G, u);
            tc::tma_load_4d(base + kSmemQ + GW * 128, &qmap, bar(kBarQ), 64, 0, h * A.G, u);
            bool ok = true;
            for (int t = 0; ok && t < nt; ++t) {
                const int st = t % kStages;
                ok = tc::mbar_wait(bar(kBarEmpty + st), ((t / kStages) & 1) ^ 1, abort_flag, A.status);
                if (!ok) break;
                const uint32_t dst = base + st * kStageBytes;
                tc::mbar_expect_tx(bar(kBarFull + st), kStageBytes);
                tc::tma_load_4d(dst, &kmap, bar(kBarFull + st), 0, t * kTile, h, u);
                tc::tma_load_4d(dst + kPanel, &kmap, bar(kBarFull + st), 64, t * kTile, h, u);
            }
            if (!ok) {       // winding down after a timeout: give copies already issued a moment to land
                for (int i = 0; i < kStages; ++i)
                    for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(bar(kBarFull + i), 0) && !tc::mbar_try_wait(bar(kBarFull + i), 1); ++s) {}
                for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(bar(kBarQ), 0); ++s) {}
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = tc::idesc_bf16(kTile, GW);
            bool ok = tc::mbar_wait(bar(kBarQ), 0, abort_flag, A.status);
            for (int t = 0; ok && t < nt; ++t) {
                const int st = t % kStages;
                ok = tc::mbar_wait(bar(kBarFull + st), (t / kStages) & 1, abort_flag, A.status);
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t a = base + st * kStageBytes;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    tc::umma_bf16(tmem + GW * t, tc::smem_desc_sw128(a + (j >> 2) * kPanel, (j & 3) * 32),
                                  tc::smem_desc_sw128(base + kSmemQ + (j >> 2) * (GW * 128), (j & 3) * 32), idesc, j > 0);
                tc::umma_commit(bar(kBarEmpty + st));
                tc::umma_commit(bar(kBarS + t));
            }
        }
    } else {
        // eight sweep warps: two per 32 TMEM lanes, each with half of the proxy rows (HC columns)
        constexpr int HC = GW / 2;
        const int e = threadIdx.x - 64;
        const int wq = warp & 3, half = (warp - 2) >> 2, cb = half * HC;   // cb: first proxy row of this thread
        const int row = 32 * wq + lane;                              // TMEM lane: key of a tile
        const uint32_t trow = tmem + ((uint32_t)(32 * wq) << 16) + cb;
        float *red = reinterpret_cast<float *>(sft_smem + kSmemRed);    // [3][4][kMaxRows]
        float *impx = reinterpret_cast<float *>(sft_smem + kSmemBar + 8 * kNumBars + 16);   // [nt][128] partial importances
        const uint8_t *mod = A.modality + (int64_t)u * A.L;
        const int first_proxy = A.L - A.W;
        // which of this thread's proxy rows belong to visual tokens: bit q for row cb + q = g W + a, token first_proxy + a
        const unsigned qvis = __ballot_sync(0xFFFFFFFFu, lane < HC && mod[first_proxy + (cb + lane) % A.W] != 0);
        // a (key, proxy row c) pair counts if key <= lim[c] = first_proxy + c % W (which also keeps key < L)
        int *lim = reinterpret_cast<int *>(red + 12 * kMaxRows);
        if (e < GW) lim[e] = first_proxy + e % A.W;
        sweep_sync();
        const int n_plain = min(nt, (first_proxy + 1) / kTile);      // leading tiles in which no pair is masked
        auto load = [&](int t, uint32_t (&r)[HC]) {
            if constexpr (HC == 16) { tc::tmem_ld16(trow + GW * t, r); } else { tc::tmem_ld32(trow + GW * t, r); }
            tc::tmem_ld_wait(r);
        };

        bool ok = true;
        float mx[HC];
#pragma unroll
        for (int q = 0; q < HC; ++q) mx[q] = kNegBig;
        for (int t = 0; t < nt; ++t) {                               // sweep A, under the K stream
            ok = ok && tc::mbar_wait(bar(kBarS + t), 0, abort_flag, A.status);
            tc::tc_fence_after();
            const int key = t * kTile + row;
            uint32_t r[HC];
            load(t, r);
            if (t < n_plain) {
#pragma unroll
                for (int q = 0; q < HC; ++q) mx[q] = fmaxf(mx[q], __uint_as_float(r[q]));
            } else {
#pragma unroll
                for (int q = 0; q < HC; ++q)
                    if (key <= lim[cb + q]) mx[q] = fmaxf(mx[q], __uint_as_float(r[q]));
            }
        }
#pragma unroll
        for (int q = 0; q < HC; ++q) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx[q] = fmaxf(mx[q], __shfl_xor_sync(0xFFFFFFFFu, mx[q], o));
            if (lane == 0) red[wq * kMaxRows + cb + q] = mx[q];
        }
        sweep_sync();
#pragma unroll
        for (int q = 0; q < HC; ++q) {   // from here on: the row's maximum in the log2 domain
            const int c = cb + q;
            mx[q] = A.scale_log2 * fmaxf(fmaxf(red[c], red[kMaxRows + c]), fmaxf(red[2 * kMaxRows + c], red[3 * kMaxRows + c]));
        }

        float lt[HC], lc[HC];                                        // sweep B: row sums, total and other-modality keys
#pragma unroll
        for (int q = 0; q < HC; ++q) { lt[q] = 0.f; lc[q] = 0.f; }
        for (int t = 0; t < nt; ++t) {
            const int key = t * kTile + row;
            const bool my_vis = key < A.L && mod[key] != 0;
            const unsigned oth = my_vis ? ~qvis : qvis;              // proxy rows of the other modality than this key's
            uint32_t r[HC];
            load(t, r);
#pragma unroll
            for (int q = 0; q < HC; ++q) {
                float p = tc::ex2(fmaf(__uint_as_float(r[q]), A.scale_log2, -mx[q]));
                if (t >= n_plain && key > lim[cb + q]) p = 0.f;
                lt[q] += p;
                lc[q] += ((oth >> q) & 1u) ? p : 0.f;
            }
        }
#pragma unroll
        for (int q = 0; q < HC; ++q) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                lt[q] += __shfl_xor_sync(0xFFFFFFFFu, lt[q], o);
                lc[q] += __shfl_xor_sync(0xFFFFFFFFu, lc[q], o);
            }
            if (lane == 0) {
                red[(4 + wq) * kMaxRows + cb + q] = lt[q];
                red[(8 + wq) * kMaxRows + cb + q] = lc[q];
            }
        }
        sweep_sync();
#pragma unroll
        for (int q = 0; q < HC; ++q) {   // from here on: 1 / row sum
            const int c = cb + q;
            lt[q] = 1.f / (red[4 * kMaxRows + c] + red[5 * kMaxRows + c] + red[6 * kMaxRows + c] + red[7 * kMaxRows + c]);
        }
        if (e < A.G && ok) {                                         // Eq. 7 for query head e of the group: sum over its rows
            float s = 0.f;
            for (int a = 0; a < A.W; ++a) {
                const int c = e * A.W + a;
                const float tot = red[4 * kMaxRows + c] + red[5 * kMaxRows + c] + red[6 * kMaxRows + c] + red[7 * kMaxRows + c];
                const float cr = red[8 * kMaxRows + c] + red[9 * kMaxRows + c] + red[10 * kMaxRows + c] + red[11 * kMaxRows + c];
                s += cr / tot;
            }
            A.cross_mass[(int64_t)u * A.Hq + h * A.G + e] = s;
        }
        float imp[kMaxTiles];                                        // sweep C: this thread's share of every key's importance
#pragma unroll
        for (int t = 0; t < kMaxTiles; ++t) {
            imp[t] = 0.f;
            if (t < nt) {
                const int key = t * kTile + row;
                uint32_t r[HC];
                load(t, r);
                if (t < n_plain) {
#pragma unroll
                    for (int q = 0; q < HC; ++q)
                        imp[t] = fmaf(tc::ex2(fmaf(__uint_as_float(r[q]), A.scale_log2, -mx[q])), lt[q], imp[t]);
                } else {
#pragma unroll
                    for (int q = 0; q < HC; ++q) {
                        const float p = tc::ex2(fmaf(__uint_as_float(r[q]), A.scale_log2, -mx[q])) * lt[q];
                        imp[t] += key <= lim[cb + q] ? p : 0.f;
                    }
                }
                if (half == 1) impx[t * kTile + row] = imp[t];
            }
        }
        sweep_sync();
        if (half == 0 && ok) {
            const float inv_g = 1.f / (float)A.G;
#pragma unroll
            for (int t = 0; t < kMaxTiles; ++t) {
                const int key = t * kTile + row;
                if (t < nt && key < A.L) A.importance[(int64_t)uh * A.L + key] = (imp[t] + impx[t * kTile + row]) * inv_g;
            }
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (warp == 1) tc::tmem_dealloc(tmem, (uint32_t)A.tmem_cols);
}

}  // namespace sft
}  // namespace flowmm
