// Window scoring (Eq. 8 with the softmax of Eq. 4, and the masses of Eq. 7) in one pass over K, for
// short contexts with few proxy rows per KV head (bf16, head_dim 128).
//
// The two-pass kernels of score_tc.cuh read K twice because a column sum needs every row's final
// normaliser first.  When all logits of a head fit in half of TMEM - ceil(L / 128) tiles x (G W) columns
// <= 256 - a CTA computes S_t = K_t Q^T once per 128-key tile (tcgen05.mma, keys as M, proxy rows as N),
// keeps every tile of the head in TMEM, and a team of eight warps sweeps them three times:
//   A  per proxy row the maximum over all keys (running while the K tiles still stream),
//   B  per proxy row the sum of exponentials, in total and over the keys of the other modality (Eq. 7),
//   C  per key the sum over proxy rows of exp / row sum: the importance (group mean over the G heads).
// Lanes are keys, so the per-row reductions of A and B cross lanes (shuffles, then shared memory across
// the warps) once per head; everything else is per thread.  K is read from HBM exactly once.
// CTAs are persistent (one per SM) and take (unit, KV head) items in turn.  Warp 0 lane 0 streams Q and the
// K tiles through a five-stage TMA ring and runs ahead of the arithmetic, warp 1 lane 0 issues the MMAs of
// item i into TMEM half i mod 2, and two teams of eight warps (two warps per 32 TMEM lanes, each with
// half of the proxy rows; their partial importances meet in shared memory) take the items alternately, so
// one head is swept while the next one streams in.
#pragma once
#include "common.cuh"
#include "decode_tc.cuh"
#include "tc_common.cuh"

namespace flowmm {
namespace sft {

constexpr int kTile = 128;
constexpr int kStages = 5;
constexpr int kRows = 32;                       // proxy rows per KV head (G W) this kernel is built for
constexpr int kMaxTiles = 8;                    // 8 x 32 columns = one half of TMEM
constexpr int kTeam = 256;                      // threads of a sweep team
constexpr int kThreads = 64 + 2 * kTeam;
constexpr uint32_t kStageBytes = kTile * 128 * 2, kPanel = kStageBytes / 2;
constexpr uint32_t kQBytes = kRows * 256;                          // Q operand of one head: two panels of 32 rows
constexpr uint32_t kSmemQ = kStages * kStageBytes;                 // two Q operands
constexpr uint32_t kSmemRed = kSmemQ + 2 * kQBytes;                // per team: float [3][4][kRows], int [kRows] mask limits
constexpr uint32_t kRedBytes = 13 * kRows * 4;
constexpr uint32_t kSmemImp = kSmemRed + 2 * kRedBytes;            // per team: float [kMaxTiles][128] partial importances
constexpr uint32_t kImpBytes = kMaxTiles * kTile * 4;
constexpr uint32_t kSmemBar = kSmemImp + 2 * kImpBytes;
constexpr int kBarFull = 0, kBarEmpty = kStages, kBarQFull = 2 * kStages, kBarQEmpty = kBarQFull + 2,
              kBarSetFree = kBarQEmpty + 2 /* 256 arrivals */, kBarS = kBarSetFree + 2 /* [2][kMaxTiles] */,
              kNumBars = kBarS + 2 * kMaxTiles;
constexpr uint32_t kSmemBytes = kSmemBar + 8 * kNumBars + 16;

struct Args {
    const uint8_t *modality;    // [U, L]
    float *importance;          // [UH, L]
    float *cross_mass;          // [U, Hq]
    int *status;
    int Hq, Hkv, G, W, L, n_items;
    float scale_log2;
};

// Reduction of 16 values per lane across the 32 lanes of a warp with 16 shuffles instead of 80: every step a lane
// hands half of its values to the partner that keeps them.  On return v[0] holds the total of value
// number (lane >> 1) & 15 (in both lanes of the pair).
template <class Op>
__device__ __forceinline__ void warp_reduce16(float (&v)[16], Op op) {
#pragma unroll
    for (int n = 8, m = 16; n >= 1; n >>= 1, m >>= 1) {
        const bool upper = (threadIdx.x & m) != 0;
#pragma unroll
        for (int i = 0; i < n; ++i) {
            const float send = upper ? v[i] : v[i + n], keep = upper ? v[i + n] : v[i];
            v[i] = op(keep, __shfl_xor_sync(0xFFFFFFFFu, send, m));
        }
    }
    v[0] = op(v[0], __shfl_xor_sync(0xFFFFFFFFu, v[0], 1));
}

__device__ __forceinline__ void team_sync(int team) { asm volatile("bar.sync %0, 256;" ::"r"(1 + team) : "memory"); }

__global__ void __launch_bounds__(kThreads, 1)
score_fused_tc_kernel(const __grid_constant__ CUtensorMap qmap, const __grid_constant__ CUtensorMap kmap, const Args A) {
    constexpr int GW = kRows, HC = GW / 2;
    extern __shared__ __align__(1024) uint8_t sft_smem[];
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
        for (int i = 0; i < kNumBars; ++i) tc::mbar_init(bar(i), (i == kBarSetFree || i == kBarSetFree + 1) ? kTeam : 1);
        *abort_flag = 0;
        tc::mbar_init_fence();
        tc::tma_prefetch_desc(&qmap);
        tc::tma_prefetch_desc(&kmap);
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), 512);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;
    const int nt = (A.L + kTile - 1) / kTile;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int i = 0, it = 0;
            for (int item = blockIdx.x; ok && item < A.n_items; item += gridDim.x, ++it) {
                const int u = item / A.Hkv, h = item % A.Hkv, set = it & 1;
                ok = tc::mbar_wait(bar(kBarQEmpty + set), ((it >> 1) & 1) ^ 1, abort_flag, A.status);
                if (!ok) break;
                const uint32_t qd = base + kSmemQ + set * kQBytes;
                tc::mbar_expect_tx(bar(kBarQFull + set), kQBytes);
                tc::tma_load_4d(qd, &qmap, bar(kBarQFull + set), 0, 0, h * A.G, u);
                tc::tma_load_4d(qd + kQBytes / 2, &qmap, bar(kBarQFull + set), 64, 0, h * A.G, u);
                for (int t = 0; ok && t < nt; ++t, ++i) {
                    const int st = i % kStages;
                    ok = tc::mbar_wait(bar(kBarEmpty + st), ((i / kStages) & 1) ^ 1, abort_flag, A.status);
                    if (!ok) break;
                    const uint32_t dst = base + st * kStageBytes;
                    tc::mbar_expect_tx(bar(kBarFull + st), kStageBytes);
                    tc::tma_load_4d(dst, &kmap, bar(kBarFull + st), 0, t * kTile, h, u);
                    tc::tma_load_4d(dst + kPanel, &kmap, bar(kBarFull + st), 64, t * kTile, h, u);
                }
            }
            if (!ok) {       // winding down after a timeout: give copies already issued a moment to land
                for (int b = 0; b < kStages; ++b)
                    for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(bar(kBarFull + b), 0) && !tc::mbar_try_wait(bar(kBarFull + b), 1); ++s) {}
                for (int b = 0; b < 2; ++b)
                    for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(bar(kBarQFull + b), 0) && !tc::mbar_try_wait(bar(kBarQFull + b), 1); ++s) {}
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = tc::idesc_bf16(kTile, GW);
            bool ok = true;
            int i = 0, it = 0;
            for (int item = blockIdx.x; ok && item < A.n_items; item += gridDim.x, ++it) {
                const int set = it & 1, use = it >> 1;
                ok = tc::mbar_wait(bar(kBarQFull + set), use & 1, abort_flag, A.status) &&
                     tc::mbar_wait(bar(kBarSetFree + set), (use & 1) ^ 1, abort_flag, A.status);   // the half's previous head is swept
                tc::tc_fence_after();
                const uint32_t qd = base + kSmemQ + set * kQBytes;
                for (int t = 0; ok && t < nt; ++t, ++i) {
                    const int st = i % kStages;
                    ok = tc::mbar_wait(bar(kBarFull + st), (i / kStages) & 1, abort_flag, A.status);
                    if (!ok) break;
                    tc::tc_fence_after();
                    const uint32_t a = base + st * kStageBytes;
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        tc::umma_bf16(tmem + 256 * set + GW * t, tc::smem_desc_sw128(a + (j >> 2) * kPanel, (j & 3) * 32),
                                      tc::smem_desc_sw128(qd + (j >> 2) * (kQBytes / 2), (j & 3) * 32), idesc, j > 0);
                    tc::umma_commit(bar(kBarEmpty + st));
                    tc::umma_commit(bar(kBarS + set * kMaxTiles + t));
                }
                if (ok) tc::umma_commit(bar(kBarQEmpty + set));
            }
        }
    } else {
        // two sweep teams of eight warps: two warps per 32 TMEM lanes, each with half of the proxy rows (HC columns)
        const int team = (warp - 2) >> 3, tw = (warp - 2) & 7;
        const int e = (threadIdx.x - 64) & (kTeam - 1);
        const int wq = warp & 3, half = tw >> 2, cb = half * HC;     // cb: first proxy row of this thread
        const int row = 32 * wq + lane;                              // TMEM lane: key of a tile
        const uint32_t trow = tmem + ((uint32_t)(32 * wq) << 16) + 256 * team + cb;
        float *red = reinterpret_cast<float *>(sft_smem + kSmemRed + team * kRedBytes);    // [3][4][kRows]
        float *impx = reinterpret_cast<float *>(sft_smem + kSmemImp + team * kImpBytes);   // [nt][128]
        int *lim = reinterpret_cast<int *>(red + 12 * kRows);
        const int first_proxy = A.L - A.W;
        // a (key, proxy row c) pair counts if key <= lim[c] = first_proxy + c % W (which also keeps key < L)
        if (e < GW) lim[e] = first_proxy + e % A.W;
        const int n_plain = min(nt, (first_proxy + 1) / kTile);      // leading tiles in which no pair is masked
        auto load = [&](int t, uint32_t (&r)[HC]) {
            tc::tmem_ld16(trow + GW * t, r);
            tc::tmem_ld_wait(r);
        };
        bool ok = true;
        int it = team;
        for (int item = blockIdx.x + team * gridDim.x; item < A.n_items; item += 2 * gridDim.x, it += 2) {
            const int uh = item, u = item / A.Hkv, h = item % A.Hkv, use = it >> 1;
            const uint8_t *mod = A.modality + (int64_t)u * A.L;
            // which of this thread's proxy rows belong to visual tokens: bit q for row cb + q = g W + a, token first_proxy + a
            const unsigned qvis = __ballot_sync(0xFFFFFFFFu, lane < HC && mod[first_proxy + (cb + lane) % A.W] != 0);
            unsigned vis_bits = 0;                                   // bit t: this thread's key of tile t is a visual token
#pragma unroll
            for (int t = 0; t < kMaxTiles; ++t)
                if (t < nt && t * kTile + row < A.L && mod[t * kTile + row] != 0) vis_bits |= 1u << t;
            team_sync(team);                                         // lim is written; the previous item's scratch is free

            float mx[HC];
#pragma unroll
            for (int q = 0; q < HC; ++q) mx[q] = kNegBig;
            for (int t = 0; t < nt; ++t) {                           // sweep A, under the K stream
                ok = ok && tc::mbar_wait(bar(kBarS + team * kMaxTiles + t), use & 1, abort_flag, A.status);
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
            warp_reduce16(mx, [](float a, float b) { return fmaxf(a, b); });
            if (!(lane & 1)) red[wq * kRows + cb + (lane >> 1)] = mx[0];
            team_sync(team);
#pragma unroll
            for (int q = 0; q < HC; ++q) {   // from here on: the row's maximum in the log2 domain
                const int c = cb + q;
                mx[q] = A.scale_log2 * fmaxf(fmaxf(red[c], red[kRows + c]), fmaxf(red[2 * kRows + c], red[3 * kRows + c]));
            }

            float lt[HC], lc[HC];                                    // sweep B: row sums, total and other-modality keys
#pragma unroll
            for (int q = 0; q < HC; ++q) { lt[q] = 0.f; lc[q] = 0.f; }
            for (int t = 0; t < nt; ++t) {
                const int key = t * kTile + row;
                const unsigned oth = ((vis_bits >> t) & 1u) ? ~qvis : qvis;   // proxy rows of the other modality than this key's
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
            warp_reduce16(lt, [](float a, float b) { return a + b; });
            warp_reduce16(lc, [](float a, float b) { return a + b; });
            if (!(lane & 1)) {
                red[(4 + wq) * kRows + cb + (lane >> 1)] = lt[0];
                red[(8 + wq) * kRows + cb + (lane >> 1)] = lc[0];
            }
            team_sync(team);
#pragma unroll
            for (int q = 0; q < HC; ++q) {   // from here on: 1 / row sum
                const int c = cb + q;
                lt[q] = 1.f / (red[4 * kRows + c] + red[5 * kRows + c] + red[6 * kRows + c] + red[7 * kRows + c]);
            }
            if (e < A.G && ok) {                                     // Eq. 7 for query head e of the group: sum over its rows
                float s = 0.f;
                for (int a = 0; a < A.W; ++a) {
                    const int c = e * A.W + a;
                    const float tot = red[4 * kRows + c] + red[5 * kRows + c] + red[6 * kRows + c] + red[7 * kRows + c];
                    const float cr = red[8 * kRows + c] + red[9 * kRows + c] + red[10 * kRows + c] + red[11 * kRows + c];
                    s += cr / tot;
                }
                A.cross_mass[(int64_t)u * A.Hq + h * A.G + e] = s;
            }
            float imp[kMaxTiles];                                    // sweep C: this thread's share of every key's importance
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
            tc::tc_fence_before();
            tc::mbar_arrive(bar(kBarSetFree + team));               // this thread has read the half for the last time
            team_sync(team);
            if (half == 0 && ok) {
                const float inv_g = 1.f / (float)A.G;
#pragma unroll
                for (int t = 0; t < kMaxTiles; ++t) {
                    const int key = t * kTile + row;
                    if (t < nt && key < A.L) A.importance[(int64_t)uh * A.L + key] = (imp[t] + impx[t * kTile + row]) * inv_g;
                }
            }
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (warp == 1) tc::tmem_dealloc(tmem, 512);
}

}  // namespace sft
}  // namespace flowmm
