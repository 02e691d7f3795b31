// Decode-step attention over a KV cache (Eq. 4) on the tensor cores, for bf16 caches with head_dim 128.
//
// One CTA takes a range of up to 15 tiles of 128 keys of one (unit, KV head) and all query heads of
// the group (up to 8, zero-padded to the 16 rows of the narrow operand).  Both contractions run with the keys on the wide side, so the
// tiny query side costs nothing and every K and V row is read from HBM exactly once:
//   phase 1   S_t[key, head] = K_t Q^T        tcgen05.mma M = 128 keys, N = 16, contraction over head_dim;
//             every tile's logits stay in TMEM (16 columns per tile)
//   reduce    the exact per-head maximum over the CTA's range, from TMEM
//   phase 2   P_t = 2^(c S_t - max) into shared memory as two bf16 rows per head (the rounded weight and
//             the rounding remainder), then O[dim, row] += V_t^T P_t^T: M = 128 dims, N = 16 = 8 heads x 2,
//             contraction over the tile's keys; a head's output is the sum of its two columns.  The V tile is the same swizzled
//             shared-memory tile a K tile is, read the other way round (MN-major operand), so V needs no
//             transposition.  O never needs rescaling because the maximum is already final.
// A head with one range is normalised and written at once.  Otherwise the CTA writes its unnormalised
// output, its maximum and its sum of weights, and whichever range of a head finishes last (a ticket per
// head) joins them all; the records it reads are L2-resident.
// Roles: warp 0 lane 0 streams K tiles then V tiles through a three-stage TMA ring, warp 1 lane 0 issues
// the MMAs, warps 2-5 (one thread per key of a tile / per output dim) do the softmax and the output.
// Two CTAs fit an SM (256 TMEM columns, about 109 KB of shared memory each), so one streams while the
// other is between its phases.  Every wait is bounded.
#pragma once
#include "common.cuh"
#include "tc_common.cuh"

namespace flowmm {
namespace dtc {

constexpr int kTile = 128;                  // keys per tile
constexpr int kStages = 3;
constexpr int kHeads = 16;                  // N of both contractions
constexpr int kMaxHeads = 8;                // query heads per KV head this kernel serves
constexpr int kMaxTiles = 15;               // 16 TMEM columns for O + 16 per score tile = 256
constexpr int kTmemCols = 256;
constexpr int kMaxJoin = 8192;               // (range, head) records the joining CTA can stage: ranges per head x heads
constexpr int kThreads = 192;
constexpr uint32_t kStageBytes = kTile * 128 * 2;            // both 64-element panels of a 128-row tile
constexpr uint32_t kPanel = kStageBytes / 2;
constexpr uint32_t kSmallPanel = kHeads * 128;               // 16 rows x 128 bytes
constexpr uint32_t kSmemQ = kStages * kStageBytes;           // Q operand: two panels of 16 rows
constexpr uint32_t kSmemP = kSmemQ + 2 * kSmallPanel;        // two P buffers of the same shape
constexpr uint32_t kSmemRed = kSmemP + 4 * kSmallPanel;      // float [4 warps][8 heads], then the last-range flag
constexpr uint32_t kSmemBar = kSmemRed + 256;
constexpr int kBarFull = 0, kBarEmpty = kStages, kBarQ = 2 * kStages, kBarS = kBarQ + 1 /* one per score tile */,
              kBarPFull = kBarS + kMaxTiles, kBarPEmpty = kBarPFull + 2, kBarO = kBarPEmpty + 2, kNumBars = kBarO + 1;
constexpr uint32_t kSmemBytes = kSmemBar + 8 * kNumBars + 16;

struct Args {
    const __nv_bfloat16 *q;     // [U, Hq, 128] dense
    float *part;                // [UH, n_split, G, 130]: unnormalised output, maximum (log2 domain), sum of weights
    float *out;                 // [U, Hq, 128]
    int *tickets;               // [UH], zero on entry and on exit: how many ranges of the head have finished
    int *status;
    int Hq, Hkv, G, N, n_split, tiles_per_split;
    float scale_log2;
};

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void epi_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ void sts128u(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void sts16(uint32_t addr, unsigned short v) {
    asm volatile("st.shared.b16 [%0], %1;" ::"r"(addr), "h"(v) : "memory");
}
// The swizzled 128-row tile read as an MN-major operand: a 128-byte row holds 64 consecutive M
// elements of one K index, eight K indices make a 1024-byte group, the second 64 M elements live
// `kPanel` bytes further on.  `byte_offset` selects the 16 K indices (rows) of one instruction.
__device__ __forceinline__ uint64_t smem_desc_sw128_mn(uint32_t tile_base, uint32_t byte_offset) {
    uint64_t d = 0;
    d |= (uint64_t)(((tile_base + byte_offset) & 0x3FFFFu) >> 4);
    d |= (uint64_t)(kPanel >> 4) << 16;                                  // between 64-element M panels
    d |= (uint64_t)(1024u >> 4) << 32;                                   // between groups of eight K indices
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
constexpr uint32_t kIdescQK = tc::idesc_bf16(kTile, kHeads);
constexpr uint32_t kIdescPV = tc::idesc_bf16(128, kHeads) | (1u << 15);   // A operand MN-major

__global__ void __launch_bounds__(kThreads, 2)
decode_tc_kernel(const __grid_constant__ CUtensorMap kmap, const __grid_constant__ CUtensorMap vmap, const Args A) {
    extern __shared__ __align__(1024) uint8_t dtc_smem[];
    const uint32_t base = tc::smem_u32(dtc_smem), bars = base + kSmemBar;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(dtc_smem + kSmemBar + 8 * kNumBars + 4);
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(dtc_smem + kSmemBar + 8 * kNumBars);
    if ((base & 1023u) != 0) {                      // the swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0) atomicCAS(A.status, 0, 6);
        return;
    }
    auto bar = [&](int i) { return bars + 8u * i; };
    if (threadIdx.x == 0) {
        for (int i = 0; i < kNumBars; ++i)
            tc::mbar_init(bar(i), (i == kBarQ || i == kBarPFull || i == kBarPFull + 1) ? 128 : 1);
        *abort_flag = 0;
        tc::mbar_init_fence();
        tc::tma_prefetch_desc(&kmap);
        tc::tma_prefetch_desc(&vmap);
    }
    if (warp == 1) tc::tmem_alloc(tc::smem_u32(tmem_slot), kTmemCols);
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int uh = blockIdx.x, u = uh / A.Hkv, h = uh % A.Hkv, split = blockIdx.y;
    const int tiles_total = (A.N + kTile - 1) / kTile;
    const int t0 = split * A.tiles_per_split, nt = min(A.tiles_per_split, tiles_total - t0);
    const int key0 = t0 * kTile;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            for (int i = 0; ok && i < 2 * nt; ++i) {                 // the K tiles, then the V tiles
                const int st = i % kStages;
                ok = tc::mbar_wait(bar(kBarEmpty + st), ((i / kStages) & 1) ^ 1, abort_flag, A.status);
                if (!ok) break;
                const CUtensorMap *m = i < nt ? &kmap : &vmap;
                const int row = key0 + (i < nt ? i : i - nt) * kTile;
                const uint32_t dst = base + st * kStageBytes;
                tc::mbar_expect_tx(bar(kBarFull + st), kStageBytes);
                tc::tma_load_4d(dst, m, bar(kBarFull + st), 0, row, h, u);
                tc::tma_load_4d(dst + kPanel, m, bar(kBarFull + st), 64, row, h, u);
            }
            if (!ok)         // winding down after a timeout: give copies already issued a moment to land
                for (int i = 0; i < kStages; ++i)
                    for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(bar(kBarFull + i), 0) && !tc::mbar_try_wait(bar(kBarFull + i), 1); ++s) {}
        }
    } else if (warp == 1) {
        if (lane == 0) {
            bool ok = tc::mbar_wait(bar(kBarQ), 0, abort_flag, A.status);
            for (int t = 0; ok && t < nt; ++t) {
                const int st = t % kStages;
                ok = tc::mbar_wait(bar(kBarFull + st), (t / kStages) & 1, abort_flag, A.status);
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t a = base + st * kStageBytes;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    tc::umma_bf16(tmem + kHeads + kHeads * t, tc::smem_desc_sw128(a + (j >> 2) * kPanel, (j & 3) * 32),
                                  tc::smem_desc_sw128(base + kSmemQ + (j >> 2) * kSmallPanel, (j & 3) * 32), kIdescQK, j > 0);
                tc::umma_commit(bar(kBarEmpty + st));
                tc::umma_commit(bar(kBarS + t));
            }
            for (int t = 0; ok && t < nt; ++t) {
                const int i = nt + t, st = i % kStages, pb = t & 1;
                ok = tc::mbar_wait(bar(kBarFull + st), (i / kStages) & 1, abort_flag, A.status) &&
                     tc::mbar_wait(bar(kBarPFull + pb), (t >> 1) & 1, abort_flag, A.status);
                if (!ok) break;
                tc::tc_fence_after();
                const uint32_t a = base + st * kStageBytes, p = base + kSmemP + pb * 2 * kSmallPanel;
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    tc::umma_bf16(tmem, smem_desc_sw128_mn(a, j * 2048),
                                  tc::smem_desc_sw128(p + (j >> 2) * kSmallPanel, (j & 3) * 32), kIdescPV, (t | j) != 0);
                tc::umma_commit(bar(kBarEmpty + st));
                tc::umma_commit(bar(kBarPEmpty + pb));
            }
            if (ok) tc::umma_commit(bar(kBarO));
        }
    } else {
        const int e = threadIdx.x - 64;                              // 0 .. 127
        const int row = 32 * (warp & 3) + lane;                      // TMEM lane this thread reads: key of a tile / output dim
        const uint32_t trow = tmem + ((uint32_t)(32 * (warp & 3)) << 16);
        const int G = A.G;
        // the Q operand (rows = heads, zero beyond G) and zeroed P buffers
        for (int c = e; c < 256; c += 128) {
            const int g = c >> 4, cc = c & 15;
            uint4 val = make_uint4(0, 0, 0, 0);
            if (g < G) val = *reinterpret_cast<const uint4 *>(A.q + ((int64_t)u * A.Hq + h * G + g) * 128 + cc * 8);
            sts128u(base + kSmemQ + (cc >> 3) * kSmallPanel + g * 128 + (((cc & 7) ^ (g & 7)) << 4), val);
        }
        for (int c = e; c < 512; c += 128) sts128u(base + kSmemP + c * 16, make_uint4(0, 0, 0, 0));
        fence_proxy_async();
        tc::mbar_arrive(bar(kBarQ));

        bool ok = true;
        float mx[kMaxHeads];
#pragma unroll
        for (int g = 0; g < kMaxHeads; ++g) mx[g] = kNegBig;
        for (int t = 0; t < nt; ++t) {                               // running maxima while the K tiles stream
            ok = ok && tc::mbar_wait(bar(kBarS + t), 0, abort_flag, A.status);
            tc::tc_fence_after();
            uint32_t r[16];
            tc::tmem_ld16(trow + kHeads + kHeads * t, r);
            tc::tmem_ld_wait(r);
            if (key0 + t * kTile + row < A.N) {
#pragma unroll
                for (int g = 0; g < kMaxHeads; ++g) mx[g] = fmaxf(mx[g], __uint_as_float(r[g]));
            }
        }
        float *red = reinterpret_cast<float *>(dtc_smem + kSmemRed);
#pragma unroll
        for (int g = 0; g < kMaxHeads; ++g) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mx[g] = fmaxf(mx[g], __shfl_xor_sync(0xFFFFFFFFu, mx[g], o));
            if (lane == 0) red[(warp & 3) * kMaxHeads + g] = mx[g];
        }
        epi_sync();
        float mref[kMaxHeads], l[kMaxHeads];
#pragma unroll
        for (int g = 0; g < kMaxHeads; ++g) {
            mref[g] = A.scale_log2 * fmaxf(fmaxf(red[g], red[kMaxHeads + g]), fmaxf(red[2 * kMaxHeads + g], red[3 * kMaxHeads + g]));
            l[g] = 0.f;
        }
        epi_sync();                                                  // red is reused for the sums below
        for (int t = 0; t < nt; ++t) {
            const int pb = t & 1;
            ok = ok && tc::mbar_wait(bar(kBarPEmpty + pb), ((t >> 1) & 1) ^ 1, abort_flag, A.status);
            uint32_t r[16];
            tc::tmem_ld16(trow + kHeads + kHeads * t, r);
            tc::tmem_ld_wait(r);
            const bool valid = key0 + t * kTile + row < A.N;
            const uint32_t prow = base + kSmemP + pb * 2 * kSmallPanel + (row >> 6) * kSmallPanel + ((row & 7) << 1);
            const int chunk = (row & 63) >> 3;
#pragma unroll
            for (int g = 0; g < kMaxHeads; ++g) {
                if (g < G) {
                    const float p = valid ? tc::ex2(fmaf(__uint_as_float(r[g]), A.scale_log2, -mref[g])) : 0.f;
                    // bf16 head and bf16 remainder in rows g and 8 + g: their two products add up in fp32, so the
                    // weight enters the second contraction with about 16 bits of mantissa
                    const __nv_bfloat16 hi = __float2bfloat16_rn(p), lo = __float2bfloat16_rn(p - __bfloat162float(hi));
                    l[g] += p;
                    const uint32_t at = prow + g * 128 + ((chunk ^ g) << 4);
                    sts16(at, __bfloat16_as_ushort(hi));
                    sts16(at + 1024, __bfloat16_as_ushort(lo));
                }
            }
            fence_proxy_async();
            tc::mbar_arrive(bar(kBarPFull + pb));
        }
#pragma unroll
        for (int g = 0; g < kMaxHeads; ++g) {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) l[g] += __shfl_xor_sync(0xFFFFFFFFu, l[g], o);
            if (lane == 0) red[(warp & 3) * kMaxHeads + g] = l[g];
        }
        epi_sync();
        ok = ok && tc::mbar_wait(bar(kBarO), 0, abort_flag, A.status);
        tc::tc_fence_after();
        uint32_t r[16];
        tc::tmem_ld16(trow, r);
        tc::tmem_ld_wait(r);
        float *out = A.out + ((int64_t)u * A.Hq + h * G) * 128 + row;
        if (A.n_split == 1) {                                        // the only range of its head: normalise and finish
#pragma unroll
            for (int g = 0; g < kMaxHeads; ++g)
                if (g < G && ok)
                    out[g * 128] = (__uint_as_float(r[g]) + __uint_as_float(r[kMaxHeads + g])) /
                                   (red[g] + red[kMaxHeads + g] + red[2 * kMaxHeads + g] + red[3 * kMaxHeads + g]);
        } else {
            float *dst = A.part + ((int64_t)uh * A.n_split + split) * G * 130;
#pragma unroll
            for (int g = 0; g < kMaxHeads; ++g) {
                if (g < G) dst[g * 130 + row] = __uint_as_float(r[g]) + __uint_as_float(r[kMaxHeads + g]);
                if (e == g && g < G) {
                    dst[g * 130 + 128] = mref[g];
                    dst[g * 130 + 129] = red[g] + red[kMaxHeads + g] + red[2 * kMaxHeads + g] + red[3 * kMaxHeads + g];
                }
            }
            // the range that finishes last joins all ranges of its head
            __threadfence();
            epi_sync();
            int *last = reinterpret_cast<int *>(red + 4 * kMaxHeads);
            if (e == 0) {
                const int done = atomicAdd(A.tickets + uh, 1);
                *last = done == A.n_split - 1;
                if (*last) A.tickets[uh] = 0;                        // ready for the next call
            }
            epi_sync();
            if (*last && *abort_flag == 0) {        // both the same for all 128 threads: the barrier below is safe
                __threadfence();
                // maxima and sums of every (range, head) go through shared memory (the tile stages are idle by
                // now), so that the long loop below is over independent loads only
                const float *rec0 = A.part + (int64_t)uh * A.n_split * G * 130;
                float *sm_m = reinterpret_cast<float *>(dtc_smem), *sm_l = sm_m + kMaxJoin;
                const int n_rec = A.n_split * G;
                for (int i = e; i < n_rec; i += 128) {
                    sm_m[i] = __ldcg(rec0 + (int64_t)i * 130 + 128);
                    sm_l[i] = __ldcg(rec0 + (int64_t)i * 130 + 129);
                }
                epi_sync();
                float m[kMaxHeads], o[kMaxHeads], ls[kMaxHeads];
#pragma unroll
                for (int g = 0; g < kMaxHeads; ++g) {
                    m[g] = kNegBig; o[g] = 0.f; ls[g] = 0.f;
                    if (g < G)
                        for (int sp = 0; sp < A.n_split; ++sp) m[g] = fmaxf(m[g], sm_m[sp * G + g]);
                }
#pragma unroll 2
                for (int sp = 0; sp < A.n_split; ++sp) {             // all heads of two ranges in flight at a time
#pragma unroll
                    for (int g = 0; g < kMaxHeads; ++g)
                        if (g < G) {
                            const float w = tc::ex2(sm_m[sp * G + g] - m[g]);
                            o[g] = fmaf(__ldcg(rec0 + ((int64_t)sp * G + g) * 130 + row), w, o[g]);
                            ls[g] = fmaf(sm_l[sp * G + g], w, ls[g]);
                        }
                }
#pragma unroll
                for (int g = 0; g < kMaxHeads; ++g)
                    if (g < G) out[g * 128] = o[g] / ls[g];
            }
        }
    }
    tc::tc_fence_before();
    __syncthreads();
    tc::tc_fence_after();
    if (warp == 1) tc::tmem_dealloc(tmem, kTmemCols);
}

}  // namespace dtc
}  // namespace flowmm
