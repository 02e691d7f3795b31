// Tensor-core path of the matching step (Eq. 9 and Eq. 10) for bf16 keys with head_dim 128.
//
// Per (unit, KV head) the admissible pivots (importance <= tau) are gathered into a dense
// candidate matrix, text candidates first and visual candidates from the next multiple of 32.
// The similarity contraction then runs as  S[128 tokens x 256 candidates] = K_tile . C_tile^T
// (two such 128-token halves per candidate tile) on tcgen05 with the token rows taken straight from the caller's K by TMA (every token of the
// head in prompt order; rows that are pivots are computed and dropped), fp32 accumulators in
// TMEM, and an epilogue that scales each column by the candidate's reciprocal norm and keeps a
// running row maximum.  Raw bf16 keys feed the MMA (their products are exact in fp32); the
// norms enter in fp32 afterwards, so no precision is lost before the argmax.
// An intra-modal layer visits only the candidate group of the row tile's modality.
#pragma once
#include <type_traits>

#include "common.cuh"
#include "tc_stream.cuh"

namespace flowmm {

constexpr int kMtRows = tcs::kRows;          // tokens per accumulator half
constexpr int kMtItemRows = tcs::kItemRows;  // tokens per item (two halves)

struct MatchPrepArgs {
    const void *k;
    const float *importance;
    const uint8_t *modality;
    const int *retained, *evicted;
    __nv_bfloat16 *cand_k;       // [UH, Ctot, 128]
    float *cand_scale;           // [UH, Ctot]
    int *cand_slot;              // [UH, Ctot]
    int *cand_count;             // [UH, 2]  admissible text / visual pivots
    int *rank;                   // [UH, L]  position in the non-pivot list, or -(s + 2) for the pivot of slot s
    uint8_t *tile_mod;           // [U, n_rt] per tile of 256 tokens; bit 0: holds text tokens, bit 1: visual tokens
    int Hkv, L, B, E, Ctot, n_rt;
    int *status;                 // device status word (index checks of the debug build report here)
    int copy_here;               // 1: this kernel also gathers the candidate rows; 0: match_gather_kernel does
    float tau_eff;
    int64_t ks[3];
};

// Copies the candidate key rows (256 bytes each) of positions [lo, hi) of one head's candidate
// list, 16 lanes per row, and takes each row's reciprocal norm on the way (0 for a zero row: its
// similarity to anything is 0).  lo, hi multiples of 16; every thread of the block takes part.
__device__ __forceinline__ void match_gather_rows(const MatchPrepArgs &A, int uh, int lo, int hi, int tid, int nthreads) {
    const int u = uh / A.Hkv, h = uh % A.Hkv;
    const int *ret = A.retained + (int64_t)uh * A.B;
    const int *slot_out = A.cand_slot + (int64_t)uh * A.Ctot;
    float *scale_out = A.cand_scale + (int64_t)uh * A.Ctot;
    const __nv_bfloat16 *kb = static_cast<const __nv_bfloat16 *>(A.k) + u * A.ks[0] + h * A.ks[1];
    uint4 *dst = reinterpret_cast<uint4 *>(A.cand_k + (int64_t)uh * A.Ctot * 128);
    const int sub = tid & 15;
    for (int pos = lo + (tid >> 4); pos < hi; pos += nthreads >> 4) {       // uniform trip count within a warp
        const int s = slot_out[pos];
        uint4 val = make_uint4(0, 0, 0, 0);
        if (s >= 0 && index_ok(s, A.B, A.status) && index_ok(ret[s], A.L, A.status))
            val = *reinterpret_cast<const uint4 *>(kb + (int64_t)ret[s] * A.ks[2] + sub * 8);
        dst[(int64_t)pos * 16 + sub] = val;
        float x[8], ssq = 0.f;
        Elem<__nv_bfloat16>::unpack(val, x);
#pragma unroll
        for (int e = 0; e < 8; ++e) ssq = fmaf(x[e], x[e], ssq);
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) ssq += __shfl_xor_sync(0xFFFFFFFFu, ssq, o);
        if (sub == 0 && s >= 0) scale_out[pos] = ssq > 0.f ? rsqrtf(ssq) : 0.f;
    }
}

// The preparation of one (unit, head) by its whole block (256 to 1024 threads, a multiple of 32); `scratch` = 33 ints
// and `s_ntext` = one int of shared memory.  Also called at the end of the selection kernel, which has just written
// this head's index lists.
__device__ __forceinline__ void match_prepare_head(const MatchPrepArgs &A, int uh, int *scratch, int *s_ntext) {
    const int tid = threadIdx.x, u = uh / A.Hkv, h = uh % A.Hkv;
    const int *ret = A.retained + (int64_t)uh * A.B;
    const int *evi = A.evicted + (int64_t)uh * A.E;
    const float *imp = A.importance + (int64_t)uh * A.L;
    const uint8_t *mod = A.modality + (int64_t)u * A.L;
    int *rank = A.rank + (int64_t)uh * A.L;
    int *slot_out = A.cand_slot + (int64_t)uh * A.Ctot;
    float *scale_out = A.cand_scale + (int64_t)uh * A.Ctot;

    for (int i = tid; i < A.Ctot; i += blockDim.x) { slot_out[i] = -1; scale_out[i] = __int_as_float(0x7FC00000); }   // NaN: no candidate here
    for (int s = tid; s < A.B; s += blockDim.x)
        if (index_ok(ret[s], A.L, A.status)) rank[ret[s]] = -(s + 2);
    for (int j = tid; j < A.E; j += blockDim.x)
        if (index_ok(evi[j], A.L, A.status)) rank[evi[j]] = j;
    if (h == 0) {
        for (int t = tid; t < A.n_rt; t += blockDim.x) {
            int bits = 0;
            const int hi = min(A.L, (t + 1) * kMtItemRows);
            for (int i = t * kMtItemRows; i < hi; ++i) bits |= mod[i] ? 2 : 1;
            A.tile_mod[(int64_t)u * A.n_rt + t] = (uint8_t)bits;
        }
    }
    // admissible text pivots first: count them to know where the visual group starts
    int n_text = 0;
    for (int s = tid; s < A.B; s += blockDim.x) {
        const int r = index_ok(ret[s], A.L, A.status) ? ret[s] : 0;
        n_text += (imp[r] <= A.tau_eff && mod[r] == 0) ? 1 : 0;
    }
    int total;
    block_exclusive_scan(n_text, scratch, total);
    if (tid == 0) *s_ntext = total;
    __syncthreads();
    const int t0 = (*s_ntext + 31) & ~31;
    int seen_t = 0, seen_v = 0;
    for (int base = 0; base < A.B; base += blockDim.x) {
        const int s = base + tid;
        int ft = 0, fv = 0, r = 0;
        if (s < A.B) {
            r = index_ok(ret[s], A.L, A.status) ? ret[s] : 0;
            const bool adm = imp[r] <= A.tau_eff;              // Eq. 10: pivots above tau are kept out of merging
            ft = adm && mod[r] == 0;
            fv = adm && mod[r] != 0;
        }
        int tot_t, tot_v;
        const int pt = seen_t + block_exclusive_scan(ft, scratch, tot_t);
        const int pv = seen_v + block_exclusive_scan(fv, scratch, tot_v);
        if (ft) slot_out[pt] = s;
        if (fv) slot_out[t0 + pv] = s;
        seen_t += tot_t;
        seen_v += tot_v;
    }
    if (tid == 0) { A.cand_count[2 * uh] = seen_t; A.cand_count[2 * uh + 1] = seen_v; }
    __syncthreads();
    if (A.copy_here) match_gather_rows(A, uh, 0, A.Ctot, tid, blockDim.x);
}

// grid = U*Hkv, block = 256 to 1024 (a multiple of 32).
__global__ void __launch_bounds__(1024) match_prepare_kernel(const MatchPrepArgs A) {
    __shared__ int scratch[33];
    __shared__ int s_ntext;
    match_prepare_head(A, blockIdx.x, scratch, &s_ntext);
}

// The gather step of the preparation as a kernel of its own for long candidate lists, so that many
// CTAs share a head's rows.  grid = (U*Hkv, ceil(Ctot / 64)), block = 256.
__global__ void __launch_bounds__(256) match_gather_kernel(const MatchPrepArgs A) {
    const int lo = blockIdx.y * 64;
    match_gather_rows(A, blockIdx.x, lo, min(A.Ctot, lo + 64), threadIdx.x, blockDim.x);
}

struct MatchTcArgs {
    const int *cand_count, *cand_slot, *rank, *strategy;
    const float *cand_scale;
    const uint8_t *modality, *tile_mod;
    int *match;
    float *match_sim;
    int *status;
    int Hkv, L, E, Ctot, n_rt, n_items;
    FastDiv by_nrt, by_hkv;      // exact division of item numbers by n_rt and of head numbers by Hkv
};

struct MatchItem {
    int u, h, uh, rt, lo, hi, n_text, t0, n_vis;
    bool intra, mixed;
    tcs::TilePlan tp;
};

// What an item's plan reads from global memory; kept apart so that a role can fetch the next item's
// values while it works on the current one.
struct MatchRaw { int n_text, n_vis, strategy, tile_mod; };

__device__ __forceinline__ MatchRaw match_raw(const MatchTcArgs &A, int item) {
    MatchRaw r = {0, 0, 1, 0};
    if (item >= A.n_items) return r;
    const int uh = (int)A.by_nrt.div(item), rt = item - uh * A.n_rt, u = (int)A.by_hkv.div(uh);
    r.n_text = A.cand_count[2 * uh]; r.n_vis = A.cand_count[2 * uh + 1];
    r.strategy = A.strategy[u];
    r.tile_mod = A.tile_mod[(int64_t)u * A.n_rt + rt];
    return r;
}

// Which candidate columns a tile of 256 tokens has to visit: everything in a cross-modal layer or
// when the tile mixes modalities, otherwise only the group of the tile's modality.
template <class S>
__device__ __forceinline__ MatchItem match_plan(const MatchTcArgs &A, int item, const MatchRaw &raw) {
    constexpr int kMtCols = S::kCols;        // candidates per column tile
    MatchItem p;
    p.uh = (int)A.by_nrt.div(item); p.rt = item - p.uh * A.n_rt;
    p.u = (int)A.by_hkv.div(p.uh); p.h = p.uh - p.u * A.Hkv;
    p.n_text = raw.n_text; p.n_vis = raw.n_vis;
    p.t0 = (p.n_text + 31) & ~31;
    p.intra = raw.strategy == 0;
    const int tm = raw.tile_mod;
    p.mixed = tm == 3;
    const int end_all = p.n_vis > 0 ? p.t0 + p.n_vis : p.n_text;
    if (!p.intra || tm == 3) { p.lo = 0; p.hi = end_all; }
    else if (tm == 1) { p.lo = 0; p.hi = p.n_text; }
    else { p.lo = p.t0; p.hi = p.t0 + p.n_vis; }
    const int cols = p.hi > p.lo ? p.hi - p.lo : 0;
    p.tp.a1 = p.rt * kMtItemRows; p.tp.a2 = p.h; p.tp.a3 = p.u;
    p.tp.h1 = kMtRows; p.tp.h2 = 0;
    p.tp.n_halves = p.tp.a1 + kMtRows < A.L ? 2 : 1;
    p.tp.b1 = p.lo; p.tp.b2 = p.uh; p.tp.b3 = 0;
    p.tp.step1 = kMtCols; p.tp.step2 = 0;
    p.tp.n_tiles = (cols + kMtCols - 1) / kMtCols;
    p.tp.cols_total = cols;
    p.tp.extra = A.cand_scale + (int64_t)p.uh * A.Ctot + p.lo;
    return p;
}
template <class S>
__device__ __forceinline__ MatchItem match_plan(const MatchTcArgs &A, int item) {
    return match_plan<S>(A, item, match_raw(A, item));
}

// The inner step of the epilogue, written out in PTX so that it stays inside what the tensor core leaves room for:
// a 128 x 256 accumulator is refilled in 1024 clocks, in which the four schedulers issue 4096 warp instructions for its
// 1024 warp-wide elements, and the tensor core's operand reads already take three quarters of the shared-memory
// bandwidth, so the epilogue must not stage anything through shared memory.
// One block of 16 accumulator columns of this thread's row: similarities = accumulators x the candidates' reciprocal
// norms (packed pairs; the norms are the block's only shared-memory reads); each similarity then carries its column in
// its four lowest mantissa bits (15 - column, so that of equal similarities the lower column is the larger number; the
// change is below 2^-19 relative, far inside the margin the decision is judged with); one maximum over the 16 tagged
// values; the block's maximum with the tag cleared is compared with the row's running maximum `best`: a block that
// beats it - strictly, so that an earlier block keeps a tie, and never with NaN (= no candidate there) - replaces it
// and `win` records where it was: 16 x block number + tag.
//   taddr   TMEM address of the block for this warp's lanes        scales   shared address of the block's 16 norms
// (TMEM is read 32 columns at a time: a read has a cost of its own that does not shrink with its width, and sixteen
// warps reading 16 columns each time kept the tensor core waiting for its accumulators.)
#define FLOWMM_MB_MUL2(i, j, k, ti, tj, MASK)                                                                  \
    "mov.b64 t0, {a" #i ", a" #j "};\n\tmul.rn.f32x2 t0, t0, s" #k ";\n\tmov.b64 {a" #i ", a" #j "}, t0;\n\t"    \
    "lop3.b32 a" #i ", a" #i ", " MASK ", " #ti ", 0xEA;\n\t"                                                   \
    "lop3.b32 a" #j ", a" #j ", " MASK ", " #tj ", 0xEA;\n\t"
#define FLOWMM_MB_LDS(OFF)                                     \
    "ld.shared.v2.b64 {s0, s1}, [%3 + " #OFF "];\n\t"          \
    "ld.shared.v2.b64 {s2, s3}, [%3 + " #OFF " + 16];\n\t"     \
    "ld.shared.v2.b64 {s4, s5}, [%3 + " #OFF " + 32];\n\t"     \
    "ld.shared.v2.b64 {s6, s7}, [%3 + " #OFF " + 48];\n\t"
// 16 columns held in registers a<c0> .. a<c15>: products, tags, maximum, comparison with the running maximum;
// WIN = 16 x block number and MASK = 0xFFFFFFF0 held in a register, as asm operand references (the tag-insertion takes
// one immediate only: with the mask as a literal too, each tag would first be moved into a register)
#define FLOWMM_MB_STEP(c0, c1, c2, c3, c4, c5, c6, c7, c8, c9, c10, c11, c12, c13, c14, c15, WIN, MASK)         \
    FLOWMM_MB_MUL2(c0, c1, 0, 15, 14, MASK) FLOWMM_MB_MUL2(c2, c3, 1, 13, 12, MASK) FLOWMM_MB_MUL2(c4, c5, 2, 11, 10, MASK) \
    FLOWMM_MB_MUL2(c6, c7, 3, 9, 8, MASK) FLOWMM_MB_MUL2(c8, c9, 4, 7, 6, MASK) FLOWMM_MB_MUL2(c10, c11, 5, 5, 4, MASK)     \
    FLOWMM_MB_MUL2(c12, c13, 6, 3, 2, MASK) FLOWMM_MB_MUL2(c14, c15, 7, 1, 0, MASK)                             \
    "max.f32 m0, a" #c0 ", a" #c1 ", a" #c2 ";\n\t"                                                             \
    "max.f32 m1, a" #c3 ", a" #c4 ", a" #c5 ";\n\t"                                                             \
    "max.f32 m2, a" #c6 ", a" #c7 ", a" #c8 ";\n\t"                                                             \
    "max.f32 m3, a" #c9 ", a" #c10 ", a" #c11 ";\n\t"                                                           \
    "max.f32 m4, a" #c12 ", a" #c13 ", a" #c14 ";\n\t"                                                          \
    "max.f32 m0, m0, m1, m2;\n\t"                                                                               \
    "max.f32 m3, m3, m4, a" #c15 ";\n\t"                                                                        \
    "max.f32 q0, m0, m3;\n\t"                                                                                   \
    "and.b32 qm, q0, " MASK ";\n\t"                                                                             \
    "setp.gt.f32 p0, qm, %0;\n\t"                                                                               \
    "@p0 mov.b32 %0, qm;\n\t"                                                                                   \
    "@p0 lop3.b32 %1, q0, 15, " WIN ", 0xEA;\n\t"
#define FLOWMM_MB_HEAD                 \
    "{\n\t"                            \
    ".reg .b32 a<32>, qm;\n\t"         \
    ".reg .b64 s<8>, t0;\n\t"          \
    ".reg .f32 m<5>, q0;\n\t"          \
    ".reg .pred p0;\n\t"

// Block number kBlk (16 columns) of the warp's share of the tile.
template <int kBlk>
__device__ __forceinline__ void match_block16(uint32_t taddr, uint32_t scales, float &best, int &win) {
    asm volatile(FLOWMM_MB_HEAD
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {a0, a1, a2, a3, a4, a5, a6, a7, a8, a9, a10, a11, a12, a13, a14, a15}, [%2];\n\t"
        FLOWMM_MB_LDS(0)
        "tcgen05.wait::ld.sync.aligned;\n\t"
        FLOWMM_MB_STEP(0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15, "%4", "%5")
        "}"
        : "+f"(best), "+r"(win)
        : "r"(taddr), "r"(scales), "n"(16 * kBlk), "r"(0xFFFFFFF0u)
        : "memory");
}

// Blocks kBlk and kBlk + 1 (32 columns) with one TMEM read.
template <int kBlk>
__device__ __forceinline__ void match_block32(uint32_t taddr, uint32_t scales, float &best, int &win) {
    asm volatile(FLOWMM_MB_HEAD
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {a0, a1, a2, a3, a4, a5, a6, a7, a8, a9, a10, a11, a12, a13, a14, a15, "
        "a16, a17, a18, a19, a20, a21, a22, a23, a24, a25, a26, a27, a28, a29, a30, a31}, [%2];\n\t"
        FLOWMM_MB_LDS(0)
        "tcgen05.wait::ld.sync.aligned;\n\t"
        FLOWMM_MB_STEP(0, 1, 2, 3, 4, 5, 6, 7, 8, 9, 10, 11, 12, 13, 14, 15, "%4", "%6")
        FLOWMM_MB_LDS(64)
        FLOWMM_MB_STEP(16, 17, 18, 19, 20, 21, 22, 23, 24, 25, 26, 27, 28, 29, 30, 31, "%5", "%6")
        "}"
        : "+f"(best), "+r"(win)
        : "r"(taddr), "r"(scales), "n"(16 * kBlk), "n"(16 * kBlk + 16), "r"(0xFFFFFFF0u)
        : "memory");
}
#undef FLOWMM_MB_MUL2
#undef FLOWMM_MB_LDS
#undef FLOWMM_MB_STEP
#undef FLOWMM_MB_HEAD

// Blocks kI .. kN - 1 of the warp's share.  (One TMEM read per block of 16 columns measured a little faster than
// one per 32 columns: the narrower read leaves the compiler more registers around it.)
template <int kN, int kI = 0>
__device__ __forceinline__ void match_blocks(uint32_t taddr, uint32_t scales, float &best, int &win) {
    if constexpr (kI < kN) {
        match_block16<kI>(taddr + 16 * kI, scales + 64 * kI, best, win);
        match_blocks<kN, kI + 1>(taddr, scales, best, win);
    }
}

// Of two (similarity, slot) results the larger similarity wins and equal similarities go to the lower slot
// (slot < 0: no result).
__device__ __forceinline__ bool match_better(float va, int sa, float vb, int sb) {
    return sa >= 0 && (sb < 0 || va > vb || (va == vb && sa < sb));
}

// Squared norm of 64 bf16 elements of a key row in an operand stage (one 128-byte swizzled row: 16-byte units
// XOR-ed with the row index), as packed pairs.
__device__ __forceinline__ float row_half_ssq(uint32_t row_addr, int row) {
    float2 acc = make_float2(0.f, 0.f);
#pragma unroll
    for (int un = 0; un < 8; ++un) {
        const float4 rawf = tc::lds128(row_addr + ((un ^ (row & 7)) << 4));
        const uint32_t w[4] = {__float_as_uint(rawf.x), __float_as_uint(rawf.y), __float_as_uint(rawf.z), __float_as_uint(rawf.w)};
#pragma unroll
        for (int i = 0; i < 4; ++i) {            // a bf16 is the upper half of the fp32 with the same value
            const float2 x = make_float2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xFFFF0000u));
            acc = tc::ffma2(x, x, acc);
        }
    }
    return acc.x + acc.y;
}

// Persistent kernel, one CTA per SM; item = (unit, head, tile of 256 tokens).
template <class S>
__global__ void __launch_bounds__(tcs::kThreads, 1)
match_tc_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap cand_map,
                const MatchTcArgs A) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    constexpr int kMtCols = S::kCols;
    constexpr int kPer = kMtCols / 32;                           // blocks of 16 columns a warp takes of a full tile
    const typename S::Ctx c = S::setup(smem_raw, &k_map, &cand_map, A.status, 8);
    if (!c.ok) return;
    auto plan = [&](int item) { return match_plan<S>(A, item).tp; };
    if (c.warp == 0) {
        if (c.lane == 0) S::producer(c, &k_map, &cand_map, A.n_items, tcs::kAHalf, S::kBStage, plan, A.status);
    } else if (c.warp == 1) {
        if (c.lane == 0) S::mma_issuer(c, A.n_items, plan, A.status);
    } else {
        const int lane = c.lane, row = c.quarter * 32 + lane;
        const int b0 = kPer * c.colhalf;                         // first block of this warp's share of a tile
        const uint32_t wrow = c.epi_addr() + row * 16;          // hand-over slot of this row
        const uint32_t prow = c.partner_addr() + row * 16;      // the other column half's
        const uint32_t t_lane = c.tmem_base + c.group * kMtCols + b0 * 16 + ((uint32_t)(c.quarter * 32) << 16);
        int k = 0, bt = 0, n_mine = 0;
        bool ok = true;
        // what an item needs from global memory is fetched one item ahead: its plan values, the token's
        // modality and its place in the non-pivot list
        auto token_of = [&](int item) { return (item - (int)A.by_nrt.div(item) * A.n_rt) * kMtItemRows + c.group * kMtRows + row; };
        auto fetch_mod = [&](int item) -> int {
            const int token = token_of(item);
            return item < A.n_items && token < A.L ? A.modality[(int64_t)A.by_hkv.div(A.by_nrt.div(item)) * A.L + token] : 0;
        };
        auto fetch_rank = [&](int item) -> int {
            const int token = token_of(item);
            return item < A.n_items && token < A.L ? A.rank[(int64_t)A.by_nrt.div(item) * A.L + token] : -1;
        };
        MatchRaw raw_next = match_raw(A, blockIdx.x);
        int mod_next = fetch_mod(blockIdx.x), rank_next = fetch_rank(blockIdx.x);
        for (int item = blockIdx.x; ok && item < A.n_items; item += gridDim.x) {
            const MatchRaw raw = raw_next;
            const int my_mod = mod_next, my_rank = rank_next;
            raw_next = match_raw(A, item + gridDim.x);
            mod_next = fetch_mod(item + gridDim.x);
            rank_next = fetch_rank(item + gridDim.x);
            const MatchItem p = match_plan<S>(A, item, raw);
            const bool active = !p.tp.empty() && c.group < p.tp.n_halves;
            const int token = p.rt * kMtItemRows + c.group * kMtRows + row;
            const bool in_range = token < A.L;
            const bool row_masked = p.intra && p.mixed;
            const int *slots = A.cand_slot + (int64_t)p.uh * A.Ctot;
            // Running winner of this row among the warp's columns: its similarity (still times the row's norm, four
            // lowest mantissa bits cleared), the tile it came from, and in `win` the block of 16 columns inside the warp's
            // share of that tile (x 16) with 15 - column inside the block.  Candidates are laid out text group first, each group by ascending
            // slot, so within a group the first maximum is the lowest slot; where a row sees both groups (a cross-modal
            // layer) the text group's winner is set aside when the first visual column comes up, and the two meet by
            // (similarity, slot).
            float best = -INFINITY, before = -INFINITY;
            int win = -1, best_tile = 0;
            float val_a = -INFINITY;                                 // the winner set aside
            int slot_a = -1;
            bool parked = p.intra;                                   // (an intra-modal row sees one group only)
            float ssq = 0.f;                                         // squared norm of this row's key, this warp's half of it
            auto resolve = [&]() -> int {                            // slot of the running winner
                if (win < 0) return -1;
                const int col = p.lo + best_tile * kMtCols + (b0 + (win >> 4)) * 16 + 15 - (win & 15);
                return index_ok(col, A.Ctot, A.status) ? slots[col] : -1;
            };
            auto park = [&](int t) {
                if (best > before) best_tile = t;                   // the winner may be of this tile's earlier blocks
                slot_a = resolve();
                val_a = best;
                best = -INFINITY; before = -INFINITY; win = -1;
                parked = true;
            };
            if (!active) {
                if (!p.tp.empty()) bt += p.tp.n_tiles;               // keep the B-tile count in step
            } else {
                {   // the token's key row sits in this half's A stage: each of the row's two warps reads one 64-element
                    // half of it for the norm while the first MMAs run, then hands the stage back
                    ok = S::a_wait(c, n_mine, A.status);
                    ssq = row_half_ssq(c.a_addr(n_mine) + c.colhalf * (tcs::kAHalf / 2) + row * 128, row);
                    S::a_release(c, n_mine++);
                }
                for (int t = 0; ok && t < p.tp.n_tiles; ++t, ++k, ++bt) {
                    const int col0 = p.lo + t * kMtCols;
                    const int ncols = min(kMtCols, p.hi - col0);
                    ok = S::extra_wait(c, bt, A.status) && S::acc_wait(c, k, A.status);
                    if (!ok) break;
                    const uint32_t scale4 = c.extra(bt);             // reciprocal norms of this tile's candidates
                    const int n_blocks = (ncols + 15) >> 4;
                    if (row_masked) {
                        // intra-modal layer, tile with tokens of both modalities: rows differ in which columns they may take
                        S::for_each_block16(c, n_blocks, [&](int bl, uint32_t (&acc)[16]) {
                            const int cc = col0 + bl * 16;
                            float v[16];
#pragma unroll
                            for (int q4 = 0; q4 < 4; ++q4) {     // a column that is no candidate has scale NaN and never wins
                                const float4 s4 = tc::lds128(scale4 + (bl * 4 + q4) * 16);
                                v[4 * q4 + 0] = __uint_as_float(acc[4 * q4 + 0]) * s4.x;
                                v[4 * q4 + 1] = __uint_as_float(acc[4 * q4 + 1]) * s4.y;
                                v[4 * q4 + 2] = __uint_as_float(acc[4 * q4 + 2]) * s4.z;
                                v[4 * q4 + 3] = __uint_as_float(acc[4 * q4 + 3]) * s4.w;
                            }
                            int r1hi = p.n_text, r2lo = p.t0, r2hi = p.t0 + p.n_vis;   // admissible columns of this row
                            if (my_mod == 0) r2hi = r2lo; else r1hi = 0;
                            float q = -INFINITY;
                            int qj = 0;
#pragma unroll
                            for (int j = 0; j < 16; ++j) {           // columns in ascending order; NaN never wins
                                const int col = cc + j;
                                const bool valid = (col < r1hi) || (col >= r2lo && col < r2hi);
                                const float x = __uint_as_float(__float_as_uint(v[j]) & 0xFFFFFFF0u);   // as the unmasked path rounds it
                                if (valid && x > q) { q = x; qj = j; }
                            }
                            if (q > best) {                          // strict: an earlier block keeps a tie
                                best = q;
                                win = (bl - b0) * 16 + 15 - qj;
                                best_tile = t;
                            }
                        });
                    } else {
                        const int nb = min(n_blocks - b0, kPer);     // blocks of this warp in this tile (may be <= 0)
                        // block before which the text group's winner is set aside (>= nb: not in this tile)
                        // (splitting a ragged last tile evenly between the row's two warps was measured and is no faster:
                        // the tile's arithmetic, not the longer of its two shares, is what takes the time)
                        const int pk = parked ? kPer : max(0, (p.t0 - (col0 + b0 * 16)) >> 4);
                        const uint32_t sc = scale4 + b0 * 64, tl = t_lane;
                        before = best;
                        if (nb == kPer && pk >= kPer) {
                            match_blocks<kPer>(tl, sc, best, win);
                        } else {
                            // (the group boundary is a multiple of 32 columns, the warp's share starts at one: pairs of blocks)
#pragma unroll
                            for (int i = 0; i < kPer; i += 2) {
                                if (i < nb) {
                                    if (i == pk) park(t);
                                    const bool two = i + 1 < nb;
                                    switch (i) {                     // (the block's number is a compile-time constant)
                                        case 0: if (two) match_block32<0>(tl, sc, best, win); else match_block16<0>(tl, sc, best, win); break;
                                        case 2: if (two) match_block32<2>(tl + 32, sc + 128, best, win); else match_block16<2>(tl + 32, sc + 128, best, win); break;
                                        case 4: if (two) match_block32<4>(tl + 64, sc + 256, best, win); else match_block16<4>(tl + 64, sc + 256, best, win); break;
                                        default: if (two) match_block32<6>(tl + 96, sc + 384, best, win); else match_block16<6>(tl + 96, sc + 384, best, win); break;
                                    }
                                }
                            }
                        }
                        if (best > before) best_tile = t;            // the winner moved into this tile
                    }
                    S::acc_release(c);
                }
            }
            // (after a wait that ran out the results are garbage, but the two meeting points below are still
            // kept so that the partner warp is never left waiting; the first one tells both warps, and the loop
            // ends for both right after them)
            // this warp's result for the row: similarity (still times the row's norm) and pivot slot
            int slot = -1;
            if (ok && active) {
                slot = resolve();
                if (match_better(val_a, slot_a, best, slot)) { best = val_a; slot = slot_a; }
            }
            // the upper column half hands its result and its half of the norm to the lower one, which owns the row's output
            if (c.colhalf == 1) tc::sts128(wrow, best, __int_as_float(slot), ssq, 0.f);
            ok = !S::pair_meet(c, !ok);                            // (both warps of a row go on, or neither)
            if (c.colhalf == 0 && ok) {
                const float4 other = tc::lds128(prow);
                if (match_better(other.x, __float_as_int(other.y), best, slot)) { best = other.x; slot = __float_as_int(other.y); }
                ssq += other.z;
                if (in_range) {
                    const int j = my_rank;
                    if (j >= 0 && index_ok(j, A.E, A.status)) {      // a non-pivot: report its match
                        float sim = 0.f;
                        if (slot >= 0 && ssq > 0.f) sim = best * rsqrtf(ssq);
                        A.match[(int64_t)p.uh * A.E + j] = slot;
                        A.match_sim[(int64_t)p.uh * A.E + j] = sim;
                    }
                }
            }
            S::pair_sync(c);                                       // the hand-over slot may be overwritten again
        }
    }
    S::teardown(c);
}

}  // namespace flowmm
