// Tensor-core path of the scoring step (Eq. 8 with the softmax of Eq. 4, and the masses of
// Eq. 7) for bf16 inputs, head_dim 128 and a window of 32, 64 or 128 tokens.
//
// The proxy attention needs every row's softmax normaliser before any column can be summed, so
// the keys are streamed twice:
//   pass 1  S = Q_group . K^T with the G*W proxy rows of a KV head as accumulator lanes (two
//           halves of 128 rows per item) and 256 keys per tile: each thread keeps the running
//           maximum and exp-sum of its own row (no cross-thread traffic);
//   pass 2  S^T = K . Q_group^T with keys as the lanes (two halves of 128 keys per item) and the
//           proxy rows as columns: each thread owns one key, recomputes its logits, normalises
//           them with the per-column constants of pass 1 and sums along its row, which is
//           exactly the key's importance; the same probabilities, split by the modality of key
//           and proxy token, give the cross-modal mass.
// Both passes run on tcgen05 with TMA-fed operands; logits never leave TMEM / registers.
#pragma once
#include "common.cuh"
#include "tc_stream.cuh"

namespace flowmm {

struct ScoreTcArgs {
    float2 *row_part;            // [UH*GW, 4*n_chunk] (max, sum) per proxy row, key chunk and column quarter, log2 domain
    float *negc;                 // [UH, GWpad] -(row max + log2 row sum); very negative for padding rows
    const uint8_t *modality;     // [U, L]
    float *importance;           // [UH, L]
    float *cross_part;           // [U*Hq, n_rt * 8] partial cross-modal mass per key tile and epilogue warp
    int *status;
    int Hq, Hkv, G, W, L, GW, GWpad;
    int n_qt;                    // 256-row tiles over the G*W proxy rows
    int n_chunk, tiles_per_chunk;   // pass 1: key chunks per row tile, 256-key tiles per chunk
    int n_rt;                    // pass 2: 256-key tiles
    int a_heads, b_heads;        // query heads one A box (pass 1) / B box (pass 2) delivers
    int n_items1, n_items2;
    float scale_log2;
    // flow-only variant of pass 1 (full-prefill flow): the row sums also split off the keys of the other modality
    float *row_cross;            // [UH*GW, 4*n_chunk] that part of the sum, same scaling as row_part
    const uint32_t *modbits;     // [U, mod_words] key modality, 32 keys per word (bit j of word w: key 32 w + j is visual)
    int mod_words, mod_pitch;    // words per unit in modbits; row pitch of `modality` (the uncut prompt's length)
};

// max of 32 values with three-input maxima
__device__ __forceinline__ float max32(const float (&v)[32]) {
    float m12[12];
#pragma unroll
    for (int i = 0; i < 10; ++i) m12[i] = tc::max3(v[3 * i], v[3 * i + 1], v[3 * i + 2]);
    m12[10] = v[30]; m12[11] = v[31];
    const float a0 = tc::max3(m12[0], m12[1], m12[2]), a1 = tc::max3(m12[3], m12[4], m12[5]);
    const float a2 = tc::max3(m12[6], m12[7], m12[8]), a3 = tc::max3(m12[9], m12[10], m12[11]);
    return fmaxf(tc::max3(a0, a1, a2), a3);
}

// ---------------------------------------------------------------------------------------------
// Pass 1.  item = (unit*head, tile of 256 proxy rows, key chunk).
// kFlow: also keep, per row, the part of the exp-sum that falls on keys of the other modality than the row's token
// (a chunk of 32 keys is usually of one modality: then it costs one comparison; only mixed chunks go element by element).
template <class S, bool kFlow = false>
__global__ void __launch_bounds__(tcs::kThreads, 1)
score_stats_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                      const ScoreTcArgs A) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const typename S::Ctx c = S::setup(smem_raw, &q_map, &k_map, A.status, 0, 16);
    if (!c.ok) return;
    auto plan = [&](int item) {
        tcs::TilePlan p;
        const int kc = item % A.n_chunk, qt = (item / A.n_chunk) % A.n_qt, uh = item / (A.n_chunk * A.n_qt);
        const int u = uh / A.Hkv, h = uh % A.Hkv;
        const int key0 = kc * A.tiles_per_chunk * S::kCols;
        const int keys = min(A.L - key0, A.tiles_per_chunk * S::kCols);
        p.a1 = 0; p.a2 = h * A.G + qt * (tcs::kItemRows / A.W); p.a3 = u;
        p.h1 = 0; p.h2 = tcs::kRows / A.W;
        p.n_halves = qt * tcs::kItemRows + tcs::kRows < A.GW ? 2 : 1;
        p.b1 = key0; p.b2 = h; p.b3 = u; p.step1 = S::kCols; p.step2 = 0;
        p.cols_total = keys > 0 ? keys : 0;
        p.n_tiles = (p.cols_total + S::kCols - 1) / S::kCols;
        p.extra = nullptr;
        return p;
    };
    const uint32_t a_bytes = (uint32_t)A.a_heads * A.W * 256u;
    if (c.warp == 0) {
        if (c.lane == 0) S::producer(c, &q_map, &k_map, A.n_items1, a_bytes, S::kBStage, plan, A.status);
    } else if (c.warp == 1) {
        if (c.lane == 0) S::mma_issuer(c, A.n_items1, plan, A.status);
    } else {
        // all sixteen warps drain one accumulator at a time: a warp owns 32 lanes x a quarter of the columns of
        // BOTH halves, so the tensor core refills one half while the other is being read
        const int row_in_half = c.quarter * 32 + c.lane, colq = (c.warp - 2) >> 2;
        int kh[2] = {0, 0};
        bool ok = true;
        for (int item = blockIdx.x; ok && item < A.n_items1; item += gridDim.x) {
            const tcs::TilePlan p = plan(item);
            if (p.empty()) continue;
            const int kc = item % A.n_chunk, qt = (item / A.n_chunk) % A.n_qt, uh = item / (A.n_chunk * A.n_qt);
            float m[2] = {kNegBig, kNegBig}, l[2] = {0.f, 0.f};
            float lc[2] = {0.f, 0.f};
            bool my_vis[2] = {false, false};
            const uint32_t *bits = nullptr;
            if constexpr (kFlow) {
                const int u = uh / A.Hkv;
                bits = A.modbits + (int64_t)u * A.mod_words;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int pa = A.L - A.W + ((qt * tcs::kItemRows + h * tcs::kRows + row_in_half) % A.W);
                    my_vis[h] = A.modality[(int64_t)u * A.mod_pitch + pa] != 0;
                }
            }
            for (int t = 0; ok && t < p.n_tiles; ++t) {
                const int kb = p.b1 + t * S::kCols;
                const int ncols = min(S::kCols, p.cols_total - t * S::kCols);
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (h >= p.n_halves || !ok) continue;
                    ok = S::acc_wait_h(c, h, kh[h]++, A.status);
                    if (!ok) continue;
                    const int r0 = qt * tcs::kItemRows + h * tcs::kRows;
                    const int pa = A.L - A.W + ((r0 + row_in_half) % A.W);   // last key this proxy row may see
                    if (r0 + c.quarter * 32 < A.GW) {
                        S::for_each_chunk_q(c, h, colq, (ncols + 31) >> 5, [&](int ch, uint32_t (&acc)[32]) {
                            const int k0 = kb + ch * 32;
                            float mx;
                            float add0 = 0.f, add1 = 0.f, add2 = 0.f, add3 = 0.f;
                            float addc = 0.f;                            // kFlow: the other-modality part of this chunk's sum
                            uint32_t other = 0;
                            if constexpr (kFlow) other = my_vis[h] ? ~bits[k0 >> 5] : bits[k0 >> 5];
                            if (k0 + 32 <= A.L - A.W + 1) {              // no key of this chunk is masked for any row
                                float raw[32];
#pragma unroll
                                for (int j = 0; j < 32; ++j) raw[j] = __uint_as_float(acc[j]);
                                mx = fmaxf(max32(raw) * A.scale_log2, m[h]);
                                const float2 neg2 = make_float2(-mx, -mx), sc2 = make_float2(A.scale_log2, A.scale_log2);
                                float2 a01 = make_float2(0.f, 0.f), a23 = make_float2(0.f, 0.f);
#pragma unroll
                                for (int j = 0; j < 32; j += 8) {        // every fourth exponential on the FMA pipe, two at a time
                                    const float2 x01 = tc::ffma2(make_float2(raw[j], raw[j + 1]), sc2, neg2);
                                    const float2 x23 = tc::ffma2(make_float2(raw[j + 2], raw[j + 3]), sc2, neg2);
                                    const float2 x45 = tc::ffma2(make_float2(raw[j + 4], raw[j + 5]), sc2, neg2);
                                    const float2 x67 = tc::ffma2(make_float2(raw[j + 6], raw[j + 7]), sc2, neg2);
                                    const float2 pf = tc::ex2_fma2(make_float2(x23.y, x67.y));
                                    a01 = tc::fadd2(a01, make_float2(tc::ex2(x01.x), tc::ex2(x01.y)));
                                    a23 = tc::fadd2(a23, make_float2(tc::ex2(x23.x), pf.x));
                                    a01 = tc::fadd2(a01, make_float2(tc::ex2(x45.x), tc::ex2(x45.y)));
                                    a23 = tc::fadd2(a23, make_float2(tc::ex2(x67.x), pf.y));
                                }
                                add0 = a01.x; add1 = a01.y; add2 = a23.x; add3 = a23.y;
                                if constexpr (kFlow) {
                                    if (other == 0xFFFFFFFFu) addc = (add0 + add1) + (add2 + add3);
                                    else if (other != 0u) {
#pragma unroll
                                        for (int j = 0; j < 32; ++j)
                                            addc += ((other >> j) & 1u) ? tc::ex2(fmaf(raw[j], A.scale_log2, -mx)) : 0.f;
                                    }
                                }
                            } else {
                                float s[32];
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    s[j] = (k0 + j <= pa) ? __uint_as_float(acc[j]) * A.scale_log2 : kNegBig;
                                mx = fmaxf(max32(s), m[h]);
#pragma unroll
                                for (int j = 0; j < 32; j += 4) {        // masked entries sit ~1e30 below: exp2 gives 0
                                    add0 += tc::ex2(s[j] - mx);
                                    add1 += tc::ex2(s[j + 1] - mx);
                                    add2 += tc::ex2(s[j + 2] - mx);
                                    add3 += tc::ex2(s[j + 3] - mx);
                                }
                                if constexpr (kFlow) {
#pragma unroll
                                    for (int j = 0; j < 32; ++j) addc += ((other >> j) & 1u) ? tc::ex2(s[j] - mx) : 0.f;
                                }
                            }
                            float add = (add0 + add1) + (add2 + add3);
                            if (mx < 0.5f * kNegBig) { add = 0.f; addc = 0.f; }   // nothing visible yet: exp2(0) terms are not real
                            const float carry = tc::ex2(m[h] - mx);
                            l[h] = l[h] * carry + add;
                            if constexpr (kFlow) lc[h] = lc[h] * carry + addc;
                            m[h] = mx;
                        });
                    }
                    S::acc_release_h(c, h);
                }
            }
            if (!ok) break;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int r = qt * tcs::kItemRows + h * tcs::kRows + row_in_half;
                if (h < p.n_halves && r < A.GW) {
                    A.row_part[((int64_t)uh * A.GW + r) * (4 * A.n_chunk) + 4 * kc + colq] = make_float2(m[h], l[h]);
                    if constexpr (kFlow) A.row_cross[((int64_t)uh * A.GW + r) * (4 * A.n_chunk) + 4 * kc + colq] = lc[h];
                }
            }
        }
    }
    S::teardown(c);
}

// Flow-only variant: joins the partial statistics of every proxy row and adds up, per query head, the share of each
// row's attention that lands on the other modality (Eq. 7 over the rows of this call).  One warp per query head.
__global__ void flow_combine_kernel(const float2 *row_part, const float *row_cross, int n_part, int G, int W, int Hkv, int n_heads,
                                    float *cross_mass) {
    const int head = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (head >= n_heads) return;                                         // head = (u * Hkv + h) * G + g
    const int uh = head / G, g = head % G;
    float s = 0.f;
    for (int a = lane; a < W; a += 32) {
        const int64_t row = ((int64_t)uh * G * W + g * W + a) * n_part;
        float mx = kNegBig;
        for (int c = 0; c < n_part; ++c) mx = fmaxf(mx, row_part[row + c].x);
        float z = 0.f, zc = 0.f;
        for (int c = 0; c < n_part; ++c) {
            const float w = exp2f(row_part[row + c].x - mx);
            z += row_part[row + c].y * w;
            zc += row_cross[row + c] * w;
        }
        s += z > 0.f ? zc / z : 0.f;
    }
    s = warp_sum(s);
    if (lane == 0) cross_mass[(int64_t)(uh / Hkv) * (Hkv * G) + (uh % Hkv) * G + g] = s;
}

// Packs the modality map: word w of a unit holds keys 32 w .. 32 w + 31 (bit set = visual; keys past the prompt: 0).
__global__ void pack_modality_kernel(const uint8_t *modality, int L, int n_words, uint32_t *bits) {
    const int u = blockIdx.x, w = blockIdx.y * (blockDim.x >> 5) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (w >= n_words) return;
    const int key = 32 * w + lane;
    const uint32_t word = __ballot_sync(0xFFFFFFFFu, key < L && modality[(int64_t)u * L + key] != 0);
    if (lane == 0) bits[(int64_t)u * n_words + w] = word;
}

// Row constants for pass 2: negc[r] = -(M_r + log2 Z_r) so that exp2(s + negc) is the softmax
// probability; padding rows get a constant that makes every probability 0.
__global__ void score_combine_kernel(const float2 *row_part, int n_chunk, int GW, int GWpad, int n_uh, float *negc) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_uh * GWpad) return;
    const int uh = i / GWpad, r = i % GWpad;
    float out = kNegBig;
    if (r < GW) {
        const float2 *part = row_part + ((int64_t)uh * GW + r) * n_chunk;
        float mx = kNegBig;
        for (int c = 0; c < n_chunk; ++c) mx = fmaxf(mx, part[c].x);
        float z = 0.f;
        for (int c = 0; c < n_chunk; ++c) z += part[c].y * exp2f(part[c].x - mx);
        out = -(mx + log2f(z));
    }
    negc[i] = out;
}

// The common case of pass 2's inner step, written out in PTX so that it costs what it must and no more: 32 accumulator
// columns of this thread's key (32 proxy rows of one query head): probability = 2^(logit * scale + row constant), with
// the row constants read as packed pairs from shared memory, the multiply-adds and the additions as packed pairs, one
// exp2 per element; returns the sum of the 32 probabilities.  No mask and no split by modality: chunks that need either
// take the general path.
//   taddr  TMEM address of the chunk for this warp's lanes     negc  shared address of its 32 row constants
// (three phases, so that no exponential's result is needed before the last one has been issued: logits in place,
// exponentials in place, then a tree of packed additions)
#define FLOWMM_CS_X(q, i0, i1, i2, i3)                                                      \
    "ld.shared.v2.b64 {n0, n1}, [%2 + " #q " * 16];\n\t"                                    \
    "mov.b64 x0, {a" #i0 ", a" #i1 "};\n\t"                                                 \
    "mov.b64 x1, {a" #i2 ", a" #i3 "};\n\t"                                                 \
    "fma.rn.f32x2 x0, x0, sc, n0;\n\t"                                                      \
    "fma.rn.f32x2 x1, x1, sc, n1;\n\t"                                                      \
    "mov.b64 {a" #i0 ", a" #i1 "}, x0;\n\t"                                                 \
    "mov.b64 {a" #i2 ", a" #i3 "}, x1;\n\t"
#define FLOWMM_CS_E(i) "ex2.approx.ftz.f32 a" #i ", a" #i ";\n\t"
// 2^x for the pair (a_i, a_j) on the FMA pipe instead of the exp2 unit (which sets this step's pace): x clamped at
// -125, n = round(x) by the 1.5 * 2^23 trick, 2^f on f = x - n in [-0.5, 0.5] by a degree-4 polynomial (own least-squares
// fit at Chebyshev nodes with the constant fixed at 1: relative error 3.6e-6), n added to the exponent field.
#define FLOWMM_CS_POLY(i, j)                                                          \
    "max.f32 a" #i ", a" #i ", 0fC2FA0000;\n\t"                                        \
    "max.f32 a" #j ", a" #j ", 0fC2FA0000;\n\t"                                        \
    "mov.b64 x0, {a" #i ", a" #j "};\n\t"                                              \
    "add.rn.f32x2 x1, x0, kmg;\n\t"          /* t = x + 1.5 * 2^23 */                  \
    "mov.b64 {f0, f1}, x1;\n\t"                                                       \
    "sub.rn.f32x2 x1, x1, kmg;\n\t"          /* n */                                   \
    "sub.rn.f32x2 x0, x0, x1;\n\t"           /* f */                                   \
    "fma.rn.f32x2 x1, kc4, x0, kc3;\n\t"                                              \
    "fma.rn.f32x2 x1, x1, x0, kc2;\n\t"                                               \
    "fma.rn.f32x2 x1, x1, x0, kc1;\n\t"                                               \
    "fma.rn.f32x2 x1, x1, x0, kone;\n\t"                                              \
    "mov.b64 {a" #i ", a" #j "}, x1;\n\t"                                              \
    "mad.lo.s32 a" #i ", f0, 8388608, a" #i ";\n\t"                                    \
    "mad.lo.s32 a" #j ", f1, 8388608, a" #j ";\n\t"
#define FLOWMM_CS_P(k, i0, i1) "mov.b64 p" #k ", {a" #i0 ", a" #i1 "};\n\t"
#define FLOWMM_CS_A(d, x, y) "add.rn.f32x2 p" #d ", p" #x ", p" #y ";\n\t"
__device__ __forceinline__ float colsum_chunk32(uint32_t taddr, uint32_t negc, float scale_log2) {
    float csum;
    asm volatile(
        "{\n\t"
        ".reg .b32 a<32>;\n\t"
        ".reg .b64 n0, n1, x0, x1, sc, p<16>, kmg, kc1, kc2, kc3, kc4, kone;\n\t"
        ".reg .b32 f0, f1;\n\t"
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {a0, a1, a2, a3, a4, a5, a6, a7, a8, a9, a10, a11, a12, a13, a14, a15, "
        "a16, a17, a18, a19, a20, a21, a22, a23, a24, a25, a26, a27, a28, a29, a30, a31}, [%1];\n\t"
        "mov.b64 sc, {%3, %3};\n\t"
        "mov.b64 kmg, 0x4B4000004B400000;\n\t"      /* 12582912.0f twice */
        "mov.b64 kone, 0x3F8000003F800000;\n\t"
        "mov.b64 kc1, 0x3F3170613F317061;\n\t"      /* 0.69312102 */
        "mov.b64 kc2, 0x3E75FCD43E75FCD4;\n\t"      /* 0.24022228 */
        "mov.b64 kc3, 0x3D650E813D650E81;\n\t"      /* 0.05592204 */
        "mov.b64 kc4, 0x3C1E78073C1E7807;\n\t"      /* 0.00967217 */
        "tcgen05.wait::ld.sync.aligned;\n\t"
        FLOWMM_CS_X(0, 0, 1, 2, 3) FLOWMM_CS_X(1, 4, 5, 6, 7) FLOWMM_CS_X(2, 8, 9, 10, 11) FLOWMM_CS_X(3, 12, 13, 14, 15)
        FLOWMM_CS_X(4, 16, 17, 18, 19) FLOWMM_CS_X(5, 20, 21, 22, 23) FLOWMM_CS_X(6, 24, 25, 26, 27) FLOWMM_CS_X(7, 28, 29, 30, 31)
        // every fourth exponential goes to the FMA pipe, placed between the others
        FLOWMM_CS_E(0) FLOWMM_CS_E(1) FLOWMM_CS_E(2) FLOWMM_CS_E(4) FLOWMM_CS_E(5) FLOWMM_CS_E(6) FLOWMM_CS_POLY(3, 7)
        FLOWMM_CS_E(8) FLOWMM_CS_E(9) FLOWMM_CS_E(10) FLOWMM_CS_E(12) FLOWMM_CS_E(13) FLOWMM_CS_E(14) FLOWMM_CS_POLY(11, 15)
        FLOWMM_CS_E(16) FLOWMM_CS_E(17) FLOWMM_CS_E(18) FLOWMM_CS_E(20) FLOWMM_CS_E(21) FLOWMM_CS_E(22) FLOWMM_CS_POLY(19, 23)
        FLOWMM_CS_E(24) FLOWMM_CS_E(25) FLOWMM_CS_E(26) FLOWMM_CS_E(28) FLOWMM_CS_E(29) FLOWMM_CS_E(30) FLOWMM_CS_POLY(27, 31)
        FLOWMM_CS_P(0, 0, 1) FLOWMM_CS_P(1, 2, 3) FLOWMM_CS_P(2, 4, 5) FLOWMM_CS_P(3, 6, 7) FLOWMM_CS_P(4, 8, 9) FLOWMM_CS_P(5, 10, 11)
        FLOWMM_CS_P(6, 12, 13) FLOWMM_CS_P(7, 14, 15) FLOWMM_CS_P(8, 16, 17) FLOWMM_CS_P(9, 18, 19) FLOWMM_CS_P(10, 20, 21)
        FLOWMM_CS_P(11, 22, 23) FLOWMM_CS_P(12, 24, 25) FLOWMM_CS_P(13, 26, 27) FLOWMM_CS_P(14, 28, 29) FLOWMM_CS_P(15, 30, 31)
        FLOWMM_CS_A(0, 0, 1) FLOWMM_CS_A(2, 2, 3) FLOWMM_CS_A(4, 4, 5) FLOWMM_CS_A(6, 6, 7) FLOWMM_CS_A(8, 8, 9) FLOWMM_CS_A(10, 10, 11)
        FLOWMM_CS_A(12, 12, 13) FLOWMM_CS_A(14, 14, 15)
        FLOWMM_CS_A(0, 0, 2) FLOWMM_CS_A(4, 4, 6) FLOWMM_CS_A(8, 8, 10) FLOWMM_CS_A(12, 12, 14)
        FLOWMM_CS_A(0, 0, 4) FLOWMM_CS_A(8, 8, 12)
        FLOWMM_CS_A(0, 0, 8)
        "mov.b64 {f0, f1}, p0;\n\t"
        "add.f32 %0, f0, f1;\n\t"
        "}"
        : "=f"(csum)
        : "r"(taddr), "r"(negc), "f"(scale_log2)
        : "memory");
    return csum;
}
#undef FLOWMM_CS_X
#undef FLOWMM_CS_E
#undef FLOWMM_CS_POLY
#undef FLOWMM_CS_P
#undef FLOWMM_CS_A

// ---------------------------------------------------------------------------------------------
// Pass 2.  item = (unit*head, tile of 256 keys); the B stream is the head group's proxy rows.
template <class S>
__global__ void __launch_bounds__(tcs::kThreads, 1)
score_colsum_tc_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap q_map,
                       const ScoreTcArgs A) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const typename S::Ctx c = S::setup(smem_raw, &k_map, &q_map, A.status);
    if (!c.ok) return;
    auto plan = [&](int item) {
        tcs::TilePlan p;
        const int kt = item % A.n_rt, uh = item / A.n_rt;
        const int u = uh / A.Hkv, h = uh % A.Hkv;
        p.a1 = kt * tcs::kItemRows; p.a2 = h; p.a3 = u;
        p.h1 = tcs::kRows; p.h2 = 0;
        p.n_halves = p.a1 + tcs::kRows < A.L ? 2 : 1;
        p.b1 = 0; p.b2 = h * A.G; p.b3 = u; p.step1 = 0; p.step2 = S::kCols / A.W;
        p.cols_total = A.GW;
        p.n_tiles = (A.GW + S::kCols - 1) / S::kCols;
        p.extra = A.negc + (int64_t)uh * A.GWpad;        // row constants of pass 1, 256 per B tile
        return p;
    };
    const uint32_t b_bytes = (uint32_t)A.b_heads * A.W * 256u;
    if (c.warp == 0) {
        if (c.lane == 0) S::producer(c, &k_map, &q_map, A.n_items2, tcs::kAHalf, b_bytes, plan, A.status);
    } else if (c.warp == 1) {
        if (c.lane == 0) S::mma_issuer(c, A.n_items2, plan, A.status);
    } else {
        const int lane = c.lane, row = c.quarter * 32 + lane;
        const uint32_t xch = c.epi_addr() + row * 4;            // hand-over slot of this row
        const uint32_t pxch = c.partner_addr() + row * 4;
        int k = 0, bt = 0, cached_u = -1;
        const int w_shift = 31 - __clz(A.W);
        uint32_t wbits[4] = {0, 0, 0, 0};                            // modality of the proxy tokens, 32 per word
        bool ok = true;
        for (int item = blockIdx.x; ok && item < A.n_items2; item += gridDim.x) {
            const tcs::TilePlan p = plan(item);
            const int kt = item % A.n_rt, uh = item / A.n_rt, u = uh / A.Hkv, h = uh % A.Hkv;
            float *cross_out = A.cross_part + ((int64_t)u * A.Hq + h * A.G) * (A.n_rt * 8) + kt * 8 + c.group * 4 + c.quarter;
            if (c.group >= p.n_halves) {                             // no keys in this half: its masses are zero
                if (lane == 0)
                    for (int g = 0; g < A.G; ++g) cross_out[(int64_t)g * (A.n_rt * 8)] = 0.f;
                bt += p.n_tiles;                                     // keep the B-tile count in step
                continue;
            }
            if (u != cached_u) {
#pragma unroll
                for (int w = 0; w < 4; ++w) {
                    const int a = w * 32 + lane;
                    const bool vis = a < A.W && A.modality[(int64_t)u * A.L + A.L - A.W + a] != 0;
                    wbits[w] = __ballot_sync(0xFFFFFFFFu, vis);
                }
                cached_u = u;
            }
            const int key0 = kt * tcs::kItemRows + c.group * tcs::kRows;
            const int key = key0 + row;
            const bool masked_tile = key0 + tcs::kRows > A.L - A.W + 1;   // some (key, proxy row) pair is masked
            const bool my_vis = key < A.L && A.modality[(int64_t)u * A.L + key] != 0;
            const int first_proxy = A.L - A.W;
            float imp = 0.f, cg = 0.f;
            int cur_g = -1;                                          // head whose mass is being summed; -1: none yet
            for (int t = 0; ok && t < p.n_tiles; ++t, ++k, ++bt) {
                const int ncols = min(S::kCols, A.GW - t * S::kCols);
                ok = S::extra_wait(c, bt, A.status) && S::acc_wait(c, k, A.status);
                if (!ok) break;
                const uint32_t negc4 = c.extra(bt);
                constexpr int kPerC = S::kCols / 64;               // 32-column chunks a warp takes of a full tile
                const int chunk_hi = min((ncols + 31) >> 5, kPerC * c.colhalf + kPerC);
                for (int ch = kPerC * c.colhalf; ch < chunk_hi; ++ch) {
                    const int col = t * S::kCols + ch * 32;        // proxy row index r = g_local * W + a
                    const int g_local = col >> w_shift, a0 = col & (A.W - 1);   // (the window is 32, 64 or 128 rows)
                    if (g_local != cur_g) {                          // a head is complete: publish its mass
                        if (cur_g >= 0) {
                            const float tot = warp_sum(cg);
                            if (lane == 0) cross_out[(int64_t)cur_g * (A.n_rt * 8)] = tot;
                        }
                        cg = 0.f;
                        cur_g = g_local;
                    }
                    // proxy tokens of the other modality than this key's
                    const uint32_t wm = a0 < 32 ? wbits[0] : a0 < 64 ? wbits[1] : a0 < 96 ? wbits[2] : wbits[3];
                    const uint32_t other = my_vis ? ~wm : wm;
                    // the common case: no causal mask inside this tile, and the chunk's proxy tokens are all of this
                    // key's modality or all of the other one (decided for the whole warp: the TMEM read is warp-wide)
                    const bool plain = !masked_tile && (other == 0u || other == 0xFFFFFFFFu);
                    if (__all_sync(0xFFFFFFFFu, plain)) {
                        const float csum = colsum_chunk32(S::acc_addr(c, ch), negc4 + ch * 128, A.scale_log2);
                        imp += csum;
                        cg += other != 0u ? csum : 0.f;
                        continue;
                    }
                    uint32_t acc[32];
                    tc::tmem_ld32(S::acc_addr(c, ch), acc);
                    tc::tmem_ld_wait(acc);
                    float pr[32];
                    const float2 sc2 = make_float2(A.scale_log2, A.scale_log2);
#pragma unroll
                    for (int q4 = 0; q4 < 8; ++q4) {
                        const float4 n4 = tc::lds128(negc4 + (ch * 8 + q4) * 16);
                        const float2 x01 = tc::ffma2(make_float2(__uint_as_float(acc[4 * q4 + 0]), __uint_as_float(acc[4 * q4 + 1])),
                                                     sc2, make_float2(n4.x, n4.y));
                        const float2 x23 = tc::ffma2(make_float2(__uint_as_float(acc[4 * q4 + 2]), __uint_as_float(acc[4 * q4 + 3])),
                                                     sc2, make_float2(n4.z, n4.w));
                        pr[4 * q4 + 0] = tc::ex2(x01.x);
                        pr[4 * q4 + 1] = tc::ex2(x01.y);
                        pr[4 * q4 + 2] = tc::ex2(x23.x);
                        pr[4 * q4 + 3] = tc::ex2(x23.y);
                    }
                    if (masked_tile) {                               // causal mask inside the window, and keys >= L
#pragma unroll
                        for (int j = 0; j < 32; ++j) pr[j] = (key <= first_proxy + a0 + j) ? pr[j] : 0.f;
                    }
                    float2 s01 = make_float2(0.f, 0.f), s23 = make_float2(0.f, 0.f);
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        s01 = tc::fadd2(s01, make_float2(pr[j], pr[j + 1]));
                        s23 = tc::fadd2(s23, make_float2(pr[j + 2], pr[j + 3]));
                    }
                    const float csum = (s01.x + s01.y) + (s23.x + s23.y);
                    imp += csum;
                    if (other == 0xFFFFFFFFu) cg += csum;
                    else if (other != 0u) {
                        float x = 0.f;
#pragma unroll
                        for (int j = 0; j < 32; ++j) x += ((other >> j) & 1u) ? pr[j] : 0.f;
                        cg += x;
                    }
                }
                S::acc_release(c);
            }
            if (ok && cur_g >= 0) {
                const float tot = warp_sum(cg);
                if (lane == 0) cross_out[(int64_t)cur_g * (A.n_rt * 8)] = tot;
            }
            // the two column halves of a key meet: the upper one hands its partial sum over (kept even after a
            // wait ran out, so that the partner warp is never left waiting)
            if (c.colhalf == 1) tc::sts32(xch, imp);
            ok = !S::pair_meet(c, !ok);                            // (both warps of a key go on, or neither)
            if (c.colhalf == 0 && ok && key < A.L) A.importance[(int64_t)uh * A.L + key] = (imp + tc::lds32(pxch)) / (float)A.G;   // group mean
            S::pair_sync(c);
        }
    }
    S::teardown(c);
}

}  // namespace flowmm
