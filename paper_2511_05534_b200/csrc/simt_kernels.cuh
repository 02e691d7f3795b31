// SIMT fp32 kernels for the two dense contractions (window scoring and pivot matching).
// They serve fp32 inputs and head_dim 64, and any shape the tensor-core kernels do not take.
// Products of the inputs are accumulated in fp32; for bf16 inputs every product is exact.
#pragma once
#include "common.cuh"

namespace flowmm {

constexpr int kTile = 64;       // rows and columns of a CTA tile
constexpr int kDChunk = 32;     // head_dim slice held in shared memory
constexpr int kPitch = 68;      // row pitch of a slice (floats): 16-byte aligned, breaks bank strides
constexpr int kSimtThreads = 256;

struct SimtTiles {
    float a[kDChunk][kPitch];
    float b[kDChunk][kPitch];
};

// acc[i][j] = sum_d A[ty*4+i][d] * B[tx*4+j][d] for a 64x64 tile; rowA(r) / rowB(r) give the
// address of tile row r (nullptr: a row of zeros).  All 256 threads of the CTA take part.
template <typename T, typename FA, typename FB>
__device__ __forceinline__ void simt_tile_dot(SimtTiles &sm, int D, FA rowA, FB rowB, float (&acc)[4][4]) {
    constexpr int V = Elem<T>::kVec;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    const int lr = tid >> 2, ld = (tid & 3) * 8;       // this thread loads 8 elements of row lr
    const T *pa = rowA(lr);
    const T *pb = rowB(lr);
    for (int d0 = 0; d0 < D; d0 += kDChunk) {
        __syncthreads();
#pragma unroll
        for (int half = 0; half < 8 / V; ++half) {
            float va[V], vb[V];
            if (pa) Elem<T>::load16(pa + d0 + ld + half * V, va);
            else {
#pragma unroll
                for (int e = 0; e < V; ++e) va[e] = 0.f;
            }
            if (pb) Elem<T>::load16(pb + d0 + ld + half * V, vb);
            else {
#pragma unroll
                for (int e = 0; e < V; ++e) vb[e] = 0.f;
            }
#pragma unroll
            for (int e = 0; e < V; ++e) {
                sm.a[ld + half * V + e][lr] = va[e];
                sm.b[ld + half * V + e][lr] = vb[e];
            }
        }
        __syncthreads();
#pragma unroll 8
        for (int d = 0; d < kDChunk; ++d) {
            const float4 a4 = *reinterpret_cast<const float4 *>(&sm.a[d][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4 *>(&sm.b[d][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w};
            const float b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
    }
}

struct ScoreArgs {
    const void *q, *k;
    const uint8_t *modality;      // [U, L]
    float *importance;            // [U, Hkv, L]
    float2 *row_part;             // [U*Hq*W, n_chunk1]: (max, sum) of a row over one key chunk, log2 domain
    float *cross_part;            // [U*Hq, n_chunk2]
    int Hq, Hkv, G, D, L, W;
    int n_chunk1, chunk1;         // pass 1: key chunks per row, keys per chunk (multiple of 64)
    int n_chunk2, chunk2;         // pass 2
    float scale_log2;             // softmax scale * log2(e)
    int64_t qs[3], ks[3];
};

// Pass 1 of Eq. 8: per proxy row the running maximum and exp-sum of its causal logits over one
// chunk of keys.  grid = (U*Hkv, row tiles of G*W, n_chunk1).
template <typename T>
__global__ void __launch_bounds__(kSimtThreads) score_stats_simt(const ScoreArgs A) {
    __shared__ SimtTiles sm;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int uh = blockIdx.x, u = uh / A.Hkv, h = uh % A.Hkv;
    const int GW = A.G * A.W;
    const int row0 = blockIdx.y * kTile;
    const int key_lo = blockIdx.z * A.chunk1, key_hi = min(A.L, key_lo + A.chunk1);
    const T *q = static_cast<const T *>(A.q) + u * A.qs[0];
    const T *k = static_cast<const T *>(A.k) + u * A.ks[0] + h * A.ks[1];

    float m[4], l[4];
    int pa[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m[i] = kNegBig; l[i] = 0.f;
        const int r = row0 + ty * 4 + i;
        pa[i] = r < GW ? A.L - A.W + (r % A.W) : -1;
    }
    auto rowA = [&](int lr) -> const T * {
        const int r = row0 + lr;
        if (r >= GW) return nullptr;
        return q + (int64_t)(h * A.G + r / A.W) * A.qs[1] + (int64_t)(r % A.W) * A.qs[2];
    };
    for (int kt = key_lo; kt < key_hi; kt += kTile) {
        auto rowB = [&](int lr) -> const T * {
            const int i = kt + lr;
            return i < key_hi ? k + (int64_t)i * A.ks[2] : nullptr;
        };
        float acc[4][4];
        simt_tile_dot<T>(sm, A.D, rowA, rowB, acc);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float s[4], mx = m[i];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int key = kt + tx * 4 + j;
                const bool ok = key < key_hi && key <= pa[i];       // causal inside the window
                s[j] = ok ? acc[i][j] * A.scale_log2 : kNegBig;
                mx = fmaxf(mx, s[j]);
            }
            float add = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) add += s[j] > 0.5f * kNegBig ? exp2f(s[j] - mx) : 0.f;
            l[i] = l[i] * exp2f(m[i] - mx) + add;
            m[i] = mx;
        }
    }
    // the 16 threads that share a row sit in one half-warp
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {
            const float mo = __shfl_xor_sync(0xFFFFFFFFu, m[i], o);
            const float lo = __shfl_xor_sync(0xFFFFFFFFu, l[i], o);
            const float mx = fmaxf(m[i], mo);
            l[i] = l[i] * exp2f(m[i] - mx) + lo * exp2f(mo - mx);
            m[i] = mx;
        }
        const int r = row0 + ty * 4 + i;
        if (tx == 0 && r < GW)
            A.row_part[((int64_t)uh * GW + r) * A.n_chunk1 + blockIdx.z] = make_float2(m[i], l[i]);
    }
}

// Pass 2 of Eq. 8 and the modality split of Eq. 7: logits are recomputed, normalised with the
// row statistics of pass 1, summed down the columns into the importance, and summed per head
// over the keys of the other modality.  grid = (U*Hkv, n_chunk2); dynamic shared memory:
// 3*G*W floats.
template <typename T>
__global__ void __launch_bounds__(kSimtThreads) score_colsum_simt(const ScoreArgs A) {
    __shared__ SimtTiles sm;
    __shared__ float colpart[16][kTile];
    extern __shared__ float dyn[];
    const int GW = A.G * A.W;
    float *row_max = dyn, *row_inv = dyn + GW, *row_cross = dyn + 2 * GW;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int uh = blockIdx.x, u = uh / A.Hkv, h = uh % A.Hkv;
    const int key_lo = blockIdx.y * A.chunk2, key_hi = min(A.L, key_lo + A.chunk2);
    const T *q = static_cast<const T *>(A.q) + u * A.qs[0];
    const T *k = static_cast<const T *>(A.k) + u * A.ks[0] + h * A.ks[1];
    const uint8_t *mod = A.modality + (int64_t)u * A.L;

    for (int r = tid; r < GW; r += kSimtThreads) {      // combine the chunk statistics of pass 1
        const float2 *part = A.row_part + ((int64_t)uh * GW + r) * A.n_chunk1;
        float mx = kNegBig;
        for (int c = 0; c < A.n_chunk1; ++c) mx = fmaxf(mx, part[c].x);
        float z = 0.f;
        for (int c = 0; c < A.n_chunk1; ++c) z += part[c].y * exp2f(part[c].x - mx);
        row_max[r] = mx;
        row_inv[r] = 1.f / z;
        row_cross[r] = 0.f;
    }
    __syncthreads();

    for (int kt = key_lo; kt < key_hi; kt += kTile) {
        auto rowB = [&](int lr) -> const T * {
            const int i = kt + lr;
            return i < key_hi ? k + (int64_t)i * A.ks[2] : nullptr;
        };
        float colacc[4] = {0.f, 0.f, 0.f, 0.f};
        uint8_t mk[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int key = kt + tx * 4 + j;
            mk[j] = key < key_hi ? mod[key] : 0;
        }
        for (int row0 = 0; row0 < GW; row0 += kTile) {
            auto rowA = [&](int lr) -> const T * {
                const int r = row0 + lr;
                if (r >= GW) return nullptr;
                return q + (int64_t)(h * A.G + r / A.W) * A.qs[1] + (int64_t)(r % A.W) * A.qs[2];
            };
            float acc[4][4];
            simt_tile_dot<T>(sm, A.D, rowA, rowB, acc);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = row0 + ty * 4 + i;
                float cr = 0.f;
                if (r < GW) {
                    const int pa = A.L - A.W + (r % A.W);
                    const uint8_t mq = mod[pa];
                    const float mx = row_max[r], inv = row_inv[r];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const int key = kt + tx * 4 + j;
                        if (key < key_hi && key <= pa) {
                            const float p = exp2f(acc[i][j] * A.scale_log2 - mx) * inv;
                            colacc[j] += p;
                            if (mk[j] != mq) cr += p;
                        }
                    }
                }
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) cr += __shfl_xor_sync(0xFFFFFFFFu, cr, o);
                if (tx == 0 && r < GW) row_cross[r] += cr;      // one owner per row: fixed order
            }
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < 4; ++j) colpart[ty][tx * 4 + j] = colacc[j];
        __syncthreads();
        if (tid < kTile) {
            float s = 0.f;
#pragma unroll
            for (int t = 0; t < 16; ++t) s += colpart[t][tid];
            const int key = kt + tid;
            if (key < key_hi) A.importance[(int64_t)uh * A.L + key] = s / (float)A.G;   // group mean
        }
    }
    __syncthreads();
    for (int g = tid; g < A.G; g += kSimtThreads) {
        float s = 0.f;
        for (int a = 0; a < A.W; ++a) s += row_cross[g * A.W + a];
        A.cross_part[((int64_t)u * A.Hq + h * A.G + g) * A.n_chunk2 + blockIdx.y] = s;
    }
}

// cross_mass[u, g] = sum of the per-chunk partial masses; one warp per head.
__global__ void cross_mass_reduce(const float *cross_part, int n_chunk, int n, float *cross_mass) {
    const int i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (i >= n) return;
    const float s = head_mass(cross_part + (int64_t)i * n_chunk, n_chunk);
    if (lane_id() == 0) cross_mass[i] = s;
}

// Eq. 6 and the theta rule: one thread per unit.
__global__ void layer_flow_kernel(const float *cross_mass, int U, int Hq, int W, float theta, int flow_mode,
                                  float *rho, int *strategy) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= U) return;
    float s = 0.f;
    for (int g = 0; g < Hq; ++g) s += cross_mass[(int64_t)u * Hq + g] / (float)W;   // a head's total mass is W
    const float r = s / (float)Hq;
    if (rho) rho[u] = r;
    strategy[u] = flow_mode == 1 ? 0 : flow_mode == 2 ? 1 : ((r > theta) != (flow_mode == 3) ? 1 : 0);
}

// Full-prefill flow: per-head masses of the query tiles added up in tile order, then Eq. 6 over all L rows
// and the theta rule.  parts [n_tiles][U * Hq]; one block per unit, one thread per query head.
__global__ void full_flow_reduce_kernel(const float *parts, int n_tiles, int n, int Hq, int L, float theta, int flow_mode,
                                        float *cross_mass, float *rho, int *strategy) {
    const int u = blockIdx.x;
    for (int g = threadIdx.x; g < Hq; g += blockDim.x) {
        float s = 0.f;
        for (int t = 0; t < n_tiles; ++t) s += parts[(int64_t)t * n + (int64_t)u * Hq + g];
        cross_mass[(int64_t)u * Hq + g] = s;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f;
        for (int g = 0; g < Hq; ++g) s += cross_mass[(int64_t)u * Hq + g] / (float)L;   // a head's total mass is L
        const float r = s / (float)Hq;
        if (rho) rho[u] = r;
        strategy[u] = flow_mode == 1 ? 0 : flow_mode == 2 ? 1 : ((r > theta) != (flow_mode == 3) ? 1 : 0);
    }
}

// Reciprocal Euclidean norm of every key row (0 for a zero row).  One group of D/kVec lanes per row.
template <typename T>
__global__ void inv_norm_kernel(const void *k_, int64_t n_rows, int Hkv, int L, int D, int64_t s0, int64_t s1,
                                int64_t s2, float *rn) {
    constexpr int V = Elem<T>::kVec;
    const int lanes = D / V;                               // 8, 16 or 32
    const int64_t gid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t row = gid / lanes;
    const int sub = (int)(gid % lanes);
    float s = 0.f;
    if (row < n_rows) {
        const int64_t u = row / ((int64_t)Hkv * L);
        const int64_t rem = row % ((int64_t)Hkv * L);
        const T *p = static_cast<const T *>(k_) + u * s0 + (rem / L) * s1 + (rem % L) * s2 + sub * V;
        float v[V];
        Elem<T>::load16(p, v);
#pragma unroll
        for (int e = 0; e < V; ++e) s = fmaf(v[e], v[e], s);
    }
    for (int o = lanes >> 1; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    if (row < n_rows && sub == 0) rn[row] = s > 0.f ? rsqrtf(s) : 0.f;
}

struct MatchArgs {
    const void *k;
    const float *importance;      // [U, Hkv, L]
    const uint8_t *modality;      // [U, L]
    const int *retained, *evicted, *strategy;
    const float *rn;              // [U, Hkv, L] reciprocal key norms
    int *match;
    float *match_sim;
    int Hkv, D, L, B, E;
    float tau_eff;
    int64_t ks[3];
};

// Eq. 9 and Eq. 10: cosine similarity of 64 non-pivots against every pivot, gated argmax per row.
// grid = (U*Hkv, ceil(E / 64)).
template <typename T>
__global__ void __launch_bounds__(kSimtThreads) match_simt(const MatchArgs A) {
    __shared__ SimtTiles sm;
    const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
    const int uh = blockIdx.x, u = uh / A.Hkv, h = uh % A.Hkv;
    const T *k = static_cast<const T *>(A.k) + u * A.ks[0] + h * A.ks[1];
    const int *ret = A.retained + (int64_t)uh * A.B;
    const int *evi = A.evicted + (int64_t)uh * A.E;
    const float *imp = A.importance + (int64_t)uh * A.L;
    const float *rn = A.rn + (int64_t)uh * A.L;
    const uint8_t *mod = A.modality + (int64_t)u * A.L;
    const bool intra = A.strategy[u] == 0;
    const int j0 = blockIdx.y * kTile;

    float rne[4], best[4];
    int bests[4];
    uint8_t me[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int j = j0 + ty * 4 + i;
        const int e = j < A.E ? evi[j] : -1;
        rne[i] = e >= 0 ? rn[e] : 0.f;
        me[i] = e >= 0 ? mod[e] : 0;
        best[i] = -INFINITY;
        bests[i] = 0x7FFFFFFF;
    }
    auto rowA = [&](int lr) -> const T * {
        const int j = j0 + lr;
        return j < A.E ? k + (int64_t)evi[j] * A.ks[2] : nullptr;
    };
    for (int s0 = 0; s0 < A.B; s0 += kTile) {
        auto rowB = [&](int lr) -> const T * {
            const int s = s0 + lr;
            return s < A.B ? k + (int64_t)ret[s] * A.ks[2] : nullptr;
        };
        float acc[4][4];
        simt_tile_dot<T>(sm, A.D, rowA, rowB, acc);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int s = s0 + tx * 4 + j;
            if (s >= A.B) continue;
            const int r = ret[s];
            if (!(imp[r] <= A.tau_eff)) continue;            // highly sensitive pivot: never a merge target
            const float rnr = rn[r];
            const uint8_t mr = mod[r];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (intra && mr != me[i]) continue;
                const float uval = acc[i][j] * rne[i] * rnr;
                if (uval > best[i] || (uval == best[i] && s < bests[i])) { best[i] = uval; bests[i] = s; }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) {
            const float bo = __shfl_xor_sync(0xFFFFFFFFu, best[i], o);
            const int so = __shfl_xor_sync(0xFFFFFFFFu, bests[i], o);
            if (bo > best[i] || (bo == best[i] && so < bests[i])) { best[i] = bo; bests[i] = so; }
        }
        const int j = j0 + ty * 4 + i;
        if (tx == 0 && j < A.E) {
            const bool none = bests[i] == 0x7FFFFFFF;
            A.match[(int64_t)uh * A.E + j] = none ? -1 : bests[i];
            A.match_sim[(int64_t)uh * A.E + j] = none ? 0.f : best[i];
        }
    }
}

}  // namespace flowmm
