// Decode-step attention over a KV cache (Eq. 4): one new query per query head against the n_keys
// rows of its KV head, all G heads of a group in one pass over K and V (each row is read once).
// HBM-bound streaming: split over key ranges (flash-decoding style), online softmax in the log2
// domain, fp32 accumulation; a second small kernel joins the key ranges.
#pragma once
#include "common.cuh"

namespace flowmm {

constexpr int kDecThreads = 128;
constexpr int kDecKeysPerStep = 4;      // rows a lane group keeps in flight (K and V each)

struct DecodeArgs {
    const void *q, *k, *v;       // q [U, Hq, D] dense
    float *part;                 // [UH, n_split, G, D + 2]: unnormalised output, running max (log2), exp-sum
    float *out;                  // [U, Hq, D]
    int Hq, Hkv, G, N, n_split, keys_per_split;
    float scale_log2;
    int64_t ks[3], vs[3];
};

__device__ __forceinline__ float dec_ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// grid = (U*Hkv, n_split), block = 128.  GP = G rounded up to 1, 2, 4 or 8; D = head_dim.
// A group of D / kVec lanes shares a row (16 bytes per lane); the groups of a block take the keys of the
// block's range in turn.  Dynamic shared memory: (rows groups per block) * GP * (D + 2) floats.
template <typename T, int D, int GP>
__global__ void __launch_bounds__(kDecThreads) decode_partial_kernel(const DecodeArgs A) {
    constexpr int V = Elem<T>::kVec, LPR = D / V, GROUPS = kDecThreads / LPR;
    extern __shared__ float dec_smem[];                              // [GROUPS][GP][D + 2]
    const int tid = threadIdx.x, sub = tid % LPR, grp = tid / LPR;
    const int uh = blockIdx.x, u = uh / A.Hkv, h = uh % A.Hkv;
    const int lo = blockIdx.y * A.keys_per_split, hi = min(A.N, lo + A.keys_per_split);
    const T *kb = static_cast<const T *>(A.k) + u * A.ks[0] + h * A.ks[1] + sub * V;
    const T *vb = static_cast<const T *>(A.v) + u * A.vs[0] + h * A.vs[1] + sub * V;
    const T *qb = static_cast<const T *>(A.q) + ((int64_t)u * A.Hq + h * A.G) * D + sub * V;

    float qf[GP][V], acc[GP][V], m[GP], l[GP];
#pragma unroll
    for (int g = 0; g < GP; ++g) {
        m[g] = kNegBig; l[g] = 0.f;
#pragma unroll
        for (int e = 0; e < V; ++e) { acc[g][e] = 0.f; qf[g][e] = 0.f; }
        if (g < A.G) {
            Elem<T>::load16(qb + (int64_t)g * D, qf[g]);
#pragma unroll
            for (int e = 0; e < V; ++e) qf[g][e] *= A.scale_log2;    // logits come out in the log2 domain
        }
    }
    for (int base = lo; base < hi; base += GROUPS * kDecKeysPerStep) {     // same trip count for every lane group
        const int key0 = base + grp * kDecKeysPerStep;                     // may lie past the range: then nothing counts
        uint4 kr[kDecKeysPerStep], vr[kDecKeysPerStep];
#pragma unroll
        for (int i = 0; i < kDecKeysPerStep; ++i) {                  // the step's row loads, back to back
            const int key = min(key0 + i, hi - 1);
            kr[i] = load_raw16(kb + (int64_t)key * A.ks[2]);
            vr[i] = load_raw16(vb + (int64_t)key * A.vs[2]);
        }
        float s[kDecKeysPerStep][GP];
#pragma unroll
        for (int i = 0; i < kDecKeysPerStep; ++i) {
            float kf[V];
            Elem<T>::unpack(kr[i], kf);
#pragma unroll
            for (int g = 0; g < GP; ++g) {
                float d = 0.f;
#pragma unroll
                for (int e = 0; e < V; ++e) d = fmaf(qf[g][e], kf[e], d);
                s[i][g] = d;
            }
        }
#pragma unroll
        for (int o = LPR >> 1; o > 0; o >>= 1)                       // every lane of the group gets the full dot products
#pragma unroll
            for (int i = 0; i < kDecKeysPerStep; ++i)
#pragma unroll
                for (int g = 0; g < GP; ++g) s[i][g] += __shfl_xor_sync(0xFFFFFFFFu, s[i][g], o);
        float p[kDecKeysPerStep][GP], corr[GP];
#pragma unroll
        for (int g = 0; g < GP; ++g) {
            float mx = m[g];
#pragma unroll
            for (int i = 0; i < kDecKeysPerStep; ++i)
                if (key0 + i < hi) mx = fmaxf(mx, s[i][g]);
            corr[g] = dec_ex2(m[g] - mx);
            float add = 0.f;
#pragma unroll
            for (int i = 0; i < kDecKeysPerStep; ++i) {
                p[i][g] = key0 + i < hi ? dec_ex2(s[i][g] - mx) : 0.f;
                add += p[i][g];
            }
            l[g] = l[g] * corr[g] + add;
            m[g] = mx;
#pragma unroll
            for (int e = 0; e < V; ++e) acc[g][e] *= corr[g];
        }
#pragma unroll
        for (int i = 0; i < kDecKeysPerStep; ++i) {
            float vf[V];
            Elem<T>::unpack(vr[i], vf);
#pragma unroll
            for (int g = 0; g < GP; ++g)
#pragma unroll
                for (int e = 0; e < V; ++e) acc[g][e] = fmaf(p[i][g], vf[e], acc[g][e]);
        }
    }
    // join the block's lane groups through shared memory
#pragma unroll
    for (int g = 0; g < GP; ++g) {
        float *rec = dec_smem + ((int64_t)grp * GP + g) * (D + 2);
#pragma unroll
        for (int e = 0; e < V; ++e) rec[sub * V + e] = acc[g][e];
        if (sub == 0) { rec[D] = m[g]; rec[D + 1] = l[g]; }
    }
    __syncthreads();
    for (int idx = tid; idx < A.G * D; idx += kDecThreads) {
        const int g = idx / D, d = idx % D;
        float mx = kNegBig;
        for (int r = 0; r < GROUPS; ++r) mx = fmaxf(mx, dec_smem[((int64_t)r * GP + g) * (D + 2) + D]);
        float o = 0.f, ls = 0.f;
        for (int r = 0; r < GROUPS; ++r) {
            const float *rec = dec_smem + ((int64_t)r * GP + g) * (D + 2);
            const float w = dec_ex2(rec[D] - mx);
            o = fmaf(rec[d], w, o);
            ls = fmaf(rec[D + 1], w, ls);
        }
        float *dst = A.part + (((int64_t)uh * A.n_split + blockIdx.y) * A.G + g) * (D + 2);
        dst[d] = o;
        if (d == 0) { dst[D] = mx; dst[D + 1] = ls; }
    }
}

// grid = U*Hq, block = D: joins the key ranges of one query head and normalises.
template <int D>
__global__ void __launch_bounds__(D) decode_combine_kernel(const DecodeArgs A) {
    const int ug = blockIdx.x, u = ug / A.Hq, gq = ug % A.Hq, h = gq / A.G, g = gq % A.G, d = threadIdx.x;
    const int uh = u * A.Hkv + h;
    float mx = kNegBig;
    for (int sp = 0; sp < A.n_split; ++sp)
        mx = fmaxf(mx, A.part[(((int64_t)uh * A.n_split + sp) * A.G + g) * (D + 2) + D]);
    float o = 0.f, ls = 0.f;
    for (int sp = 0; sp < A.n_split; ++sp) {
        const float *rec = A.part + (((int64_t)uh * A.n_split + sp) * A.G + g) * (D + 2);
        const float w = dec_ex2(rec[D] - mx);
        o = fmaf(rec[d], w, o);
        ls = fmaf(rec[D + 1], w, ls);
    }
    A.out[(int64_t)ug * D + d] = o / ls;
}

}  // namespace flowmm
