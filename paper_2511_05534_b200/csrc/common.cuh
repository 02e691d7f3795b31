// Shared device helpers for the FlowMM kernels: element types, vector loads, warp reductions.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace flowmm {

constexpr float kLog2e = 1.4426950408889634f;
constexpr float kNegBig = -1.0e30f;   // "minus infinity" that stays finite under subtraction
constexpr int kStatusIndex = 10;      // FLOWMM_ERR_INDEX

// Range check of an index that is about to address memory.  In a build with -DFLOWMM_DEBUG a bad index is recorded
// in the status word (first error wins) and reported to the caller, which skips the access; otherwise the check
// compiles to nothing.
#ifdef FLOWMM_DEBUG
__device__ __forceinline__ bool index_ok(long long i, long long n, int *status) {
    if (i >= 0 && i < n) return true;
    if (status) atomicCAS(status, 0, kStatusIndex);
    return false;
}
#else
__device__ __forceinline__ constexpr bool index_ok(long long, long long, int *) { return true; }
#endif

// ---- element access -------------------------------------------------------------------------
template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kVec = 4;    // elements per 16-byte vector
    __device__ static void load16(const float *p, float (&out)[4]) {
        const float4 v = *reinterpret_cast<const float4 *>(p);
        out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
    }
    __device__ static void unpack(const uint4 &v, float (&out)[4]) {
        out[0] = __uint_as_float(v.x); out[1] = __uint_as_float(v.y);
        out[2] = __uint_as_float(v.z); out[3] = __uint_as_float(v.w);
    }
    __device__ static void store16(float *p, const float (&in)[4]) {
        *reinterpret_cast<float4 *>(p) = make_float4(in[0], in[1], in[2], in[3]);
    }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kVec = 8;
    __device__ static void load16(const __nv_bfloat16 *p, float (&out)[8]) {
        const uint4 v = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {           // a bf16 is the upper half of the fp32 with the same value
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static void unpack(const uint4 &v, float (&out)[8]) {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            out[2 * i] = __uint_as_float(w[i] << 16);
            out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
        }
    }
    __device__ static void store16(__nv_bfloat16 *p, const float (&in)[8]) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(in[2 * i], in[2 * i + 1]);   // round to nearest even
            w[i] = *reinterpret_cast<const uint32_t *>(&h);
        }
        *reinterpret_cast<uint4 *>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// 16 bytes of a row as they are in memory; Elem<T>::unpack turns them into floats
template <typename T> __device__ __forceinline__ uint4 load_raw16(const T *p) {
    return *reinterpret_cast<const uint4 *>(p);
}

// Division of a 32-bit unsigned number by a divisor known on the host (Granlund-Montgomery, round-up multiplier):
// q = n / d exactly for every n < 2^32.  Replaces the ~20-instruction integer division in per-item index arithmetic.
struct FastDiv {
    uint32_t mul, shift, d;      // d == 1: shift == 0 and the multiplier is not used
    __device__ __forceinline__ uint32_t div(uint32_t n) const {
        if (shift == 0) return n;
        const uint32_t t = __umulhi(n, mul);
        return (t + ((n - t) >> 1)) >> (shift - 1);
    }
};
inline FastDiv make_fastdiv(uint32_t d) {
    FastDiv f;
    f.d = d;
    if (d <= 1) { f.mul = 0; f.shift = 0; return f; }
    uint32_t s = 0;
    while ((1ull << s) < d) ++s;                                   // s = ceil(log2 d), 1 .. 32
    const unsigned long long m = ((1ull << 32) * ((1ull << s) - d)) / d + 1;   // multiplier minus 2^32
    f.mul = (uint32_t)m;
    f.shift = s;
    return f;
}

// ---- warp helpers ---------------------------------------------------------------------------
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}


__device__ __forceinline__ int lane_id() { return threadIdx.x & 31; }

// Sum of one head's partial masses: lanes take the parts with a stride of 32, then a shuffle
// tree; the order is fixed, so every caller gets the same bits.  Call with the whole warp.
__device__ __forceinline__ float head_mass(const float *parts, int n_chunk) {
    float s = 0.f;
    for (int c = lane_id(); c < n_chunk; c += 32) s += parts[c];
    return warp_sum(s);
}
__device__ __forceinline__ uint32_t lanemask_lt() {
    uint32_t m;
    asm volatile("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
    return m;
}

// Exclusive prefix sum of one int per thread over a block of up to 1024 threads.
// `scratch` has room for 33 ints; returns the exclusive prefix and writes the block total.
__device__ __forceinline__ int block_exclusive_scan(int v, int *scratch, int &total) {
    const int lane = lane_id(), warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();                       // scratch may still be read from a previous call
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < nwarps ? scratch[lane] : 0;
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
            if (lane >= o) wi += t;
        }
        scratch[lane] = wi - w;            // exclusive prefix of the warp totals
        if (lane == 31) scratch[32] = wi;
    }
    __syncthreads();
    total = scratch[32];
    return scratch[warp] + incl - v;
}

}  // namespace flowmm
