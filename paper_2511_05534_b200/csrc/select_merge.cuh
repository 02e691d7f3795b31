// Pivot selection (top-B per KV head) and the merge / compaction stage.
#pragma once
#include "common.cuh"

namespace flowmm {

constexpr int kSelectThreads = 1024;

// Order-preserving integer key of an importance (a non-negative float); window tokens forced
// into the pivot set get the largest key.
__device__ __forceinline__ uint32_t select_key(float v, bool forced) {
    if (forced) return 0xFFFFFFFFu;
    const uint32_t b = __float_as_uint(v);
    return (b & 0x80000000u) ? 0u : b;        // -0 and (never expected) negatives sort lowest
}

// Section 3.3.1 pivot selection: a radix select finds the B-th largest key, then one ordered
// sweep writes the pivot positions and the non-pivot positions, both ascending.  Ties at the
// threshold go to the lower positions.  grid = U*Hkv, block = 1024.
__global__ void __launch_bounds__(kSelectThreads)
select_topb_kernel(const float *importance, int L, int B, int W, int keep_window, int *retained, int *evicted) {
    __shared__ int hist[256];
    __shared__ int scratch[33];
    __shared__ uint32_t s_prefix;
    __shared__ int s_need;
    const int tid = threadIdx.x;
    const float *imp = importance + (int64_t)blockIdx.x * L;
    int *ret = retained + (int64_t)blockIdx.x * B;
    int *evi = evicted + (int64_t)blockIdx.x * (L - B);
    const int first_forced = keep_window ? L - W : L;

    // radix select, most significant byte first: after the loop `prefix` is the B-th largest key
    uint32_t prefix = 0, mask = 0;
    int need = B;                                    // how many keys to take among those matching prefix
    for (int shift = 24; shift >= 0; shift -= 8) {
        if (tid < 256) hist[tid] = 0;
        __syncthreads();
        for (int i = tid; i < L; i += kSelectThreads) {
            const uint32_t key = select_key(imp[i], i >= first_forced);
            if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
        }
        __syncthreads();
        if (tid == 0) {
            int acc = 0, d = 255;
            for (; d > 0; --d) {                     // walk down from the largest digit
                if (acc + hist[d] >= need) break;
                acc += hist[d];
            }
            s_prefix = prefix | ((uint32_t)d << shift);
            s_need = need - acc;
        }
        __syncthreads();
        prefix = s_prefix;
        need = s_need;
        mask |= 0xFFu << shift;
        __syncthreads();
    }
    // keys > prefix are all kept; of the keys == prefix the first `need` (by position) are kept
    int eq_seen = 0, kept_seen = 0;
    for (int base = 0; base < L; base += kSelectThreads) {
        const int i = base + tid;
        uint32_t key = 0;
        bool valid = i < L;
        if (valid) key = select_key(imp[i], i >= first_forced);
        const int is_eq = valid && key == prefix;
        int total_eq;
        const int eq_rank = eq_seen + block_exclusive_scan(is_eq, scratch, total_eq);
        const int keep = valid && (key > prefix || (is_eq && eq_rank < need));
        int total_keep;
        const int pos = kept_seen + block_exclusive_scan(keep, scratch, total_keep);
        if (valid) {
            if (keep) ret[pos] = i;
            else evi[i - pos] = i;
        }
        eq_seen += total_eq;
        kept_seen += total_keep;
    }
}

// ---------------------------------------------------------------------------------------------
// Merge stage.  The match array maps non-pivot j to a slot (or -1).  The members of every slot
// are needed in a fixed order, so the non-pivot positions j are sorted by slot with a stable
// LSD radix sort (ascending j inside a slot); slot s then owns sorted[off[s] .. off[s+1]).
// Long member lists are cut into pieces of kPiece so that many warps share a popular pivot.
// ---------------------------------------------------------------------------------------------
constexpr int kCsrThreads = 1024;
constexpr int kPiece = 64;

struct CsrArgs {
    const int *match;        // [UH, E]
    int *sort_a, *sort_b;    // [UH, E] ping-pong buffers of non-pivot positions
    int *off;                // [UH, B+1] first member of each slot in the sorted order
    int *piece_off;          // [UH, B+1] first piece of each slot
    int *part_off;           // [UH, B+1] first partial-sum record of each slot (multi-piece slots only)
    int B, E, n_pass;
};

__device__ __forceinline__ int csr_key(int m, int B) { return m < 0 ? B : m; }   // dropped tokens sort last

// grid = U*Hkv, block = 1024 (32 warps; warp w owns a contiguous range of the input).
__global__ void __launch_bounds__(kCsrThreads) build_csr_kernel(const CsrArgs A) {
    __shared__ int counters[32][257];               // [warp][digit], padded
    __shared__ int scratch[33];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int uh = blockIdx.x;
    const int *match = A.match + (int64_t)uh * A.E;
    int *bufs[2] = {A.sort_a + (int64_t)uh * A.E, A.sort_b + (int64_t)uh * A.E};
    const int per_warp = ((A.E + 31) / 32 + 31) / 32 * 32;     // multiple of 32
    const int lo = warp * per_warp, hi = min(A.E, lo + per_warp);

    for (int pass = 0; pass < A.n_pass; ++pass) {
        const int shift = 8 * pass;
        const int *src = pass == 0 ? nullptr : bufs[(pass - 1) & 1];
        int *dst = bufs[pass & 1];
        for (int i = tid; i < 32 * 257; i += kCsrThreads) (&counters[0][0])[i] = 0;
        __syncthreads();
        // count digits, warp-private counters
        for (int t = lo; t < lo + per_warp && t < ((hi + 31) / 32) * 32; t += 32) {
            const int idx = t + lane;
            const bool valid = idx < hi;
            const int j = valid ? (src ? src[idx] : idx) : 0;
            const int digit = valid ? (csr_key(match[j], A.B) >> shift) & 255 : 256 + lane;
            const uint32_t peers = __match_any_sync(0xFFFFFFFFu, digit);
            if (valid && lane == __ffs(peers) - 1) counters[warp][digit] += __popc(peers);
            __syncwarp();
        }
        __syncthreads();
        // exclusive scan in (digit, warp) order: thread t covers 8 consecutive entries
        int vals[8], sum = 0;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int idx = tid * 8 + e;            // idx = digit * 32 + warp
            vals[e] = counters[idx & 31][idx >> 5];
            sum += vals[e];
        }
        int total;
        int run = block_exclusive_scan(sum, scratch, total);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const int idx = tid * 8 + e;
            counters[idx & 31][idx >> 5] = run;
            run += vals[e];
        }
        __syncthreads();
        // scatter, in order inside each warp's range
        for (int t = lo; t < lo + per_warp && t < ((hi + 31) / 32) * 32; t += 32) {
            const int idx = t + lane;
            const bool valid = idx < hi;
            const int j = valid ? (src ? src[idx] : idx) : 0;
            const int digit = valid ? (csr_key(match[j], A.B) >> shift) & 255 : 256 + lane;
            const uint32_t peers = __match_any_sync(0xFFFFFFFFu, digit);
            const int rank = __popc(peers & lanemask_lt());
            if (valid) dst[counters[warp][digit] + rank] = j;
            __syncwarp();
            if (valid && lane == __ffs(peers) - 1) counters[warp][digit] += __popc(peers);
            __syncwarp();
        }
        __syncthreads();
        __threadfence_block();
    }
    const int *sorted = bufs[(A.n_pass - 1) & 1];
    int *off = A.off + (int64_t)uh * (A.B + 1);
    int *piece_off = A.piece_off + (int64_t)uh * (A.B + 1);
    int *part_off = A.part_off + (int64_t)uh * (A.B + 1);
    // off[s] = number of sorted entries with key < s (binary search on the sorted order)
    for (int s = tid; s <= A.B; s += kCsrThreads) {
        int a = 0, b = A.E;
        while (a < b) {
            const int mid = (a + b) >> 1;
            if (csr_key(match[sorted[mid]], A.B) < s) a = mid + 1; else b = mid;
        }
        off[s] = a;
    }
    __syncthreads();
    // pieces per slot and partial records per slot, exclusive scans over the slots
    int piece_seen = 0, part_seen = 0;
    for (int base = 0; base <= A.B; base += kCsrThreads) {
        const int s = base + tid;
        int np = 0, npart = 0;
        if (s < A.B) {
            const int n = off[s + 1] - off[s];
            np = n > kPiece ? (n + kPiece - 1) / kPiece : 1;
            npart = np > 1 ? np : 0;
        }
        int tot_p, tot_q;
        const int pp = piece_seen + block_exclusive_scan(np, scratch, tot_p);
        const int qq = part_seen + block_exclusive_scan(npart, scratch, tot_q);
        if (s <= A.B) { piece_off[s] = pp; part_off[s] = qq; }
        piece_seen += tot_p;
        part_seen += tot_q;
    }
}

struct MergeArgs {
    const void *k, *v;
    void *k_out, *v_out;
    const int *retained, *evicted;    // [UH, B], [UH, E]
    const float *match_sim;           // [UH, E]
    const int *sorted, *off, *piece_off, *part_off;   // CSR arrays; all nullptr when E == 0
    float *partial;                   // [UH, max_parts, 2*D + 4] fp32 partial sums
    int Hkv, D, L, B, E, max_pieces, max_parts, merge_mode;
    int64_t ks[3], vs[3], kos[3], vos[3];
};

// One warp per piece of a slot.  A 16-byte vector of a K row or V row per lane: with D*sizeof(T)
// = 256 bytes lanes 0-15 carry the K row and lanes 16-31 the V row.  A single-piece slot is
// finished here (pivot row with weight 1, Eq. 5 weights, normalise, round once); a piece of a
// multi-piece slot stores its fp32 partial sums for merge_finish_kernel.
// grid = (ceil(max_pieces / warps per block), U*Hkv).
template <typename T>
__global__ void __launch_bounds__(256) merge_pieces_kernel(const MergeArgs A) {
    constexpr int V = Elem<T>::kVec;
    const int lane = lane_id();
    const int uh = blockIdx.y, u = uh / A.Hkv, h = uh % A.Hkv;
    const int piece = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int rv = A.D / V;                                   // 16-byte vectors per row
    int slot = piece, first = 0, count = 0, n_pieces = 1, part_base = 0, piece_in_slot = 0;
    if (A.sorted) {
        const int *poff = A.piece_off + (int64_t)uh * (A.B + 1);
        if (piece >= poff[A.B]) return;
        int a = 0, b = A.B;                                   // largest s with piece_off[s] <= piece
        while (b - a > 1) {
            const int mid = (a + b) >> 1;
            if (poff[mid] <= piece) a = mid; else b = mid;
        }
        slot = a;
        const int *off = A.off + (int64_t)uh * (A.B + 1);
        const int n = off[slot + 1] - off[slot];
        n_pieces = poff[slot + 1] - poff[slot];
        piece_in_slot = piece - poff[slot];
        first = off[slot] + piece_in_slot * kPiece;
        count = min(kPiece, n - piece_in_slot * kPiece);
        part_base = A.part_off[(int64_t)uh * (A.B + 1) + slot];
    } else if (piece >= A.B) {
        return;
    }
    const T *kb = static_cast<const T *>(A.k) + u * A.ks[0] + h * A.ks[1];
    const T *vb = static_cast<const T *>(A.v) + u * A.vs[0] + h * A.vs[1];
    const int *evi = A.evicted + (int64_t)uh * A.E;
    const int *sorted = A.sorted ? A.sorted + (int64_t)uh * A.E : nullptr;
    const float *sim = A.match_sim + (int64_t)uh * A.E;

    for (int vec = lane; vec < 2 * rv; vec += 32) {           // which vector of the (K row, V row) pair
        const bool is_v = vec >= rv;
        const int c0 = (is_v ? vec - rv : vec) * V;
        const T *src = is_v ? vb : kb;
        const int64_t tstride = is_v ? A.vs[2] : A.ks[2];
        float acc[V];
#pragma unroll
        for (int e = 0; e < V; ++e) acc[e] = 0.f;
        float wsum = 0.f;
        int t = 0;
        for (; t + 4 <= count; t += 4) {                      // four rows in flight
            int j[4]; float w[4]; float x[4][V];
#pragma unroll
            for (int q = 0; q < 4; ++q) j[q] = sorted[first + t + q];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                Elem<T>::load16(src + (int64_t)evi[j[q]] * tstride + c0, x[q]);
                w[q] = A.merge_mode == 1 ? 1.f : __expf(sim[j[q]] - 1.f);
            }
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                wsum += w[q];
#pragma unroll
                for (int e = 0; e < V; ++e) acc[e] = fmaf(w[q], x[q][e], acc[e]);
            }
        }
        for (; t < count; ++t) {
            const int j = sorted[first + t];
            float x[V];
            Elem<T>::load16(src + (int64_t)evi[j] * tstride + c0, x);
            const float w = A.merge_mode == 1 ? 1.f : __expf(sim[j] - 1.f);
            wsum += w;
#pragma unroll
            for (int e = 0; e < V; ++e) acc[e] = fmaf(w, x[e], acc[e]);
        }
        if (n_pieces == 1) {
            const int r = A.retained[(int64_t)uh * A.B + slot];
            float x[V];
            Elem<T>::load16(src + (int64_t)r * tstride + c0, x);
            T *dst = is_v ? static_cast<T *>(A.v_out) + u * A.vos[0] + h * A.vos[1] + (int64_t)slot * A.vos[2]
                          : static_cast<T *>(A.k_out) + u * A.kos[0] + h * A.kos[1] + (int64_t)slot * A.kos[2];
            if (count == 0) {
                Elem<T>::store16(dst + c0, x);                // nothing merged in: the pivot row, bit for bit
            } else {
                const float inv = 1.f / (1.f + wsum);
                float o[V];
#pragma unroll
                for (int e = 0; e < V; ++e) o[e] = (x[e] + acc[e]) * inv;
                Elem<T>::store16(dst + c0, o);
            }
        } else {
            float *rec = A.partial + ((int64_t)uh * A.max_parts + part_base + piece_in_slot) * (2 * A.D + 4);
#pragma unroll
            for (int e = 0; e < V; ++e) rec[(is_v ? A.D : 0) + c0 + e] = acc[e];
            if (vec == 0) rec[2 * A.D] = wsum;
        }
    }
}

// Slots whose members were cut into several pieces: add the pieces' partial sums in piece
// order, then the pivot row, normalise and store.  One warp per slot; grid = (ceil(B/8), U*Hkv).
template <typename T>
__global__ void __launch_bounds__(256) merge_finish_kernel(const MergeArgs A) {
    constexpr int V = Elem<T>::kVec;
    const int lane = lane_id();
    const int uh = blockIdx.y, u = uh / A.Hkv, h = uh % A.Hkv;
    const int slot = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (slot >= A.B) return;
    const int *poff = A.piece_off + (int64_t)uh * (A.B + 1);
    const int n_pieces = poff[slot + 1] - poff[slot];
    if (n_pieces <= 1) return;
    const int part_base = A.part_off[(int64_t)uh * (A.B + 1) + slot];
    const float *rec0 = A.partial + ((int64_t)uh * A.max_parts + part_base) * (2 * A.D + 4);
    const int rv = A.D / V;
    const int r = A.retained[(int64_t)uh * A.B + slot];
    float wsum = 0.f;
    for (int p = 0; p < n_pieces; ++p) wsum += rec0[(int64_t)p * (2 * A.D + 4) + 2 * A.D];
    const float inv = 1.f / (1.f + wsum);
    for (int vec = lane; vec < 2 * rv; vec += 32) {
        const bool is_v = vec >= rv;
        const int c0 = (is_v ? vec - rv : vec) * V;
        float acc[V];
#pragma unroll
        for (int e = 0; e < V; ++e) acc[e] = 0.f;
        for (int p = 0; p < n_pieces; ++p) {
            const float *rec = rec0 + (int64_t)p * (2 * A.D + 4) + (is_v ? A.D : 0) + c0;
#pragma unroll
            for (int e = 0; e < V; ++e) acc[e] += rec[e];
        }
        const T *src = is_v ? static_cast<const T *>(A.v) + u * A.vs[0] + h * A.vs[1] + (int64_t)r * A.vs[2]
                            : static_cast<const T *>(A.k) + u * A.ks[0] + h * A.ks[1] + (int64_t)r * A.ks[2];
        T *dst = is_v ? static_cast<T *>(A.v_out) + u * A.vos[0] + h * A.vos[1] + (int64_t)slot * A.vos[2]
                      : static_cast<T *>(A.k_out) + u * A.kos[0] + h * A.kos[1] + (int64_t)slot * A.kos[2];
        float x[V], o[V];
        Elem<T>::load16(src + c0, x);
#pragma unroll
        for (int e = 0; e < V; ++e) o[e] = (x[e] + acc[e]) * inv;
        Elem<T>::store16(dst + c0, o);
    }
}

}  // namespace flowmm
