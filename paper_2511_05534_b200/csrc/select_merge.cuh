// Pivot selection (top-B per KV head) and the merge / compaction stage.
#pragma once
#include <type_traits>
#include "common.cuh"
#include "match_tc.cuh"

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
// threshold go to the lower positions.  grid = U*Hkv, block = any multiple of 32 up to 1024.
// Eq. 6 and the theta rule riding along with the selection (cross_mass == nullptr: not asked for): the block of a
// unit's first KV head applies them, one thread, same arithmetic as layer_flow_kernel.
struct SelectFlow {
    const float *cross_part;     // nullptr, or [U * Hq, n_parts] partial masses that are first added up into cross_mass
    int n_parts;
    float *cross_mass;           // [U, Hq] per-head masses (read; written first when cross_part is given)
    float *rho;                  // [U] or nullptr
    int *strategy;               // [U]
    int Hq, Hkv;
    float theta;
    int flow_mode;
};

// with_prepare: the block goes on to lay out the head's matching candidates (match_prepare_head) from the lists it has
// just written, which saves the short-context workloads a launch and a second pass over the same few kilobytes.
__global__ void __launch_bounds__(kSelectThreads)
select_topb_kernel(const float *importance, int L, int B, int W, int keep_window, int *retained, int *evicted,
                   const SelectFlow F, const MatchPrepArgs P, int with_prepare) {
    __shared__ int hist[256];
    __shared__ int scratch[33];
    __shared__ uint32_t s_prefix;
    __shared__ int s_need;
    const int tid = threadIdx.x, nthreads = blockDim.x, lane = tid & 31;
    const float *imp = importance + (int64_t)blockIdx.x * L;
    int *ret = retained + (int64_t)blockIdx.x * B;
    int *evi = evicted + (int64_t)blockIdx.x * (L - B);
    const int first_forced = keep_window ? L - W : L;
    if (F.cross_part && blockIdx.x % F.Hkv == 0) {                   // (the same for every thread of the block)
        const int u = blockIdx.x / F.Hkv;
        for (int g = tid >> 5; g < F.Hq; g += nthreads >> 5) {      // same sums in the same order as cross_mass_reduce
            const int64_t i = (int64_t)u * F.Hq + g;
            const float s = head_mass(F.cross_part + i * F.n_parts, F.n_parts);
            if (lane == 0) F.cross_mass[i] = s;
        }
        __syncthreads();
    }
    if (F.cross_mass && blockIdx.x % F.Hkv == 0 && tid == nthreads - 1) {
        const int u = blockIdx.x / F.Hkv;
        float s = 0.f;
        for (int g = 0; g < F.Hq; ++g) s += F.cross_mass[(int64_t)u * F.Hq + g] / (float)W;   // a head's total mass is W
        const float r = s / (float)F.Hq;
        if (F.rho) F.rho[u] = r;
        F.strategy[u] = F.flow_mode == 1 ? 0 : F.flow_mode == 2 ? 1 : ((r > F.theta) != (F.flow_mode == 3) ? 1 : 0);
    }

    // radix select, most significant byte first: after the loop `prefix` is the B-th largest key
    uint32_t prefix = 0, mask = 0;
    int need = B;                                    // how many keys to take among those matching prefix
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += nthreads) hist[i] = 0;
        __syncthreads();
        // Eight keys per thread are in flight at a time, and a thread adds runs of equal digits at once: the first
        // digits (sign and exponent) are nearly the same for all keys, which would put every thread's every add on one counter.
        {
            int run_bin = -1, run_cnt = 0;
            for (int base = 0; base < L; base += 8 * nthreads) {
                uint32_t keys[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int i = base + e * nthreads + tid;
                    keys[e] = i < L ? select_key(imp[i], i >= first_forced) : 0u;
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const int i = base + e * nthreads + tid;
                    if (i < L && (keys[e] & mask) == prefix) {
                        const int bin = (keys[e] >> shift) & 255;
                        if (bin != run_bin) {
                            if (run_cnt > 0) atomicAdd(&hist[run_bin], run_cnt);
                            run_bin = bin; run_cnt = 0;
                        }
                        ++run_cnt;
                    }
                }
            }
            if (run_cnt > 0) atomicAdd(&hist[run_bin], run_cnt);
        }
        __syncthreads();
        if (tid < 32) {                              // walk down from the largest digit, 8 digits per lane
            int local[8], lsum = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) { local[e] = hist[255 - (lane * 8 + e)]; lsum += local[e]; }
            int incl = lsum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
                if (lane >= o) incl += t;
            }
            int acc = incl - lsum;                   // keys with a larger digit than this lane's first
            if (acc < need && need <= incl) {        // the B-th largest key has one of this lane's digits
                int e = 0;
                for (; e < 7; ++e) {
                    if (acc + local[e] >= need) break;
                    acc += local[e];
                }
                s_prefix = prefix | ((uint32_t)(255 - (lane * 8 + e)) << shift);
                s_need = need - acc;
            }
        }
        __syncthreads();
        prefix = s_prefix;
        need = s_need;
        mask |= 0xFFu << shift;
    }
    // keys > prefix are all kept; of the keys == prefix the first `need` (by position) are kept
    // (four consecutive positions per thread and iteration: a quarter of the block-wide scans)
    int eq_seen = 0, kept_seen = 0;
    for (int base = 0; base < L; base += 4 * nthreads) {
        const int i0 = base + 4 * tid;
        uint32_t key[4];
        int n_eq = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            key[e] = i0 + e < L ? select_key(imp[i0 + e], i0 + e >= first_forced) : 0u;
            n_eq += i0 + e < L && key[e] == prefix;
        }
        int total_eq;
        int eq_rank = eq_seen + block_exclusive_scan(n_eq, scratch, total_eq);
        int keep[4], n_keep = 0;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const bool valid = i0 + e < L, is_eq = valid && key[e] == prefix;
            keep[e] = valid && (key[e] > prefix || (is_eq && eq_rank < need));
            eq_rank += is_eq;
            n_keep += keep[e];
        }
        int total_keep;
        int pos = kept_seen + block_exclusive_scan(n_keep, scratch, total_keep);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (i0 + e < L) {
                if (keep[e]) ret[pos] = i0 + e;
                else evi[i0 + e - pos] = i0 + e;
            }
            pos += keep[e];
        }
        eq_seen += total_eq;
        kept_seen += total_keep;
    }
    if (with_prepare) {
        __syncthreads();                                 // this block's lists are complete and visible to all its threads
        match_prepare_head(P, blockIdx.x, scratch, &s_need);
    }
}

// ---------------------------------------------------------------------------------------------
// Merge stage.  The match array maps non-pivot j to a slot (or -1).  The members of every slot
// are needed in a fixed order, so the non-pivot positions j are sorted by slot with a stable
// LSD radix sort (ascending j inside a slot); slot s then owns entries off[s] .. off[s+1] of the
// sorted order, for which the kernel writes the member's token position and Eq. 5 weight.
// Long member lists are cut into pieces of kPiece so that many warps share a popular pivot; one
// descriptor per piece tells its warp what to do without any search.
// ---------------------------------------------------------------------------------------------
constexpr int kPiece = 64;

struct CsrArgs {
    const int *match;        // [UH, E]
    const int *evicted;      // [UH, E]
    const float *match_sim;  // [UH, E]
    int *sort_a, *sort_b;    // [UH, E] ping-pong buffers of non-pivot positions
    int *mem_tok;            // [UH, E] token position of the i-th member in slot order
    float *mem_w;            // [UH, E] its merge weight
    int *off;                // [UH, B+1] first member of each slot in the sorted order
    int *piece_off;          // [UH, B+1] first piece of each slot
    int *part_off;           // [UH, B+1] first partial-sum record of each slot (multi-piece slots only)
    int4 *piece_desc;        // [UH, max_pieces] (slot, first member, members, partial record or -1)
    unsigned *ticket;        // work counter of the merge kernel, cleared here
    int *slot_done;          // [UH, B] pieces of a slot that have stored their partial sums, cleared here
    int B, E, n_pass, max_pieces, merge_mode;
};

__device__ __forceinline__ int csr_key(int m, int B) { return m < 0 ? B : m; }   // dropped tokens sort last

constexpr int kCsrBits = 6, kCsrBins = 1 << kCsrBits;      // digit width of the sort

// Lanes of the warp that hold the same digit as this one, among the valid lanes: a vote per bit and as many logic
// operations (the match instruction gives the same set, but its unit is slow and shared by the SM's warps).
__device__ __forceinline__ uint32_t digit_peers(int digit, bool valid) {
    uint32_t mine = __ballot_sync(0xFFFFFFFFu, valid);
#pragma unroll
    for (int b = 0; b < kCsrBits; ++b) {
        const uint32_t vote = __ballot_sync(0xFFFFFFFFu, (digit >> b) & 1);
        mine &= ((digit >> b) & 1) ? vote : ~vote;
    }
    return mine;
}

// grid = U*Hkv, block = 32 * NW threads (warp w owns a contiguous range of the input).  n_pass passes of kCsrBits bits.
// The sort gathers keys by position and scatters positions, 4 or 2 bytes at a time, which an SM's global-memory path
// takes at about one access per clock: with kStaged (E and B below 65536 and 6 E bytes of dynamic shared memory) the
// keys and both position buffers are 16-bit arrays in shared memory and only the results touch global memory.
template <int NW, bool kStaged>
__global__ void __launch_bounds__(32 * NW) build_csr_kernel(const CsrArgs A) {
    constexpr int kThreads = 32 * NW;
    constexpr int kBatch = 8;                       // steps of 32 positions whose loads are in flight together
    using Pos = std::conditional_t<kStaged, uint16_t, int>;
    extern __shared__ __align__(16) uint16_t csr_smem[];   // kStaged: keys[Ep], positions[2][Ep], Ep = E rounded up to 8
    __shared__ int counters[NW][kCsrBins + 1];      // [warp][digit], padded
    __shared__ int scratch[33];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int uh = blockIdx.x;
    if (uh == 0 && tid == 0) *A.ticket = 0u;
    const int *match = A.match + (int64_t)uh * A.E;
    const int Ep = (A.E + 7) & ~7;
    Pos *bufs[2];
    if constexpr (kStaged) {
        // (the buffer that holds the final order comes last: keys and the other buffer are then one free region of 4 Ep bytes)
        const int fin = (A.n_pass - 1) & 1;
        bufs[fin] = csr_smem + 2 * Ep; bufs[fin ^ 1] = csr_smem + Ep;
        for (int i = tid; i < A.E; i += kThreads) csr_smem[i] = (uint16_t)csr_key(match[i], A.B);
        __syncthreads();
    } else {
        bufs[0] = A.sort_a + (int64_t)uh * A.E; bufs[1] = A.sort_b + (int64_t)uh * A.E;
    }
    auto key_of = [&](int j) -> int {
        if constexpr (kStaged) return csr_smem[j]; else return csr_key(match[j], A.B);
    };
    const int per_warp = ((A.E + NW - 1) / NW + 31) / 32 * 32;     // multiple of 32
    const int lo = warp * per_warp, hi = min(A.E, lo + per_warp);
    const int end = min(lo + per_warp, ((hi + 31) / 32) * 32);

    for (int pass = 0; pass < A.n_pass; ++pass) {
        const int shift = kCsrBits * pass;
        const Pos *src = pass == 0 ? nullptr : bufs[(pass - 1) & 1];
        Pos *dst = bufs[pass & 1];
        // The positions and their keys are fetched kBatch steps at a time (the loads of a step depend on each other,
        // those of different steps do not); a step past the warp's range has no valid lane and changes nothing.
        auto fetch = [&](int t0, int (&jv)[kBatch], int (&dg)[kBatch]) {
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const int idx = t0 + 32 * b + lane;
                jv[b] = idx < hi ? (src ? (int)src[idx] : idx) : -1;
            }
#pragma unroll
            for (int b = 0; b < kBatch; ++b) dg[b] = jv[b] >= 0 ? (key_of(jv[b]) >> shift) & (kCsrBins - 1) : 0;
        };
        // count the warp's positions by digit (order does not matter here: shared-memory atomics on the warp's own counters)
        for (int d = lane; d < kCsrBins; d += 32) counters[warp][d] = 0;
        __syncwarp();
        for (int t0 = lo; t0 < end; t0 += 32 * kBatch) {
            int jv[kBatch], dg[kBatch];
            fetch(t0, jv, dg);
#pragma unroll
            for (int b = 0; b < kBatch; ++b)
                if (jv[b] >= 0) atomicAdd(&counters[warp][dg[b]], 1);
        }
        __syncthreads();
        // exclusive scan in (digit, warp) order: thread t holds the kPerThread consecutive entries from kPerThread t on,
        // entry e being digit = e / NW, warp = e % NW
        {
            constexpr int kPerThread = kCsrBins / 32;
            int vals[kPerThread], sum = 0;
#pragma unroll
            for (int e = 0; e < kPerThread; ++e) {
                const int idx = tid * kPerThread + e;
                vals[e] = counters[idx % NW][idx / NW];
                sum += vals[e];
            }
            int total;
            int run = block_exclusive_scan(sum, scratch, total);
            __syncthreads();
#pragma unroll
            for (int e = 0; e < kPerThread; ++e) {
                const int idx = tid * kPerThread + e;
                counters[idx % NW][idx / NW] = run;
                run += vals[e];
            }
        }
        __syncthreads();
        // scatter, in order inside each warp's range: the warp's counters now hold the next free place of each digit
        for (int t0 = lo; t0 < end; t0 += 32 * kBatch) {
            int jv[kBatch], dg[kBatch];
            fetch(t0, jv, dg);
#pragma unroll
            for (int b = 0; b < kBatch; ++b) {
                const bool valid = jv[b] >= 0;
                const uint32_t mine = digit_peers(dg[b], valid);
                if (valid) dst[counters[warp][dg[b]] + __popc(mine & lanemask_lt())] = (Pos)jv[b];
                __syncwarp();
                if (valid && lane == __ffs(mine) - 1) counters[warp][dg[b]] += __popc(mine);
                __syncwarp();
            }
        }
        __syncthreads();
        __threadfence_block();
    }
    const Pos *sorted = bufs[(A.n_pass - 1) & 1];
    int *off = A.off + (int64_t)uh * (A.B + 1);
    int *piece_off = A.piece_off + (int64_t)uh * (A.B + 1);
    int *part_off = A.part_off + (int64_t)uh * (A.B + 1);
    // token position and weight of every member, in slot order
    {
        const int *evi = A.evicted + (int64_t)uh * A.E;
        const float *sim = A.match_sim + (int64_t)uh * A.E;
        int *mem_tok = A.mem_tok + (int64_t)uh * A.E;
        float *mem_w = A.mem_w + (int64_t)uh * A.E;
        // ... and off[s] = number of sorted entries with key < s: entry i starts every slot above its predecessor's
        // key up to its own, the last entry also ends the slots above its key (E > 0: the kernel is not launched otherwise)
        for (int i = tid; i < A.E; i += kThreads) {
            const int j = sorted[i];
            const int key = key_of(j);
            const int prev = i > 0 ? key_of(sorted[i - 1]) : -1;
            if constexpr (!kStaged) {
                mem_tok[i] = evi[j];
                mem_w[i] = A.merge_mode == 1 ? 1.f : __expf(sim[j] - 1.f);
            }
            for (int s2 = prev + 1; s2 <= key; ++s2) off[s2] = i;
            if (i == A.E - 1)
                for (int s2 = key + 1; s2 <= A.B; ++s2) off[s2] = A.E;
        }
        if constexpr (kStaged) {
            // the gathers by position go through shared memory as well: the token positions, then the similarities, are
            // copied in order into the region the keys and the spare buffer have left, and picked from there
            int *stage_i = reinterpret_cast<int *>(csr_smem);
            float *stage_f = reinterpret_cast<float *>(csr_smem);
            __syncthreads();                                     // the keys are not read any more
            for (int i = tid; i < A.E; i += kThreads) stage_i[i] = evi[i];
            __syncthreads();
            for (int i = tid; i < A.E; i += kThreads) mem_tok[i] = stage_i[sorted[i]];
            __syncthreads();
            if (A.merge_mode == 1) {
                for (int i = tid; i < A.E; i += kThreads) mem_w[i] = 1.f;
            } else {
                for (int i = tid; i < A.E; i += kThreads) stage_f[i] = sim[i];
                __syncthreads();
                for (int i = tid; i < A.E; i += kThreads) mem_w[i] = __expf(stage_f[sorted[i]] - 1.f);
            }
        }
    }
    __syncthreads();
    // pieces per slot and partial records per slot, exclusive scans over the slots
    int4 *desc = A.piece_desc + (int64_t)uh * A.max_pieces;
    int piece_seen = 0, part_seen = 0;
    for (int base = 0; base <= A.B; base += kThreads) {
        const int s = base + tid;
        int n = 0, np = 0, npart = 0;
        if (s < A.B) {
            n = off[s + 1] - off[s];
            np = n > kPiece ? (n + kPiece - 1) / kPiece : 1;
            npart = np > 1 ? np : 0;
        }
        int tot_p, tot_q;
        const int pp = piece_seen + block_exclusive_scan(np, scratch, tot_p);
        const int qq = part_seen + block_exclusive_scan(npart, scratch, tot_q);
        if (s <= A.B) { piece_off[s] = pp; part_off[s] = qq; }
        if (s < A.B) A.slot_done[(int64_t)uh * A.B + s] = 0;
        for (int q = 0; q < np; ++q)
            desc[pp + q] = make_int4(s, off[s] + q * kPiece, min(kPiece, n - q * kPiece), np > 1 ? qq + q : -1);
        piece_seen += tot_p;
        part_seen += tot_q;
    }
    for (int i = piece_seen + tid; i < A.max_pieces; i += kThreads) desc[i] = make_int4(0, 0, -1, -1);   // unused entries
}

struct MergeArgs {
    const void *k, *v;
    void *k_out, *v_out;
    const int *retained;              // [UH, B]
    const int *mem_tok;               // [UH, E] member token positions in slot order; nullptr when E == 0
    const float *mem_w;               // [UH, E] member weights
    const int4 *piece_desc;           // [UH, max_pieces]
    const int *piece_off, *part_off;  // [UH, B+1]
    float *partial;                   // [UH, max_parts, 2*D + 4] fp32 partial sums
    unsigned *ticket;                 // shared work counter (pieces are handed out in table order); nullptr: fixed stride
    int *slot_done;                   // [UH, B] arrival counters of multi-piece slots
    int Hkv, D, L, B, E, max_pieces, max_parts;
    int64_t ks[3], vs[3], kos[3], vos[3];
};

// A slot whose members were cut into several pieces: add the pieces' partial sums in piece order,
// then the pivot row, normalise and store.  Run by the warp whose piece was the last to arrive;
// the partial records come from other SMs, so they are read past L1.
template <typename T>
__device__ __forceinline__ void merge_finish_slot(const MergeArgs &A, int uh, int slot, int lane) {
    constexpr int V = Elem<T>::kVec;
    const int u = uh / A.Hkv, h = uh % A.Hkv;
    const int *poff = A.piece_off + (int64_t)uh * (A.B + 1);
    const int n_pieces = poff[slot + 1] - poff[slot];
    const int part_base = A.part_off[(int64_t)uh * (A.B + 1) + slot];
    const float *rec0 = A.partial + ((int64_t)uh * A.max_parts + part_base) * (2 * A.D + 4);
    const int rv = A.D / V;
    const int r = A.retained[(int64_t)uh * A.B + slot];
    float wsum = 0.f;
    for (int p = 0; p < n_pieces; ++p) wsum += __ldcg(rec0 + (int64_t)p * (2 * A.D + 4) + 2 * A.D);
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
            for (int e = 0; e < V; ++e) acc[e] += __ldcg(rec + e);
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

constexpr int kMergeBatch = 8;        // member rows a warp keeps in flight

// One warp per piece of a slot, persistent: a warp walks the flat piece table with a stride and
// fetches the next piece's descriptor, member list and pivot index while it streams the rows of
// the current one, so the row loads never wait on index loads.  A 16-byte vector of a K row or V
// row per lane: with D*sizeof(T) = 256 bytes lanes 0-15 carry the K row and lanes 16-31 the V
// row.  A single-piece slot is finished here (pivot row with weight 1, Eq. 5 weights, normalise,
// round once); a piece of a multi-piece slot stores its fp32 partial sums, and the piece that arrives
// last adds them up in piece order (so the result does not depend on which piece that was).
template <typename T>
__global__ void __launch_bounds__(256) merge_pieces_kernel(const MergeArgs A, int n_uh) {
    constexpr int V = Elem<T>::kVec;
    const int lane = lane_id();
    const unsigned n_warps = gridDim.x * (blockDim.x >> 5);
    const unsigned total = (unsigned)n_uh * (unsigned)A.max_pieces;
    const int rv = A.D / V;                                   // 16-byte vectors per row
    const int n_vec = 2 * rv;

    struct Piece { int4 d; int tok_lo, tok_hi, r; float w_lo, w_hi; };
    auto fetch_desc = [&](unsigned g) -> int4 {              // (slot, first, count, part); count < 0: no such piece
        if (g >= total) return make_int4(0, 0, -1, -1);
        if (!A.piece_desc) return make_int4((int)(g % (unsigned)A.max_pieces), 0, 0, -1);   // E == 0: plain copy of the pivots
        return A.piece_desc[g];
    };
    auto fetch_members = [&](unsigned g, Piece &pc) {        // needs pc.d
        pc.tok_lo = pc.tok_hi = pc.r = 0; pc.w_lo = pc.w_hi = 0.f;
        if (pc.d.z < 0) return;
        const int64_t uh = g / (unsigned)A.max_pieces;
        if (pc.d.z > 0) {
            const int *mt = A.mem_tok + uh * A.E + pc.d.y;
            const float *mw = A.mem_w + uh * A.E + pc.d.y;
            if (lane < pc.d.z) { pc.tok_lo = mt[lane]; pc.w_lo = mw[lane]; }
            if (lane + 32 < pc.d.z) { pc.tok_hi = mt[lane + 32]; pc.w_hi = mw[lane + 32]; }
        }
        if (pc.d.w < 0) pc.r = A.retained[uh * A.B + pc.d.x];
    };
    // the next piece of this warp: from the shared counter (warps that drew light pieces come back sooner, so
    // the last pieces end together), or with a fixed stride when there is no counter
    unsigned stride_next = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    unsigned drawn = 0, drawn_left = 0;                       // pieces are drawn kDraw at a time
    constexpr unsigned kDraw = 4;
    auto next_piece = [&]() -> unsigned {
        if (!A.ticket) { const unsigned g = stride_next; stride_next = g + n_warps < g ? 0xFFFFFFFFu : g + n_warps; return g; }
        if (drawn_left == 0) {
            unsigned g = 0;
            if (lane == 0) g = atomicAdd(A.ticket, kDraw);
            drawn = __shfl_sync(0xFFFFFFFFu, g, 0);
            drawn_left = kDraw;
        }
        --drawn_left;
        return drawn++;
    };

    unsigned g = next_piece(), g_nxt = next_piece();
    Piece cur, nxt;
    cur.d = fetch_desc(g);
    nxt.d = fetch_desc(g_nxt);
    fetch_members(g, cur);
    while (g < total) {
        const unsigned g_d2 = next_piece();
        const int4 d2 = fetch_desc(g_d2);                     // two pieces ahead
        fetch_members(g_nxt, nxt);                            // one piece ahead
        const int slot = cur.d.x, count = cur.d.z, part = cur.d.w;
        if (count >= 0) {
            const int uh = (int)(g / (unsigned)A.max_pieces), u = uh / A.Hkv, h = uh % A.Hkv;
            const T *kb = static_cast<const T *>(A.k) + u * A.ks[0] + h * A.ks[1];
            const T *vb = static_cast<const T *>(A.v) + u * A.vs[0] + h * A.vs[1];
            for (int vec0 = 0; vec0 < n_vec; vec0 += 32) {    // which vector of the (K row, V row) pair
                const int vec = vec0 + lane;
                const bool on = vec < n_vec;
                const bool is_v = vec >= rv;
                const int c0 = on ? (is_v ? vec - rv : vec) * V : 0;
                const T *src = is_v ? vb : kb;
                const int64_t tstride = is_v ? A.vs[2] : A.ks[2];
                float acc[V];
#pragma unroll
                for (int e = 0; e < V; ++e) acc[e] = 0.f;
                float wsum = 0.f;
                uint4 xr = make_uint4(0, 0, 0, 0);
                if (on && part < 0) xr = load_raw16(src + (int64_t)cur.r * tstride + c0);    // the pivot row, early
                for (int t0 = 0; t0 < count; t0 += kMergeBatch) {
                    uint4 x[kMergeBatch];
                    int tok[kMergeBatch];
                    float w[kMergeBatch];
#pragma unroll
                    for (int q = 0; q < kMergeBatch; ++q) {   // this batch's positions and weights from the lanes that hold them
                        const int t = t0 + q;
                        tok[q] = __shfl_sync(0xFFFFFFFFu, t < 32 ? cur.tok_lo : cur.tok_hi, t & 31);
                        w[q] = __shfl_sync(0xFFFFFFFFu, t < 32 ? cur.w_lo : cur.w_hi, t & 31);
                    }
#pragma unroll
                    for (int q = 0; q < kMergeBatch; ++q)     // the batch's row loads, back to back
                        x[q] = (t0 + q < count && on) ? load_raw16(src + (int64_t)tok[q] * tstride + c0) : make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int q = 0; q < kMergeBatch; ++q) {   // fixed order: ascending member index
                        if (t0 + q < count) {
                            float xf[V];
                            Elem<T>::unpack(x[q], xf);
                            wsum += w[q];
#pragma unroll
                            for (int e = 0; e < V; ++e) acc[e] = fmaf(w[q], xf[e], acc[e]);
                        }
                    }
                }
                if (!on) continue;
                if (part < 0) {
                    T *dst = is_v ? static_cast<T *>(A.v_out) + u * A.vos[0] + h * A.vos[1] + (int64_t)slot * A.vos[2]
                                  : static_cast<T *>(A.k_out) + u * A.kos[0] + h * A.kos[1] + (int64_t)slot * A.kos[2];
                    if (count == 0) {
                        *reinterpret_cast<uint4 *>(dst + c0) = xr;   // nothing merged in: the pivot row, bit for bit
                    } else {
                        const float inv = 1.f / (1.f + wsum);
                        float xf[V], o[V];
                        Elem<T>::unpack(xr, xf);
#pragma unroll
                        for (int e = 0; e < V; ++e) o[e] = (xf[e] + acc[e]) * inv;
                        Elem<T>::store16(dst + c0, o);
                    }
                } else {
                    float *rec = A.partial + ((int64_t)uh * A.max_parts + part) * (2 * A.D + 4);
#pragma unroll
                    for (int e = 0; e < V; ++e) rec[(is_v ? A.D : 0) + c0 + e] = acc[e];
                    if (vec == 0) rec[2 * A.D] = wsum;
                }
            }
            if (part >= 0) {                                  // multi-piece slot: was this the last piece to arrive?
                __threadfence();
                __syncwarp();
                int prev = 0;
                if (lane == 0) prev = atomicAdd(&A.slot_done[(int64_t)uh * A.B + slot], 1);
                prev = __shfl_sync(0xFFFFFFFFu, prev, 0);
                const int *poff = A.piece_off + (int64_t)uh * (A.B + 1);
                if (prev == poff[slot + 1] - poff[slot] - 1) {
                    __threadfence();
                    merge_finish_slot<T>(A, uh, slot, lane);
                }
            }
        }
        cur = nxt;
        g = g_nxt;
        nxt.d = d2;
        g_nxt = g_d2;
    }
}

}  // namespace flowmm
