// Weighted merge (Eq. 5) + compaction, gather form, for rows of 256 bytes (bf16 at head_dim 128): the same
// pieces, order of accumulation and results as merge_pieces_kernel, with the member rows brought into shared
// memory by asynchronous bulk copies instead of register loads.
//
// merge_pieces_kernel is bound by latency: a warp has one batch of row loads in flight, then computes, then
// stores, and only then starts the next piece.  Here every warp owns two row buffers in shared memory and a
// pair of mbarriers; while it accumulates one batch (pivot row + up to 8 member rows, K and V side by side)
// the next batch - of the same piece or already of the next piece - is on its way (cp.async.bulk, 256 bytes
// per row and tensor, one copy per lane).  The rows cost no registers while in flight, so three CTAs of
// eight warps fit an SM and each warp keeps up to 9 KB coming.
#pragma once
#include "common.cuh"
#include "select_merge.cuh"
#include "tc_common.cuh"

namespace flowmm {
namespace mstg {

constexpr int kThreads = 256;
constexpr int kBatch = 8;                                    // member rows per batch
constexpr uint32_t kRowBytes = 512;                          // a token's K row and V row
constexpr uint32_t kBufBytes = (kBatch + 1) * kRowBytes;     // + the pivot row
constexpr uint32_t kWarpBytes = 2 * kBufBytes;
constexpr uint32_t kSmemBytes = (kThreads / 32) * kWarpBytes + (kThreads / 32) * 16 + 16;

template <typename T>
__global__ void __launch_bounds__(kThreads, 3) merge_staged_kernel(const MergeArgs A, int n_uh, int *status,
                                                                   const FastDiv by_pieces, const FastDiv by_hkv) {
    static_assert(sizeof(T) * 128 == 256 || sizeof(T) * 64 == 256, "rows of 256 bytes");
    constexpr int V = Elem<T>::kVec;
    extern __shared__ __align__(128) uint8_t mstg_smem[];
    const int lane = lane_id(), warp = threadIdx.x >> 5;
    const uint32_t bufs = tc::smem_u32(mstg_smem) + warp * kWarpBytes;
    const uint32_t bar0 = tc::smem_u32(mstg_smem) + (kThreads / 32) * kWarpBytes + warp * 16;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(mstg_smem + (kThreads / 32) * (kWarpBytes + 16));
    if (threadIdx.x == 0) *abort_flag = 0;
    if (lane == 0) {
        tc::mbar_init(bar0, 1);
        tc::mbar_init(bar0 + 8, 1);
        tc::mbar_init_fence();
    }
    __syncthreads();
    const unsigned total = (unsigned)n_uh * (unsigned)A.max_pieces;
    const bool is_v = lane >= 16;                             // lanes 0-15: the K row, 16-31: the V row, 16 bytes each
    const int c0 = (lane & 15) * V;

    struct Piece { int4 d; int tok_lo, tok_hi, r; float w_lo, w_hi; };
    auto fetch_desc = [&](unsigned g) -> int4 {              // (slot, first, count, part); count < 0: no such piece
        if (g >= total) return make_int4(0, 0, -1, -1);
        return A.piece_desc[g];
    };
    auto fetch_members = [&](unsigned g, Piece &pc) {        // needs pc.d
        pc.tok_lo = pc.tok_hi = pc.r = 0; pc.w_lo = pc.w_hi = 0.f;
        if (pc.d.z < 0) return;
        const int64_t uh = by_pieces.div(g);
        if (pc.d.z > 0) {
            const int *mt = A.mem_tok + uh * A.E + pc.d.y;
            const float *mw = A.mem_w + uh * A.E + pc.d.y;
            if (lane < pc.d.z) { pc.tok_lo = mt[lane]; pc.w_lo = mw[lane]; }
            if (lane + 32 < pc.d.z) { pc.tok_hi = mt[lane + 32]; pc.w_hi = mw[lane + 32]; }
        }
        if (pc.d.w < 0) pc.r = A.retained[uh * A.B + pc.d.x];
    };
    unsigned drawn = 0, drawn_left = 0;                       // pieces are drawn kDraw at a time from the shared counter
    constexpr unsigned kDraw = 4;
    auto next_piece = [&]() -> unsigned {
        if (drawn_left == 0) {
            unsigned g = 0;
            if (lane == 0) g = atomicAdd(A.ticket, kDraw);
            drawn = __shfl_sync(0xFFFFFFFFu, g, 0);
            drawn_left = kDraw;
        }
        --drawn_left;
        return drawn++;
    };
    // Starts the copies of batch `b` of a piece into buffer `j & 1` (j = batches this warp has started so far):
    // row slot 0 = the pivot (first batch of a single-piece slot only), slots 1.. = members 8 b .. 8 b + 7.
    // this lane's source rows (K for lanes 0-15, V for 16-31) and output rows of one (unit, head), kept until the head changes
    int src_uh = -1, dst_uh = -1;
    const T *src_base = nullptr;
    T *dst_base = nullptr;
    const int64_t tstride = is_v ? A.vs[2] : A.ks[2], ostride = is_v ? A.vos[2] : A.kos[2];
    auto issue = [&](const Piece &pc, unsigned g, int b, int j) {
        const int uh = (int)by_pieces.div(g);
        if (uh != src_uh) {
            const int u = (int)by_hkv.div(uh), h = uh - u * A.Hkv;
            src_base = is_v ? static_cast<const T *>(A.v) + u * A.vs[0] + h * A.vs[1]
                            : static_cast<const T *>(A.k) + u * A.ks[0] + h * A.ks[1];
            src_uh = uh;
        }
        const int n_mem = min(kBatch, pc.d.z - b * kBatch);
        const bool pivot = b == 0 && pc.d.w < 0;
        const uint32_t buf = bufs + (j & 1) * kBufBytes, bar = bar0 + (j & 1) * 8;
        // (the buffer was read by this warp two batches ago; order those reads before the copies' writes)
        __syncwarp();
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (lane == 0) tc::mbar_expect_tx(bar, (uint32_t)(n_mem + (pivot ? 1 : 0)) * kRowBytes);
        __syncwarp();
        // lane l < 16 copies a row's K part, lane 16 + l its V part: rows l = 0 .. 8 (0 = pivot)
        const int rowslot = lane & 15;
        const int t = b * kBatch + rowslot - 1;               // member index of this lane's row
        // (every lane asks for another member, so both halves of the list are offered and the asker picks)
        const int tok_a = __shfl_sync(0xFFFFFFFFu, pc.tok_lo, t & 31), tok_b = __shfl_sync(0xFFFFFFFFu, pc.tok_hi, t & 31);
        int tok = t < 32 ? tok_a : tok_b;
        bool go = rowslot >= 1 && rowslot <= n_mem;
        if (rowslot == 0) { tok = pc.r; go = pivot; }
        if (go && !index_ok(tok, A.L, status)) tok = 0;     // (debug build: a bad row number is recorded; row 0 stands in so that the byte count still arrives)
        if (go) tc::bulk_load(buf + rowslot * kRowBytes + (is_v ? 256u : 0u), src_base + (int64_t)tok * tstride, 256u, bar);
    };

    unsigned g = next_piece(), g_nxt = next_piece();
    Piece cur, nxt;
    cur.d = fetch_desc(g);
    nxt.d = fetch_desc(g_nxt);
    fetch_members(g, cur);
    int j = 0, jc = 0;                                        // batches started / taken so far
    bool started = false;                                     // the first batch of `cur` is already on its way
    bool ok = true;
    while (ok && g < total) {
        const unsigned g_d2 = next_piece();
        const int4 d2 = fetch_desc(g_d2);                     // two pieces ahead
        fetch_members(g_nxt, nxt);                            // one piece ahead
        const int slot = cur.d.x, count = cur.d.z, part = cur.d.w;
        bool next_started = false;
        if (count >= 0) {
            const int uh = (int)by_pieces.div(g);
            const int nb = count > 0 ? (count + kBatch - 1) / kBatch : 1;
            if (!started) { issue(cur, g, 0, j); ++j; }
            float acc[V];
#pragma unroll
            for (int e = 0; e < V; ++e) acc[e] = 0.f;
            float wsum = 0.f;
            uint4 xr = make_uint4(0, 0, 0, 0);
            for (int b = 0; ok && b < nb; ++b) {
                // the next batch starts before this one is worked on: of this piece, else the next piece's first
                if (b + 1 < nb) { issue(cur, g, b + 1, j); ++j; }
                else if (g_nxt < total && nxt.d.z >= 0) { issue(nxt, g_nxt, 0, j); ++j; next_started = true; }
                ok = tc::mbar_wait(bar0 + (jc & 1) * 8, (jc >> 1) & 1, abort_flag, status);
                if (!ok) break;
                const uint32_t buf = bufs + (jc & 1) * kBufBytes + lane * 16;
                ++jc;
                if (b == 0 && part < 0) {
                    const float4 f = tc::lds128(buf);
                    xr = make_uint4(__float_as_uint(f.x), __float_as_uint(f.y), __float_as_uint(f.z), __float_as_uint(f.w));
                }
                const int n_mem = min(kBatch, count - b * kBatch);
#pragma unroll
                for (int q = 0; q < kBatch; ++q) {            // fixed order: ascending member index
                    if (q < n_mem) {
                        const int t = b * kBatch + q;
                        const float w = __shfl_sync(0xFFFFFFFFu, t < 32 ? cur.w_lo : cur.w_hi, t & 31);
                        const float4 f = tc::lds128(buf + (q + 1) * kRowBytes);
                        float xf[V];
                        Elem<T>::unpack(make_uint4(__float_as_uint(f.x), __float_as_uint(f.y), __float_as_uint(f.z), __float_as_uint(f.w)), xf);
                        wsum += w;
#pragma unroll
                        for (int e = 0; e < V; ++e) acc[e] = fmaf(w, xf[e], acc[e]);
                    }
                }
            }
            if (!ok) break;
            if (part < 0) {
                if (uh != dst_uh) {
                    const int u = (int)by_hkv.div(uh), h = uh - u * A.Hkv;
                    dst_base = is_v ? static_cast<T *>(A.v_out) + u * A.vos[0] + h * A.vos[1]
                                    : static_cast<T *>(A.k_out) + u * A.kos[0] + h * A.kos[1];
                    dst_uh = uh;
                }
                T *dst = dst_base + (int64_t)slot * ostride;
                if (count == 0) {
                    *reinterpret_cast<uint4 *>(dst + c0) = xr;       // nothing merged in: the pivot row, bit for bit
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
                if (lane == 0) rec[2 * A.D] = wsum;
                // multi-piece slot: was this the last piece to arrive?
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
        started = next_started;
    }
    if (!ok) {               // winding down after a timeout: give copies already started a moment to land
        for (int b = 0; b < 2; ++b)
            for (int s = 0; s < (1 << 16) && !tc::mbar_try_wait(bar0 + b * 8, 0) && !tc::mbar_try_wait(bar0 + b * 8, 1); ++s) {}
    }
}

}  // namespace mstg
}  // namespace flowmm
