// C ABI of the FlowMM compression library: validation, workspace layout and kernel launches.
// Declarations and the meaning of every argument are in include/flowmm.h.
#include "flowmm.h"

#include <cuda_runtime.h>
#include <math.h>
#include <string.h>

#include <mutex>

#include "common.cuh"
#include "decode.cuh"
#include "decode_tc.cuh"
#include "match_small_tc.cuh"
#include "merge_staged.cuh"
#include "merge_tc.cuh"
#include "score_fused_tc.cuh"
#include "match_tc.cuh"
#include "score_tc.cuh"
#include "select_merge.cuh"
#include "simt_kernels.cuh"
#include "tc_host.cuh"

using namespace flowmm;

namespace {

thread_local int32_t g_launches = 0;

// Optional per-kernel timing: one event before the first kernel of an entry point, one after each.
constexpr int kMaxProfiled = 32;
struct Profile {
    bool on = false, have_events = false;
    cudaEvent_t ev[kMaxProfiled + 1];
    const char *name[kMaxProfiled];
    int n = 0;
};
thread_local Profile g_prof;

inline void profile_begin(cudaStream_t st) {
    g_launches = 0;
    g_prof.n = 0;
    if (g_prof.on) cudaEventRecord(g_prof.ev[0], st);
}
inline void profile_mark(const char *name, cudaStream_t st) {
    if (g_prof.on && g_prof.n < kMaxProfiled) {
        g_prof.name[g_prof.n] = name;
        cudaEventRecord(g_prof.ev[++g_prof.n], st);
    }
}

#define FLOWMM_LAUNCHED(name)                                          \
    do {                                                               \
        ++g_launches;                                                  \
        if (cudaGetLastError() != cudaSuccess) return FLOWMM_ERR_CUDA; \
        profile_mark(name, st);                                        \
    } while (0)

#define FLOWMM_TRY(expr)                         \
    do {                                         \
        const flowmm_status _s = (expr);         \
        if (_s != FLOWMM_OK) return _s;          \
    } while (0)

inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

// (unit, head) pairs per call: they index grid.x of several launches and 32-bit item counters
// (items = pairs x row tiles), so the bound is generous rather than a grid limit of 65535.
constexpr int64_t kMaxHeadsPerCall = 1 << 22;

// Where everything lives inside the caller's workspace.  One layout serves every entry point.
struct Layout {
    size_t status, importance, cross_mass, rho, strategy, retained, evicted, match, match_sim;
    size_t row_cross;          // flow-only statistics pass: the other-modality part of every partial row sum
    size_t row_part, cross_part, rn, sort_a, sort_b, mem_tok, mem_w, piece_desc, off, piece_off, part_off, partial, ticket, slot_done;
    size_t cand_k, cand_scale, cand_slot, cand_count, rank, tile_mod, negc;
    size_t tokmap;             // [UH, L] (slot, weight) of every token position, for the tensor-core merge
    size_t merge_status;       // status word the merge kernels report to (the workspace's own, or one of the merge scratch)
    int tc_n_qt, tc_n_chunk, tc_tiles_per_chunk, gw_pad;
    size_t total;
    int n_chunk1, chunk1, n_chunk2, chunk2, max_pieces, max_parts, csr_passes, c_tot, n_rt;
};

int chunks_for(int L, int other_ctas, int &chunk) {
    // enough CTAs to fill the GPU about twice, at least 64 keys per chunk
    int want = (2 * 148 + other_ctas - 1) / other_ctas;
    const int max_chunks = (L + kTile - 1) / kTile;
    if (want < 1) want = 1;
    if (want > max_chunks) want = max_chunks;
    chunk = ((L + want - 1) / want + kTile - 1) / kTile * kTile;
    return (L + chunk - 1) / chunk;
}

// The part of the workspace that the merge step uses (CSR of the match, piece table, partial sums).
template <class Take>
void layout_merge(Layout &y, const flowmm_params &p, Take take) {
    const size_t UH = (size_t)p.n_units * p.n_kv_heads, B = p.n_keep, E = (size_t)p.seq_len - B, D = p.head_dim;
    y.max_pieces = (int)(B + E / kPiece + 1);
    y.max_parts = (int)(2 * (E / kPiece) + 2);
    y.csr_passes = 1;                                        // digits of kCsrBits bits over the keys 0 .. B
    while (y.csr_passes < 6 && (B >> (kCsrBits * y.csr_passes)) != 0) ++y.csr_passes;
    y.sort_a = take(UH * E * 4);
    y.sort_b = take(UH * E * 4);
    y.mem_tok = take(UH * E * 4);
    y.mem_w = take(UH * E * 4);
    y.piece_desc = take(UH * (size_t)y.max_pieces * 16);
    y.off = take(UH * (B + 1) * 4);
    y.piece_off = take(UH * (B + 1) * 4);
    y.part_off = take(UH * (B + 1) * 4);
    y.partial = take(UH * (size_t)y.max_parts * (2 * D + 4) * 4);
    y.ticket = take(256);
    y.slot_done = take(UH * B * 4);
    y.merge_status = take(256);
    y.tokmap = take(UH * (size_t)p.seq_len * 8);
}

Layout make_layout(const flowmm_params &p) {
    Layout y;
    const size_t U = p.n_units, Hq = p.n_q_heads, Hkv = p.n_kv_heads, L = p.seq_len, W = p.window;
    const size_t B = p.n_keep, E = L - B, D = p.head_dim, G = Hq / Hkv;
    const int row_tiles = (int)((G * W + kTile - 1) / kTile);
    y.n_chunk1 = chunks_for((int)L, (int)(U * Hkv) * row_tiles, y.chunk1);
    y.n_chunk2 = chunks_for((int)L, (int)(U * Hkv), y.chunk2);
    size_t o = 0;
    auto take = [&](size_t bytes) { const size_t at = o; o += align256(bytes); return at; };
    y.status = take(256);
    y.importance = take(U * Hkv * L * 4);
    y.cross_mass = take(U * Hq * 4);
    y.rho = take(U * 4);
    y.strategy = take(U * 4);
    y.retained = take(U * Hkv * B * 4);
    y.evicted = take(U * Hkv * E * 4);
    y.match = take(U * Hkv * E * 4);
    y.match_sim = take(U * Hkv * E * 4);
    y.n_rt = (int)((L + tcs::kItemRows - 1) / tcs::kItemRows);
    {   // pass 1 of the tensor-core scoring: key chunks of whole 256-key tiles, sized so that the
        // persistent CTAs (one per SM, 148 on B200) finish their last round together
        y.tc_n_qt = (int)((G * W + tcs::kItemRows - 1) / tcs::kItemRows);
        const int key_tiles = (int)((L + tcs::Big::kCols - 1) / tcs::Big::kCols);
        const long base_items = (long)(U * Hkv) * y.tc_n_qt;
        double best_cost = 1e300;
        y.tc_tiles_per_chunk = key_tiles;
        for (int want = 1; want <= key_tiles; ++want) {
            const int tpc = (key_tiles + want - 1) / want;
            const int nc = (key_tiles + tpc - 1) / tpc;
            const long rounds = (base_items * nc + 147) / 148;
            const double cost = (double)rounds * (tpc + 0.75);     // 0.75 tile: per-item start-up
            if (cost < best_cost - 1e-9) { best_cost = cost; y.tc_tiles_per_chunk = tpc; }
        }
        y.tc_n_chunk = (key_tiles + y.tc_tiles_per_chunk - 1) / y.tc_tiles_per_chunk;
        y.gw_pad = (int)((G * W + tcs::Big::kCols - 1) / tcs::Big::kCols * tcs::Big::kCols);
    }
    const size_t max_chunk1 = (size_t)(y.n_chunk1 > 4 * y.tc_n_chunk ? y.n_chunk1 : 4 * y.tc_n_chunk);
    const size_t max_chunk2 = (size_t)(y.n_chunk2 > 8 * y.n_rt ? y.n_chunk2 : 8 * y.n_rt);
    y.row_part = take(U * Hq * W * max_chunk1 * 8);
    y.row_cross = take(U * Hq * W * max_chunk1 * 4);
    y.cross_part = take(U * Hq * max_chunk2 * 4);
    y.negc = take(U * Hkv * (size_t)y.gw_pad * 4);
    y.rn = take(U * Hkv * L * 4);
    layout_merge(y, p, take);
    y.merge_status = y.status;
    y.c_tot = (int)((B + 31) / 32 * 32 + 32);
    y.cand_k = take(U * Hkv * (size_t)y.c_tot * 128 * 2);
    y.cand_scale = take(U * Hkv * (size_t)y.c_tot * 4 + 1024);   // + one tile of slack: whole 256-column slices are copied
    y.cand_slot = take(U * Hkv * (size_t)y.c_tot * 4);
    y.cand_count = take(U * Hkv * 2 * 4);
    y.rank = take(U * Hkv * L * 4);
    y.tile_mod = take(U * (size_t)y.n_rt);
    y.total = o;
    return y;
}

flowmm_status validate(const flowmm_params *p) {
    if (!p) return FLOWMM_ERR_NULL;
    if (p->n_units < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1) return FLOWMM_ERR_SHAPE;
    if (p->n_q_heads % p->n_kv_heads != 0) return FLOWMM_ERR_SHAPE;
    if (p->head_dim != 64 && p->head_dim != 128) return FLOWMM_ERR_SHAPE;
    if (p->seq_len < 1 || p->window < 1 || p->window > p->seq_len) return FLOWMM_ERR_SHAPE;
    if ((int64_t)p->n_units * p->n_kv_heads > kMaxHeadsPerCall) return FLOWMM_ERR_SHAPE;
    {   // work items (pairs x 128-row tiles of the context x 128-row tiles of a head's proxy rows) are counted in 32 bits
        const int64_t tiles = (int64_t)p->n_units * p->n_kv_heads * ((p->seq_len + 127) / 128) *
                              (((int64_t)p->n_q_heads / p->n_kv_heads * p->window + 127) / 128);
        if (tiles > 0x7FFFFFFFll) return FLOWMM_ERR_SHAPE;
    }
    if (p->n_keep < 1 || p->n_keep > p->seq_len) return FLOWMM_ERR_BUDGET;
    if (p->keep_window && p->n_keep < p->window) return FLOWMM_ERR_BUDGET;
    if (p->dtype != FLOWMM_F32 && p->dtype != FLOWMM_BF16) return FLOWMM_ERR_DTYPE;
    if (p->tau_mode < 0 || p->tau_mode > 1 || p->flow_mode < 0 || p->flow_mode > 3 || p->merge_mode < 0 ||
        p->merge_mode > 1 || p->path < 0 || p->path > 1)
        return FLOWMM_ERR_SHAPE;
    if (!(p->softmax_scale >= 0.f) || isnan(p->theta) || isnan(p->tau)) return FLOWMM_ERR_SHAPE;
    return FLOWMM_OK;
}

bool strides_ok(const int64_t s[3], int head_dim) {
    for (int i = 0; i < 3; ++i)
        if (s[i] < 0 || s[i] % 8 != 0) return false;
    return s[2] >= head_dim;
}
bool aligned16(const void *ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15) == 0; }

flowmm_status check_device() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FLOWMM_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return FLOWMM_ERR_CUDA;
    return major == 10 ? FLOWMM_OK : FLOWMM_ERR_UNSUPPORTED_DEVICE;
}

flowmm_status check_ws(const flowmm_params *p, const void *ws, size_t ws_bytes, Layout &y) {
    if (!ws) return FLOWMM_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(ws) & 255) return FLOWMM_ERR_ALIGN;
    y = make_layout(*p);
    if (ws_bytes < y.total) return FLOWMM_ERR_WORKSPACE;
    return FLOWMM_OK;
}

template <typename X> X *at(void *ws, size_t off) { return reinterpret_cast<X *>(static_cast<char *>(ws) + off); }

float tau_effective(const flowmm_params &p) {
    return p.tau_mode == FLOWMM_TAU_REL ? (float)((double)p.tau * (double)p.window / (double)p.seq_len) : p.tau;
}

// ---- debug build: the index lists a caller hands in are checked before any kernel uses them ---------
#ifdef FLOWMM_DEBUG
// One block per (unit, head): pivots and non-pivots inside [0, L) and strictly ascending, matches inside [-1, B).
__global__ void debug_check_lists_kernel(const int32_t *retained, const int32_t *evicted, const int32_t *match,
                                         int L, int B, int E, int *status) {
    const int uh = blockIdx.x;
    bool bad = false;
    if (retained)
        for (int s = threadIdx.x; s < B; s += blockDim.x) {
            const int r = retained[(int64_t)uh * B + s];
            bad |= r < 0 || r >= L || (s > 0 && retained[(int64_t)uh * B + s - 1] >= r);
        }
    if (evicted)
        for (int j = threadIdx.x; j < E; j += blockDim.x) {
            const int e = evicted[(int64_t)uh * E + j];
            bad |= e < 0 || e >= L || (j > 0 && evicted[(int64_t)uh * E + j - 1] >= e);
        }
    if (match)
        for (int j = threadIdx.x; j < E; j += blockDim.x) {
            const int m = match[(int64_t)uh * E + j];
            bad |= m < -1 || m >= B;
        }
    if (bad) atomicCAS(status, 0, kStatusIndex);
}

// Runs the check, waits for it and reports: the entry point launches nothing else when a list is bad.
flowmm_status debug_check_lists(const flowmm_params &p, const int32_t *retained, const int32_t *evicted,
                                const int32_t *match, int *status, cudaStream_t st) {
    debug_check_lists_kernel<<<p.n_units * p.n_kv_heads, 256, 0, st>>>(retained, evicted, match, p.seq_len, p.n_keep,
                                                                        p.seq_len - p.n_keep, status);
    if (cudaGetLastError() != cudaSuccess) return FLOWMM_ERR_CUDA;
    int32_t word = 0;
    if (cudaMemcpyAsync(&word, status, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return FLOWMM_ERR_CUDA;
    return word == kStatusIndex ? FLOWMM_ERR_INDEX : FLOWMM_OK;
}
#define FLOWMM_DEBUG_LISTS(p, ret, evi, mt, status, st) FLOWMM_TRY(debug_check_lists(p, ret, evi, mt, status, st))
#else
#define FLOWMM_DEBUG_LISTS(p, ret, evi, mt, status, st) do { } while (0)
#endif

// ---- step launchers (no validation; the entry points below validate) --------------------------

bool use_tc(const flowmm_params &p) {
    return p.path == FLOWMM_PATH_AUTO && p.dtype == FLOWMM_BF16 && p.head_dim == 128;
}
bool use_tc_score(const flowmm_params &p) {
    const int gw = p.n_q_heads / p.n_kv_heads * p.window;
    return use_tc(p) && (p.window == 32 || p.window == 64 || p.window == 128) && gw <= 1024;
}

flowmm_status run_score_tc(const flowmm_params &p, const Layout &y, const void *q, const void *k, const uint8_t *mod,
                           float *importance, float *cross_mass, void *ws, cudaStream_t st, int *parts_out) {
    const int UH = p.n_units * p.n_kv_heads, G = p.n_q_heads / p.n_kv_heads, W = p.window;
    ScoreTcArgs a;
    a.row_part = at<float2>(ws, y.row_part); a.negc = at<float>(ws, y.negc); a.modality = mod;
    a.importance = importance; a.cross_part = at<float>(ws, y.cross_part); a.status = at<int>(ws, y.status);
    a.Hq = p.n_q_heads; a.Hkv = p.n_kv_heads; a.G = G; a.W = W; a.L = p.seq_len; a.GW = G * W; a.GWpad = y.gw_pad;
    a.n_qt = y.tc_n_qt; a.n_chunk = y.tc_n_chunk; a.tiles_per_chunk = y.tc_tiles_per_chunk; a.n_rt = y.n_rt;
    a.a_heads = G < tcs::kRows / W ? G : tcs::kRows / W;        // one A half holds 128 proxy rows
    // pass 2 streams the keys as the A operand; with few proxy rows per KV head the small shape (two A stages)
    // keeps the key loads in flight across items
    const bool small2 = a.GW <= 128 && W <= 64;
    const int nb2 = small2 ? tcs::Small::kCols : tcs::Big::kCols;
    a.b_heads = G < nb2 / W ? G : nb2 / W;
    a.n_items1 = UH * a.n_qt * a.n_chunk; a.n_items2 = UH * a.n_rt;
    const float scale = p.softmax_scale != 0.f ? p.softmax_scale : 1.f / sqrtf((float)p.head_dim);
    a.scale_log2 = scale * kLog2e;

    CUtensorMap qa, qb, k128, k256;
    const uint64_t qd[4] = {128, (uint64_t)W, (uint64_t)p.n_q_heads, (uint64_t)p.n_units};
    const uint64_t qs[3] = {(uint64_t)p.q_stride[2] * 2, (uint64_t)p.q_stride[1] * 2, (uint64_t)p.q_stride[0] * 2};
    const uint64_t kd[4] = {128, (uint64_t)p.seq_len, (uint64_t)p.n_kv_heads, (uint64_t)p.n_units};
    const uint64_t ks[3] = {(uint64_t)p.k_stride[2] * 2, (uint64_t)p.k_stride[1] * 2, (uint64_t)p.k_stride[0] * 2};
    const uint32_t bqa[4] = {64, (uint32_t)W, (uint32_t)a.a_heads, 1}, bqb[4] = {64, (uint32_t)W, (uint32_t)a.b_heads, 1};
    const uint32_t bk128[4] = {64, tcs::kRows, 1, 1}, bk256[4] = {64, tcs::Big::kCols, 1, 1};
    if (!tc::make_bf16_map(&qa, q, 4, qd, qs, bqa) || !tc::make_bf16_map(&qb, q, 4, qd, qs, bqb) ||
        !tc::make_bf16_map(&k128, k, 4, kd, ks, bk128) || !tc::make_bf16_map(&k256, k, 4, kd, ks, bk256))
        return FLOWMM_ERR_CUDA;
    if (cudaFuncSetAttribute(score_stats_tc_kernel<tcs::Big>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tcs::Big::kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(score_colsum_tc_kernel<tcs::Big>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tcs::Big::kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(score_colsum_tc_kernel<tcs::Small>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tcs::Small::kSmemBytes) != cudaSuccess)
        return FLOWMM_ERR_CUDA;
    const int sms = tc::sm_count();
    score_stats_tc_kernel<tcs::Big><<<a.n_items1 < sms ? a.n_items1 : sms, tcs::kThreads, tcs::Big::kSmemBytes, st>>>(qa, k256, a);
    FLOWMM_LAUNCHED("score_stats_tc");
    const int n_negc = UH * a.GWpad;
    score_combine_kernel<<<(n_negc + 255) / 256, 256, 0, st>>>(a.row_part, 4 * a.n_chunk, a.GW, a.GWpad, UH, a.negc);
    FLOWMM_LAUNCHED("score_combine");
    if (small2)
        score_colsum_tc_kernel<tcs::Small><<<a.n_items2 < sms ? a.n_items2 : sms, tcs::kThreads, tcs::Small::kSmemBytes, st>>>(k128, qb, a);
    else
        score_colsum_tc_kernel<tcs::Big><<<a.n_items2 < sms ? a.n_items2 : sms, tcs::kThreads, tcs::Big::kSmemBytes, st>>>(k128, qb, a);
    FLOWMM_LAUNCHED("score_colsum_tc");
    if (parts_out) { *parts_out = a.n_rt * 8; return FLOWMM_OK; }     // the caller reduces the partial masses itself
    const int n = p.n_units * p.n_q_heads;
    cross_mass_reduce<<<(n + 7) / 8, 256, 0, st>>>(a.cross_part, a.n_rt * 8, n, cross_mass);
    FLOWMM_LAUNCHED("cross_mass_reduce");
    return FLOWMM_OK;
}

// Short contexts with 32 proxy rows per KV head: every logit of a head fits in half of TMEM, K is read once.
bool use_fused_score(const flowmm_params &p) {
    const int gw = p.n_q_heads / p.n_kv_heads * p.window, nt = (p.seq_len + sft::kTile - 1) / sft::kTile;
    return use_tc(p) && gw == sft::kRows && nt <= sft::kMaxTiles;
}

flowmm_status run_score_fused(const flowmm_params &p, const Layout &y, const void *q, const void *k, const uint8_t *mod,
                              float *importance, float *cross_mass, void *ws, cudaStream_t st) {
    const int UH = p.n_units * p.n_kv_heads, G = p.n_q_heads / p.n_kv_heads, W = p.window;
    CUtensorMap qmap, kmap;
    const uint64_t qd[4] = {128, (uint64_t)W, (uint64_t)p.n_q_heads, (uint64_t)p.n_units};
    const uint64_t qs[3] = {(uint64_t)p.q_stride[2] * 2, (uint64_t)p.q_stride[1] * 2, (uint64_t)p.q_stride[0] * 2};
    const uint64_t kd[4] = {128, (uint64_t)p.seq_len, (uint64_t)p.n_kv_heads, (uint64_t)p.n_units};
    const uint64_t ks[3] = {(uint64_t)p.k_stride[2] * 2, (uint64_t)p.k_stride[1] * 2, (uint64_t)p.k_stride[0] * 2};
    const uint32_t bq[4] = {64, (uint32_t)W, (uint32_t)G, 1}, bk[4] = {64, sft::kTile, 1, 1};
    if (!tc::make_bf16_map(&qmap, q, 4, qd, qs, bq) || !tc::make_bf16_map(&kmap, k, 4, kd, ks, bk)) return FLOWMM_ERR_CUDA;
    sft::Args a;
    a.modality = mod; a.importance = importance; a.cross_mass = cross_mass; a.status = at<int>(ws, y.status);
    a.Hq = p.n_q_heads; a.Hkv = p.n_kv_heads; a.G = G; a.W = W; a.L = p.seq_len; a.n_items = UH;
    const float scale = p.softmax_scale != 0.f ? p.softmax_scale : 1.f / sqrtf((float)p.head_dim);
    a.scale_log2 = scale * kLog2e;
    if (cudaFuncSetAttribute(sft::score_fused_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)sft::kSmemBytes) != cudaSuccess)
        return FLOWMM_ERR_CUDA;
    const int grid = UH < tc::sm_count() ? UH : tc::sm_count();
    sft::score_fused_tc_kernel<<<grid, sft::kThreads, sft::kSmemBytes, st>>>(qmap, kmap, a);
    FLOWMM_LAUNCHED("score_fused_tc");
    return FLOWMM_OK;
}

// parts_out: the caller reduces the partial cross-modal masses itself; set to 0 when cross_mass is already final
flowmm_status run_score(const flowmm_params &p, const Layout &y, const void *q, const void *k, const uint8_t *mod,
                        float *importance, float *cross_mass, void *ws, cudaStream_t st, int *parts_out = nullptr) {
    if (use_fused_score(p)) {
        if (parts_out) *parts_out = 0;
        return run_score_fused(p, y, q, k, mod, importance, cross_mass, ws, st);
    }
    if (use_tc_score(p)) return run_score_tc(p, y, q, k, mod, importance, cross_mass, ws, st, parts_out);
    ScoreArgs a;
    a.q = q; a.k = k; a.modality = mod; a.importance = importance;
    a.row_part = at<float2>(ws, y.row_part);
    a.cross_part = at<float>(ws, y.cross_part);
    a.Hq = p.n_q_heads; a.Hkv = p.n_kv_heads; a.G = p.n_q_heads / p.n_kv_heads;
    a.D = p.head_dim; a.L = p.seq_len; a.W = p.window;
    a.n_chunk1 = y.n_chunk1; a.chunk1 = y.chunk1; a.n_chunk2 = y.n_chunk2; a.chunk2 = y.chunk2;
    const float scale = p.softmax_scale != 0.f ? p.softmax_scale : 1.f / sqrtf((float)p.head_dim);
    a.scale_log2 = scale * kLog2e;
    for (int i = 0; i < 3; ++i) { a.qs[i] = p.q_stride[i]; a.ks[i] = p.k_stride[i]; }
    const int GW = a.G * a.W;
    const int UH = p.n_units * p.n_kv_heads;
    const dim3 g1(UH, (GW + kTile - 1) / kTile, y.n_chunk1), g2(UH, y.n_chunk2);
    const size_t dyn = (size_t)3 * GW * sizeof(float);
    if (p.dtype == FLOWMM_BF16) {
        score_stats_simt<__nv_bfloat16><<<g1, kSimtThreads, 0, st>>>(a);
        FLOWMM_LAUNCHED("score_stats_simt");
        score_colsum_simt<__nv_bfloat16><<<g2, kSimtThreads, dyn, st>>>(a);
        FLOWMM_LAUNCHED("score_colsum_simt");
    } else {
        score_stats_simt<float><<<g1, kSimtThreads, 0, st>>>(a);
        FLOWMM_LAUNCHED("score_stats_simt");
        score_colsum_simt<float><<<g2, kSimtThreads, dyn, st>>>(a);
        FLOWMM_LAUNCHED("score_colsum_simt");
    }
    if (parts_out) { *parts_out = y.n_chunk2; return FLOWMM_OK; }
    const int n = p.n_units * p.n_q_heads;
    cross_mass_reduce<<<(n + 7) / 8, 256, 0, st>>>(a.cross_part, y.n_chunk2, n, cross_mass);
    FLOWMM_LAUNCHED("cross_mass_reduce");
    return FLOWMM_OK;
}

flowmm_status run_layer_flow(const flowmm_params &p, const float *cross_mass, float *rho, int32_t *strategy,
                             cudaStream_t st) {
    layer_flow_kernel<<<(p.n_units + 127) / 128, 128, 0, st>>>(cross_mass, p.n_units, p.n_q_heads, p.window, p.theta,
                                                                p.flow_mode, rho, strategy);
    FLOWMM_LAUNCHED("layer_flow");
    return FLOWMM_OK;
}

// What the preparation of the tensor-core matching step needs (candidate layout per head; see match_tc.cuh).
MatchPrepArgs match_prep_args(const flowmm_params &p, const Layout &y, const void *k, const float *importance,
                              const uint8_t *mod, const int32_t *retained, const int32_t *evicted, void *ws) {
    MatchPrepArgs g;
    g.k = k; g.importance = importance; g.modality = mod;
    g.retained = retained; g.evicted = evicted;
    g.cand_k = at<__nv_bfloat16>(ws, y.cand_k); g.cand_scale = at<float>(ws, y.cand_scale);
    g.cand_slot = at<int>(ws, y.cand_slot); g.cand_count = at<int>(ws, y.cand_count);
    g.rank = at<int>(ws, y.rank); g.tile_mod = at<uint8_t>(ws, y.tile_mod);
    g.Hkv = p.n_kv_heads; g.L = p.seq_len; g.B = p.n_keep; g.E = p.seq_len - p.n_keep; g.Ctot = y.c_tot; g.n_rt = y.n_rt;
    g.tau_eff = tau_effective(p);
    for (int i = 0; i < 3; ++i) g.ks[i] = p.k_stride[i];
    g.copy_here = y.c_tot <= 256;
    g.status = at<int>(ws, y.status);
    return g;
}

// cross_mass != nullptr: the launch also applies Eq. 6 and the theta rule to the final masses (rho may be nullptr)
// prep != nullptr: each block goes on to prepare its head's matching candidates (the fused call, tensor-core matching)
flowmm_status run_select(const flowmm_params &p, const float *importance, int32_t *retained, int32_t *evicted,
                         cudaStream_t st, float *cross_mass = nullptr, float *rho = nullptr,
                         int32_t *strategy = nullptr, const float *cross_part = nullptr, int n_parts = 0,
                         const MatchPrepArgs *prep = nullptr) {
    const int few = p.n_units * p.n_kv_heads < 2 * tc::sm_count();       // few heads: more threads per head
    const int threads = few ? (p.seq_len <= 512 ? 256 : kSelectThreads) : p.seq_len <= 2048 ? 256 : p.seq_len <= 8192 ? 512 : kSelectThreads;
    SelectFlow f;
    f.cross_part = cross_part; f.n_parts = n_parts; f.cross_mass = cross_mass; f.rho = rho; f.strategy = strategy; f.Hq = p.n_q_heads; f.Hkv = p.n_kv_heads;
    f.theta = p.theta; f.flow_mode = p.flow_mode;
    MatchPrepArgs none = {};
    select_topb_kernel<<<p.n_units * p.n_kv_heads, threads, 0, st>>>(importance, p.seq_len, p.n_keep, p.window,
                                                                           p.keep_window, retained, evicted, f,
                                                                           prep ? *prep : none, prep ? 1 : 0);
    FLOWMM_LAUNCHED("select_topb");
    return FLOWMM_OK;
}


flowmm_status run_match_tc(const flowmm_params &p, const Layout &y, const void *k, const float *importance,
                           const uint8_t *mod, const int32_t *retained, const int32_t *evicted,
                           const int32_t *strategy, int32_t *match, float *match_sim, void *ws, cudaStream_t st,
                           int2 *tokmap, bool prepared) {
    const int UH = p.n_units * p.n_kv_heads, E = p.seq_len - p.n_keep;
    const MatchPrepArgs g = match_prep_args(p, y, k, importance, mod, retained, evicted, ws);
    if (!prepared) {                                 // (the fused call's selection launch has done it already)
        // few heads: a head's lists are walked by more threads, the GPU is not full either way
        const int prep_threads = UH >= 4 * tc::sm_count() ? 256 : UH >= 2 * tc::sm_count() ? 512 : 1024;
        match_prepare_kernel<<<UH, prep_threads, 0, st>>>(g);
        FLOWMM_LAUNCHED("match_prepare");
    }
    if (!g.copy_here) {
        match_gather_kernel<<<dim3(UH, (y.c_tot + 63) / 64), 256, 0, st>>>(g);
        FLOWMM_LAUNCHED("match_gather");
    }

    CUtensorMap k_map, cand_map;
    const uint64_t kd[4] = {128, (uint64_t)p.seq_len, (uint64_t)p.n_kv_heads, (uint64_t)p.n_units};
    const uint64_t ks[3] = {(uint64_t)p.k_stride[2] * 2, (uint64_t)p.k_stride[1] * 2, (uint64_t)p.k_stride[0] * 2};
    const uint64_t cd[4] = {128, (uint64_t)y.c_tot, (uint64_t)UH, 1};
    const uint64_t cs[3] = {256, (uint64_t)y.c_tot * 256, (uint64_t)y.c_tot * 256 * (uint64_t)UH};
    if (y.c_tot <= mst::kMaxCols) {      // the whole candidate list of a head is one operand tile
        const uint32_t box_t[4] = {64, mst::kTile, 1, 1}, box_c[4] = {64, (uint32_t)y.c_tot, 1, 1};
        if (!tc::make_bf16_map(&k_map, k, 4, kd, ks, box_t) || !tc::make_bf16_map(&cand_map, g.cand_k, 4, cd, cs, box_c))
            return FLOWMM_ERR_CUDA;
        mst::Args a;
        a.cand_count = g.cand_count; a.cand_slot = g.cand_slot; a.rank = g.rank; a.strategy = strategy;
        a.cand_scale = g.cand_scale; a.modality = mod; a.match = match; a.match_sim = match_sim;
        a.tokmap = tokmap; a.merge_mode = p.merge_mode;
        a.status = at<int>(ws, y.status);
        a.Hkv = p.n_kv_heads; a.L = p.seq_len; a.E = E; a.Ctot = y.c_tot; a.n_heads = UH;
        if (cudaFuncSetAttribute(mst::match_small_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)mst::kSmemBytes) != cudaSuccess)
            return FLOWMM_ERR_CUDA;
        mst::match_small_tc_kernel<<<UH < tc::sm_count() ? UH : tc::sm_count(), mst::kThreads, mst::kSmemBytes, st>>>(k_map, cand_map, a);
        FLOWMM_LAUNCHED("match_small_tc");
        return FLOWMM_OK;
    }
    // few candidates per head: the token rows are the stream, take the shape with two A stages
    const bool small = y.c_tot <= 128;
    const uint32_t box_a[4] = {64, kMtRows, 1, 1};
    const uint32_t box_b[4] = {64, (uint32_t)(small ? tcs::Small::kCols : tcs::Big::kCols), 1, 1};
    if (!tc::make_bf16_map(&k_map, k, 4, kd, ks, box_a) || !tc::make_bf16_map(&cand_map, g.cand_k, 4, cd, cs, box_b))
        return FLOWMM_ERR_CUDA;
    MatchTcArgs a;
    a.cand_count = g.cand_count; a.cand_slot = g.cand_slot; a.rank = g.rank; a.strategy = strategy;
    a.cand_scale = g.cand_scale; a.modality = mod; a.tile_mod = g.tile_mod;
    a.match = match; a.match_sim = match_sim; a.status = at<int>(ws, y.status);
    a.Hkv = p.n_kv_heads; a.L = p.seq_len; a.E = E; a.Ctot = y.c_tot; a.n_rt = y.n_rt; a.n_items = UH * y.n_rt;
    a.by_nrt = make_fastdiv((uint32_t)y.n_rt); a.by_hkv = make_fastdiv((uint32_t)p.n_kv_heads);
    if (cudaFuncSetAttribute(match_tc_kernel<tcs::Big>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tcs::Big::kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(match_tc_kernel<tcs::Small>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tcs::Small::kSmemBytes) != cudaSuccess)
        return FLOWMM_ERR_CUDA;
    const int grid = a.n_items < tc::sm_count() ? a.n_items : tc::sm_count();
    if (small) match_tc_kernel<tcs::Small><<<grid, tcs::kThreads, tcs::Small::kSmemBytes, st>>>(k_map, cand_map, a);
    else match_tc_kernel<tcs::Big><<<grid, tcs::kThreads, tcs::Big::kSmemBytes, st>>>(k_map, cand_map, a);
    FLOWMM_LAUNCHED("match_tc");
    return FLOWMM_OK;
}

// tokmap != nullptr (only with the short-list tensor-core kernel): also write the tensor-core merge's table
flowmm_status run_match(const flowmm_params &p, const Layout &y, const void *k, const float *importance,
                        const uint8_t *mod, const int32_t *retained, const int32_t *evicted, const int32_t *strategy,
                        int32_t *match, float *match_sim, void *ws, cudaStream_t st, int2 *tokmap = nullptr,
                        bool prepared = false) {
    const int E = p.seq_len - p.n_keep;
    if (E == 0) return FLOWMM_OK;
    if (use_tc(p)) return run_match_tc(p, y, k, importance, mod, retained, evicted, strategy, match, match_sim, ws, st, tokmap, prepared);
    float *rn = at<float>(ws, y.rn);
    const int64_t rows = (int64_t)p.n_units * p.n_kv_heads * p.seq_len;
    const int lanes = p.head_dim / (p.dtype == FLOWMM_BF16 ? 8 : 4);
    const int64_t threads = rows * lanes;
    const unsigned blocks = (unsigned)((threads + 255) / 256);
    if (p.dtype == FLOWMM_BF16)
        inv_norm_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(k, rows, p.n_kv_heads, p.seq_len, p.head_dim,
                                                               p.k_stride[0], p.k_stride[1], p.k_stride[2], rn);
    else
        inv_norm_kernel<float><<<blocks, 256, 0, st>>>(k, rows, p.n_kv_heads, p.seq_len, p.head_dim, p.k_stride[0],
                                                       p.k_stride[1], p.k_stride[2], rn);
    FLOWMM_LAUNCHED("inv_norm");
    MatchArgs a;
    a.k = k; a.importance = importance; a.modality = mod; a.retained = retained; a.evicted = evicted;
    a.strategy = strategy; a.rn = rn; a.match = match; a.match_sim = match_sim;
    a.Hkv = p.n_kv_heads; a.D = p.head_dim; a.L = p.seq_len; a.B = p.n_keep; a.E = E;
    a.tau_eff = tau_effective(p);
    for (int i = 0; i < 3; ++i) a.ks[i] = p.k_stride[i];
    const dim3 grid(p.n_units * p.n_kv_heads, (E + kTile - 1) / kTile);
    if (p.dtype == FLOWMM_BF16) match_simt<__nv_bfloat16><<<grid, kSimtThreads, 0, st>>>(a);
    else match_simt<float><<<grid, kSimtThreads, 0, st>>>(a);
    FLOWMM_LAUNCHED("match_simt");
    return FLOWMM_OK;
}

// Few slots per head: Eq. 5 as a product with the slot-by-token weight matrix on the tensor cores.
// (Below 65536 tokens a slot's fixed-point weight sum cannot overflow.)
bool merge_is_tc(const flowmm_params &p) {
    return p.seq_len > p.n_keep && p.dtype == FLOWMM_BF16 && p.head_dim == 128 && p.n_keep <= mtc::kMaxSlots &&
           p.seq_len < 65536 && p.path != FLOWMM_PATH_SIMT;
}

// map_ready: the (slot, weight) table of the tensor-core merge has been written already (by the matching kernel)
flowmm_status run_merge(const flowmm_params &p, const Layout &y, const void *k, const void *v,
                        const int32_t *retained, const int32_t *evicted, const int32_t *match, const float *match_sim,
                        void *k_out, void *v_out, void *ws, cudaStream_t st, bool map_ready = false) {
    const int E = p.seq_len - p.n_keep, UH = p.n_units * p.n_kv_heads;
    MergeArgs m;
    m.k = k; m.v = v; m.k_out = k_out; m.v_out = v_out; m.retained = retained;
    m.mem_tok = nullptr; m.mem_w = nullptr; m.piece_desc = nullptr; m.piece_off = nullptr; m.part_off = nullptr;
    m.partial = at<float>(ws, y.partial); m.ticket = nullptr; m.slot_done = nullptr;
    m.Hkv = p.n_kv_heads; m.D = p.head_dim; m.L = p.seq_len; m.B = p.n_keep; m.E = E;
    m.max_pieces = E == 0 ? p.n_keep : y.max_pieces; m.max_parts = y.max_parts;
    for (int i = 0; i < 3; ++i) {
        m.ks[i] = p.k_stride[i]; m.vs[i] = p.v_stride[i]; m.kos[i] = p.ko_stride[i]; m.vos[i] = p.vo_stride[i];
    }
    // few slots per head: Eq. 5 as a product with the slot-by-token weight matrix on the tensor cores
    if (merge_is_tc(p)) {
        mtc::MapArgs ma;
        ma.retained = retained; ma.evicted = evicted; ma.match = match; ma.match_sim = match_sim;
        ma.tokmap = at<int2>(ws, y.tokmap); ma.L = p.seq_len; ma.B = p.n_keep; ma.E = E; ma.merge_mode = p.merge_mode;
        const int longest = E > p.n_keep ? E : p.n_keep;
        if (!map_ready) {
            mtc::merge_map_kernel<<<dim3(UH, (longest + 255) / 256), 256, 0, st>>>(ma);
            FLOWMM_LAUNCHED("merge_map");
        }
        CUtensorMap kmap, vmap;
        const uint64_t dims[4] = {128, (uint64_t)p.seq_len, (uint64_t)p.n_kv_heads, (uint64_t)p.n_units};
        const uint64_t ksb[3] = {(uint64_t)p.k_stride[2] * 2, (uint64_t)p.k_stride[1] * 2, (uint64_t)p.k_stride[0] * 2};
        const uint64_t vsb[3] = {(uint64_t)p.v_stride[2] * 2, (uint64_t)p.v_stride[1] * 2, (uint64_t)p.v_stride[0] * 2};
        const uint32_t box[4] = {64, mtc::kTile, 1, 1};
        if (!tc::make_bf16_map(&kmap, k, 4, dims, ksb, box) || !tc::make_bf16_map(&vmap, v, 4, dims, vsb, box))
            return FLOWMM_ERR_CUDA;
        mtc::Args a;
        a.tokmap = ma.tokmap; a.k_out = k_out; a.v_out = v_out; a.status = at<int>(ws, y.merge_status);
        a.Hkv = p.n_kv_heads; a.L = p.seq_len; a.B = p.n_keep; a.n_items = UH; a.n_stages = p.n_keep <= 128 ? mtc::kMaxStages : 3;
        for (int i = 0; i < 3; ++i) { a.kos[i] = p.ko_stride[i]; a.vos[i] = p.vo_stride[i]; }
        const uint32_t smem = mtc::smem_bytes(p.n_keep, a.n_stages);
        if (cudaFuncSetAttribute(mtc::merge_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return FLOWMM_ERR_CUDA;
        const int grid = UH < tc::sm_count() ? UH : tc::sm_count();
        mtc::merge_tc_kernel<<<grid, mtc::kThreads, smem, st>>>(kmap, vmap, a);
        FLOWMM_LAUNCHED("merge_tc");
        return FLOWMM_OK;
    }
    if (E > 0) {
        CsrArgs c;
        c.match = match; c.evicted = evicted; c.match_sim = match_sim;
        c.sort_a = at<int>(ws, y.sort_a); c.sort_b = at<int>(ws, y.sort_b);
        c.mem_tok = at<int>(ws, y.mem_tok); c.mem_w = at<float>(ws, y.mem_w);
        c.off = at<int>(ws, y.off); c.piece_off = at<int>(ws, y.piece_off); c.part_off = at<int>(ws, y.part_off);
        c.piece_desc = at<int4>(ws, y.piece_desc); c.ticket = at<unsigned>(ws, y.ticket); c.slot_done = at<int>(ws, y.slot_done);
        c.B = p.n_keep; c.E = E; c.n_pass = y.csr_passes; c.max_pieces = y.max_pieces; c.merge_mode = p.merge_mode;
        // positions and keys as 16-bit arrays in shared memory when they fit (6 bytes per non-pivot), else through global memory
        const size_t csr_smem = 6 * (((size_t)E + 7) & ~(size_t)7);
        const bool staged = E < 65536 && p.n_keep < 65535 && csr_smem <= 200 * 1024;
        if (staged) {
            if (E <= 4096) {
                if (cudaFuncSetAttribute(build_csr_kernel<8, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)csr_smem) != cudaSuccess) return FLOWMM_ERR_CUDA;
                build_csr_kernel<8, true><<<UH, 256, csr_smem, st>>>(c);
            } else {
                if (cudaFuncSetAttribute(build_csr_kernel<32, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)csr_smem) != cudaSuccess) return FLOWMM_ERR_CUDA;
                build_csr_kernel<32, true><<<UH, 1024, csr_smem, st>>>(c);
            }
        } else if (E <= 4096) build_csr_kernel<8, false><<<UH, 256, 0, st>>>(c);
        else build_csr_kernel<32, false><<<UH, 1024, 0, st>>>(c);
        FLOWMM_LAUNCHED("build_csr");
        m.mem_tok = c.mem_tok; m.mem_w = c.mem_w; m.piece_desc = c.piece_desc;
        m.piece_off = c.piece_off; m.part_off = c.part_off; m.ticket = c.ticket; m.slot_done = c.slot_done;
    }
    const int64_t total_pieces = (int64_t)UH * m.max_pieces;
    if (total_pieces > 0xFFFF0000ll) return FLOWMM_ERR_SHAPE;           // the piece table is indexed with 32 bits
    const int64_t want_blocks = (total_pieces + 7) / 8;
    const int gp = (int)(want_blocks < 2 * tc::sm_count() ? want_blocks : 2 * tc::sm_count());   // persistent warps
    if (p.dtype == FLOWMM_BF16 && p.head_dim == 128 && E > 0 && p.path != FLOWMM_PATH_SIMT) {
        // rows of 256 bytes: member rows staged through shared memory by asynchronous copies, three CTAs per SM
        if (cudaFuncSetAttribute(mstg::merge_staged_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)mstg::kSmemBytes) != cudaSuccess)
            return FLOWMM_ERR_CUDA;
        const int gs = (int)(want_blocks < 3 * tc::sm_count() ? want_blocks : 3 * tc::sm_count());
        mstg::merge_staged_kernel<__nv_bfloat16><<<gs, mstg::kThreads, mstg::kSmemBytes, st>>>(
            m, UH, at<int>(ws, y.merge_status), make_fastdiv((uint32_t)m.max_pieces), make_fastdiv((uint32_t)p.n_kv_heads));
        FLOWMM_LAUNCHED("merge_staged");
    } else if (p.dtype == FLOWMM_BF16) {
        merge_pieces_kernel<__nv_bfloat16><<<gp, 256, 0, st>>>(m, UH);
        FLOWMM_LAUNCHED("merge_pieces");
    } else {
        merge_pieces_kernel<float><<<gp, 256, 0, st>>>(m, UH);
        FLOWMM_LAUNCHED("merge_pieces");
    }
    return FLOWMM_OK;
}

}  // namespace

extern "C" {

flowmm_status flowmm_workspace_bytes(const flowmm_params *p, size_t *bytes) {
    if (!bytes) return FLOWMM_ERR_NULL;
    FLOWMM_TRY(validate(p));
    *bytes = make_layout(*p).total;
    return FLOWMM_OK;
}

flowmm_status flowmm_score(const flowmm_params *p, const void *q_win, const void *k, const uint8_t *modality,
                           float *importance, float *cross_mass, void *ws, size_t ws_bytes, void *cuda_stream) {
    profile_begin(static_cast<cudaStream_t>(cuda_stream));
    FLOWMM_TRY(validate(p));
    if (!q_win || !k || !modality || !importance || !cross_mass) return FLOWMM_ERR_NULL;
    if (!aligned16(q_win) || !aligned16(k) || !strides_ok(p->q_stride, p->head_dim) ||
        !strides_ok(p->k_stride, p->head_dim))
        return FLOWMM_ERR_ALIGN;
    Layout y;
    FLOWMM_TRY(check_ws(p, ws, ws_bytes, y));
    FLOWMM_TRY(check_device());
    return run_score(*p, y, q_win, k, modality, importance, cross_mass, ws, static_cast<cudaStream_t>(cuda_stream));
}

flowmm_status flowmm_layer_flow(const flowmm_params *p, const float *cross_mass, float *rho, int32_t *strategy,
                                void *cuda_stream) {
    profile_begin(static_cast<cudaStream_t>(cuda_stream));
    FLOWMM_TRY(validate(p));
    if (!cross_mass || !rho || !strategy) return FLOWMM_ERR_NULL;
    FLOWMM_TRY(check_device());
    return run_layer_flow(*p, cross_mass, rho, strategy, static_cast<cudaStream_t>(cuda_stream));
}

flowmm_status flowmm_select(const flowmm_params *p, const float *importance, int32_t *retained_idx,
                            int32_t *evicted_idx, void *ws, size_t ws_bytes, void *cuda_stream) {
    profile_begin(static_cast<cudaStream_t>(cuda_stream));
    FLOWMM_TRY(validate(p));
    if (!importance || !retained_idx || (!evicted_idx && p->n_keep < p->seq_len)) return FLOWMM_ERR_NULL;
    Layout y;
    FLOWMM_TRY(check_ws(p, ws, ws_bytes, y));
    FLOWMM_TRY(check_device());
    return run_select(*p, importance, retained_idx, evicted_idx, static_cast<cudaStream_t>(cuda_stream));
}

flowmm_status flowmm_match(const flowmm_params *p, const void *k, const float *importance, const uint8_t *modality,
                           const int32_t *retained_idx, const int32_t *evicted_idx, const int32_t *strategy,
                           int32_t *match, float *match_sim, void *ws, size_t ws_bytes, void *cuda_stream) {
    profile_begin(static_cast<cudaStream_t>(cuda_stream));
    FLOWMM_TRY(validate(p));
    const bool has_e = p->n_keep < p->seq_len;
    if (!k || !importance || !modality || !retained_idx || !strategy) return FLOWMM_ERR_NULL;
    if (has_e && (!evicted_idx || !match || !match_sim)) return FLOWMM_ERR_NULL;
    if (!aligned16(k) || !strides_ok(p->k_stride, p->head_dim)) return FLOWMM_ERR_ALIGN;
    Layout y;
    FLOWMM_TRY(check_ws(p, ws, ws_bytes, y));
    FLOWMM_TRY(check_device());
    FLOWMM_DEBUG_LISTS(*p, retained_idx, evicted_idx, nullptr, at<int>(ws, y.status), static_cast<cudaStream_t>(cuda_stream));
    return run_match(*p, y, k, importance, modality, retained_idx, evicted_idx, strategy, match, match_sim, ws,
                     static_cast<cudaStream_t>(cuda_stream));
}

flowmm_status flowmm_merge(const flowmm_params *p, const void *k, const void *v, const int32_t *retained_idx,
                           const int32_t *evicted_idx, const int32_t *match, const float *match_sim, void *k_out,
                           void *v_out, void *ws, size_t ws_bytes, void *cuda_stream) {
    profile_begin(static_cast<cudaStream_t>(cuda_stream));
    FLOWMM_TRY(validate(p));
    const bool has_e = p->n_keep < p->seq_len;
    if (!k || !v || !retained_idx || !k_out || !v_out) return FLOWMM_ERR_NULL;
    if (has_e && (!evicted_idx || !match || !match_sim)) return FLOWMM_ERR_NULL;
    if (!aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out) ||
        !strides_ok(p->k_stride, p->head_dim) || !strides_ok(p->v_stride, p->head_dim) ||
        !strides_ok(p->ko_stride, p->head_dim) || !strides_ok(p->vo_stride, p->head_dim))
        return FLOWMM_ERR_ALIGN;
    Layout y;
    FLOWMM_TRY(check_ws(p, ws, ws_bytes, y));
    FLOWMM_TRY(check_device());
    FLOWMM_DEBUG_LISTS(*p, retained_idx, evicted_idx, match, at<int>(ws, y.status), static_cast<cudaStream_t>(cuda_stream));
    return run_merge(*p, y, k, v, retained_idx, evicted_idx, match, match_sim, k_out, v_out, ws,
                     static_cast<cudaStream_t>(cuda_stream));
}

flowmm_status flowmm_compress_layer(const flowmm_params *p, const void *q_win, const void *k, const void *v,
                                    const uint8_t *modality, void *k_out, void *v_out, float *importance, float *rho,
                                    int32_t *strategy, int32_t *retained_idx, int32_t *evicted_idx, int32_t *match,
                                    float *match_sim, void *ws, size_t ws_bytes, void *cuda_stream) {
    profile_begin(static_cast<cudaStream_t>(cuda_stream));
    FLOWMM_TRY(validate(p));
    if (!q_win || !k || !v || !modality || !k_out || !v_out) return FLOWMM_ERR_NULL;
    if (!aligned16(q_win) || !aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out) ||
        !strides_ok(p->q_stride, p->head_dim) || !strides_ok(p->k_stride, p->head_dim) ||
        !strides_ok(p->v_stride, p->head_dim) || !strides_ok(p->ko_stride, p->head_dim) ||
        !strides_ok(p->vo_stride, p->head_dim))
        return FLOWMM_ERR_ALIGN;
    Layout y;
    FLOWMM_TRY(check_ws(p, ws, ws_bytes, y));
    FLOWMM_TRY(check_device());
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (!importance) importance = at<float>(ws, y.importance);
    if (!rho) rho = at<float>(ws, y.rho);
    if (!strategy) strategy = at<int32_t>(ws, y.strategy);
    if (!retained_idx) retained_idx = at<int32_t>(ws, y.retained);
    if (!evicted_idx) evicted_idx = at<int32_t>(ws, y.evicted);
    if (!match) match = at<int32_t>(ws, y.match);
    if (!match_sim) match_sim = at<float>(ws, y.match_sim);
    float *cross_mass = at<float>(ws, y.cross_mass);
    int n_parts = 0;
    FLOWMM_TRY(run_score(*p, y, q_win, k, modality, importance, cross_mass, ws, st, &n_parts));
    // Eq. 6 and the theta rule ride along with the selection launch (which first adds up the partial masses, if any)
    // ... and so does the candidate layout of the tensor-core matching step
    const bool prep_in_select = p->seq_len > p->n_keep && use_tc(*p);
    const MatchPrepArgs prep = match_prep_args(*p, y, k, importance, modality, retained_idx, evicted_idx, ws);
    FLOWMM_TRY(run_select(*p, importance, retained_idx, evicted_idx, st, cross_mass, rho, strategy,
                          n_parts > 0 ? at<float>(ws, y.cross_part) : nullptr, n_parts, prep_in_select ? &prep : nullptr));
    // when both the short-list matching kernel and the tensor-core merge apply, the former writes the latter's table
    const bool map_in_match = p->seq_len > p->n_keep && use_tc(*p) && y.c_tot <= mst::kMaxCols && merge_is_tc(*p);
    FLOWMM_TRY(run_match(*p, y, k, importance, modality, retained_idx, evicted_idx, strategy, match, match_sim, ws, st,
                         map_in_match ? at<int2>(ws, y.tokmap) : nullptr, prep_in_select));
    FLOWMM_TRY(run_merge(*p, y, k, v, retained_idx, evicted_idx, match, match_sim, k_out, v_out, ws, st, map_in_match));
    return FLOWMM_OK;
}

flowmm_status flowmm_last_device_status(void *ws, void *cuda_stream) {
    if (!ws) return FLOWMM_ERR_NULL;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int32_t word = 0;
    if (cudaMemcpyAsync(&word, ws, sizeof(word), cudaMemcpyDeviceToHost, st) != cudaSuccess) return FLOWMM_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return FLOWMM_ERR_CUDA;
    if (word != 0) {
        if (cudaMemsetAsync(ws, 0, sizeof(word), st) != cudaSuccess) return FLOWMM_ERR_CUDA;
        if (cudaStreamSynchronize(st) != cudaSuccess) return FLOWMM_ERR_CUDA;
    }
    return word >= 0 && word <= FLOWMM_ERR_INDEX ? static_cast<flowmm_status>(word) : FLOWMM_ERR_CUDA;
}

int32_t flowmm_last_launch_count(void) { return g_launches; }

int32_t flowmm_debug_build(void) {
#ifdef FLOWMM_DEBUG
    return 1;
#else
    return 0;
#endif
}

flowmm_status flowmm_profile_enable(int32_t on) {
    if (on && !g_prof.have_events) {
        for (int i = 0; i <= kMaxProfiled; ++i)
            if (cudaEventCreate(&g_prof.ev[i]) != cudaSuccess) return FLOWMM_ERR_CUDA;
        g_prof.have_events = true;
    }
    g_prof.on = on != 0;
    g_prof.n = 0;
    return FLOWMM_OK;
}

int32_t flowmm_profile_read(const char **names, float *ms, int32_t max_entries) {
    if (!g_prof.on || g_prof.n == 0) return 0;
    if (cudaEventSynchronize(g_prof.ev[g_prof.n]) != cudaSuccess) return -1;
    const int n = g_prof.n < max_entries ? g_prof.n : max_entries;
    for (int i = 0; i < n; ++i) {
        if (names) names[i] = g_prof.name[i];
        if (ms && cudaEventElapsedTime(&ms[i], g_prof.ev[i], g_prof.ev[i + 1]) != cudaSuccess) return -1;
    }
    return n;
}

const char *flowmm_status_string(flowmm_status s) {
    switch (s) {
        case FLOWMM_OK: return "ok";
        case FLOWMM_ERR_NULL: return "null pointer";
        case FLOWMM_ERR_SHAPE: return "inconsistent shape or parameter";
        case FLOWMM_ERR_BUDGET: return "retention budget out of range";
        case FLOWMM_ERR_DTYPE: return "unsupported dtype";
        case FLOWMM_ERR_WORKSPACE: return "workspace too small";
        case FLOWMM_ERR_ALIGN: return "pointer or stride not aligned";
        case FLOWMM_ERR_CUDA: return "CUDA error";
        case FLOWMM_ERR_TIMEOUT: return "device-side wait timed out";
        case FLOWMM_ERR_UNSUPPORTED_DEVICE: return "device is not compute capability 10.x";
        case FLOWMM_ERR_INDEX: return "index out of range (debug build)";
    }
    return "unknown status";
}

}  // extern "C"

// ---- full-prefill information flow ---------------------------------------------------------------
namespace {

constexpr int kFlowTile = 128;      // query rows per scoring call

// Query tile t of n: rows [lo, hi); the first tile takes the remainder so that all others are full.
void flow_tile(int L, int t, int &lo, int &hi) {
    const int rem = L % kFlowTile, n_full = L / kFlowTile;
    if (rem == 0) { lo = t * kFlowTile; hi = lo + kFlowTile; return; }
    if (t == 0) { lo = 0; hi = rem; return; }
    lo = rem + (t - 1) * kFlowTile; hi = lo + kFlowTile;
    (void)n_full;
}
int flow_tiles(int L) { return (L + kFlowTile - 1) / kFlowTile; }

// The scoring step's parameters for one query tile: the prompt cut after the tile's last row, the tile as window.
flowmm_params flow_tile_params(const flowmm_params &p, const int64_t qs[3], int lo, int hi) {
    flowmm_params t = p;
    t.seq_len = hi; t.window = hi - lo; t.n_keep = 1; t.keep_window = 0; t.tau = 0.f; t.tau_mode = FLOWMM_TAU_ABS;
    for (int i = 0; i < 3; ++i) t.q_stride[i] = qs[i];
    return t;
}

struct FlowLayout { size_t std_bytes, mod, imp, parts, bits, total; };

// One query tile of the full-prefill flow on the tensor cores: the statistics pass alone, with the row sums split by
// key modality, then the per-head join.  `tp` is the tile's scoring problem (prompt cut after the tile, tile = window).
flowmm_status run_flow_tile_tc(const flowmm_params &tp, const Layout &y, const void *q_tile, const void *k,
                               const uint8_t *modality, int mod_pitch, const uint32_t *modbits, int mod_words,
                               float *cross_out, void *ws, cudaStream_t st) {
    const int UH = tp.n_units * tp.n_kv_heads, G = tp.n_q_heads / tp.n_kv_heads, W = tp.window;
    ScoreTcArgs a = {};
    a.row_part = at<float2>(ws, y.row_part); a.row_cross = at<float>(ws, y.row_cross); a.modality = modality;
    a.modbits = modbits; a.mod_words = mod_words; a.mod_pitch = mod_pitch; a.status = at<int>(ws, y.status);
    a.Hq = tp.n_q_heads; a.Hkv = tp.n_kv_heads; a.G = G; a.W = W; a.L = tp.seq_len; a.GW = G * W; a.GWpad = y.gw_pad;
    a.n_qt = y.tc_n_qt; a.n_chunk = y.tc_n_chunk; a.tiles_per_chunk = y.tc_tiles_per_chunk; a.n_rt = y.n_rt;
    a.a_heads = G < tcs::kRows / W ? G : tcs::kRows / W;
    a.n_items1 = UH * a.n_qt * a.n_chunk;
    const float scale = tp.softmax_scale != 0.f ? tp.softmax_scale : 1.f / sqrtf((float)tp.head_dim);
    a.scale_log2 = scale * kLog2e;
    CUtensorMap qa, k256;
    const uint64_t qd[4] = {128, (uint64_t)W, (uint64_t)tp.n_q_heads, (uint64_t)tp.n_units};
    const uint64_t qs[3] = {(uint64_t)tp.q_stride[2] * 2, (uint64_t)tp.q_stride[1] * 2, (uint64_t)tp.q_stride[0] * 2};
    const uint64_t kd[4] = {128, (uint64_t)tp.seq_len, (uint64_t)tp.n_kv_heads, (uint64_t)tp.n_units};
    const uint64_t ks[3] = {(uint64_t)tp.k_stride[2] * 2, (uint64_t)tp.k_stride[1] * 2, (uint64_t)tp.k_stride[0] * 2};
    const uint32_t bqa[4] = {64, (uint32_t)W, (uint32_t)a.a_heads, 1}, bk256[4] = {64, tcs::Big::kCols, 1, 1};
    if (!tc::make_bf16_map(&qa, q_tile, 4, qd, qs, bqa) || !tc::make_bf16_map(&k256, k, 4, kd, ks, bk256)) return FLOWMM_ERR_CUDA;
    if (cudaFuncSetAttribute(score_stats_tc_kernel<tcs::Big, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)tcs::Big::kSmemBytes) != cudaSuccess)
        return FLOWMM_ERR_CUDA;
    const int sms = tc::sm_count();
    score_stats_tc_kernel<tcs::Big, true><<<a.n_items1 < sms ? a.n_items1 : sms, tcs::kThreads, tcs::Big::kSmemBytes, st>>>(qa, k256, a);
    FLOWMM_LAUNCHED("flow_stats_tc");
    const int n_heads = tp.n_units * tp.n_q_heads;
    flow_combine_kernel<<<(n_heads + 7) / 8, 256, 0, st>>>(a.row_part, a.row_cross, 4 * a.n_chunk, G, W, tp.n_kv_heads, n_heads, cross_out);
    FLOWMM_LAUNCHED("flow_combine");
    return FLOWMM_OK;
}

FlowLayout flow_layout(const flowmm_params &p, const int64_t qs[3]) {
    FlowLayout f = {};
    const int n = flow_tiles(p.seq_len);
    for (int t = 0; t < n; ++t) {
        int lo, hi;
        flow_tile(p.seq_len, t, lo, hi);
        const size_t need = make_layout(flow_tile_params(p, qs, lo, hi)).total;
        if (need > f.std_bytes) f.std_bytes = need;
    }
    size_t o = align256(f.std_bytes);
    f.mod = o; o += align256((size_t)p.n_units * p.seq_len);
    f.imp = o; o += align256((size_t)p.n_units * p.n_kv_heads * p.seq_len * 4);
    f.parts = o; o += align256((size_t)n * p.n_units * p.n_q_heads * 4);
    f.bits = o; o += align256((size_t)p.n_units * ((p.seq_len + 31) / 32 + 8) * 4);
    f.total = o;
    return f;
}

flowmm_status validate_flow(const flowmm_params *p) {
    if (!p) return FLOWMM_ERR_NULL;
    flowmm_params t = *p;
    t.window = 1; t.n_keep = 1; t.keep_window = 0; t.tau = 0.f; t.tau_mode = FLOWMM_TAU_ABS;   // not used here
    return validate(&t);
}

}  // namespace

extern "C" flowmm_status flowmm_full_flow_workspace_bytes(const flowmm_params *p, size_t *bytes) {
    if (!bytes) return FLOWMM_ERR_NULL;
    FLOWMM_TRY(validate_flow(p));
    const int64_t dense[3] = {(int64_t)p->n_q_heads * p->seq_len * p->head_dim, (int64_t)p->seq_len * p->head_dim, p->head_dim};
    *bytes = flow_layout(*p, dense).total;
    return FLOWMM_OK;
}

extern "C" flowmm_status flowmm_full_flow(const flowmm_params *p, const void *q_full, const int64_t q_full_stride[3],
                                          const void *k, const uint8_t *modality, float *cross_mass, float *rho,
                                          int32_t *strategy, void *ws, size_t ws_bytes, void *cuda_stream) {
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    profile_begin(st);
    FLOWMM_TRY(validate_flow(p));
    if (!q_full || !q_full_stride || !k || !modality || !cross_mass || !strategy || !ws) return FLOWMM_ERR_NULL;
    if (!aligned16(q_full) || !aligned16(k) || !strides_ok(q_full_stride, p->head_dim) || !strides_ok(p->k_stride, p->head_dim) ||
        (reinterpret_cast<uintptr_t>(ws) & 255))
        return FLOWMM_ERR_ALIGN;
    const FlowLayout f = flow_layout(*p, q_full_stride);
    if (ws_bytes < f.total) return FLOWMM_ERR_WORKSPACE;
    FLOWMM_TRY(check_device());
    if (cudaMemsetAsync(ws, 0, 4, st) != cudaSuccess) return FLOWMM_ERR_CUDA;       // the status word
    const int n_tiles = flow_tiles(p->seq_len), n = p->n_units * p->n_q_heads;
    const size_t esize = p->dtype == FLOWMM_BF16 ? 2 : 4;
    uint8_t *mod = at<uint8_t>(ws, f.mod);
    float *imp = at<float>(ws, f.imp), *parts = at<float>(ws, f.parts);
    uint32_t *bits = at<uint32_t>(ws, f.bits);
    const int mod_words = (p->seq_len + 31) / 32 + 8;                  // + slack: whole 256-key tiles are indexed
    if (use_tc(*p)) {
        pack_modality_kernel<<<dim3(p->n_units, (mod_words + 7) / 8), 256, 0, st>>>(modality, p->seq_len, mod_words, bits);
        FLOWMM_LAUNCHED("pack_modality");
    }
    for (int t = 0; t < n_tiles; ++t) {
        int lo, hi;
        flow_tile(p->seq_len, t, lo, hi);
        const flowmm_params tp = flow_tile_params(*p, q_full_stride, lo, hi);
        const Layout y = make_layout(tp);
        const char *q_tile_tc = static_cast<const char *>(q_full) + (size_t)lo * (size_t)q_full_stride[2] * esize;
        if (use_tc_score(tp)) {            // full tiles on the tensor cores: one pass, no importance
            FLOWMM_TRY(run_flow_tile_tc(tp, y, q_tile_tc, k, modality, p->seq_len, bits, mod_words, parts + (size_t)t * n, ws, st));
            continue;
        }
        // the scoring kernels index the modality map with the cut prompt's length as the row pitch
        if (cudaMemcpy2DAsync(mod, (size_t)hi, modality, (size_t)p->seq_len, (size_t)hi, (size_t)p->n_units,
                              cudaMemcpyDeviceToDevice, st) != cudaSuccess)
            return FLOWMM_ERR_CUDA;
        const char *q_tile = static_cast<const char *>(q_full) + (size_t)lo * (size_t)q_full_stride[2] * esize;
        FLOWMM_TRY(run_score(tp, y, q_tile, k, mod, imp, parts + (size_t)t * n, ws, st));
    }
    full_flow_reduce_kernel<<<p->n_units, 64, 0, st>>>(parts, n_tiles, n, p->n_q_heads, p->seq_len, p->theta, p->flow_mode,
                                                       cross_mass, rho, strategy);
    FLOWMM_LAUNCHED("full_flow_reduce");
    return FLOWMM_OK;
}

// ---- decode-step attention over a cache ---------------------------------------------------------
namespace {

flowmm_status validate_decode(const flowmm_decode_params *p) {
    if (!p) return FLOWMM_ERR_NULL;
    if (p->n_units < 1 || p->n_q_heads < 1 || p->n_kv_heads < 1 || p->n_keys < 1) return FLOWMM_ERR_SHAPE;
    if (p->n_q_heads % p->n_kv_heads != 0 || p->n_q_heads / p->n_kv_heads > 8) return FLOWMM_ERR_SHAPE;
    if (p->head_dim != 64 && p->head_dim != 128) return FLOWMM_ERR_SHAPE;
    if ((int64_t)p->n_units * p->n_kv_heads > kMaxHeadsPerCall) return FLOWMM_ERR_SHAPE;
    if (p->dtype != FLOWMM_F32 && p->dtype != FLOWMM_BF16) return FLOWMM_ERR_DTYPE;
    if (!(p->softmax_scale >= 0.f)) return FLOWMM_ERR_SHAPE;
    if (p->path != FLOWMM_PATH_AUTO && p->path != FLOWMM_PATH_SIMT) return FLOWMM_ERR_SHAPE;
    return FLOWMM_OK;
}

// How a call is cut into key ranges, and where its scratch lives:
// [status word, 256 bytes][one ticket per (unit, KV head)][partial records].
struct DecodePlan {
    bool tc;                 // tensor-core kernel (bf16, head_dim 128) or the SIMT one
    int n_split, per_split;  // ranges per (unit, KV head); keys (SIMT) or 128-key tiles (tensor core) per range
    size_t part_off, bytes;
};

DecodePlan decode_plan(const flowmm_decode_params &p) {
    DecodePlan d;
    const int uh = p.n_units * p.n_kv_heads, g = p.n_q_heads / p.n_kv_heads;
    d.tc = p.dtype == FLOWMM_BF16 && p.head_dim == 128 && p.path != FLOWMM_PATH_SIMT;
    if (d.tc) {
        // Two CTAs share an SM.  Of the range lengths TMEM allows, take the one with the least work per CTA
        // slot when the CTAs run in rounds; a CTA's fixed cost (set-up, the pause between its two phases)
        // counts like a tile and a half.
        const int tiles = (p.n_keys + dtc::kTile - 1) / dtc::kTile;
        const int64_t slots = 2 * (int64_t)tc::sm_count();
        double best = 0.0;
        d.per_split = 1;
        for (int per = 1; per <= dtc::kMaxTiles && per <= tiles; ++per) {
            const int64_t ctas = (int64_t)uh * ((tiles + per - 1) / per);
            const double cost = (double)((ctas + slots - 1) / slots) * (per + 1.5);
            if (per == 1 || cost < best) { best = cost; d.per_split = per; }
        }
        d.n_split = (tiles + d.per_split - 1) / d.per_split;
        if ((int64_t)d.n_split * g > dtc::kMaxJoin) d.tc = false;      // more ranges than the joining CTA can stage
    }
    if (!d.tc) {
        // enough CTAs for about four per SM, at least 64 keys each
        int want = (4 * 148 + uh - 1) / uh;
        const int max_split = (p.n_keys + 63) / 64;
        want = want < 1 ? 1 : (want > max_split ? max_split : want);
        d.per_split = (p.n_keys + want - 1) / want;
        d.n_split = (p.n_keys + d.per_split - 1) / d.per_split;
    }
    d.part_off = 256 + align256((size_t)uh * sizeof(int));
    d.bytes = d.part_off + align256((size_t)uh * d.n_split * g * (p.head_dim + 2) * sizeof(float));
    return d;
}

template <typename T, int D>
flowmm_status launch_decode(const DecodeArgs &a, int uh, int n_q, cudaStream_t st) {
    constexpr int groups = kDecThreads / (D / Elem<T>::kVec);
    const dim3 grid(uh, a.n_split);
    const int gp = a.G <= 1 ? 1 : a.G <= 2 ? 2 : a.G <= 4 ? 4 : 8;
    const size_t smem = (size_t)groups * gp * (D + 2) * sizeof(float);
    switch (gp) {
        case 1: decode_partial_kernel<T, D, 1><<<grid, kDecThreads, smem, st>>>(a); break;
        case 2: decode_partial_kernel<T, D, 2><<<grid, kDecThreads, smem, st>>>(a); break;
        case 4: decode_partial_kernel<T, D, 4><<<grid, kDecThreads, smem, st>>>(a); break;
        default: decode_partial_kernel<T, D, 8><<<grid, kDecThreads, smem, st>>>(a); break;
    }
    FLOWMM_LAUNCHED("decode_partial");
    decode_combine_kernel<D><<<n_q, D, 0, st>>>(a);
    FLOWMM_LAUNCHED("decode_combine");
    return FLOWMM_OK;
}

flowmm_status launch_decode_tc(const flowmm_decode_params &p, const DecodeArgs &a, int *status, int uh, cudaStream_t st) {
    CUtensorMap kmap, vmap;
    const uint64_t dims[4] = {128, (uint64_t)p.n_keys, (uint64_t)p.n_kv_heads, (uint64_t)p.n_units};
    const uint64_t ks[3] = {(uint64_t)p.k_stride[2] * 2, (uint64_t)p.k_stride[1] * 2, (uint64_t)p.k_stride[0] * 2};
    const uint64_t vs[3] = {(uint64_t)p.v_stride[2] * 2, (uint64_t)p.v_stride[1] * 2, (uint64_t)p.v_stride[0] * 2};
    const uint32_t box[4] = {64, dtc::kTile, 1, 1};
    if (!tc::make_bf16_map(&kmap, a.k, 4, dims, ks, box) || !tc::make_bf16_map(&vmap, a.v, 4, dims, vs, box))
        return FLOWMM_ERR_CUDA;
    // (function attributes belong to the current device: set on every call, like the other launchers)
    if (cudaFuncSetAttribute(dtc::decode_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)dtc::kSmemBytes) != cudaSuccess ||
        cudaFuncSetAttribute(dtc::decode_tc_kernel, cudaFuncAttributePreferredSharedMemoryCarveout,
                             cudaSharedmemCarveoutMaxShared) != cudaSuccess)
        return FLOWMM_ERR_CUDA;
    dtc::Args t;
    t.q = static_cast<const __nv_bfloat16 *>(a.q); t.part = a.part; t.out = a.out; t.status = status;
    t.tickets = status + 64;
    t.Hq = a.Hq; t.Hkv = a.Hkv; t.G = a.G; t.N = a.N; t.n_split = a.n_split; t.tiles_per_split = a.keys_per_split;
    t.scale_log2 = a.scale_log2;
    dtc::decode_tc_kernel<<<dim3(uh, a.n_split), dtc::kThreads, dtc::kSmemBytes, st>>>(kmap, vmap, t);
    FLOWMM_LAUNCHED("decode_tc");
    return FLOWMM_OK;
}

}  // namespace

extern "C" flowmm_status flowmm_decode_workspace_bytes(const flowmm_decode_params *p, size_t *bytes) {
    if (!bytes) return FLOWMM_ERR_NULL;
    FLOWMM_TRY(validate_decode(p));
    *bytes = decode_plan(*p).bytes;
    return FLOWMM_OK;
}

extern "C" flowmm_status flowmm_decode_attention(const flowmm_decode_params *p, const void *q, const void *k,
                                                 const void *v, float *out, void *ws, size_t ws_bytes,
                                                 void *cuda_stream) {
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    profile_begin(st);
    FLOWMM_TRY(validate_decode(p));
    if (!q || !k || !v || !out || !ws) return FLOWMM_ERR_NULL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !strides_ok(p->k_stride, p->head_dim) ||
        !strides_ok(p->v_stride, p->head_dim) || (reinterpret_cast<uintptr_t>(ws) & 255))
        return FLOWMM_ERR_ALIGN;
    const DecodePlan plan = decode_plan(*p);
    if (ws_bytes < plan.bytes) return FLOWMM_ERR_WORKSPACE;
    FLOWMM_TRY(check_device());
    if (cudaMemsetAsync(ws, 0, plan.part_off, st) != cudaSuccess) return FLOWMM_ERR_CUDA;   // status word and tickets
    DecodeArgs a;
    a.q = q; a.k = k; a.v = v; a.part = reinterpret_cast<float *>(static_cast<char *>(ws) + plan.part_off); a.out = out;
    a.Hq = p->n_q_heads; a.Hkv = p->n_kv_heads; a.G = p->n_q_heads / p->n_kv_heads; a.N = p->n_keys;
    a.n_split = plan.n_split; a.keys_per_split = plan.per_split;
    const float scale = p->softmax_scale != 0.f ? p->softmax_scale : 1.f / sqrtf((float)p->head_dim);
    a.scale_log2 = scale * kLog2e;
    for (int i = 0; i < 3; ++i) { a.ks[i] = p->k_stride[i]; a.vs[i] = p->v_stride[i]; }
    const int uh = p->n_units * p->n_kv_heads, n_q = p->n_units * p->n_q_heads;
    if (plan.tc) return launch_decode_tc(*p, a, static_cast<int *>(ws), uh, st);
    if (p->dtype == FLOWMM_BF16)
        return p->head_dim == 128 ? launch_decode<__nv_bfloat16, 128>(a, uh, n_q, st) : launch_decode<__nv_bfloat16, 64>(a, uh, n_q, st);
    return p->head_dim == 128 ? launch_decode<float, 128>(a, uh, n_q, st) : launch_decode<float, 64>(a, uh, n_q, st);
}

// ---- re-compression of a cache that grew during decoding ----------------------------------------
namespace {

// strategy of a unit copied to each of its KV heads (the per-head problems below take one strategy each)
__global__ void expand_strategy_kernel(const int32_t *strategy, int n_units, int n_kv_heads, int32_t *per_head) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_units * n_kv_heads) per_head[i] = strategy[i / n_kv_heads];
}

// modality of the rows that were kept: out[uh, s] = row_modality[uh, retained[uh, s]]
__global__ void gather_row_modality_kernel(const uint8_t *row_modality, const int32_t *retained, int64_t n, int L, int B,
                                           uint8_t *out) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) out[i] = row_modality[(i / B) * L + retained[i]];
}

// Every (unit, KV head) of the cache as a problem of its own: one KV head, its G query heads, its own row modalities.
// Needs the unit stride of every tensor to be heads x head stride (one stride then steps through units and heads).
bool per_head_params(const flowmm_params &p, flowmm_params &ph) {
    const int G = p.n_q_heads / p.n_kv_heads;
    if (p.q_stride[0] != (int64_t)p.n_q_heads * p.q_stride[1] || p.k_stride[0] != (int64_t)p.n_kv_heads * p.k_stride[1] ||
        p.v_stride[0] != (int64_t)p.n_kv_heads * p.v_stride[1] || p.ko_stride[0] != (int64_t)p.n_kv_heads * p.ko_stride[1] ||
        p.vo_stride[0] != (int64_t)p.n_kv_heads * p.vo_stride[1])
        return false;
    ph = p;
    ph.n_units = p.n_units * p.n_kv_heads; ph.n_q_heads = G; ph.n_kv_heads = 1;
    ph.q_stride[0] = (int64_t)G * p.q_stride[1];
    ph.k_stride[0] = p.k_stride[1]; ph.v_stride[0] = p.v_stride[1];
    ph.ko_stride[0] = p.ko_stride[1]; ph.vo_stride[0] = p.vo_stride[1];
    return true;
}

struct RecompressLayout { size_t strategy_h, total; };
RecompressLayout recompress_layout(const flowmm_params &ph) {
    RecompressLayout r;
    r.strategy_h = align256(make_layout(ph).total);
    r.total = r.strategy_h + align256((size_t)ph.n_units * 4);
    return r;
}

}  // namespace

extern "C" flowmm_status flowmm_recompress_workspace_bytes(const flowmm_params *p, size_t *bytes) {
    if (!bytes) return FLOWMM_ERR_NULL;
    FLOWMM_TRY(validate(p));
    flowmm_params ph;
    if (!per_head_params(*p, ph)) return FLOWMM_ERR_ALIGN;
    FLOWMM_TRY(validate(&ph));
    *bytes = recompress_layout(ph).total;
    return FLOWMM_OK;
}

extern "C" flowmm_status flowmm_recompress(const flowmm_params *p, const void *q_win, const void *k_cache,
                                           const void *v_cache, const uint8_t *row_modality, void *k_out, void *v_out,
                                           uint8_t *row_modality_out, float *importance, float *rho, int32_t *strategy,
                                           int32_t *retained_idx, int32_t *evicted_idx, int32_t *match, float *match_sim,
                                           void *ws, size_t ws_bytes, void *cuda_stream) {
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    profile_begin(st);
    FLOWMM_TRY(validate(p));
    if (!q_win || !k_cache || !v_cache || !row_modality || !k_out || !v_out || !row_modality_out) return FLOWMM_ERR_NULL;
    if (!aligned16(q_win) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(k_out) || !aligned16(v_out) ||
        !strides_ok(p->q_stride, p->head_dim) || !strides_ok(p->k_stride, p->head_dim) ||
        !strides_ok(p->v_stride, p->head_dim) || !strides_ok(p->ko_stride, p->head_dim) ||
        !strides_ok(p->vo_stride, p->head_dim))
        return FLOWMM_ERR_ALIGN;
    flowmm_params ph;
    if (!per_head_params(*p, ph)) return FLOWMM_ERR_ALIGN;
    FLOWMM_TRY(validate(&ph));
    if (!ws) return FLOWMM_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(ws) & 255) return FLOWMM_ERR_ALIGN;
    const Layout y = make_layout(ph);
    const RecompressLayout r = recompress_layout(ph);
    if (ws_bytes < r.total) return FLOWMM_ERR_WORKSPACE;
    FLOWMM_TRY(check_device());
    if (!importance) importance = at<float>(ws, y.importance);
    if (!rho) rho = at<float>(ws, y.rho);
    if (!strategy) strategy = at<int32_t>(ws, y.strategy);
    if (!retained_idx) retained_idx = at<int32_t>(ws, y.retained);
    if (!evicted_idx) evicted_idx = at<int32_t>(ws, y.evicted);
    if (!match) match = at<int32_t>(ws, y.match);
    if (!match_sim) match_sim = at<float>(ws, y.match_sim);
    float *cross_mass = at<float>(ws, y.cross_mass);             // [U * Hkv, G] = [U, Hq]
    int32_t *strategy_h = at<int32_t>(ws, r.strategy_h);
    // scoring per (unit, KV head) against that head's own row modalities; Eq. 6 over all query heads of the layer
    FLOWMM_TRY(run_score(ph, y, q_win, k_cache, row_modality, importance, cross_mass, ws, st));
    FLOWMM_TRY(run_layer_flow(*p, cross_mass, rho, strategy, st));
    expand_strategy_kernel<<<(ph.n_units + 255) / 256, 256, 0, st>>>(strategy, p->n_units, p->n_kv_heads, strategy_h);
    FLOWMM_LAUNCHED("expand_strategy");
    FLOWMM_TRY(run_select(ph, importance, retained_idx, evicted_idx, st));
    FLOWMM_TRY(run_match(ph, y, k_cache, importance, row_modality, retained_idx, evicted_idx, strategy_h, match, match_sim, ws, st));
    FLOWMM_TRY(run_merge(ph, y, k_cache, v_cache, retained_idx, evicted_idx, match, match_sim, k_out, v_out, ws, st));
    const int64_t n = (int64_t)ph.n_units * p->n_keep;
    gather_row_modality_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(row_modality, retained_idx, n, p->seq_len, p->n_keep,
                                                                            row_modality_out);
    FLOWMM_LAUNCHED("gather_row_modality");
    return FLOWMM_OK;
}

// ---- bounded-wait self-test ----------------------------------------------------------------------
namespace {
// One CTA waits on an mbarrier phase that nothing completes, with the same bounded wait the
// tensor-core kernels use: after the limit the first waiter records FLOWMM_ERR_TIMEOUT, raises the
// CTA's abort flag, and every thread returns.
__global__ void wait_timeout_selftest_kernel(int *status) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0;
        tc::mbar_init(tc::smem_u32(&bar), 1);
        tc::mbar_init_fence();
    }
    __syncthreads();
    tc::mbar_wait(tc::smem_u32(&bar), 0, &abort_flag, status);
}
}  // namespace

extern "C" flowmm_status flowmm_selftest_wait_timeout(void *ws, void *cuda_stream) {
    profile_begin(static_cast<cudaStream_t>(cuda_stream));
    if (!ws) return FLOWMM_ERR_NULL;
    FLOWMM_TRY(check_device());
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    wait_timeout_selftest_kernel<<<1, 64, 0, st>>>(static_cast<int *>(ws));
    FLOWMM_LAUNCHED("wait_timeout_selftest");
    return FLOWMM_OK;
}

// ---- merge without caller scratch --------------------------------------------------------------
// Scratch of flowmm_merge_static: lives in the library image, one copy per GPU that loads it.
static __device__ __align__(256) unsigned char g_merge_static_scratch[FLOWMM_MERGE_STATIC_BYTES];

namespace {

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
void *g_static_ptr[kMaxDevices] = {};          // device address of the array, per device ordinal

// The array's name is only a handle in host code; the address a kernel can use comes from the
// runtime, once per device, with that device current.
flowmm_status merge_static_base(void **base) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FLOWMM_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return FLOWMM_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_merge_static_scratch) != cudaSuccess || !ptr) return FLOWMM_ERR_CUDA;
        g_static_ptr[dev] = ptr;
    }
    *base = g_static_ptr[dev];
    return FLOWMM_OK;
}

// The part of the workspace layout that the merge step touches, packed behind the array's status word
// (the first 256 bytes, where flowmm_merge_static_status finds it whatever the problem's shape).
Layout make_merge_layout(const flowmm_params &p) {
    Layout y = {};
    size_t o = 256;
    layout_merge(y, p, [&](size_t bytes) { const size_t at = o; o += align256(bytes); return at; });
    y.merge_status = 0;
    y.total = o;
    return y;
}

}  // namespace

extern "C" flowmm_status flowmm_merge_static(const flowmm_params *p, const void *k, const void *v,
                                             const int32_t *retained_idx, const int32_t *evicted_idx,
                                             const int32_t *match, const float *match_sim, void *k_out, void *v_out,
                                             void *cuda_stream) {
    profile_begin(static_cast<cudaStream_t>(cuda_stream));
    FLOWMM_TRY(validate(p));
    const bool has_e = p->n_keep < p->seq_len;
    if (!k || !v || !retained_idx || !k_out || !v_out) return FLOWMM_ERR_NULL;
    if (has_e && (!evicted_idx || !match || !match_sim)) return FLOWMM_ERR_NULL;
    if (!aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out) ||
        !strides_ok(p->k_stride, p->head_dim) || !strides_ok(p->v_stride, p->head_dim) ||
        !strides_ok(p->ko_stride, p->head_dim) || !strides_ok(p->vo_stride, p->head_dim))
        return FLOWMM_ERR_ALIGN;
    const Layout y = make_merge_layout(*p);
    if (y.total > (size_t)FLOWMM_MERGE_STATIC_BYTES) return FLOWMM_ERR_WORKSPACE;   // problem too large for the array
    FLOWMM_TRY(check_device());
    void *base = nullptr;
    FLOWMM_TRY(merge_static_base(&base));
    FLOWMM_DEBUG_LISTS(*p, retained_idx, evicted_idx, match, static_cast<int *>(base), static_cast<cudaStream_t>(cuda_stream));
    // Nothing in this scratch has to start at zero: the slot lists, the piece table, the work counter and
    // the arrival counters are written (or cleared) by this call's first kernel before they are read, a
    // partial-sum record is only read for pieces that wrote it in the same call, and the status word is
    // sticky on purpose (the loader zero-fills the array; flowmm_merge_static_status clears the word).
    return run_merge(*p, y, k, v, retained_idx, evicted_idx, match, match_sim, k_out, v_out, base,
                     static_cast<cudaStream_t>(cuda_stream));
}

extern "C" flowmm_status flowmm_merge_static_status(void *cuda_stream) {
    FLOWMM_TRY(check_device());
    void *base = nullptr;
    FLOWMM_TRY(merge_static_base(&base));
    return flowmm_last_device_status(base, cuda_stream);
}

// Test hook of the reader above: stores `word` in the array's status word from the host, in stream order.
extern "C" flowmm_status flowmm_merge_static_poke_status(int32_t word, void *cuda_stream) {
    FLOWMM_TRY(check_device());
    void *base = nullptr;
    FLOWMM_TRY(merge_static_base(&base));
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(base, &word, sizeof(word), cudaMemcpyHostToDevice, st) != cudaSuccess) return FLOWMM_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? FLOWMM_OK : FLOWMM_ERR_CUDA;
}
