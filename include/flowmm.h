/*
 * flowmm.h - C ABI of the FlowMM KV-cache compression library for NVIDIA B200 (sm_100a).
 *
 * FlowMM (arXiv 2511.05534, Section 3.3) compresses each transformer layer's KV cache once,
 * after multimodal prefill, per KV head:
 *   1. score   - attention of the proxy tokens (the last W prompt positions) over all context
 *                keys gives every token an importance (Eq. 8); the same attention, split by
 *                modality, gives the layer's cross-modal interaction ratio rho (Eq. 6-7);
 *   2. flow    - rho against the threshold theta picks cross-modal or intra-modal merging;
 *   3. select  - the B most important tokens form the pivot set, the rest the non-pivot set;
 *   4. match   - each non-pivot finds the pivot of largest key cosine similarity (Eq. 9)
 *                among pivots whose importance does not exceed the sensitivity threshold
 *                tau (Eq. 10) and, in an intra-modal layer, that share its modality;
 *   5. merge   - non-pivots are folded into their pivots (Eq. 5) and the B merged rows are
 *                written out as the compressed cache.
 *
 * Conventions for every entry point
 *   - A "unit" is one (layer, sequence) pair; units are independent problems and a call
 *     processes n_units of them at once.  G = n_q_heads / n_kv_heads query heads share KV
 *     head h = g / G.  L = seq_len, W = window, B = n_keep, E = L - B.
 *   - Every tensor pointer is a DEVICE pointer owned by the caller; the library allocates
 *     and frees nothing.  Scratch memory comes from the caller as `ws` / `ws_bytes`
 *     (size from flowmm_workspace_bytes, 256-byte aligned); its first word is a sticky
 *     device status, so the caller zero-fills the first 256 bytes once after allocating
 *     it.  Inputs are never written; outputs must not alias inputs.
 *   - n_units * n_kv_heads must not exceed 4 194 304 per call, and that product times the number of
 *     128-token tiles of the context times the number of 128-row tiles of a KV head's proxy rows must
 *     stay below 2^31 (work items are counted in 32 bits); else FLOWMM_ERR_SHAPE.
 *   - Q, K, V and the outputs have the element type `dtype`, head_dim contiguous, and the
 *     element strides given in the params (unit, head, token).  Base pointers must be
 *     16-byte aligned and every stride a multiple of 8 elements, else FLOWMM_ERR_ALIGN.
 *     All other arrays are dense in the stated shape.
 *   - Calls enqueue work on `cuda_stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and return without waiting.  The return value reports host-side validation
 *     and launch errors.  Problems found on the device (a bounded wait that ran out) set
 *     the status word, which flowmm_last_device_status reads back.
 *   - There is no CPU fallback: on a device that is not compute capability 10.x every
 *     compute entry point returns FLOWMM_ERR_UNSUPPORTED_DEVICE.
 */
#ifndef FLOWMM_H_
#define FLOWMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    FLOWMM_OK = 0,
    FLOWMM_ERR_NULL = 1,               /* a required pointer is NULL */
    FLOWMM_ERR_SHAPE = 2,              /* sizes inconsistent (heads, head_dim, window, ...) */
    FLOWMM_ERR_BUDGET = 3,             /* n_keep outside [1, L], or below W with keep_window */
    FLOWMM_ERR_DTYPE = 4,
    FLOWMM_ERR_WORKSPACE = 5,          /* ws_bytes smaller than flowmm_workspace_bytes */
    FLOWMM_ERR_ALIGN = 6,
    FLOWMM_ERR_CUDA = 7,               /* a CUDA runtime call or launch failed */
    FLOWMM_ERR_TIMEOUT = 8,            /* device status: a bounded wait inside a kernel ran out */
    FLOWMM_ERR_UNSUPPORTED_DEVICE = 9,
    FLOWMM_ERR_INDEX = 10              /* debug build only: an index list or a computed index was out of range */
} flowmm_status;

typedef enum { FLOWMM_F32 = 0, FLOWMM_BF16 = 1 } flowmm_dtype;
typedef enum { FLOWMM_INTRA = 0, FLOWMM_CROSS = 1 } flowmm_strategy;
/* Eq. 5 leaves the merge functions open.  EXPSIM: pivot weight 1, non-pivot weight
 * exp(u - 1) with u its cosine similarity to the pivot; MEAN: all weights 1.  Weights are
 * normalised to sum to one per output row. */
typedef enum { FLOWMM_MERGE_EXPSIM = 0, FLOWMM_MERGE_MEAN = 1 } flowmm_merge_mode;
/* ABS: tau is compared with the importance directly.  REL: tau is in units of the
 * importance a uniform attention would give, tau_eff = tau * W / L. */
typedef enum { FLOWMM_TAU_ABS = 0, FLOWMM_TAU_REL = 1 } flowmm_tau_mode;
/* AUTO: the theta rule on rho (aligned merging).  FORCE_*: one strategy for every layer.  MISALIGNED: the
 * reverse of the rule (intra-modal where rho > theta, cross-modal elsewhere), the contrast case of the paper's
 * study of flow-aligned merging. */
typedef enum { FLOWMM_FLOW_AUTO = 0, FLOWMM_FLOW_FORCE_INTRA = 1, FLOWMM_FLOW_FORCE_CROSS = 2,
               FLOWMM_FLOW_MISALIGNED = 3 } flowmm_flow_mode;
/* Which kernels do the two dense contractions.  AUTO: tensor-core (tcgen05) kernels when
 * dtype is bf16 and head_dim is 128, SIMT fp32 kernels otherwise.  SIMT forces the latter. */
typedef enum { FLOWMM_PATH_AUTO = 0, FLOWMM_PATH_SIMT = 1 } flowmm_path;

typedef struct {
    int32_t n_units;                    /* independent (layer, sequence) problems */
    int32_t n_q_heads, n_kv_heads;      /* n_q_heads must be a multiple of n_kv_heads */
    int32_t head_dim;                   /* 64 or 128 */
    int32_t seq_len, window;            /* L, W with 1 <= W <= L */
    int32_t n_keep;                     /* B with 1 <= B <= L */
    int32_t dtype;                      /* flowmm_dtype of Q, K, V, K_out, V_out */
    float softmax_scale;                /* 0 selects 1/sqrt(head_dim) */
    float theta;                        /* cross-modal merging threshold of Section 3.3.1 */
    float tau;                          /* sensitivity threshold of Eq. 10; +inf disables it */
    int32_t tau_mode;                   /* flowmm_tau_mode */
    int32_t flow_mode;                  /* flowmm_flow_mode */
    int32_t merge_mode;                 /* flowmm_merge_mode */
    int32_t keep_window;                /* 1: the W proxy tokens are always pivots (needs B >= W) */
    int32_t path;                       /* flowmm_path */
    /* element strides of (unit, head, token); head_dim stride is 1 */
    int64_t q_stride[3];                /* Q_win [U, Hq,  W, D] */
    int64_t k_stride[3];                /* K     [U, Hkv, L, D] */
    int64_t v_stride[3];                /* V     [U, Hkv, L, D] */
    int64_t ko_stride[3];               /* K_out [U, Hkv, B, D] */
    int64_t vo_stride[3];               /* V_out [U, Hkv, B, D] */
} flowmm_params;

/* Scratch size in bytes that any entry point below needs for these params.  Host only; makes
 * no CUDA call.  Fails with the same validation errors as the compute entry points. */
flowmm_status flowmm_workspace_bytes(const flowmm_params *p, size_t *bytes);

/*
 * Step 1, Eq. 8 (with the causal softmax of Eq. 4 on the proxy rows) and the masses of Eq. 7.
 *   q_win      [U, Hq, W, D]   queries of the last W prompt positions
 *   k          [U, Hkv, L, D]  layer keys
 *   modality   [U, L] uint8    0 = text token, 1 = visual token
 *   importance [U, Hkv, L] f32 out: I[h,i] = (1/G) sum_{g in h} sum_a alpha[g,a,i]
 *   cross_mass [U, Hq] f32     out: sum_a sum_{i: m_i != m_(p_a)} alpha[g,a,i]; the total mass
 *                              of a head is W because every softmax row sums to one.
 */
flowmm_status flowmm_score(const flowmm_params *p, const void *q_win, const void *k, const uint8_t *modality,
                           float *importance, float *cross_mass, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Step 2, Eq. 6 and the threshold rule after Eq. 7.
 *   rho      [U] f32   out: mean over query heads of cross_mass / W
 *   strategy [U] int32 out: FLOWMM_CROSS if rho > theta else FLOWMM_INTRA (or as flow_mode forces)
 */
flowmm_status flowmm_layer_flow(const flowmm_params *p, const float *cross_mass, float *rho, int32_t *strategy,
                                void *cuda_stream);

/*
 * Step 3, pivot selection of Section 3.3.1: the B largest importances per KV head, ties to the
 * lower index.
 *   retained_idx [U, Hkv, B] int32 out: pivot token positions, ascending; slot s holds r_s
 *   evicted_idx  [U, Hkv, E] int32 out: non-pivot token positions, ascending
 */
flowmm_status flowmm_select(const flowmm_params *p, const float *importance, int32_t *retained_idx,
                            int32_t *evicted_idx, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Step 4, Eq. 9 and Eq. 10.  For the j-th non-pivot e = evicted_idx[j]:
 *   match     [U, Hkv, E] int32 out: slot of the admissible pivot with the largest cosine
 *                                    similarity (ties to the lower slot), or -1 if none
 *   match_sim [U, Hkv, E] f32   out: that similarity, 0 where match is -1
 * A pivot r_s is admissible if importance[r_s] <= tau_eff and, when strategy[u] is
 * FLOWMM_INTRA, modality[r_s] == modality[e].  A key of zero norm has similarity 0.
 */
flowmm_status flowmm_match(const flowmm_params *p, const void *k, const float *importance, const uint8_t *modality,
                           const int32_t *retained_idx, const int32_t *evicted_idx, const int32_t *strategy,
                           int32_t *match, float *match_sim, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Step 5, Eq. 5 and compaction.  Output row s (s in [0, B), ascending token position) is
 *   (x[r_s] + sum_{j: match[j] = s} w_j x[e_j]) / (1 + sum w_j),  x in {K, V},
 * with w_j = exp(match_sim[j] - 1) (EXPSIM) or 1 (MEAN); non-pivots with match -1 are dropped.
 * Accumulation is fp32 in a fixed order (results are bit-reproducible), rounded once to dtype.
 *   k_out, v_out [U, Hkv, B, D]
 */
flowmm_status flowmm_merge(const flowmm_params *p, const void *k, const void *v, const int32_t *retained_idx,
                           const int32_t *evicted_idx, const int32_t *match, const float *match_sim,
                           void *k_out, void *v_out, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * flowmm_merge without a caller-provided workspace.  (The paper has no counterpart: this is a
 * packaging variant of step 5 for callers that cannot allocate device memory - a plugin running
 * inside another runtime's memory pool, code running while that pool is frozen, a host that is
 * handed fixed buffers only.  They still pass the inputs and the two output tensors; what they
 * cannot provide is the scratch flowmm_merge needs for its slot lists and partial sums.)
 *
 * The scratch is a fixed array of FLOWMM_MERGE_STATIC_BYTES inside the library image; every GPU
 * that loads the library holds one copy until the process exits.  The call makes no cudaMalloc
 * or cudaFree and calls no allocating routine.  Arguments, outputs and results are those of
 * flowmm_merge (same kernels, same fixed accumulation order, so the outputs are bit-identical).
 *
 * Limits and rules:
 *   - The scratch a problem needs, per (unit, KV head): 16 E + 16 (B + E / 64 + 1) + 12 (B + 1) + 4 B
 *     bytes of slot lists, piece table and counters, 8 L bytes of per-token (slot, weight) pairs,
 *     and (2 (E / 64) + 2) * (8 head_dim + 16) bytes of partial sums; every part is rounded up
 *     to 256 bytes and 768 bytes are fixed.  If that exceeds the array the call returns
 *     FLOWMM_ERR_WORKSPACE and launches nothing.
 *   - A problem found on the device (a bounded wait that ran out) is recorded in a status word
 *     inside the array, since there is no workspace to carry it: flowmm_merge_static_status
 *     waits for the stream, returns that word (FLOWMM_OK or the first error recorded by any
 *     call since the last read) and clears it.  Outputs of a call that reported an error are
 *     not valid.
 *   - The first call on a device looks up the array's device address (once per device, with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents;
 *     nothing in it needs clearing between calls.  Two calls that overlap on the GPU (different
 *     streams, or graphs replayed concurrently) race on it: keep them ordered.
 */
#define FLOWMM_MERGE_STATIC_BYTES (8u << 20)
flowmm_status flowmm_merge_static(const flowmm_params *p, const void *k, const void *v, const int32_t *retained_idx,
                                  const int32_t *evicted_idx, const int32_t *match, const float *match_sim,
                                  void *k_out, void *v_out, void *cuda_stream);
flowmm_status flowmm_merge_static_status(void *cuda_stream);
/* Test aid for the reader above: waits for the stream and stores `word` in the array's status word
 * from the host, so that reading and clearing can be checked without making a kernel fail. */
flowmm_status flowmm_merge_static_poke_status(int32_t word, void *cuda_stream);

/*
 * Steps 1-5 in order on one stream: the whole per-layer FlowMM compression of Section 3.3.
 * The diagnostic outputs (importance ... match_sim, layouts as above) may each be NULL, in
 * which case the intermediate lives in the workspace only.
 */
flowmm_status flowmm_compress_layer(const flowmm_params *p, const void *q_win, const void *k, const void *v,
                                    const uint8_t *modality, void *k_out, void *v_out,
                                    float *importance, float *rho, int32_t *strategy,
                                    int32_t *retained_idx, int32_t *evicted_idx,
                                    int32_t *match, float *match_sim,
                                    void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * Re-compression of a cache that has grown during decoding.  Eq. 3 appends one key / value row per decoded token;
 * the paper runs the compression of Section 3.3 once, after prefill, and does not say what follows.  The reading
 * offered here: the current cache of a KV head - the rows an earlier compression left, in order, then the rows
 * appended since - is treated as that head's context of L = seq_len rows, and steps 1-5 run on it again with the
 * proxy window taken from the W most recent queries.  A row that came out of an earlier merge is an ordinary token
 * with the modality of the pivot it was merged into; after a compression the heads of a layer no longer hold the
 * same tokens, so modality is given per head and row.  Importance is taken afresh from the window (the causal mask
 * follows the row order, exact once at least W rows have been appended); rho is still the layer's, the mean over
 * all query heads (Eq. 6), each head measured against its own rows; merge weights as in flowmm_merge.
 *   q_win            [U, Hq, W, D]   queries of the W most recent positions
 *   k_cache, v_cache [U, Hkv, L, D]  the cache rows, strides p->k_stride / p->v_stride
 *   row_modality     [U, Hkv, L] uint8
 *   k_out, v_out     [U, Hkv, B, D]; row_modality_out [U, Hkv, B] uint8 (the kept rows' modalities, for the next round)
 *   importance ... match_sim: optional diagnostics (may be NULL), shaped as in flowmm_compress_layer but per
 *   KV head throughout; rho, strategy [U].
 * The unit stride of q, k, v and the outputs must equal heads x head stride (dense over heads), else
 * FLOWMM_ERR_ALIGN.  Scratch: flowmm_recompress_workspace_bytes.  B == L returns the cache unchanged (the plain
 * append of Eq. 3).
 */
flowmm_status flowmm_recompress_workspace_bytes(const flowmm_params *p, size_t *bytes);
flowmm_status flowmm_recompress(const flowmm_params *p, const void *q_win, const void *k_cache, const void *v_cache,
                                const uint8_t *row_modality, void *k_out, void *v_out, uint8_t *row_modality_out,
                                float *importance, float *rho, int32_t *strategy, int32_t *retained_idx,
                                int32_t *evicted_idx, int32_t *match, float *match_sim,
                                void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The step before the compression path: the cross-modal interaction ratio of Eq. 6 and Eq. 7 taken
 * literally, over every query row of the prefill (both the text-to-visual and the visual-to-text
 * term), instead of over the proxy window that flowmm_score uses.  Causal softmax attention of all
 * L queries; per query head the attention mass that lands on keys of the other modality than the
 * query's, summed over the rows; rho = mean over heads of that mass / L; strategy by theta.
 *   q_full [U, Hq, L, D] with the element strides q_full_stride (unit, head, token); head_dim contiguous
 *   k      [U, Hkv, L, D] with p->k_stride
 *   cross_mass [U, Hq] f32 out;  rho [U] f32 out (may be NULL);  strategy [U] int32 out
 * Of p, the fields n_units, n_q_heads, n_kv_heads, head_dim, seq_len, dtype, softmax_scale, theta,
 * flow_mode, k_stride and path are used (window, n_keep, tau, q_stride are not).  The work is the
 * scoring step applied to query tiles of 128 rows, each against the keys up to its last row, so it
 * costs O(L^2 D) per head.  Scratch: flowmm_full_flow_workspace_bytes; its first word is the device status.
 */
flowmm_status flowmm_full_flow_workspace_bytes(const flowmm_params *p, size_t *bytes);
flowmm_status flowmm_full_flow(const flowmm_params *p, const void *q_full, const int64_t q_full_stride[3],
                               const void *k, const uint8_t *modality, float *cross_mass, float *rho,
                               int32_t *strategy, void *ws, size_t ws_bytes, void *cuda_stream);

/*
 * The step after the compression path: decode-time attention of one new query per query head over a
 * cache of n_keys rows, Eq. 4 - o = softmax(q . K^T * scale) V - for the full cache or for the
 * compressed one that flowmm_compress_layer wrote.  Every cache row is read once for all G query
 * heads of its KV head.
 *   q   [U, Hq, D]  dense, element type `dtype`
 *   k,v [U, Hkv, n_keys, D] with the element strides given (unit, head, token); head_dim contiguous
 *   out [U, Hq, D]  f32
 * n_q_heads / n_kv_heads must be at most 8; head_dim 64 or 128.  Scratch: flowmm_decode_workspace_bytes
 * (its first word is a device status like the compression workspace's, see flowmm_last_device_status).
 * `path` as in flowmm_params: AUTO runs both contractions on the tensor cores (tcgen05) when dtype is
 * bf16 and head_dim is 128, and SIMT fp32 kernels otherwise; SIMT forces the latter.
 * Same conventions as above (device pointers, caller-owned memory, asynchronous on the stream).
 */
typedef struct {
    int32_t n_units, n_q_heads, n_kv_heads, head_dim;
    int32_t n_keys;                     /* rows of the cache to attend to (L, or B after compression) */
    int32_t dtype;                      /* flowmm_dtype of q, k, v */
    float softmax_scale;                /* 0 selects 1/sqrt(head_dim) */
    int32_t path;                       /* flowmm_path */
    int64_t k_stride[3], v_stride[3];   /* element strides of (unit, head, token) */
} flowmm_decode_params;

flowmm_status flowmm_decode_workspace_bytes(const flowmm_decode_params *p, size_t *bytes);
flowmm_status flowmm_decode_attention(const flowmm_decode_params *p, const void *q, const void *k, const void *v,
                                      float *out, void *ws, size_t ws_bytes, void *cuda_stream);

/* Waits for `cuda_stream`, then returns the device status word at the start of `ws`
 * (FLOWMM_OK, or the first error a kernel recorded) and clears it. */
flowmm_status flowmm_last_device_status(void *ws, void *cuda_stream);

/*
 * Self-test of the bounded device-side waits (every mbarrier wait inside the tensor-core kernels
 * gives up after about two seconds instead of hanging the GPU).  Enqueues one small kernel whose
 * threads wait for an event that never comes; it returns by itself after the limit and leaves
 * FLOWMM_ERR_TIMEOUT in the status word at the start of `ws`, which flowmm_last_device_status then
 * reports and clears.  The CUDA context stays usable.
 */
flowmm_status flowmm_selftest_wait_timeout(void *ws, void *cuda_stream);

/* Number of kernels the most recent compute entry point of this thread enqueued. */
int32_t flowmm_last_launch_count(void);

/*
 * 1 if the library was compiled with -DFLOWMM_DEBUG, else 0.  The debug build stands in for a memory checker:
 * flowmm_match, flowmm_merge and flowmm_merge_static first check the index lists they are given (inside
 * [0, L), strictly ascending; matches inside [-1, B)), wait for that check and return FLOWMM_ERR_INDEX without
 * launching anything else when a list is bad; inside the kernels every index taken from a list or computed for a
 * gather is range-checked before use, a bad one is skipped and recorded as FLOWMM_ERR_INDEX in the status word.
 * Results of good inputs are the same as the release build's.
 */
int32_t flowmm_debug_build(void);

/*
 * Profiling aid, per host thread, off by default.  While on, every compute entry point records
 * a CUDA event on its stream before its first kernel and after each kernel (one extra event
 * record per launch).  flowmm_profile_read waits for the last of them and fills, in launch
 * order, a static kernel name and the kernel's duration in milliseconds for the most recent
 * entry point; it returns the number of entries written (0 when off, -1 on a CUDA error).
 * The first enable creates the events.
 */
flowmm_status flowmm_profile_enable(int32_t on);
int32_t flowmm_profile_read(const char **names, float *ms, int32_t max_entries);

/* Static, human-readable name of a status code. */
const char *flowmm_status_string(flowmm_status s);

#ifdef __cplusplus
}
#endif
#endif /* FLOWMM_H_ */
