/*
 * FlowMM KV-cache compression: reference oracle (TEST INFRASTRUCTURE, not the product).
 *
 * A plain, slow, fp64 CPU restatement of the per-layer compression that FlowMM
 * runs once after multimodal prefill, written from the paper's definitions step
 * by step, in the paper's order.  It exists so that the CUDA library can be
 * checked against something that can be read against the paper by eye.  Only
 * the tests, the smoke check and the benchmark's CPU-baseline leg may call it;
 * it shares no code with the CUDA path and the CUDA path never calls it.
 *
 * Inputs are float32 arrays holding the exact values the GPU receives (for
 * bf16 workloads: bf16 values widened to float32); all arithmetic is double.
 * OpenMP only spreads independent work over cores: (unit, head) problems, or,
 * when a call has fewer of those than cores, the independent dot products of
 * one attention row and the independent non-pivot rows of the matching step.
 * Every value is computed by the same operations in the same order either way;
 * there is no blocking, fusion or reordering inside a problem.
 *
 * Steps (notation: unit u, query head g, KV head h = g / G, window row a at
 * prompt position p_a = L - W + a, token i, modality m[i] in {0 text, 1 visual}):
 *   score       Eq. 4 applied to the proxy rows of Eq. 8: causal logits
 *               s = scale * q.k, row softmax alpha, importance
 *               I[h,i] = (1/G) sum_{g in h} sum_a alpha[g,a,i]          (Eq. 8)
 *               and per head the cross-modal mass sum_a sum_{m_i != m_{p_a}} alpha
 *               and the total mass sum_a sum_i alpha                    (Eq. 7)
 *   layer_flow  rho = mean over heads of cross / total, strategy by theta (Eq. 6)
 *   select      top-B importance per KV head -> pivot set, rest non-pivot (Sec. 3.3.1)
 *   match       cosine similarity of each non-pivot key to the admissible
 *               pivots and its argmax                                   (Eq. 9, Eq. 10)
 *   merge       weighted consolidation of non-pivots into their pivots and
 *               compaction to B rows                                    (Eq. 5)
 *   decode      (the step after the path) one new query's attention over the
 *               cache, full or compressed                               (Eq. 4)
 *
 * Readings where the paper is silent (all listed in the design notes): group
 * mean for GQA importance; rho restricted to the proxy rows; rho == theta is
 * intra-modal; intra-modal merging only pairs tokens of equal modality; the
 * gate I_j <= tau applies to pivots; ties go to the lower index; a non-pivot
 * without an admissible pivot is dropped; merge weights are 1 for the pivot and
 * exp(u - 1) for a non-pivot with similarity u (or all 1 in MEAN mode),
 * normalised to sum to one.  PARITY UNPINNED for those merge weights, the
 * keep_window option and the scale of tau: the paper gives no value or formula.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t n_units, n_q_heads, n_kv_heads, head_dim, seq_len, window, n_keep;
    double softmax_scale;   /* 0 -> 1/sqrt(head_dim) */
    double theta, tau;
    int32_t tau_mode;       /* 0 absolute, 1 relative: tau_eff = tau * W / L */
    int32_t flow_mode;      /* 0 auto, 1 force intra, 2 force cross, 3 misaligned (the reverse of auto) */
    int32_t merge_mode;     /* 0 exp-similarity weights, 1 uniform mean */
    int32_t keep_window;    /* 1: the last W tokens are always pivots */
} oracle_params;

int flowmm_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static double dotd(const float *a, const float *b, int n)
{
    double s = 0.0;
    for (int c = 0; c < n; ++c) s += (double)a[c] * (double)b[c];
    return s;
}

/* Eq. 9 for one pair of rows; a zero-norm row has similarity 0 to everything. */
double flowmm_oracle_cosine(int32_t head_dim, const float *ki, const float *kj)
{
    double ni = sqrt(dotd(ki, ki, head_dim));
    double nj = sqrt(dotd(kj, kj, head_dim));
    if (ni == 0.0 || nj == 0.0) return 0.0;
    return dotd(ki, kj, head_dim) / (ni * nj);
}

/*
 * Eq. 8 (with the softmax of Eq. 4) and the masses of Eq. 7, proxy rows only.
 * q [U,Hq,W,D], k [U,Hkv,L,D], modality [U,L] ->
 * importance [U,Hkv,L], cross [U,Hq], total [U,Hq].
 */
int flowmm_oracle_score(const oracle_params *p, const float *q, const float *k, const uint8_t *modality,
                        double *importance, double *cross, double *total)
{
    const int U = p->n_units, Hq = p->n_q_heads, Hkv = p->n_kv_heads, D = p->head_dim;
    const int L = p->seq_len, W = p->window;
    if (Hkv <= 0 || Hq % Hkv != 0 || W < 1 || W > L) return 1;
    const int G = Hq / Hkv;
    const double scale = p->softmax_scale != 0.0 ? p->softmax_scale : 1.0 / sqrt((double)D);
    /* few (unit, head) problems: the cores share the independent logits of one row instead */
    const int by_head = U * Hkv >= flowmm_oracle_threads();

#pragma omp parallel for collapse(2) schedule(dynamic, 1) if (by_head)
    for (int u = 0; u < U; ++u) {
        for (int h = 0; h < Hkv; ++h) {
            const uint8_t *m = modality + (size_t)u * L;
            const float *kh = k + ((size_t)u * Hkv + h) * (size_t)L * D;
            double *imp = importance + ((size_t)u * Hkv + h) * (size_t)L;
            double *alpha = (double *)malloc(sizeof(double) * (size_t)L);
            for (int i = 0; i < L; ++i) imp[i] = 0.0;
            for (int g = h * G; g < (h + 1) * G; ++g) {
                double cr = 0.0, tot = 0.0;
                for (int a = 0; a < W; ++a) {
                    const int pa = L - W + a;               /* prompt position of this proxy token */
                    const float *qa = q + (((size_t)u * Hq + g) * W + a) * (size_t)D;
                    double mx = -INFINITY;
#pragma omp parallel for schedule(static) if (!by_head)
                    for (int i = 0; i <= pa; ++i)            /* causal: keys after p_a are masked */
                        alpha[i] = scale * dotd(qa, kh + (size_t)i * D, D);
                    for (int i = 0; i <= pa; ++i)
                        if (alpha[i] > mx) mx = alpha[i];
                    double z = 0.0;
                    for (int i = 0; i <= pa; ++i) { alpha[i] = exp(alpha[i] - mx); z += alpha[i]; }
                    for (int i = 0; i <= pa; ++i) {
                        const double al = alpha[i] / z;
                        imp[i] += al;
                        tot += al;
                        if (m[i] != m[pa]) cr += al;
                    }
                }
                cross[(size_t)u * Hq + g] = cr;
                total[(size_t)u * Hq + g] = tot;
            }
            for (int i = 0; i < L; ++i) imp[i] /= (double)G;   /* group mean */
            free(alpha);
        }
    }
    return 0;
}

/* Eq. 6 and the threshold rule that follows Eq. 7: strategy 1 = cross-modal, 0 = intra-modal. */
int flowmm_oracle_layer_flow(const oracle_params *p, const double *cross, const double *total,
                             double *rho, int32_t *strategy)
{
    const int U = p->n_units, Hq = p->n_q_heads;
    for (int u = 0; u < U; ++u) {
        double s = 0.0;
        for (int g = 0; g < Hq; ++g) {
            const double t = total[(size_t)u * Hq + g];
            s += t > 0.0 ? cross[(size_t)u * Hq + g] / t : 0.0;
        }
        rho[u] = s / (double)Hq;
        if (p->flow_mode == 1) strategy[u] = 0;
        else if (p->flow_mode == 2) strategy[u] = 1;
        else if (p->flow_mode == 3) strategy[u] = rho[u] > p->theta ? 0 : 1;   /* the misaligned contrast of the flow-merging study */
        else strategy[u] = rho[u] > p->theta ? 1 : 0;
    }
    return 0;
}

typedef struct { double imp; int32_t idx; int32_t forced; } rank_item;

static int rank_cmp(const void *pa, const void *pb)
{
    const rank_item *a = (const rank_item *)pa, *b = (const rank_item *)pb;
    if (a->forced != b->forced) return b->forced - a->forced;   /* forced pivots first */
    if (a->imp > b->imp) return -1;                             /* importance descending */
    if (a->imp < b->imp) return 1;
    return a->idx - b->idx;                                     /* ties: lower index first */
}

static int int_cmp(const void *pa, const void *pb)
{
    return *(const int32_t *)pa - *(const int32_t *)pb;
}

/* Pivot selection (Sec. 3.3.1): top-B importance per KV head; both index lists ascending. */
int flowmm_oracle_select(const oracle_params *p, const double *importance,
                         int32_t *retained, int32_t *evicted)
{
    const int U = p->n_units, Hkv = p->n_kv_heads, L = p->seq_len, W = p->window, B = p->n_keep;
    if (B < 1 || B > L) return 3;
    if (p->keep_window && B < W) return 3;
    const int E = L - B;
#pragma omp parallel for collapse(2)
    for (int u = 0; u < U; ++u) {
        for (int h = 0; h < Hkv; ++h) {
            const double *imp = importance + ((size_t)u * Hkv + h) * (size_t)L;
            rank_item *it = (rank_item *)malloc(sizeof(rank_item) * (size_t)L);
            for (int i = 0; i < L; ++i) {
                it[i].imp = imp[i];
                it[i].idx = i;
                it[i].forced = (p->keep_window && i >= L - W) ? 1 : 0;
            }
            qsort(it, (size_t)L, sizeof(rank_item), rank_cmp);
            int32_t *r = retained + ((size_t)u * Hkv + h) * (size_t)B;
            int32_t *e = evicted + ((size_t)u * Hkv + h) * (size_t)E;
            for (int j = 0; j < B; ++j) r[j] = it[j].idx;
            for (int j = 0; j < E; ++j) e[j] = it[B + j].idx;
            qsort(r, (size_t)B, sizeof(int32_t), int_cmp);
            if (E > 0) qsort(e, (size_t)E, sizeof(int32_t), int_cmp);
            free(it);
        }
    }
    return 0;
}

static double tau_effective(const oracle_params *p)
{
    return p->tau_mode == 1 ? p->tau * (double)p->window / (double)p->seq_len : p->tau;
}

/*
 * Eq. 9 and Eq. 10: for every non-pivot e the admissible pivot of largest
 * cosine similarity.  Admissible: importance <= tau_eff, and of e's modality
 * when the unit's strategy is intra-modal.  match = slot in [0,B) or -1,
 * sim = the winning similarity (0 when there is none), runner_up = the second
 * largest admissible similarity (-2 when there is none; used by tests to
 * measure how close a decision was).  row_select (optional, [U,Hkv,E] bytes)
 * limits the work to the non-pivots whose byte is non-zero; the others are
 * marked match = -2.
 */
int flowmm_oracle_match(const oracle_params *p, const float *k, const double *importance, const uint8_t *modality,
                        const int32_t *retained, const int32_t *evicted, const int32_t *strategy,
                        const uint8_t *row_select, int32_t *match, double *sim, double *runner_up)
{
    const int U = p->n_units, Hkv = p->n_kv_heads, D = p->head_dim, L = p->seq_len, B = p->n_keep;
    const int E = L - B;
    const double tau = tau_effective(p);
    /* every non-pivot row of every (unit, head) is an independent problem */
    const long long n_rows = (long long)U * Hkv * E;
#pragma omp parallel for schedule(dynamic, 16)
    for (long long row = 0; row < n_rows; ++row) {
        const int j = (int)(row % E);
        const int h = (int)(row / E % Hkv);
        const int u = (int)(row / E / Hkv);
        const uint8_t *m = modality + (size_t)u * L;
        const float *kh = k + ((size_t)u * Hkv + h) * (size_t)L * D;
        const double *imp = importance + ((size_t)u * Hkv + h) * (size_t)L;
        const int32_t *r = retained + ((size_t)u * Hkv + h) * (size_t)B;
        const int32_t *ev = evicted + ((size_t)u * Hkv + h) * (size_t)E;
        const size_t base = ((size_t)u * Hkv + h) * (size_t)E;
        if (row_select && !row_select[base + j]) {
            match[base + j] = -2; sim[base + j] = 0.0;
            if (runner_up) runner_up[base + j] = -2.0;
            continue;
        }
        const int e = ev[j];
        int best = -1;
        double ubest = 0.0, usecond = -2.0;
        for (int s = 0; s < B; ++s) {
            const int rs = r[s];
            if (!(imp[rs] <= tau)) continue;                       /* highly sensitive pivot: kept intact */
            if (strategy[u] == 0 && m[rs] != m[e]) continue;       /* intra-modal layer */
            const double us = flowmm_oracle_cosine(D, kh + (size_t)e * D, kh + (size_t)rs * D);
            if (best < 0) { best = s; ubest = us; }
            else if (us > ubest) { usecond = ubest; best = s; ubest = us; }   /* strict: ties keep lower slot */
            else if (us > usecond) usecond = us;
        }
        match[base + j] = best;
        sim[base + j] = best >= 0 ? ubest : 0.0;
        if (runner_up) runner_up[base + j] = usecond;
    }
    return 0;
}

/*
 * Eq. 5 with the weights stated in the header, then compaction: slot s of the
 * output holds pivot r_s merged with every non-pivot matched to it, taken in
 * ascending token order.  k, v [U,Hkv,L,D] -> k_out, v_out [U,Hkv,B,D] (double).
 * weight_sum (optional) [U,Hkv,B] returns each slot's normaliser Z_s.
 */
int flowmm_oracle_merge(const oracle_params *p, const float *k, const float *v,
                        const int32_t *retained, const int32_t *evicted, const int32_t *match, const double *sim,
                        double *k_out, double *v_out, double *weight_sum)
{
    const int U = p->n_units, Hkv = p->n_kv_heads, D = p->head_dim, L = p->seq_len, B = p->n_keep;
    const int E = L - B;
#pragma omp parallel for collapse(2)
    for (int u = 0; u < U; ++u) {
        for (int h = 0; h < Hkv; ++h) {
            const size_t uh = (size_t)u * Hkv + h;
            const float *kh = k + uh * (size_t)L * D;
            const float *vh = v + uh * (size_t)L * D;
            const int32_t *r = retained + uh * (size_t)B;
            const int32_t *ev = evicted + uh * (size_t)E;
            double *ko = k_out + uh * (size_t)B * D;
            double *vo = v_out + uh * (size_t)B * D;
            double *z = (double *)malloc(sizeof(double) * (size_t)B);
            for (int s = 0; s < B; ++s) {                 /* the pivot itself, weight 1 */
                z[s] = 1.0;
                for (int c = 0; c < D; ++c) {
                    ko[(size_t)s * D + c] = (double)kh[(size_t)r[s] * D + c];
                    vo[(size_t)s * D + c] = (double)vh[(size_t)r[s] * D + c];
                }
            }
            for (int j = 0; j < E; ++j) {                 /* non-pivots in ascending token order */
                const int s = match[uh * (size_t)E + j];
                if (s < 0) continue;                      /* no admissible pivot: dropped */
                const int e = ev[j];
                const double w = p->merge_mode == 1 ? 1.0 : exp(sim[uh * (size_t)E + j] - 1.0);
                z[s] += w;
                for (int c = 0; c < D; ++c) {
                    ko[(size_t)s * D + c] += w * (double)kh[(size_t)e * D + c];
                    vo[(size_t)s * D + c] += w * (double)vh[(size_t)e * D + c];
                }
            }
            for (int s = 0; s < B; ++s) {
                for (int c = 0; c < D; ++c) {
                    ko[(size_t)s * D + c] /= z[s];
                    vo[(size_t)s * D + c] /= z[s];
                }
                if (weight_sum) weight_sum[uh * (size_t)B + s] = z[s];
            }
            free(z);
        }
    }
    return 0;
}

/*
 * Decode-step attention over a (compressed or full) cache, Eq. 4: for the one new query of head g,
 * o = softmax(q . K^T / sqrt(d)) V over the n_keys rows of its KV head h = g / G.  No mask: the
 * query comes after every cached token.  scale 0 selects 1/sqrt(head_dim).
 *   q   [U, Hq, D]      k, v [U, Hkv, n_keys, D]      out [U, Hq, D] (double)
 */
int flowmm_oracle_decode_attention(int32_t n_units, int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim,
                                   int32_t n_keys, double scale, const float *q, const float *k, const float *v,
                                   double *out)
{
    if (n_units < 1 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads != 0 || head_dim < 1 || n_keys < 1)
        return 1;
    const int G = n_q_heads / n_kv_heads, D = head_dim, N = n_keys;
    if (scale == 0.0) scale = 1.0 / sqrt((double)D);
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int u = 0; u < n_units; ++u) {
        for (int g = 0; g < n_q_heads; ++g) {
            const int h = g / G;
            const float *qg = q + ((size_t)u * n_q_heads + g) * D;
            const float *kh = k + ((size_t)u * n_kv_heads + h) * (size_t)N * D;
            const float *vh = v + ((size_t)u * n_kv_heads + h) * (size_t)N * D;
            double *o = out + ((size_t)u * n_q_heads + g) * D;
            double *s = (double *)malloc(sizeof(double) * (size_t)N);
            double mx = -INFINITY;
            for (int i = 0; i < N; ++i) {
                s[i] = scale * dotd(qg, kh + (size_t)i * D, D);
                if (s[i] > mx) mx = s[i];
            }
            double z = 0.0;
            for (int i = 0; i < N; ++i) { s[i] = exp(s[i] - mx); z += s[i]; }
            for (int c = 0; c < D; ++c) o[c] = 0.0;
            for (int i = 0; i < N; ++i) {
                const double a = s[i] / z;
                for (int c = 0; c < D; ++c) o[c] += a * (double)vh[(size_t)i * D + c];
            }
            free(s);
        }
    }
    return 0;
}
