/*
 * CPU oracle for one action-guided sparse denoising step (Sparse-WAM).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * method computes, written from the paper in fp64.  It shares no code with the
 * CUDA library and must never be used by the product path; only the tests, the
 * smoke check and the benchmark's CPU-baseline leg call it.
 *
 * Tensors are [B, n, N_h, D], token-major, passed as float32 (bf16 and fp32
 * inputs are both exactly representable in float32); all arithmetic is double.
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC
 * (-ffp-contract=off keeps every multiply and add separately rounded, which the
 * anchor statistic relies on for bit-reproducibility).
 *
 * Pins (tests, CPU only): attention against a library fp64 softmax-attention
 * and closed forms; score against the full-softmax definition (Eq. 1 + Eq. 2)
 * and the all-zero-query closed form; selection against a brute-force stable
 * sort, the all-equal closed form and the paper's set guarantees; maps against
 * their inverse/identity properties.  Unpinned: how well the sparse output
 * approximates the dense one (the paper reports task success only), which is
 * reported as a number and never asserted.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------
 * Softmax attention, plain definition (Sec. 3.1; the compact sequence of
 * Sec. 4.2 is the same operation on fewer tokens).
 *   x_c = scale * sum_d Q[r,d] K[c,d];  lambda_r = log sum_c exp(x_c)
 *   O[r,:] = sum_c exp(x_c - lambda_r) V[c,:]
 * The sums run over the keys visible to the row: all n of them when
 * key_limit is NULL (full visibility), else the first key_limit[i] keys of
 * the sequence for the i-th listed row (the backbone's visibility
 * constraints of App. A.2, read as: a token sees a prefix of the sequence).
 * rows: [n_rows, 2] pairs (b, r).  out_rows: [n_rows, N_h, D];
 * lse_rows: [n_rows, N_h] (may be NULL).
 * ------------------------------------------------------------------------ */
void oracle_attention_rows(const float* q, const float* k, const float* v,
                           int n, int n_heads, int head_dim, double scale,
                           const int32_t* rows, int64_t n_rows,
                           double* out_rows, double* lse_rows, const int32_t* key_limit)
{
    const int64_t tok = (int64_t)n_heads * head_dim;
    const int64_t work = n_rows * n_heads;
#pragma omp parallel
    {
        double* x = (double*)malloc(sizeof(double) * (size_t)n);
#pragma omp for schedule(dynamic, 4)
        for (int64_t w = 0; w < work; ++w) {
            const int64_t ri = w / n_heads;
            const int h = (int)(w % n_heads);
            const int64_t b = rows[2 * ri], r = rows[2 * ri + 1];
            const float* qr = q + (b * n + r) * tok + (int64_t)h * head_dim;
            const float* kb = k + b * n * tok + (int64_t)h * head_dim;
            const float* vb = v + b * n * tok + (int64_t)h * head_dim;
            const int nv = key_limit ? key_limit[ri] : n;   /* visible keys of this row */
            double m = -INFINITY;
            for (int c = 0; c < nv; ++c) {
                const float* kc = kb + (int64_t)c * tok;
                double dot = 0.0;
                for (int d = 0; d < head_dim; ++d) dot += (double)qr[d] * (double)kc[d];
                x[c] = scale * dot;
                if (x[c] > m) m = x[c];
            }
            double sum = 0.0;
            for (int c = 0; c < nv; ++c) sum += exp(x[c] - m);
            const double lambda = m + log(sum);
            double* o = out_rows + (ri * n_heads + h) * head_dim;
            for (int d = 0; d < head_dim; ++d) o[d] = 0.0;
            for (int c = 0; c < nv; ++c) {
                const double p = exp(x[c] - lambda);
                const float* vc = vb + (int64_t)c * tok;
                for (int d = 0; d < head_dim; ++d) o[d] += p * (double)vc[d];
            }
            if (lse_rows) lse_rows[ri * n_heads + h] = lambda;
        }
        free(x);
    }
}

/* ------------------------------------------------------------------------
 * Spatial score in the extraction form of Eq. 12:
 *   S(f,j) = 1/N_h * sum_{i in I_f} sum_h alpha_i exp(x_h(i,f,j) - lambda_h(i))
 * with I_f the f-th consecutive group of H/F action queries (Eq. 8) and
 * lambda the log-sum-exp over ALL keys of the full sequence.
 * q, k: full tensors [B, L, N_h, D], L = n_obs + F*N_s + H, order
 * [observed | future | action].  lse: [B, N_h, H].  alpha: [H/F].
 * scores: [B, F, N_s] double.
 * ------------------------------------------------------------------------ */
void oracle_score(const float* q, const float* k, const double* lse, const double* alpha,
                  int batch, int n_obs, int n_frames, int n_spatial, int n_action,
                  int n_heads, int head_dim, double scale, double* scores)
{
    const int64_t L = (int64_t)n_obs + (int64_t)n_frames * n_spatial + n_action;
    const int64_t tok = (int64_t)n_heads * head_dim;
    const int g = n_action / n_frames;
    const int64_t act0 = (int64_t)n_obs + (int64_t)n_frames * n_spatial;
    const int64_t work = (int64_t)batch * n_frames * n_spatial;
#pragma omp parallel for schedule(static)
    for (int64_t w = 0; w < work; ++w) {
        const int64_t b = w / ((int64_t)n_frames * n_spatial);
        const int f = (int)((w / n_spatial) % n_frames);
        const int j = (int)(w % n_spatial);
        const float* kt = k + (b * L + n_obs + (int64_t)f * n_spatial + j) * tok;
        double s = 0.0;
        for (int a = 0; a < g; ++a) {
            const int i = f * g + a;
            const float* qt = q + (b * L + act0 + i) * tok;
            for (int h = 0; h < n_heads; ++h) {
                double dot = 0.0;
                for (int d = 0; d < head_dim; ++d)
                    dot += (double)qt[h * head_dim + d] * (double)kt[h * head_dim + d];
                s += alpha[a] * exp(scale * dot - lse[(b * n_heads + h) * n_action + i]);
            }
        }
        scores[w] = s / (double)n_heads;
    }
}

/* Layer quality of Eq. 9 for one sample: R, E, Q = R (1 - E); 0 log 0 = 0. */
void oracle_quality(const float* scores, int n_frames, int n_spatial, double* rq /* [3] */)
{
    double total = 0.0, ent = 0.0;
    for (int f = 0; f < n_frames; ++f) {
        double fs = 0.0;
        for (int j = 0; j < n_spatial; ++j) fs += (double)scores[f * n_spatial + j];
        total += fs;
        for (int j = 0; j < n_spatial; ++j) {
            const double p = fs > 0.0 ? (double)scores[f * n_spatial + j] / fs : 0.0;
            if (p > 0.0) ent -= p * log(p);
        }
    }
    const double R = total / (double)n_frames;
    const double E = ent / ((double)n_frames * log((double)n_spatial));
    rq[0] = R; rq[1] = E; rq[2] = R * (1.0 - E);
}

/* ------------------------------------------------------------------------
 * TopK: indices of the n largest keys; equal keys go to the lower index.
 * Defined through a full sort by (key descending, index ascending).
 * ------------------------------------------------------------------------ */
typedef struct { double key; int idx; } keyed;

static int by_key_desc_idx_asc(const void* a, const void* b)
{
    const keyed* x = (const keyed*)a; const keyed* y = (const keyed*)b;
    if (x->key > y->key) return -1;
    if (x->key < y->key) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

/* sorts cand[0..n_cand) in place; the first n entries are the TopK; returns the relative gap between
 * the last kept and the first dropped key (infinity when nothing is dropped) */
static double topk_sorted(keyed* cand, int n_cand, int n)
{
    qsort(cand, (size_t)n_cand, sizeof(keyed), by_key_desc_idx_asc);
    if (n <= 0 || n >= n_cand) return INFINITY;
    const double in = cand[n - 1].key, out = cand[n].key;
    const double den = fabs(in) > 0.0 ? fabs(in) : 1.0;
    return (in - out) / den;
}

/* ------------------------------------------------------------------------
 * Selection for one sample with a single profiled layer, so V = V_all = S
 * (Eq. 3 and Eq. 11 reduce to S when only one layer contributes).
 *   pool  P   = TopK_j( max_f S(f,j), N_s - K_s )             (Eq. 4)
 *   core  C_f = TopK_{j in P}( S(f,j), K_c )                   (Eq. 5)
 *   E         = J \ union_f C_f                                (Eq. 10)
 *   mu_j = mean_f S(f,j); CV_j = Std_f / mu_j (population std; mu_j = 0 -> CV_j = 0)
 *   anchors A = TopK_{j in E}( mu_j / (1 + beta CV_j), K_s )   (Eq. 6, Eq. 11)
 *   retained_f = ascending( C_f  union  A ), exactly K_c + K_s  (Sec. 4.1)
 * scores are the fp32-stored values; pool and core rank them as they are,
 * the anchor key is computed in double in the order written below.
 * Outputs: sel_idx [F, K]; optional pool [N_s], core [F, N_s] (0/1), anchors
 * [K_s] (ascending), anchor_key [N_s], margins [3] = smallest relative gap at
 * the cut of the pool / core / anchor TopK.
 * ------------------------------------------------------------------------ */
void oracle_select(const float* scores, int n_frames, int n_spatial, int k_core, int k_anchor,
                   double beta, int32_t* sel_idx, uint8_t* pool_out, uint8_t* core_out,
                   int32_t* anchors_out, double* anchor_key_out, double* margins)
{
    const int F = n_frames, N = n_spatial, K = k_core + k_anchor;
    keyed* cand = (keyed*)malloc(sizeof(keyed) * (size_t)N);
    uint8_t* pool = (uint8_t*)calloc((size_t)N, 1);
    uint8_t* core = (uint8_t*)calloc((size_t)F * N, 1);
    uint8_t* in_any_core = (uint8_t*)calloc((size_t)N, 1);
    uint8_t* anchor = (uint8_t*)calloc((size_t)N, 1);
    double* akey = (double*)malloc(sizeof(double) * (size_t)N);
    double gap_pool = INFINITY, gap_core = INFINITY, gap_anchor = INFINITY;

    /* candidate pool */
    for (int j = 0; j < N; ++j) {
        double m = (double)scores[j];
        for (int f = 1; f < F; ++f) if ((double)scores[f * N + j] > m) m = (double)scores[f * N + j];
        cand[j].key = m; cand[j].idx = j;
    }
    gap_pool = topk_sorted(cand, N, N - k_anchor);
    for (int r = 0; r < N - k_anchor; ++r) pool[cand[r].idx] = 1;

    /* frame-specific core tokens */
    for (int f = 0; f < F; ++f) {
        int nc = 0;
        for (int j = 0; j < N; ++j) if (pool[j]) { cand[nc].key = (double)scores[f * N + j]; cand[nc].idx = j; ++nc; }
        const double gap = topk_sorted(cand, nc, k_core);
        if (gap < gap_core) gap_core = gap;
        for (int r = 0; r < k_core; ++r) { core[f * N + cand[r].idx] = 1; in_any_core[cand[r].idx] = 1; }
    }

    /* anchor statistic */
    for (int j = 0; j < N; ++j) {
        double sum = 0.0;
        for (int f = 0; f < F; ++f) sum = sum + (double)scores[f * N + j];
        const double mu = sum / (double)F;
        double ss = 0.0;
        for (int f = 0; f < F; ++f) { const double d = (double)scores[f * N + j] - mu; ss = ss + d * d; }
        const double sd = sqrt(ss / (double)F);
        const double cv = (mu == 0.0) ? 0.0 : sd / mu;
        akey[j] = mu / (1.0 + beta * cv);
    }
    int ne = 0;
    for (int j = 0; j < N; ++j) if (!in_any_core[j]) { cand[ne].key = akey[j]; cand[ne].idx = j; ++ne; }
    gap_anchor = topk_sorted(cand, ne, k_anchor);
    for (int r = 0; r < k_anchor; ++r) anchor[cand[r].idx] = 1;

    /* retained positions, ascending */
    for (int f = 0; f < F; ++f) {
        int n = 0;
        for (int j = 0; j < N; ++j) if (core[f * N + j] || anchor[j]) { if (n < K) sel_idx[f * K + n] = j; ++n; }
        if (n != K) sel_idx[0] = -1;  /* cannot happen: core and anchor sets are disjoint */
    }
    if (pool_out) memcpy(pool_out, pool, (size_t)N);
    if (core_out) memcpy(core_out, core, (size_t)F * N);
    if (anchors_out) { int n = 0; for (int j = 0; j < N; ++j) if (anchor[j]) anchors_out[n++] = j; }
    if (anchor_key_out) memcpy(anchor_key_out, akey, sizeof(double) * (size_t)N);
    if (margins) { margins[0] = gap_pool; margins[1] = gap_core; margins[2] = gap_anchor; }
    free(cand); free(pool); free(core); free(in_any_core); free(anchor); free(akey);
}

/* ------------------------------------------------------------------------
 * Packing metadata (Sec. 4.2): original positions of the compact sequence,
 *   pack_map = [observed rows] ++ [n_obs + f N_s + j for f, for j in retained_f] ++ [action rows]
 * and its inverse, -1 on omitted rows.
 * ------------------------------------------------------------------------ */
void oracle_maps(const int32_t* sel_idx, int n_obs, int n_frames, int n_spatial, int n_action, int k_keep,
                 int32_t* pack_map, int32_t* inv_map)
{
    const int L = n_obs + n_frames * n_spatial + n_action;
    int p = 0;
    for (int t = 0; t < L; ++t) inv_map[t] = -1;
    for (int t = 0; t < n_obs; ++t) pack_map[p++] = t;
    for (int f = 0; f < n_frames; ++f)
        for (int r = 0; r < k_keep; ++r) pack_map[p++] = n_obs + f * n_spatial + sel_idx[f * k_keep + r];
    for (int t = 0; t < n_action; ++t) pack_map[p++] = n_obs + n_frames * n_spatial + t;
    for (int i = 0; i < p; ++i) inv_map[pack_map[i]] = i;
}

/* ------------------------------------------------------------------------
 * Multi-layer aggregation for one sample (Eq. 3 and the first line of Eq. 11).
 * layer_scores: [n_layers, F*N_s] stored fp32 scores S_l; layer_q: [n_layers] layer qualities Q_l (Eq. 9).
 *   L_core = the k_layer layers with the largest Q_l (equal Q_l: lower layer index)
 *   V      = sum_{l in L_core} Q_l S_l / sum_{l in L_core} Q_l        (Eq. 3)
 *   V_all  = sum_l Q_l S_l / sum_l Q_l                               (Eq. 11)
 * Sums run over layers in ascending order in double; results are stored as fp32.  When the weights of a set
 * sum to zero (every layer uniform) the plain mean over that set is used.
 * core_layers: [k_layer] ascending layer indices (may be NULL).
 * ------------------------------------------------------------------------ */
void oracle_aggregate(const float* layer_scores, const float* layer_q, int n_layers, int k_layer, int n_elems,
                      float* v_core, float* v_all, int32_t* core_layers)
{
    keyed* cand = (keyed*)malloc(sizeof(keyed) * (size_t)n_layers);
    uint8_t* in_core = (uint8_t*)calloc((size_t)n_layers, 1);
    for (int l = 0; l < n_layers; ++l) { cand[l].key = (double)layer_q[l]; cand[l].idx = l; }
    qsort(cand, (size_t)n_layers, sizeof(keyed), by_key_desc_idx_asc);
    for (int r = 0; r < k_layer && r < n_layers; ++r) in_core[cand[r].idx] = 1;
    double wc = 0.0, wa = 0.0;
    int nc = 0;
    for (int l = 0; l < n_layers; ++l) {
        wa = wa + (double)layer_q[l];
        if (in_core[l]) { wc = wc + (double)layer_q[l]; ++nc; }
    }
    for (int e = 0; e < n_elems; ++e) {
        double sc = 0.0, sa = 0.0;
        for (int l = 0; l < n_layers; ++l) {
            const double s = (double)layer_scores[(size_t)l * n_elems + e];
            const double w = (double)layer_q[l];
            const double wa_l = (wa == 0.0) ? 1.0 : w;
            const double wc_l = (wc == 0.0) ? 1.0 : w;
            sa = sa + wa_l * s;
            if (in_core[l]) sc = sc + wc_l * s;
        }
        v_all[e] = (float)(sa / ((wa == 0.0) ? (double)n_layers : wa));
        v_core[e] = (float)(sc / ((wc == 0.0) ? (double)nc : wc));
    }
    if (core_layers) { int n = 0; for (int l = 0; l < n_layers; ++l) if (in_core[l]) core_layers[n++] = l; }
    free(cand); free(in_core);
}

/* Selection with separate score maps: pool and cores rank v_core (Eq. 4-5), anchors use v_all (Eq. 11, Eq. 6). */
void oracle_select2(const float* v_core, const float* v_all, int n_frames, int n_spatial, int k_core, int k_anchor,
                    double beta, int32_t* sel_idx)
{
    const int F = n_frames, N = n_spatial, K = k_core + k_anchor;
    keyed* cand = (keyed*)malloc(sizeof(keyed) * (size_t)N);
    uint8_t* pool = (uint8_t*)calloc((size_t)N, 1);
    uint8_t* core = (uint8_t*)calloc((size_t)F * N, 1);
    uint8_t* in_any_core = (uint8_t*)calloc((size_t)N, 1);
    uint8_t* anchor = (uint8_t*)calloc((size_t)N, 1);
    for (int j = 0; j < N; ++j) {
        double m = (double)v_core[j];
        for (int f = 1; f < F; ++f) if ((double)v_core[f * N + j] > m) m = (double)v_core[f * N + j];
        cand[j].key = m; cand[j].idx = j;
    }
    topk_sorted(cand, N, N - k_anchor);
    for (int r = 0; r < N - k_anchor; ++r) pool[cand[r].idx] = 1;
    for (int f = 0; f < F; ++f) {
        int nc = 0;
        for (int j = 0; j < N; ++j) if (pool[j]) { cand[nc].key = (double)v_core[f * N + j]; cand[nc].idx = j; ++nc; }
        topk_sorted(cand, nc, k_core);
        for (int r = 0; r < k_core; ++r) { core[f * N + cand[r].idx] = 1; in_any_core[cand[r].idx] = 1; }
    }
    int ne = 0;
    for (int j = 0; j < N; ++j) {
        if (in_any_core[j]) continue;
        double sum = 0.0;
        for (int f = 0; f < F; ++f) sum = sum + (double)v_all[f * N + j];
        const double mu = sum / (double)F;
        double ss = 0.0;
        for (int f = 0; f < F; ++f) { const double d = (double)v_all[f * N + j] - mu; ss = ss + d * d; }
        const double sd = sqrt(ss / (double)F);
        const double cv = (mu == 0.0) ? 0.0 : sd / mu;
        cand[ne].key = mu / (1.0 + beta * cv); cand[ne].idx = j; ++ne;
    }
    topk_sorted(cand, ne, k_anchor);
    for (int r = 0; r < k_anchor; ++r) anchor[cand[r].idx] = 1;
    for (int f = 0; f < F; ++f) {
        int n = 0;
        for (int j = 0; j < N; ++j) if (core[f * N + j] || anchor[j]) { if (n < K) sel_idx[f * K + n] = j; ++n; }
        if (n != K) sel_idx[0] = -1;
    }
    free(cand); free(pool); free(core); free(in_any_core); free(anchor);
}
