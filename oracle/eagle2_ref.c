/*
 * EAGLE-2 draft-and-verify hot path: plain CPU oracle.
 *
 * THIS IS TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  It exists so that the CUDA
 * library can be checked element by element against an implementation that a
 * reader can compare with the paper by eye.  Only the tests, the smoke check
 * and the CPU-baseline leg of the benchmark may call it.  It shares no code,
 * header, table or constant generator with the CUDA library.
 *
 * Everything is computed in double precision on the same fp32 / bf16 arrays
 * the GPU sees.  There is no blocking, fusion or reordering beyond what the
 * definitions state; the only concession to speed is an OpenMP loop over
 * independent sequences (or independent queries in attention).
 *
 * Index conventions (shared with the CUDA library because they are part of the
 * interface, not of the arithmetic):
 *   level l = 1..D.  Level-1 nodes have candidate index c in [0,k).
 *   A level-l node (l >= 2) has index  k + (l-2)k^2 + j*k + c  where j is the
 *   slot of its parent in the frontier chosen from level l-1 and c is the rank
 *   of the child within its parent's draft distribution.  parent = -1 is the
 *   root (the last committed token).  Draft row 0 produces level 1; draft row
 *   1 + (s-1)k + j is the row of frontier slot j at expansion step s >= 1.
 *   N = k + (D-1)k^2 candidate nodes, R = 1 + (D-1)k draft rows per cycle.
 *
 * Parity pins (tests/test_oracle_*.py): log-softmax and per-row top-k against
 * numpy/scipy; node values against brute-force products of probabilities
 * along every root path (Section 4.1 value equation); frontier and rerank
 * selection against brute-force sorts, the closure invariant of Section 4.2
 * and exhaustive optimality over connected subsets; the mask against the
 * ancestor definition of Section 4.2 and the causal special case; attention
 * against closed forms and a library causal attention; greedy acceptance
 * against brute force; temperature-1 acceptance against exact enumeration of
 * the output law, the chain rule of Section 2.1 and a chi-square test; the
 * LM head against a library matrix product.
 * The worked example of the paper's method figure is an image that is not
 * available, so no printed value pins the oracle: "parity unpinned" by
 * printed values for that example only.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ST_NONFINITE_LOGIT 1
#define ST_NOT_CLOSED 2
#define ST_KV_OVERFLOW 4
#define ST_BAD_TREE 32

#define ERR_NULL (-1)
#define ERR_SHAPE (-2)

static long long n_nodes(int k, int D) { return (long long)k + (long long)(D - 1) * k * k; }

/* level (1-based) of candidate index i */
static int level_of(int i, int k) { return i < k ? 1 : 2 + (i - k) / (k * k); }

/* ---------- small helpers ------------------------------------------------ */

typedef struct {
    double key;
    int idx;
} keyed_t;

/* descending key, ascending index on equal keys */
static int cmp_desc_key_asc_idx(const void* a, const void* b) {
    const keyed_t* x = (const keyed_t*)a;
    const keyed_t* y = (const keyed_t*)b;
    if (x->key > y->key) return -1;
    if (x->key < y->key) return 1;
    return (x->idx > y->idx) - (x->idx < y->idx);
}

static int cmp_int_asc(const void* a, const void* b) {
    int x = *(const int*)a, y = *(const int*)b;
    return (x > y) - (x < y);
}

/* log sum_v exp(z_v) in double; returns 0 on success, 1 if a logit is NaN or +Inf. */
static int log_sum_exp(const float* z, int V, double inv_t, double* out) {
    double mx = -INFINITY;
    for (int v = 0; v < V; ++v) {
        double x = (double)z[v] * inv_t;
        if (isnan(x) || x == INFINITY) return 1;
        if (x > mx) mx = x;
    }
    if (mx == -INFINITY) return 1; /* every logit is -Inf: no distribution */
    double sum = 0.0;
    for (int v = 0; v < V; ++v) sum += exp((double)z[v] * inv_t - mx);
    *out = mx + log(sum);
    return 0;
}

/* ---------- step 1: expansion (Section 4.1) ------------------------------ */
/*
 * For every input row: log-softmax over the vocabulary, the k most probable
 * tokens become children (ties: lower token id), child value = parent value +
 * log-probability (the log of the product in the value equation; the root
 * contributes a factor 1).  Then the k best new candidates by value (ties:
 * lower candidate index) become the next frontier.
 */
static int expand_impl(const float* draft_logits, long long batch_stride, int B, int V, int k, int D,
                       int s, int by_confidence, int32_t* tree_token, int32_t* tree_parent,
                       double* tree_value, int32_t* frontier, int32_t* status) {
    if (!draft_logits || !tree_token || !tree_parent || !tree_value || !frontier || !status)
        return ERR_NULL;
    if (B < 0 || V < 1 || k < 1 || k > V || D < 1 || s < 0 || s >= D) return ERR_SHAPE;
    const long long N = n_nodes(k, D);
    const int n_rows = s ? k : 1;
    const long long base = s ? (long long)k + (long long)(s - 1) * k * k : 0;

#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        const float* rows = draft_logits + (long long)b * batch_stride;
        int32_t* tok = tree_token + (long long)b * N;
        int32_t* par = tree_parent + (long long)b * N;
        double* val = tree_value + (long long)b * N;
        int32_t* fr = frontier + (long long)b * k;
        keyed_t* order = (keyed_t*)malloc(sizeof(keyed_t) * (size_t)V);
        double* conf = (double*)malloc(sizeof(double) * (size_t)n_rows * (size_t)k);
        int st = 0;

        for (int r = 0; r < n_rows; ++r) {
            const float* z = rows + (long long)r * V;
            const int parent = s ? fr[r] : -1;
            const double parent_value = s ? val[parent] : 0.0;
            double lse = 0.0;
            if (log_sum_exp(z, V, 1.0, &lse)) {
                st |= ST_NONFINITE_LOGIT;
                lse = NAN;
            }
            for (int v = 0; v < V; ++v) {
                order[v].key = (double)z[v];
                order[v].idx = v;
            }
            qsort(order, (size_t)V, sizeof(keyed_t), cmp_desc_key_asc_idx);
            for (int c = 0; c < k; ++c) {
                const long long node = base + (long long)r * k + c;
                tok[node] = order[c].idx;
                par[node] = parent;
                val[node] = parent_value + (order[c].key - lse);
                conf[r * k + c] = order[c].key - lse; /* the node's own confidence, log c_i */
            }
        }
        free(order);

        /* next frontier: best k of this step's k*n_rows new candidates */
        const int n_new = n_rows * k;
        keyed_t* cand = (keyed_t*)malloc(sizeof(keyed_t) * (size_t)n_new);
        for (int i = 0; i < n_new; ++i) {
            cand[i].key = by_confidence ? conf[i] : val[base + i];
            cand[i].idx = (int)(base + i);
        }
        qsort(cand, (size_t)n_new, sizeof(keyed_t), cmp_desc_key_asc_idx);
        for (int j = 0; j < k; ++j) fr[j] = cand[j].idx;
        free(cand);
        free(conf);
        if (st) {
#pragma omp atomic
            *status |= st;
        }
    }
    return 0;
}

int eagle2_expand_ref(const float* draft_logits, long long batch_stride, int B, int V, int k, int D,
                      int s, int32_t* tree_token, int32_t* tree_parent, double* tree_value,
                      int32_t* frontier, int32_t* status) {
    return expand_impl(draft_logits, batch_stride, B, V, k, D, s, 0, tree_token, tree_parent, tree_value,
                       frontier, status);
}

/*
 * The ablation of Section 5.2 "w/o value", which the text describes as expanding on the confidence
 * score instead of the value: with by_confidence != 0 the k nodes to expand next are the step's best
 * by their own confidence c_i (the draft model's probability of the token given its path) instead
 * of by V_i, the product of the confidences along the path.  Only that choice changes: the stored
 * value of every node is still V_i, so a later reranking ranks by value as the paper's reranking
 * does.  by_confidence == 0 is eagle2_expand_ref.
 */
int eagle2_expand_variant_ref(const float* draft_logits, long long batch_stride, int B, int V, int k,
                              int D, int s, int by_confidence, int32_t* tree_token,
                              int32_t* tree_parent, double* tree_value, int32_t* frontier,
                              int32_t* status) {
    return expand_impl(draft_logits, batch_stride, B, V, k, D, s, by_confidence != 0, tree_token, tree_parent,
                       tree_value, frontier, status);
}

/* ---------- step 2a: reranking (Section 4.2) ----------------------------- */
/*
 * Top-m of all candidate nodes by value; equal values prefer the shallower
 * node, which under level-major indexing is the lower index.  The effective
 * value min(value, effective value of the parent) equals the value itself for
 * trees built by the expansion above (a node never beats its parent) and
 * makes the closure property hold for arbitrary caller-supplied values.
 * The selection is emitted in ascending candidate index, a topological order.
 */
static int rerank_impl(const int32_t* tree_token, const int32_t* tree_parent,
                       const double* tree_value, const int32_t* frontier, int B, int k, int D, int m,
                       int32_t* sel_index, int32_t* sel_parent, int32_t* sel_token,
                       int32_t* sel_depth, int32_t* n_sel, int32_t* status) {
    if (!tree_token || !tree_parent || !tree_value || !sel_index || !sel_parent || !sel_token ||
        !sel_depth || !n_sel || !status)
        return ERR_NULL;
    if (B < 0 || k < 1 || D < 1 || m < 1) return ERR_SHAPE;
    const long long N = n_nodes(k, D);
    const int most = (long long)m < N ? m : (int)N;

#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        int keep = most;
        const int32_t* tok = tree_token + (long long)b * N;
        const int32_t* par = tree_parent + (long long)b * N;
        const double* val = tree_value + (long long)b * N;
        int st = 0;
        double* v_eff = (double*)malloc(sizeof(double) * (size_t)N);
        keyed_t* order = (keyed_t*)malloc(sizeof(keyed_t) * (size_t)N);
        int* flat_of = (int*)malloc(sizeof(int) * (size_t)N);
        int* chosen = (int*)malloc(sizeof(int) * (size_t)most);

        for (int i = 0; i < N; ++i) {
            int p = par[i];
            if (p < -1 || p >= i) { /* parents precede children in level-major order */
                st |= ST_BAD_TREE;
                p = -1;
            }
            double v = val[i];
            if (isnan(v)) {
                st |= ST_NONFINITE_LOGIT;
                v = -INFINITY;
            }
            v_eff[i] = (p >= 0 && v_eff[p] < v) ? v_eff[p] : v;
            order[i].key = v_eff[i];
            order[i].idx = i;
            flat_of[i] = -1;
        }
        if (!frontier) {
            qsort(order, (size_t)N, sizeof(keyed_t), cmp_desc_key_asc_idx);
            for (int j = 0; j < keep; ++j) chosen[j] = order[j].idx;
            qsort(chosen, (size_t)keep, sizeof(int), cmp_int_asc);
        } else {
            /* No reranking: the draft is what the expansion phase itself selected, the frontier of
             * every step.  A frontier node of an earlier step is one that was expanded, i.e. one
             * that some node names as its parent; the last step's frontier is passed in.  Lowest
             * indices (shallowest) first if there are more than m. */
            char* picked = (char*)calloc((size_t)N, 1);
            for (int i = 0; i < N; ++i) {
                const int p = par[i];
                if (p >= 0 && p < i) picked[p] = 1;
            }
            for (int j = 0; j < k; ++j) {
                const int f = frontier[(long long)b * k + j];
                if (f < 0 || f >= N) st |= ST_BAD_TREE;
                else picked[f] = 1;
            }
            keep = 0;
            for (int i = 0; i < N && keep < most; ++i)
                if (picked[i]) chosen[keep++] = i;
            free(picked);
        }
        for (int j = 0; j < keep; ++j) flat_of[chosen[j]] = j;

        int32_t* o_idx = sel_index + (long long)b * m;
        int32_t* o_par = sel_parent + (long long)b * m;
        int32_t* o_tok = sel_token + (long long)b * m;
        int32_t* o_dep = sel_depth + (long long)b * m;
        for (int j = 0; j < m; ++j) {
            if (j < keep) {
                const int i = chosen[j];
                int p = par[i];
                if (p < -1 || p >= i) p = -1;
                o_idx[j] = i;
                o_tok[j] = tok[i];
                o_dep[j] = level_of(i, k) - 1;
                if (p < 0) {
                    o_par[j] = -1;
                } else if (flat_of[p] >= 0) {
                    o_par[j] = flat_of[p];
                } else {
                    st |= ST_NOT_CLOSED;
                    o_par[j] = -1;
                }
            } else { /* padding rows */
                o_idx[j] = -1;
                o_par[j] = -1;
                o_tok[j] = 0;
                o_dep[j] = 0;
            }
        }
        n_sel[b] = keep;
        free(v_eff);
        free(order);
        free(flat_of);
        free(chosen);
        if (st) {
#pragma omp atomic
            *status |= st;
        }
    }
    return 0;
}

int eagle2_rerank_ref(const int32_t* tree_token, const int32_t* tree_parent,
                      const double* tree_value, int B, int k, int D, int m, int32_t* sel_index,
                      int32_t* sel_parent, int32_t* sel_token, int32_t* sel_depth, int32_t* n_sel,
                      int32_t* status) {
    return rerank_impl(tree_token, tree_parent, tree_value, NULL, B, k, D, m, sel_index, sel_parent,
                       sel_token, sel_depth, n_sel, status);
}

/*
 * The ablation of Section 5.2 "w/o reranking": the tree sent to verification is the set of nodes the
 * expansion phase selected (k per step, at most kD), flattened exactly as above.  `frontier` is the
 * last step's frontier [B][k].  The paper does not spell this set out; this is the reading taken.
 */
int eagle2_rerank_skipped_ref(const int32_t* tree_token, const int32_t* tree_parent,
                              const double* tree_value, const int32_t* frontier, int B, int k, int D,
                              int m, int32_t* sel_index, int32_t* sel_parent, int32_t* sel_token,
                              int32_t* sel_depth, int32_t* n_sel, int32_t* status) {
    if (!frontier) return ERR_NULL;
    return rerank_impl(tree_token, tree_parent, tree_value, frontier, B, k, D, m, sel_index, sel_parent,
                       sel_token, sel_depth, n_sel, status);
}

/* ---------- step 2b: tree mask and position ids (Section 4.2) ------------ */
/*
 * Row i of the mask holds bit i and the bit of every ancestor of i: a draft
 * token sees itself and its ancestors only.  Position id = committed length +
 * depth (the root is the last committed token, so a level-1 node is the next
 * position).  Padding rows (>= n_sel) see only themselves.
 */
int eagle2_tree_mask_ref(const int32_t* sel_parent, const int32_t* sel_depth, const int32_t* n_sel,
                         const int32_t* kv_len, int B, int m, uint64_t* mask_bits,
                         uint8_t* mask_dense, int32_t* pos_ids, int32_t* status) {
    if (!sel_parent || !sel_depth || !n_sel || !kv_len || !mask_bits || !pos_ids || !status)
        return ERR_NULL;
    if (B < 0 || m < 1) return ERR_SHAPE;
    const int W = (m + 63) / 64;
    for (int b = 0; b < B; ++b) {
        const int32_t* par = sel_parent + (long long)b * m;
        const int32_t* dep = sel_depth + (long long)b * m;
        uint64_t* bits = mask_bits + (long long)b * m * W;
        const int ns = n_sel[b];
        for (int i = 0; i < m; ++i) {
            uint64_t* row = bits + (long long)i * W;
            for (int w = 0; w < W; ++w) row[w] = 0;
            int a = i;
            int steps = 0;
            while (a >= 0) {
                row[a / 64] |= (uint64_t)1 << (a % 64);
                if (i >= ns) break;
                const int p = par[a];
                if (p >= a || p < -1 || ++steps > m) {
                    *status |= ST_BAD_TREE;
                    break;
                }
                a = p;
            }
            pos_ids[(long long)b * m + i] = kv_len[b] + (i < ns ? dep[i] : 0);
            if (mask_dense) {
                uint8_t* drow = mask_dense + ((long long)b * m + i) * m;
                for (int j = 0; j < m; ++j) drow[j] = (uint8_t)((row[j / 64] >> (j % 64)) & 1);
            }
        }
    }
    return 0;
}

/* ---------- step 3: tree-masked attention (Section 4.2) ------------------ */

static double bf16_to_double(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* round to nearest even bf16 */
static uint16_t double_to_bf16(double x) {
    float f = (float)x;
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40); /* NaN */
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

/*
 * One query row: softmax over the visible keys of (scale * q.k), times v.
 * Visible keys of tree token i of sequence b: every committed cache row
 * [0, L_b) and the tree rows j whose bit is set in mask row i; the K/V of
 * tree row j sit at local cache row L_b + j.
 */
static void attention_one_query(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                                const int64_t* kv_off, const int32_t* kv_len,
                                const uint64_t* mask_bits, int m, int Hq, int Hkv, int d,
                                double scale, int b, int h, int i, double* out, double* lse_out) {
    const int W = (m + 63) / 64;
    const int g = Hq / Hkv;
    const int hk = h / g;
    const int L = kv_len[b];
    const int n_keys = L + m;
    const uint16_t* qv = q + (((long long)b * m + i) * Hq + h) * d;
    const uint64_t* mrow = mask_bits + ((long long)b * m + i) * W;
    double* score = (double*)malloc(sizeof(double) * (size_t)n_keys);
    double mx = -INFINITY;
    for (int j = 0; j < n_keys; ++j) {
        int visible = j < L;
        if (!visible) {
            const int t = j - L;
            visible = (int)((mrow[t / 64] >> (t % 64)) & 1);
        }
        if (!visible) {
            score[j] = -INFINITY;
            continue;
        }
        const uint16_t* kv = k_cache + ((kv_off[b] + j) * Hkv + hk) * (long long)d;
        double dot = 0.0;
        for (int e = 0; e < d; ++e) dot += bf16_to_double(qv[e]) * bf16_to_double(kv[e]);
        score[j] = scale * dot;
        if (score[j] > mx) mx = score[j];
    }
    double denom = 0.0;
    for (int e = 0; e < d; ++e) out[e] = 0.0;
    for (int j = 0; j < n_keys; ++j) {
        if (score[j] == -INFINITY) continue;
        const double w = exp(score[j] - mx);
        denom += w;
        const uint16_t* vv = v_cache + ((kv_off[b] + j) * Hkv + hk) * (long long)d;
        for (int e = 0; e < d; ++e) out[e] += w * bf16_to_double(vv[e]);
    }
    for (int e = 0; e < d; ++e) out[e] /= denom;
    if (lse_out) *lse_out = mx + log(denom);
    free(score);
}

/*
 * Full form (samples == NULL): out is bf16 [B,m,Hq,d], out_f64 (nullable) the
 * unrounded values, lse (nullable) [B,Hq,m].
 * Sampled form: samples is [n_samples,3] = (b, h, i); outputs are indexed by
 * sample: out [n_samples,d], out_f64 [n_samples,d], lse [n_samples].
 */
int eagle2_tree_attention_ref(const uint16_t* q, const uint16_t* k_cache, const uint16_t* v_cache,
                              const int64_t* kv_off, const int32_t* kv_len,
                              const uint64_t* mask_bits, int B, int m, int Hq, int Hkv, int d,
                              double scale, const int32_t* samples, int n_samples, uint16_t* out,
                              double* out_f64, double* lse, int32_t* status) {
    if (!q || !k_cache || !v_cache || !kv_off || !kv_len || !mask_bits || !status) return ERR_NULL;
    if (!out && !out_f64) return ERR_NULL;
    if (B < 0 || m < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv || d < 1) return ERR_SHAPE;
    (void)status;
    const long long total = samples ? n_samples : (long long)B * m * Hq;
#pragma omp parallel for schedule(dynamic)
    for (long long t = 0; t < total; ++t) {
        int b, h, i;
        long long o_row, lse_idx;
        if (samples) {
            b = samples[3 * t];
            h = samples[3 * t + 1];
            i = samples[3 * t + 2];
            o_row = t;
            lse_idx = t;
        } else {
            b = (int)(t / ((long long)m * Hq));
            i = (int)((t / Hq) % m);
            h = (int)(t % Hq);
            o_row = ((long long)b * m + i) * Hq + h;
            lse_idx = ((long long)b * Hq + h) * m + i;
        }
        double* tmp = (double*)malloc(sizeof(double) * (size_t)d);
        double l = 0.0;
        attention_one_query(q, k_cache, v_cache, kv_off, kv_len, mask_bits, m, Hq, Hkv, d, scale, b,
                            h, i, tmp, &l);
        for (int e = 0; e < d; ++e) {
            if (out) out[o_row * d + e] = double_to_bf16(tmp[e]);
            if (out_f64) out_f64[o_row * d + e] = tmp[e];
        }
        if (lse) lse[lse_idx] = l;
        free(tmp);
    }
    return 0;
}

/* ---------- step 4: acceptance (Sections 2.1 and 2.2) -------------------- */

static void softmax_row(const float* z, int V, double inv_t, double* p, int* nonfinite) {
    double lse = 0.0;
    if (log_sum_exp(z, V, inv_t, &lse)) {
        *nonfinite = 1;
        for (int v = 0; v < V; ++v) p[v] = 0.0;
        return;
    }
    for (int v = 0; v < V; ++v) p[v] = exp((double)z[v] * inv_t - lse);
}

static int argmax_row(const float* z, int V, int* nonfinite) {
    int best = 0;
    for (int v = 0; v < V; ++v) {
        if (isnan(z[v])) *nonfinite = 1;
        if (z[v] > z[best]) best = v; /* strict: lowest id wins ties */
    }
    return best;
}

/* draft row that produced the children of the node whose first child has candidate index i */
static int draft_row_of_child(int i, int k) {
    if (i < k) return 0;
    const int l = 2 + (i - k) / (k * k); /* level of the child */
    const int j = ((i - k) % (k * k)) / k;
    return 1 + (l - 2) * k + j;
}

/*
 * Walk from the root.  Rows of target_logits: row 0 belongs to the root, row
 * 1+x to flat node x.  Children of a node are the selected nodes whose
 * sel_parent is that node, in ascending flat position.
 *
 * temperature == 0: follow the child whose token is the argmax of the target
 * row of the current node; stop when there is none; the extra token is that
 * argmax.  (Limit of the rule of Section 2.1 when the target is one-hot.)
 *
 * temperature > 0: at the current node p = softmax(target/T), q =
 * softmax(draft/T); each child x in order is accepted with probability
 * min(1, p(x)/q(x)) using u_accept[x]; after a rejection p <- norm(max(p-q,0))
 * and the rejected token is removed from q, which is renormalised.  When
 * draft_logits_all == NULL the proposal is the point mass on the candidate
 * (q = indicator of the child's token): accept with probability p(x) and
 * remove x from p.  The extra token is drawn from the p in force when the
 * walk stops, by inverse CDF in ascending token id with u_bonus.
 *
 * margins (nullable) [B,2]: min |u - a| over the tested children, and the
 * distance of u_bonus*Z from the nearest CDF boundary of the drawn token,
 * relative to Z; both tell the caller when rounding could flip a decision.
 * dbg_accept_prob (nullable) [B,m]: the acceptance probability a of every
 * child that was tested (NaN elsewhere).  dbg_p_final (nullable) [B,V]: the
 * distribution the extra token is drawn from (temperature > 0 only).  Both
 * exist so that tests can integrate the output law exactly.
 */
int eagle2_accept_ref(const float* target_logits, long long t_stride, const float* draft_logits_all,
                      long long d_stride, const int32_t* sel_index, const int32_t* sel_parent,
                      const int32_t* sel_token, const int32_t* n_sel, int B, int V, int k, int D,
                      int m, double temperature, const float* u_accept, const float* u_bonus,
                      int32_t* acc_len, int32_t* acc_path, int32_t* bonus_token, double* margins,
                      double* dbg_accept_prob, double* dbg_p_final, int32_t* status) {
    if (!target_logits || !sel_index || !sel_parent || !sel_token || !n_sel || !acc_len ||
        !acc_path || !bonus_token || !status)
        return ERR_NULL;
    if (temperature > 0.0 && (!u_accept || !u_bonus)) return ERR_NULL;
    if (B < 0 || V < 1 || k < 1 || D < 1 || m < 1 || temperature < 0.0 || isnan(temperature))
        return ERR_SHAPE;

#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        const float* trows = target_logits + (long long)b * t_stride;
        const float* drows = draft_logits_all ? draft_logits_all + (long long)b * d_stride : NULL;
        const int32_t* s_idx = sel_index + (long long)b * m;
        const int32_t* s_par = sel_parent + (long long)b * m;
        const int32_t* s_tok = sel_token + (long long)b * m;
        const int ns = n_sel[b];
        int32_t* path = acc_path + (long long)b * D;
        for (int j = 0; j < D; ++j) path[j] = -1;
        if (dbg_accept_prob)
            for (int x = 0; x < m; ++x) dbg_accept_prob[(long long)b * m + x] = NAN;
        int len = 0, cur = -1, nonfinite = 0, bonus = 0;
        double margin_u = INFINITY, margin_cdf = INFINITY;

        if (temperature == 0.0) {
            for (;;) {
                const int a = argmax_row(trows + (long long)(cur + 1) * V, V, &nonfinite);
                bonus = a;
                int next = -1;
                for (int x = cur + 1; x < ns && next < 0; ++x)
                    if (s_par[x] == cur && s_tok[x] == a) next = x;
                if (next < 0 || len >= D) break;
                path[len++] = next;
                cur = next;
            }
        } else {
            const double inv_t = 1.0 / temperature;
            double* p = (double*)malloc(sizeof(double) * (size_t)V);
            double* q = (double*)malloc(sizeof(double) * (size_t)V);
            double* r = (double*)malloc(sizeof(double) * (size_t)V);
            for (;;) {
                softmax_row(trows + (long long)(cur + 1) * V, V, inv_t, p, &nonfinite);
                int first_child = -1;
                for (int x = cur + 1; x < ns && first_child < 0; ++x)
                    if (s_par[x] == cur) first_child = x;
                if (first_child < 0 || len >= D) break;
                if (drows) {
                    const int row = draft_row_of_child(s_idx[first_child], k);
                    softmax_row(drows + (long long)row * V, V, inv_t, q, &nonfinite);
                }
                int accepted = -1;
                for (int x = first_child; x < ns; ++x) {
                    if (s_par[x] != cur) continue;
                    const int tok = s_tok[x];
                    const double qx = drows ? q[tok] : 1.0;
                    double a;
                    if (qx > 0.0)
                        a = p[tok] / qx < 1.0 ? p[tok] / qx : 1.0;
                    else
                        a = p[tok] > 0.0 ? 1.0 : 0.0;
                    const double u = (double)u_accept[(long long)b * m + x];
                    if (fabs(u - a) < margin_u) margin_u = fabs(u - a);
                    if (dbg_accept_prob) dbg_accept_prob[(long long)b * m + x] = a;
                    if (u < a) {
                        accepted = x;
                        break;
                    }
                    /* rejected: residual target, proposal without the rejected token */
                    double z = 0.0;
                    for (int v = 0; v < V; ++v) {
                        const double qv = drows ? q[v] : (v == tok ? 1.0 : 0.0);
                        r[v] = p[v] - qv > 0.0 ? p[v] - qv : 0.0;
                        z += r[v];
                    }
                    if (z > 0.0)
                        for (int v = 0; v < V; ++v) p[v] = r[v] / z;
                    if (drows) {
                        q[tok] = 0.0;
                        double zq = 0.0;
                        for (int v = 0; v < V; ++v) zq += q[v];
                        if (zq > 0.0)
                            for (int v = 0; v < V; ++v) q[v] /= zq;
                    }
                }
                if (accepted < 0) break;
                path[len++] = accepted;
                cur = accepted;
            }
            /* extra token: inverse CDF of the p in force */
            double total = 0.0;
            for (int v = 0; v < V; ++v) total += p[v];
            const double thr = (double)u_bonus[b] * total;
            double cum = 0.0;
            int drawn = -1, last_positive = 0;
            for (int v = 0; v < V; ++v) {
                if (p[v] > 0.0) last_positive = v;
                const double before = cum;
                cum += p[v];
                if (cum > thr) {
                    drawn = v;
                    const double lo = fabs(thr - before), hi = fabs(cum - thr);
                    margin_cdf = (lo < hi ? lo : hi) / (total > 0.0 ? total : 1.0);
                    break;
                }
            }
            bonus = drawn >= 0 ? drawn : last_positive;
            if (dbg_p_final)
                for (int v = 0; v < V; ++v) dbg_p_final[(long long)b * V + v] = p[v];
            free(p);
            free(q);
            free(r);
        }
        acc_len[b] = len;
        bonus_token[b] = bonus;
        if (margins) {
            margins[2 * (long long)b] = margin_u;
            margins[2 * (long long)b + 1] = margin_cdf;
        }
        if (nonfinite) {
#pragma omp atomic
            *status |= ST_NONFINITE_LOGIT;
        }
    }
    return 0;
}

/* ---------- step 5: KV compaction (Section 2.1 discard; Appendix A cache) - */
/*
 * For every layer, K and V: tree row acc_path[j] (local cache row L+acc_path[j])
 * moves to local row L+j, j ascending, then kv_len += acc_len.  Rows beyond the
 * new length are don't-care.  Elements are 2-byte (bf16) and moved verbatim.
 */
int eagle2_kv_compact_ref(uint16_t* const* k_layers, uint16_t* const* v_layers, int n_layers,
                          const int64_t* kv_off, int32_t* kv_len, const int32_t* acc_path,
                          const int32_t* acc_len, int B, int m, int D, int Hkv, int d,
                          int32_t* status) {
    if (!k_layers || !v_layers || !kv_off || !kv_len || !acc_path || !acc_len || !status)
        return ERR_NULL;
    if (B < 0 || n_layers < 0 || m < 1 || D < 1 || Hkv < 1 || d < 1) return ERR_SHAPE;
    const long long row_elems = (long long)Hkv * d;
    for (int b = 0; b < B; ++b) {
        const int L = kv_len[b];
        int len = acc_len[b];
        if (len < 0 || len > D) {
            *status |= ST_BAD_TREE;
            continue;
        }
        int ok = 1;
        for (int j = 0; j < len; ++j) {
            const int src = acc_path[(long long)b * D + j];
            if (src < j || src >= m || (j > 0 && src <= acc_path[(long long)b * D + j - 1])) ok = 0;
        }
        if (!ok) {
            *status |= ST_BAD_TREE;
            continue;
        }
        for (int layer = 0; layer < n_layers; ++layer) {
            for (int which = 0; which < 2; ++which) {
                uint16_t* base = which ? v_layers[layer] : k_layers[layer];
                for (int j = 0; j < len; ++j) {
                    const int src = acc_path[(long long)b * D + j];
                    if (src == j) continue;
                    memmove(base + (kv_off[b] + L + j) * row_elems,
                            base + (kv_off[b] + L + src) * row_elems,
                            sizeof(uint16_t) * (size_t)row_elems);
                }
            }
        }
        kv_len[b] = L + len;
    }
    return 0;
}

int eagle2_ref_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Threads the loops over independent sequences / queries may use from now on (timing only: the
 * arithmetic of every unit is the same whatever the count).  Returns the count in force before. */
int eagle2_ref_set_threads(int n) {
#ifdef _OPENMP
    const int before = omp_get_max_threads();
    if (n >= 1) omp_set_num_threads(n);
    return before;
#else
    (void)n;
    return 1;
#endif
}

/* ---------- before step 1: the LM head (Section 4.1) --------------------- */
/*
 * The draft model's feature of each frontier token goes through the LM head of the original LLM
 * to give the draft distribution that step 1 ranks: logits[r][v] = sum_h hidden[r][h] * weight[v][h]
 * (no bias).  bf16 operands as the GPU sees them, every product and the sum in double precision.
 *   hidden [rows][H], weight [V][H]: bf16 bit patterns; logits [rows][V] double.
 * Pins: numpy's matrix product on the same values; a one-hot feature selects a weight column.
 */
int eagle2_lm_head_ref(const uint16_t* hidden, const uint16_t* weight, int rows, int H, int V,
                       double* logits) {
    if (!hidden || !weight || !logits) return ERR_NULL;
    if (rows < 0 || H < 1 || V < 1) return ERR_SHAPE;
#pragma omp parallel for schedule(static)
    for (int v = 0; v < V; ++v) {
        const uint16_t* w = weight + (long long)v * H;
        for (int r = 0; r < rows; ++r) {
            const uint16_t* x = hidden + (long long)r * H;
            double acc = 0.0;
            for (int h = 0; h < H; ++h) acc += bf16_to_double(x[h]) * bf16_to_double(w[h]);
            logits[(long long)r * V + v] = acc;
        }
    }
    return 0;
}
