/*
 * CPU oracle for the verification step of speculative decoding (Hawk).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the verify step
 * computes; the tests, the smoke check and the benchmark's CPU-baseline leg call it.  It shares
 * no code with the CUDA library and the CUDA library never calls it.
 *
 * Precision: every sum, product, exponential and division below is fp64, with two stated
 * exceptions where an integer decision depends on the value and both sides must take it on the
 * same number:
 *   - the guided logit l = lu + s*(lc - lu), then l / T, is evaluated in fp32 (subtract, fused
 *     multiply-add, divide: three correctly rounded fp32 operations), because l decides which
 *     ids survive the top-k filter;
 *   - the head projection's result is rounded once from fp64 to fp32 (its storage type).
 *
 * Parity pins (tests marked "not gpu"): brute-force attention, uniform-weights closed form,
 * causality, numpy GEMM, identity weight, softmax special cases, q == p accepts all, disjoint
 * support accepts none, acceptance rate = sum min(p,q), distribution-preservation identity,
 * chi-square of the emitted token, inverse-CDF end points, a hand-computed worked example; for the
 * candidate tree: a hand-computed walk, equality with the chain on chain-shaped trees, chi-square of
 * the first emitted token with three different draft heads, all-rejected rate = prod(1 - alpha_j),
 * candidates drawn from the (refined) target always pass; for tree attention: brute force with a
 * boolean visibility matrix, chain mask = causal attention, rows off a node's path never reach it.
 * For the draw of the candidates from the pool: point mass, a boundary straddled from both sides, no
 * mass inside the valid ids, uniform closed form, both end points, chi-square against the row.
 * Nothing here is "parity unpinned".
 *
 * OpenMP is used only across independent units (stream x head, token row, sequence).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_FLAG_BAD_DRAFT 2   /* a draft id outside [v_begin, v_end) was clamped */
#define ORACLE_FLAG_NONFINITE 4   /* a NaN or +inf logit was treated as -inf */

static double bf16_to_double(uint16_t h)
{
    uint32_t bits = (uint32_t)h << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------------------------------
 * Step 1 of verification: attention of the K draft queries against the cached context
 * (Sec. 3, "Speculative Sampling": one forward pass of the target model verifies the drafted
 * tokens in parallel; App. C mentions the KV cache).  Plain definition of causal softmax
 * attention: query i of stream s sees keys j < prefix_len[s] + i + 1.
 *
 *   q        bf16 [S][K][H][D]
 *   k_cache  bf16 [S][H_kv][L_cap][D]   (the block's own rows already stored at prefix_len[s]+i)
 *   v_cache  bf16 same layout
 *   out      fp64 [S][K][H*D]
 * Query head h reads key/value head h / (H / H_kv).
 * ------------------------------------------------------------------------------------------ */
void hawk_oracle_verify_attn(const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                             const int32_t *prefix_len, double *out, int S, int K, int H, int H_kv,
                             int D, int L_cap, double sm_scale)
{
    int group = H / H_kv;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int s = 0; s < S; ++s) {
        for (int h = 0; h < H; ++h) {
            int hk = h / group;
            const uint16_t *kb = k_cache + ((size_t)s * H_kv + hk) * (size_t)L_cap * D;
            const uint16_t *vb = v_cache + ((size_t)s * H_kv + hk) * (size_t)L_cap * D;
            double *e = (double *)malloc(sizeof(double) * (size_t)(L_cap > 0 ? L_cap : 1));
            for (int i = 0; i < K; ++i) {
                int n = prefix_len[s] + i + 1;
                const uint16_t *qv = q + (((size_t)s * K + i) * H + h) * (size_t)D;
                double m = -INFINITY;
                for (int j = 0; j < n; ++j) {
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d)
                        dot += bf16_to_double(qv[d]) * bf16_to_double(kb[(size_t)j * D + d]);
                    e[j] = sm_scale * dot;
                    if (e[j] > m) m = e[j];
                }
                double z = 0.0;
                for (int j = 0; j < n; ++j) {
                    e[j] = exp(e[j] - m);
                    z += e[j];
                }
                double *o = out + ((size_t)s * K + i) * (size_t)H * D + (size_t)h * D;
                for (int d = 0; d < D; ++d) {
                    double acc = 0.0;
                    for (int j = 0; j < n; ++j) acc += e[j] * bf16_to_double(vb[(size_t)j * D + d]);
                    o[d] = acc / z;
                }
            }
            free(e);
        }
    }
}

/* ------------------------------------------------------------------------------------------
 * Step 2: output head (Sec. 3: decoding heads sit after the final hidden layer and map a hidden
 * state onto the image-token codebook).  logits[m][v] = sum_c X[m][c] * W[v][c] for v in
 * [v_begin, v_end); other columns are left untouched.
 *   x bf16 [M][hidden], w bf16 [V][hidden], logits fp32 [M][V]
 * ------------------------------------------------------------------------------------------ */
void hawk_oracle_head_proj(const uint16_t *x, const uint16_t *w, float *logits, int M, int hidden,
                           int V, int v_begin, int v_end)
{
#pragma omp parallel for schedule(static)
    for (int m = 0; m < M; ++m) {
        double *xr = (double *)malloc(sizeof(double) * (size_t)hidden);
        for (int c = 0; c < hidden; ++c) xr[c] = bf16_to_double(x[(size_t)m * hidden + c]);
        for (int v = v_begin; v < v_end; ++v) {
            const uint16_t *wr = w + (size_t)v * hidden;
            double acc = 0.0;
            for (int c = 0; c < hidden; ++c) acc += xr[c] * bf16_to_double(wr[c]);
            logits[(size_t)m * V + v] = (float)acc;
        }
        free(xr);
    }
}

/* ------------------------------------------------------------------------------------------
 * Step 3a: the target distribution of one position (generation settings of Sec. 5: guidance
 * scale, temperature, top-k).  The paper names the settings but not the formulas; the reading
 * taken: guidance on logits, l = lu + s*(lc - lu); then l / T; then keep every l >= the top_k-th
 * largest finite l (ties at the threshold are all kept); then softmax over what is kept.
 * -inf in either stream gives -inf; NaN or +inf is treated as -inf and flagged.
 *
 *   lc, lu : fp32 rows of length V (conditional / unconditional); only [v_begin, v_end) is read
 *   p      : fp64 row of length V; ids outside the valid range get 0
 * returns flags.
 * ------------------------------------------------------------------------------------------ */
static int cmp_float_desc(const void *a, const void *b)
{
    float x = *(const float *)a, y = *(const float *)b;
    return (x < y) - (x > y);
}

int hawk_oracle_target_probs(const float *lc, const float *lu, int V, int v_begin, int v_end,
                             float cfg_scale, float temperature, int top_k, double *p)
{
    int flags = 0;
    int n = v_end - v_begin;
    float *l = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    float *sorted = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    int n_finite = 0;
    for (int v = 0; v < V; ++v) p[v] = 0.0;
    for (int t = 0; t < n; ++t) {
        float c = lc[v_begin + t], u = lu[v_begin + t];
        int bad_c = isnan(c) || (isinf(c) && c > 0), bad_u = isnan(u) || (isinf(u) && u > 0);
        if (bad_c || bad_u) flags |= ORACLE_FLAG_NONFINITE;
        if (bad_c || bad_u || isinf(c) || isinf(u)) {
            l[t] = -INFINITY;
            continue;
        }
        volatile float diff = c - u;                       /* fp32 subtract            */
        volatile float g = fmaf(cfg_scale, diff, u);       /* fp32 fused multiply-add  */
        volatile float scaled = g / temperature;           /* fp32 divide              */
        float r = scaled;
        if (isnan(r) || (isinf(r) && r > 0)) {             /* overflow of the combine  */
            flags |= ORACLE_FLAG_NONFINITE;
            r = -INFINITY;
        }
        l[t] = r;
        if (!isinf(r)) sorted[n_finite++] = r;
    }
    if (top_k > 0 && top_k < n_finite) {
        qsort(sorted, (size_t)n_finite, sizeof(float), cmp_float_desc);
        float tau = sorted[top_k - 1];
        for (int t = 0; t < n; ++t)
            if (l[t] < tau) l[t] = -INFINITY;
    }
    double m = -INFINITY;
    for (int t = 0; t < n; ++t)
        if ((double)l[t] > m) m = (double)l[t];
    if (!isinf(m)) {
        double z = 0.0;
        for (int t = 0; t < n; ++t)
            if (!isinf(l[t])) z += exp((double)l[t] - m);
        for (int t = 0; t < n; ++t)
            if (!isinf(l[t])) p[v_begin + t] = exp((double)l[t] - m) / z;
    }
    free(l);
    free(sorted);
    return flags;
}

/* ------------------------------------------------------------------------------------------
 * Step 3b: draw from a non-negative weight vector by inverse CDF in ascending token id:
 * the smallest v whose running sum strictly exceeds u * total; if rounding leaves none, the
 * largest v with positive weight.  Also reports the distance of u*total from the two running-sum
 * boundaries of the chosen id, as a fraction of total.
 * ------------------------------------------------------------------------------------------ */
static int inverse_cdf(const double *w, int v_begin, int v_end, double u, double total,
                       double *margin)
{
    double t = u * total, run = 0.0;
    int last_pos = -1;
    for (int v = v_begin; v < v_end; ++v) {
        if (w[v] > 0.0) last_pos = v;
        double prev = run;
        run += w[v];
        if (run > t) {
            if (margin) {
                double lo = t - prev, hi = run - t;
                *margin = (lo < hi ? lo : hi) / total;
            }
            return v;
        }
    }
    if (margin) *margin = 0.0;
    return last_pos;
}

/* ------------------------------------------------------------------------------------------
 * Step 3c: the residual of one rejection (Sec. 3 and Eq. "recur" of Sec. 4.2, written in App. A
 * as (p - min(q,p)) / sum(p - min(q,p))): r[v] = max(0, p[v] - q[v]) over the valid ids, left
 * un-normalised; returns its total mass.
 * ------------------------------------------------------------------------------------------ */
double hawk_oracle_residual(const double *p, const float *q, int V, int v_begin, int v_end,
                            double *r)
{
    double total = 0.0;
    for (int v = 0; v < V; ++v) r[v] = 0.0;
    for (int v = v_begin; v < v_end; ++v) {
        double d = p[v] - (double)q[v];
        r[v] = d > 0.0 ? d : 0.0;
        total += r[v];
    }
    return total;
}

/* ------------------------------------------------------------------------------------------
 * Step 3: verification of a chain of K drafts per sequence (Sec. 3: accept draft x with
 * probability min(1, p(x)/q(x)); Sec. 4.2: on a pass go one position deeper, on the first
 * rejection update the target to norm(max(0, p - q)) and resample from it).
 *
 *   logits      fp32 [2B][rows][V], rows = K + has_bonus_row; stream b conditional, B+b unconditional
 *   q_probs     fp32 [B][K][V]      draft probabilities
 *   draft       int32 [B][K]
 *   u_accept    fp32 [B][K]   in [0,1): accept iff u * q(x) < p(x)
 *   u_resample  fp32 [B][K+1] in [0,1): entry i drives the resample after a rejection at i,
 *                                        entry K the bonus row
 *   accept_len  int32 [B]  number of accepted drafts (the paper's "accept length" minus 1)
 *   out_token   int32 [B]  correction token; -1 when all K passed and there is no bonus row
 * Optional diagnostics (may be NULL):
 *   ratio           fp64 [B][K]  p(x)/q(x) of each position examined (NaN if not examined)
 *   accept_margin   fp64 [B][K]  |u - min(1, ratio)| (inf if not examined)
 *   resample_margin fp64 [B]     distance of the resample draw from a CDF boundary / total mass
 * returns OR of flags over all sequences.
 * ------------------------------------------------------------------------------------------ */
int hawk_oracle_cfg_accept(const float *logits, const float *q_probs, const int32_t *draft,
                           const float *u_accept, const float *u_resample, int B, int K, int V,
                           int v_begin, int v_end, float cfg_scale, float temperature, int top_k,
                           int has_bonus_row, int32_t *accept_len, int32_t *out_token,
                           double *ratio, double *accept_margin, double *resample_margin)
{
    int rows = K + (has_bonus_row ? 1 : 0);
    int all_flags = 0;
#pragma omp parallel for schedule(dynamic) reduction(| : all_flags)
    for (int b = 0; b < B; ++b) {
        double *p = (double *)malloc(sizeof(double) * (size_t)V);
        double *r = (double *)malloc(sizeof(double) * (size_t)V);
        int flags = 0, done = 0;
        if (resample_margin) resample_margin[b] = INFINITY;
        for (int i = 0; i < K; ++i) {
            if (ratio) ratio[(size_t)b * K + i] = NAN;
            if (accept_margin) accept_margin[(size_t)b * K + i] = INFINITY;
        }
        for (int i = 0; i < K && !done; ++i) {
            const float *lc = logits + ((size_t)b * rows + i) * (size_t)V;
            const float *lu = logits + ((size_t)(B + b) * rows + i) * (size_t)V;
            const float *q = q_probs + ((size_t)b * K + i) * (size_t)V;
            flags |= hawk_oracle_target_probs(lc, lu, V, v_begin, v_end, cfg_scale, temperature,
                                              top_k, p);
            int x = draft[(size_t)b * K + i];
            if (x < v_begin || x >= v_end) {
                flags |= ORACLE_FLAG_BAD_DRAFT;
                x = x < v_begin ? v_begin : v_end - 1;
            }
            double u = (double)u_accept[(size_t)b * K + i];
            double qx = (double)q[x], px = p[x];
            if (ratio) ratio[(size_t)b * K + i] = px / qx;
            if (accept_margin) {
                double rr = qx > 0.0 ? px / qx : (px > 0.0 ? INFINITY : 0.0);
                accept_margin[(size_t)b * K + i] = fabs(u - (rr < 1.0 ? rr : 1.0));
            }
            if (u * qx < px) continue;                       /* accepted: go one deeper */
            /* first rejection: resample from the residual, discard the later drafts */
            double total = hawk_oracle_residual(p, q, V, v_begin, v_end, r);
            const double *w = r;
            if (!(total > 0.0)) {                            /* p <= q everywhere: fall back to p */
                w = p;
                total = 1.0;
            }
            accept_len[b] = i;
            out_token[b] = inverse_cdf(w, v_begin, v_end, (double)u_resample[(size_t)b * (K + 1) + i],
                                       total, resample_margin ? &resample_margin[b] : NULL);
            done = 1;
        }
        if (!done) {
            accept_len[b] = K;
            out_token[b] = -1;
            if (has_bonus_row) {
                const float *lc = logits + ((size_t)b * rows + K) * (size_t)V;
                const float *lu = logits + ((size_t)(B + b) * rows + K) * (size_t)V;
                flags |= hawk_oracle_target_probs(lc, lu, V, v_begin, v_end, cfg_scale, temperature,
                                                  top_k, p);
                out_token[b] = inverse_cdf(p, v_begin, v_end,
                                           (double)u_resample[(size_t)b * (K + 1) + K], 1.0,
                                           resample_margin ? &resample_margin[b] : NULL);
            }
        }
        all_flags |= flags;
        free(p);
        free(r);
    }
    return all_flags;
}

/* Target probabilities of every row (for element-wise parity of p): p_out fp64 [B][rows][V]. */
int hawk_oracle_target_probs_rows(const float *logits, int B, int rows, int V, int v_begin,
                                  int v_end, float cfg_scale, float temperature, int top_k,
                                  double *p_out)
{
    int all_flags = 0;
#pragma omp parallel for collapse(2) schedule(dynamic) reduction(| : all_flags)
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < rows; ++i) {
            const float *lc = logits + ((size_t)b * rows + i) * (size_t)V;
            const float *lu = logits + ((size_t)(B + b) * rows + i) * (size_t)V;
            all_flags |= hawk_oracle_target_probs(lc, lu, V, v_begin, v_end, cfg_scale, temperature,
                                                  top_k, p_out + ((size_t)b * rows + i) * (size_t)V);
        }
    return all_flags;
}

/* ------------------------------------------------------------------------------------------
 * Step 3 with several candidates per depth: verification of a candidate TREE (Sec. 4.2,
 * "Sampling and Verification", Eq. "recur"; proof of distribution preservation in App. A).
 * Candidates at the same depth are verified one after the other.  A candidate x drawn from its
 * draft distribution q passes with probability min(1, p(x)/q(x)); when it passes, decoding moves to
 * that node and one level deeper; each rejection replaces the target by
 *     p <- norm(max(0, p - q))            (q: the distribution the rejected candidate came from)
 * and when every candidate of a level is rejected (or the node has none), the correction token is
 * drawn from the target as refined so far.  q may differ from candidate to candidate (horizontal or
 * vertical draft head).  A residual without mass (p <= q everywhere) leaves p as it is.
 *
 * The tree is shared by the batch.  Node 0 is the root (the last committed token); the children of
 * node n are the nodes child_begin[n] .. child_begin[n+1]-1, in verification order.
 *   logits      fp32 [2B][N][V]  row n: target logits for the token that follows node n
 *   q_probs     fp32 [B][NQ][V]  draft distributions
 *   node_token  int32 [B][N]     candidate token of node n (entry 0 unused)
 *   node_q      int32 [N]        row of q_probs that node n's token was drawn from (entry 0 unused)
 *   child_begin int32 [N+1]
 *   u_accept    fp32 [B][N]      one uniform per candidate node (entry 0 unused)
 *   u_resample  fp32 [B][N]      entry n drives the draw if the walk stops at node n
 *   accept_len  int32 [B]        number of accepted candidates = depth of the node the walk stops at
 *   out_token   int32 [B]        the correction token (-1 if the refined target has no mass at all)
 *   path        int32 [B][max_depth]  accepted nodes in order, -1 beyond accept_len (may be NULL)
 * Optional diagnostics (may be NULL): accept_margin fp64 [B][N] = |u - min(1, p(x)/q(x))| of every
 * candidate examined (inf otherwise); resample_margin fp64 [B].
 * returns OR of flags.
 * ------------------------------------------------------------------------------------------ */
int hawk_oracle_tree_accept(const float *logits, const float *q_probs, const int32_t *node_token,
                            const int32_t *node_q, const int32_t *child_begin,
                            const float *u_accept, const float *u_resample, int B, int N, int NQ,
                            int V, int v_begin, int v_end, float cfg_scale, float temperature,
                            int top_k, int32_t *accept_len, int32_t *out_token, int32_t *path,
                            int max_depth, double *accept_margin, double *resample_margin)
{
    int all_flags = 0;
    (void)NQ;
#pragma omp parallel for schedule(dynamic) reduction(| : all_flags)
    for (int b = 0; b < B; ++b) {
        double *p = (double *)malloc(sizeof(double) * (size_t)V);
        double *r = (double *)malloc(sizeof(double) * (size_t)V);
        int flags = 0, n = 0, depth = 0;
        if (resample_margin) resample_margin[b] = INFINITY;
        if (accept_margin)
            for (int c = 0; c < N; ++c) accept_margin[(size_t)b * N + c] = INFINITY;
        if (path)
            for (int d = 0; d < max_depth; ++d) path[(size_t)b * max_depth + d] = -1;
        for (;;) {
            const float *lc = logits + ((size_t)b * N + n) * (size_t)V;
            const float *lu = logits + ((size_t)(B + b) * N + n) * (size_t)V;
            flags |= hawk_oracle_target_probs(lc, lu, V, v_begin, v_end, cfg_scale, temperature,
                                              top_k, p);
            int next = -1;
            for (int c = child_begin[n]; c < child_begin[n + 1] && next < 0; ++c) {
                const float *q = q_probs + ((size_t)b * NQ + node_q[c]) * (size_t)V;
                int x = node_token[(size_t)b * N + c];
                if (x < v_begin || x >= v_end) {
                    flags |= ORACLE_FLAG_BAD_DRAFT;
                    x = x < v_begin ? v_begin : v_end - 1;
                }
                double u = (double)u_accept[(size_t)b * N + c];
                double qx = (double)q[x], px = p[x];
                if (accept_margin) {
                    double rr = qx > 0.0 ? px / qx : (px > 0.0 ? INFINITY : 0.0);
                    accept_margin[(size_t)b * N + c] = fabs(u - (rr < 1.0 ? rr : 1.0));
                }
                if (u * qx < px) {
                    next = c;                                  /* passed: one level deeper */
                    break;
                }
                double total = hawk_oracle_residual(p, q, V, v_begin, v_end, r);
                if (total > 0.0)                               /* p <- norm(max(0, p - q)) */
                    for (int v = v_begin; v < v_end; ++v) p[v] = r[v] / total;
            }
            if (next >= 0) {
                if (path && depth < max_depth) path[(size_t)b * max_depth + depth] = next;
                ++depth;
                n = next;
                continue;
            }
            accept_len[b] = depth;
            out_token[b] = inverse_cdf(p, v_begin, v_end, (double)u_resample[(size_t)b * N + n], 1.0,
                                       resample_margin ? &resample_margin[b] : NULL);
            break;
        }
        all_flags |= flags;
        free(p);
        free(r);
    }
    return all_flags;
}

/* ------------------------------------------------------------------------------------------
 * Step 1 for a candidate tree (Sec. 4.2: the candidates form a tree so that more of them can be
 * verified at once, all in one forward pass of the target model): the N tree nodes of a stream are N
 * queries; node i attends to the whole cached prefix and, inside the block, only to the nodes on its
 * own path from the root.
 * Plain definition of masked softmax attention:
 *   key j <  prefix_len[s]                      visible to every node
 *   key j =  prefix_len[s] + m, 0 <= m < N      visible to node i iff bit m of anc_mask[i] is set
 * (node i's own key/value row is cache row prefix_len[s] + i; anc_mask[i] has bit i set).
 * The chain of K drafts is the tree with anc_mask[i] = 2^(i+1) - 1.
 *   q bf16 [S][N][H][D]; caches bf16 [S][H_kv][L_cap][D]; anc_mask uint64 [N], N <= 64; out fp64 [S][N][H*D]
 * ------------------------------------------------------------------------------------------ */
void hawk_oracle_verify_attn_tree(const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                                  const int32_t *prefix_len, const uint64_t *anc_mask, double *out,
                                  int S, int N, int H, int H_kv, int D, int L_cap, double sm_scale)
{
    int group = H / H_kv;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int s = 0; s < S; ++s) {
        for (int h = 0; h < H; ++h) {
            int hk = h / group;
            const uint16_t *kb = k_cache + ((size_t)s * H_kv + hk) * (size_t)L_cap * D;
            const uint16_t *vb = v_cache + ((size_t)s * H_kv + hk) * (size_t)L_cap * D;
            double *e = (double *)malloc(sizeof(double) * (size_t)(L_cap > 0 ? L_cap : 1));
            for (int i = 0; i < N; ++i) {
                int pl = prefix_len[s], n = pl + N;
                const uint16_t *qv = q + (((size_t)s * N + i) * H + h) * (size_t)D;
                double m = -INFINITY;
                for (int j = 0; j < n; ++j) {
                    int visible = j < pl || (int)((anc_mask[i] >> (j - pl)) & 1u);
                    if (!visible) {
                        e[j] = -INFINITY;
                        continue;
                    }
                    double dot = 0.0;
                    for (int d = 0; d < D; ++d)
                        dot += bf16_to_double(qv[d]) * bf16_to_double(kb[(size_t)j * D + d]);
                    e[j] = sm_scale * dot;
                    if (e[j] > m) m = e[j];
                }
                double z = 0.0;
                for (int j = 0; j < n; ++j) {
                    e[j] = isinf(e[j]) ? 0.0 : exp(e[j] - m);
                    z += e[j];
                }
                double *o = out + ((size_t)s * N + i) * (size_t)H * D + (size_t)h * D;
                for (int d = 0; d < D; ++d) {
                    double acc = 0.0;
                    for (int j = 0; j < n; ++j)
                        if (e[j] != 0.0) acc += e[j] * bf16_to_double(vb[(size_t)j * D + d]);
                    o[d] = acc / z;
                }
            }
            free(e);
        }
    }
}

/* ------------------------------------------------------------------------------------------
 * Candidates from the spatial sampling pool (Sec. 4.2, "Spatial Sampling Pool": the candidate
 * tree is built from the sampling results of the pool's distributions at each speculation
 * position): one draw per pool distribution, by inverse CDF in ascending id over the valid ids,
 * negative or NaN weights counting as zero.  A row without mass yields -1.
 *   pool_q fp32 [R][V]; u fp32 [R]; row_token int32 [R]; margin fp64 [R] or NULL
 * ------------------------------------------------------------------------------------------ */
void hawk_oracle_pool_sample(const float *pool_q, const float *u, int R, int V, int v_begin, int v_end,
                             int32_t *row_token, double *margin)
{
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < R; ++r) {
        double *w = (double *)calloc((size_t)V, sizeof(double));
        double total = 0.0;
        for (int v = v_begin; v < v_end; ++v) {
            double x = (double)pool_q[(size_t)r * V + v];
            w[v] = x > 0.0 ? x : 0.0;
            total += w[v];
        }
        if (total > 0.0)
            row_token[r] = inverse_cdf(w, v_begin, v_end, (double)u[r], total, margin ? &margin[r] : NULL);
        else {
            row_token[r] = -1;
            if (margin) margin[r] = 1.0;
        }
        free(w);
    }
}

/* ------------------------------------------------------------------------------------------
 * Steps 2 and 3a's first half in one: the output head followed by the guidance combine and the
 * temperature (generation settings of Sec. 5), for callers that never need the two logit rows:
 *   guided[b*rows + i][v] = (lu + s*(lc - lu)) / T,  lc / lu the head's logits (rounded to fp32 as
 *   hawk_oracle_head_proj returns them) of rows (b, i) and (B + b, i) of x,
 * evaluated in fp32 as subtract, fused multiply-add, divide like hawk_oracle_target_probs.
 *   x bf16 [2B][rows][hidden], w bf16 [V][hidden], guided fp32 [B][rows][V]
 * ------------------------------------------------------------------------------------------ */
void hawk_oracle_head_proj_cfg(const uint16_t *x, const uint16_t *w, float *guided, int B, int rows,
                               int hidden, int V, int v_begin, int v_end, float cfg_scale,
                               float temperature)
{
    int pairs = B * rows;
#pragma omp parallel for schedule(static)
    for (int m = 0; m < pairs; ++m) {
        const uint16_t *xc = x + (size_t)m * hidden, *xu = x + (size_t)(pairs + m) * hidden;
        for (int v = v_begin; v < v_end; ++v) {
            const uint16_t *wr = w + (size_t)v * hidden;
            double acc_c = 0.0, acc_u = 0.0;
            for (int c = 0; c < hidden; ++c) {
                acc_c += bf16_to_double(xc[c]) * bf16_to_double(wr[c]);
                acc_u += bf16_to_double(xu[c]) * bf16_to_double(wr[c]);
            }
            float lc = (float)acc_c, lu = (float)acc_u;
            volatile float diff = lc - lu;
            volatile float g = fmaf(cfg_scale, diff, lu);
            volatile float scaled = g / temperature;
            guided[(size_t)m * V + v] = scaled;
        }
    }
}
