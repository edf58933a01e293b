/*
 * s4c_oracle.c -- slow, plain, float64 CPU oracle for the S4C verify step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the checker the CUDA library is
 * compared against.  It shares no code, header, table or helper with the CUDA
 * path and the product never calls it.  Only the tests, the smoke check and the
 * "cpu_baseline" / "--impl reference" legs of the benchmark may load it.
 *
 * What it computes (each function cites the passage of the S4C paper,
 * arXiv 2506.14158, that defines the operation):
 *
 *   s4c_oracle_tree_attention  Section 3.2 (the verification pass uses a tree
 *                              mask) and Figure 3 (where the mask is drawn): every
 *                              tree token attends the cached prefix and its own
 *                              root path.  Written out as the definition of
 *                              masked softmax attention; no tiling, no online
 *                              softmax.
 *   s4c_oracle_accept_greedy   Section 4.1.2 (all experiments decode greedily)
 *                              and Section 3.2 (longest accepted path).
 *   s4c_oracle_accept_stochastic
 *                              Section 2 "Speculative Sampling" (accept with
 *                              probability min(1, p/q), resample from
 *                              norm(max(0, p - q))), Eq. 11 and Eq. 12 of
 *                              Section 3.2 (the correction at fork positions).
 *                              Taken step by step, in the paper's order.
 *   s4c_oracle_accept_filtered the same walk against a top-k / nucleus filtered
 *                              target distribution (the sampling regime of the
 *                              temperature study, Section 4; the filter itself
 *                              is the usual chain of logit warpers, restated).
 *   s4c_oracle_kv_compact      Section 3.2, last paragraph (accepted tokens and
 *                              their features are kept for the next drafting
 *                              phase): a gather from a snapshot.
 *   s4c_oracle_build_tree      Section 3.2 and Figure 3 (left): the continuous
 *                              verification tree -- a vertical chain of top-1
 *                              drafts, then horizontal top-k alternatives at
 *                              every position -- built step by step as the
 *                              section tells it, then numbered breadth-first.
 *
 * Readings of silent or garbled points (symbols follow Section 2: p = target,
 * q = draft):
 *   - Eq. 11 prints q(x)/p(x) and then calls q the target and p the draft; with
 *     the symbols untangled the ratio is target/draft, as in Section 2.
 *   - Eq. 12 prints norm(max(q_c, p_c)); Section 2 gives the rule it stands for:
 *     norm(max(0, p_target - p_draft)).
 *   - Several siblings at one position are tried one after another in index
 *     order; after each rejection the target distribution is replaced by the
 *     normalised residual and the rejected token is removed from the draft
 *     distribution, which is renormalised (the multi-candidate correction the
 *     paper cites for trees).
 *   - Comparison is strict (r < min(1, ratio)), as printed in Eq. 11.
 *   - A token is always emitted at the end of the walk: from the residual at the
 *     fork, or from the unmodified target distribution at a leaf.
 *   - Ties in argmax go to the lowest index.
 *
 * Pins (see tests/test_oracle_*.py): chain tree == causal attention, star tree,
 * path equivalence against a library SDPA, constant-V, GQA == repeated MHA;
 * greedy verify == token-by-token greedy decoding, planted trees; exact
 * enumeration on dyadic tiny-vocab cases and chi-square Monte-Carlo showing the
 * emitted token follows the target distribution; compaction against a library
 * gather; tree construction against the example of Figure 3 as Section 3.2
 * describes it, an independently written construction plus a library sort,
 * and the structural facts (first sibling = top-1, rank order, breadth-first).  The paper prints no worked numeric example for any of these steps,
 * so config-level values are: parity unpinned by printed numbers (pinned by the
 * invariants above instead).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* per-sequence status bit flags (kept numerically equal to the public header's
 * values by a test, not by a shared include) */
#define ORC_SEQ_OK 0
#define ORC_SEQ_BAD_PARENT 1
#define ORC_SEQ_TOKEN_RANGE 2
#define ORC_SEQ_CAPACITY 4
#define ORC_SEQ_DEPTH 8
#define ORC_SEQ_BAD_PATH 16
#define ORC_SEQ_NONFINITE 64

int s4c_oracle_max_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void s4c_oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* A tree is given in topological order: parent[0] = -1, 0 <= parent[i] < i. */
static int tree_is_valid(const int32_t* parent, int n) {
    if (n < 1) return 0;
    if (parent[0] != -1) return 0;
    for (int i = 1; i < n; ++i)
        if (parent[i] < 0 || parent[i] >= i) return 0;
    return 1;
}

static int node_count(const int32_t* n_nodes, int b, int T) {
    return n_nodes ? n_nodes[b] : T;
}

/* ------------------------------------------------------------------------- */
/* Tree-masked attention (Section 3.2; Figure 3, tree mask matrix).            */
/*                                                                           */
/* q      [B,Hq,T,d]   float64                                               */
/* k, v   [B,Hkv,C,d]  float64; the tree's own K/V sit at slots L_b..L_b+T-1 */
/* out    [B,Hq,T,d]   float64                                               */
/* Node i of sequence b sees slots 0..L_b-1 (the committed prefix) and slot   */
/* L_b+t for every t on the path root..i (i included).  Weights are a softmax */
/* of scale * <q,k> over exactly that set.                                    */
/* Rows of padding nodes (i >= n_nodes[b]) are set to zero.  A sequence with  */
/* a malformed tree or L_b + n > C gets a status flag and its rows untouched. */
/* ------------------------------------------------------------------------- */
int s4c_oracle_tree_attention(const double* q, const double* k, const double* v,
                              const int32_t* cache_len, const int32_t* parent,
                              const int32_t* n_nodes, double* out, int32_t* status,
                              int B, int T, int Hq, int Hkv, int d, int C, double scale) {
    if (!q || !k || !v || !cache_len || !parent || !out) return 1;
    if (B < 0 || T < 1 || Hq < 1 || Hkv < 1 || d < 1 || C < 1 || Hq % Hkv) return 2;
    const int G = Hq / Hkv;
    if (scale == 0.0) scale = 1.0 / sqrt((double)d);
    for (int b = 0; b < B; ++b) {
        const int n = node_count(n_nodes, b, T);
        const int L = cache_len[b];
        const int32_t* par = parent + (size_t)b * T;
        int st = ORC_SEQ_OK;
        if (n < 1 || n > T || !tree_is_valid(par, n)) st |= ORC_SEQ_BAD_PARENT;
        if (L < 0 || (long)L + (n > 0 ? n : 0) > (long)C) st |= ORC_SEQ_CAPACITY;
        if (status) status[b] = st;
        if (st) continue;

        /* visible[i*n + t] = 1 iff t is i or an ancestor of i */
        unsigned char* visible = (unsigned char*)calloc((size_t)n * n, 1);
        for (int i = 0; i < n; ++i)
            for (int t = i; t >= 0; t = par[t]) visible[(size_t)i * n + t] = 1;

#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic)
#endif
        for (int h = 0; h < Hq; ++h) {
            const int hk = h / G;
            const double* kb = k + ((size_t)b * Hkv + hk) * C * d;
            const double* vb = v + ((size_t)b * Hkv + hk) * C * d;
            double* s = (double*)malloc(sizeof(double) * (size_t)(L + n));
            for (int i = 0; i < T; ++i) {
                double* o = out + (((size_t)b * Hq + h) * T + i) * d;
                for (int c = 0; c < d; ++c) o[c] = 0.0;
                if (i >= n) continue;
                const double* qi = q + (((size_t)b * Hq + h) * T + i) * d;
                double mx = -INFINITY;
                for (int j = 0; j < L + n; ++j) {
                    if (j >= L && !visible[(size_t)i * n + (j - L)]) {
                        s[j] = -INFINITY;
                        continue;
                    }
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += qi[c] * kb[(size_t)j * d + c];
                    s[j] = scale * acc;
                    if (s[j] > mx) mx = s[j];
                }
                double den = 0.0;
                for (int j = 0; j < L + n; ++j) {
                    s[j] = (s[j] == -INFINITY) ? 0.0 : exp(s[j] - mx);
                    den += s[j];
                }
                for (int j = 0; j < L + n; ++j) {
                    if (s[j] == 0.0) continue;
                    const double w = s[j] / den;
                    for (int c = 0; c < d; ++c) o[c] += w * vb[(size_t)j * d + c];
                }
            }
            free(s);
        }
        free(visible);
    }
    return 0;
}

/* depth of every node, root = 0 */
static void tree_depths(const int32_t* par, int n, int* depth) {
    depth[0] = 0;
    for (int i = 1; i < n; ++i) depth[i] = depth[par[i]] + 1;
}

/* writes root..e into path (max_depth+1 entries, -1 padded); returns depth of e */
static int write_path(const int32_t* par, int e, const int* depth, int max_depth, int32_t* path) {
    for (int j = 0; j <= max_depth; ++j) path[j] = -1;
    for (int t = e; t >= 0; t = par[t]) path[depth[t]] = t;
    return depth[e];
}

static int validate_accept_inputs(const int32_t* par, const int32_t* tok, int n, int T, int V,
                                  int max_depth, int* depth) {
    int st = ORC_SEQ_OK;
    if (n < 1 || n > T || !tree_is_valid(par, n)) return ORC_SEQ_BAD_PARENT;
    for (int i = 0; i < n; ++i)
        if (tok[i] < 0 || tok[i] >= V) st |= ORC_SEQ_TOKEN_RANGE;
    tree_depths(par, n, depth);
    for (int i = 0; i < n; ++i)
        if (depth[i] > max_depth) st |= ORC_SEQ_DEPTH;
    return st;
}

/* Input validation of the acceptance calls, not a step of the method: a target-logit row of a real
 * node (i < n) is unusable when it holds a NaN or +Inf (the maximum-subtracted exponent would be
 * Inf - Inf) or nothing but -Inf (no token has mass).  A -Inf logit beside finite ones is fine: the
 * token simply has probability 0.  Such a sequence is flagged and skipped like a malformed tree. */
static int logits_unusable(const float* logits, int n, int V) {
    for (int i = 0; i < n; ++i) {
        const float* row = logits + (size_t)i * V;
        int any_finite = 0;
        for (int v = 0; v < V; ++v) {
            if (isnan(row[v]) || (isinf(row[v]) && row[v] > 0)) return 1;
            if (!isinf(row[v])) any_finite = 1;
        }
        if (!any_finite) return 1;
    }
    return 0;
}

static int argmax_lowest(const float* row, int V) {
    int best = 0;
    for (int v = 1; v < V; ++v)
        if (row[v] > row[best]) best = v;
    return best;
}

/* ------------------------------------------------------------------------- */
/* Greedy verification (Section 4.1.2: greedy decoding; Section 3.2: longest   */
/* accepted path).                                                           */
/*                                                                           */
/* g[n] = argmax_v logits[n,v].  Node i is accepted iff its parent is and    */
/* tokens[i] == g[parent[i]]; the root is accepted by definition.  The result */
/* is the accepted node of greatest depth (lowest index among equals), the    */
/* path to it, and the target's own next token g[e] after it.                 */
/* ------------------------------------------------------------------------- */
int s4c_oracle_accept_greedy(const float* logits, const int32_t* tokens, const int32_t* parent,
                             const int32_t* n_nodes, int B, int T, int V, int max_depth,
                             int32_t* accept_len, int32_t* path, int32_t* next_token,
                             int32_t* status) {
    if (!logits || !tokens || !parent || !accept_len || !path || !next_token) return 1;
    if (B < 0 || T < 1 || V < 1 || max_depth < 0) return 2;
    for (int b = 0; b < B; ++b) {
        const int n = node_count(n_nodes, b, T);
        const int32_t* par = parent + (size_t)b * T;
        const int32_t* tok = tokens + (size_t)b * T;
        int32_t* pth = path + (size_t)b * (max_depth + 1);
        int* depth = (int*)malloc(sizeof(int) * (size_t)T);
        int st = validate_accept_inputs(par, tok, n, T, V, max_depth, depth);
        if (!(st & ORC_SEQ_BAD_PARENT) && logits_unusable(logits + (size_t)b * T * V, n, V)) st |= ORC_SEQ_NONFINITE;
        if (status) status[b] = st;
        if (st) {
            accept_len[b] = -1;
            next_token[b] = -1;
            for (int j = 0; j <= max_depth; ++j) pth[j] = -1;
            free(depth);
            continue;
        }
        int* g = (int*)malloc(sizeof(int) * (size_t)n);
        unsigned char* ok = (unsigned char*)calloc((size_t)n, 1);
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic)
#endif
        for (int i = 0; i < n; ++i) g[i] = argmax_lowest(logits + ((size_t)b * T + i) * V, V);
        ok[0] = 1;
        int e = 0;
        for (int i = 1; i < n; ++i) {
            ok[i] = ok[par[i]] && tok[i] == g[par[i]];
            if (ok[i] && depth[i] > depth[e]) e = i;
        }
        accept_len[b] = write_path(par, e, depth, max_depth, pth);
        next_token[b] = g[e];
        free(g);
        free(ok);
        free(depth);
    }
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Stochastic verification (Section 2 "Speculative Sampling"; Eq. 11, Eq. 12). */
/*                                                                           */
/* logits  [B,T,V] float32: row n = target logits for the token after node n  */
/* dprobs  [B,T,V] float32: row n = draft distribution the children of n were */
/*                          proposed from (already at this temperature)       */
/* uniforms[B,T]   float32 in [0,1): entry i>=1 is node i's acceptance draw,  */
/*                          entry 0 is the draw for the final token           */
/* Steps per sequence, cur = root:                                            */
/*  S1  p = softmax(logits[cur]/tau), q = dprobs[cur]; children of cur in     */
/*      index order.                                                          */
/*  S2  for each child c with token x: ratio = p(x)/q(x) (q(x)=0: +inf if     */
/*      p(x)>0 else 0); accept iff u_c < min(1, ratio); on accept cur = c and */
/*      back to S1.                                                           */
/*  S3  on reject: p <- norm(max(p-q,0)) (kept if the mass is 0); q(x) <- 0,  */
/*      q <- q/sum(q) (if the sum is 0 no further sibling is tried).           */
/*  S4  no child accepted: next token = smallest v whose running sum of p     */
/*      exceeds u_0 * sum(p).                                                 */
/* near_tie[b,i] = 1 where |ratio - u_i| < 1e-6 at node i's test.             */
/* ------------------------------------------------------------------------- */
/*                                                                           */
/* Filtered variant (top_k > 0): the sampling regime of the temperature study */
/* (Section 4, RQ5) as samplers usually run it.  Between S1 and S2 the target */
/* distribution is replaced, as by a chain of logit warpers (temperature,     */
/* then top-k, then nucleus):                                                 */
/*  F1  rank the tokens by target logit, higher first, equal logits by lower  */
/*      token index; keep the first top_k;                                     */
/*  F2  renormalise p over the kept tokens;                                    */
/*  F3  if top_p < 1: keep the shortest prefix, in rank order, whose          */
/*      cumulative (renormalised) probability reaches top_p; renormalise.      */
/* Every other token gets p = 0.  top_k = 0 leaves p as it is (top_p unused). */
/* The paper does not define filtering; F1-F3 restate, in their usual order,   */
/* the usual top-k / nucleus samplers, and the accept / resample steps then    */
/* preserve the FILTERED target distribution.                                  */
static int accept_sampling(const float* logits, const float* dprobs, const int32_t* tokens,
                           const int32_t* parent, const int32_t* n_nodes, double tau, int top_k, double top_p,
                           const float* uniforms, int B, int T, int V, int max_depth,
                           int32_t* accept_len, int32_t* path, int32_t* next_token,
                           uint8_t* near_tie, int32_t* status) {
    if (!logits || !dprobs || !tokens || !parent || !uniforms || !accept_len || !path ||
        !next_token)
        return 1;
    if (B < 0 || T < 1 || V < 1 || max_depth < 0 || !(tau > 0.0)) return 2;
    if (top_k < 0 || (top_k > 0 && !(top_p > 0.0 && top_p <= 1.0))) return 2;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic)
#endif
    for (int b = 0; b < B; ++b) {
        const int n = node_count(n_nodes, b, T);
        const int32_t* par = parent + (size_t)b * T;
        const int32_t* tok = tokens + (size_t)b * T;
        const float* u = uniforms + (size_t)b * T;
        int32_t* pth = path + (size_t)b * (max_depth + 1);
        uint8_t* tie = near_tie ? near_tie + (size_t)b * T : NULL;
        if (tie) memset(tie, 0, (size_t)T);
        int* depth = (int*)malloc(sizeof(int) * (size_t)T);
        int st = validate_accept_inputs(par, tok, n, T, V, max_depth, depth);
        if (!(st & ORC_SEQ_BAD_PARENT) && logits_unusable(logits + (size_t)b * T * V, n, V)) st |= ORC_SEQ_NONFINITE;
        if (status) status[b] = st;
        if (st) {
            accept_len[b] = -1;
            next_token[b] = -1;
            for (int j = 0; j <= max_depth; ++j) pth[j] = -1;
            free(depth);
            continue;
        }
        double* p = (double*)malloc(sizeof(double) * (size_t)V);
        double* q = (double*)malloc(sizeof(double) * (size_t)V);
        int cur = 0;
        for (;;) {
            /* S1 */
            const float* x = logits + ((size_t)b * T + cur) * V;
            const float* dq = dprobs + ((size_t)b * T + cur) * V;
            double mx = -INFINITY;
            for (int v = 0; v < V; ++v)
                if ((double)x[v] > mx) mx = (double)x[v];
            double den = 0.0;
            for (int v = 0; v < V; ++v) {
                p[v] = exp(((double)x[v] - mx) / tau);
                den += p[v];
            }
            for (int v = 0; v < V; ++v) {
                p[v] /= den;
                q[v] = (double)dq[v];
            }
            if (top_k > 0) {
                /* F1: selection by repeated maximum over the tokens not taken yet */
                const int k = top_k < V ? top_k : V;
                int* ord = (int*)malloc(sizeof(int) * (size_t)k);
                unsigned char* taken = (unsigned char*)calloc((size_t)V, 1);
                for (int j = 0; j < k; ++j) {
                    int best = -1;
                    for (int v = 0; v < V; ++v)
                        if (!taken[v] && (best < 0 || x[v] > x[best])) best = v;
                    taken[best] = 1;
                    ord[j] = best;
                }
                /* F2 */
                double kept_mass = 0.0;
                for (int j = 0; j < k; ++j) kept_mass += p[ord[j]];
                int m = k;
                if (top_p < 1.0) { /* F3 */
                    double cum = 0.0;
                    for (int j = 0; j < k; ++j) {
                        cum += p[ord[j]] / kept_mass;
                        if (cum >= top_p) {
                            m = j + 1;
                            break;
                        }
                    }
                    kept_mass = 0.0;
                    for (int j = 0; j < m; ++j) kept_mass += p[ord[j]];
                }
                double* keep = (double*)malloc(sizeof(double) * (size_t)m);
                for (int j = 0; j < m; ++j) keep[j] = p[ord[j]] / kept_mass;
                for (int v = 0; v < V; ++v) p[v] = 0.0;
                for (int j = 0; j < m; ++j) p[ord[j]] = keep[j];
                free(keep), free(taken), free(ord);
            }
            /* S2 / S3 */
            int accepted = -1;
            for (int c = cur + 1; c < n && accepted < 0; ++c) {
                if (par[c] != cur) continue;
                const int xt = tok[c];
                double ratio;
                if (q[xt] > 0.0)
                    ratio = p[xt] / q[xt];
                else
                    ratio = (p[xt] > 0.0) ? INFINITY : 0.0;
                const double uc = (double)u[c];
                if (tie && fabs(ratio - uc) < 1e-6) tie[c] = 1;
                const double thr = ratio < 1.0 ? ratio : 1.0;
                if (uc < thr) {
                    accepted = c;
                    break;
                }
                double mass = 0.0;
                for (int v = 0; v < V; ++v) {
                    const double r = p[v] - q[v];
                    mass += (r > 0.0) ? r : 0.0;
                }
                if (mass > 0.0)
                    for (int v = 0; v < V; ++v) {
                        const double r = p[v] - q[v];
                        p[v] = (r > 0.0) ? r / mass : 0.0;
                    }
                q[xt] = 0.0;
                double qs = 0.0;
                for (int v = 0; v < V; ++v) qs += q[v];
                if (!(qs > 0.0)) break;
                for (int v = 0; v < V; ++v) q[v] /= qs;
            }
            if (accepted >= 0) {
                cur = accepted;
                continue;
            }
            /* S4 */
            double tot = 0.0;
            for (int v = 0; v < V; ++v) tot += p[v];
            const double target = (double)u[0] * tot;
            double run = 0.0;
            int pick = -1, last_pos = 0;
            for (int v = 0; v < V; ++v) {
                if (p[v] > 0.0) last_pos = v;
                run += p[v];
                if (run > target) {
                    pick = v;
                    break;
                }
            }
            next_token[b] = (pick >= 0) ? pick : last_pos;
            break;
        }
        accept_len[b] = write_path(par, cur, depth, max_depth, pth);
        free(p);
        free(q);
        free(depth);
    }
    return 0;
}

int s4c_oracle_accept_stochastic(const float* logits, const float* dprobs, const int32_t* tokens,
                                 const int32_t* parent, const int32_t* n_nodes, double tau,
                                 const float* uniforms, int B, int T, int V, int max_depth,
                                 int32_t* accept_len, int32_t* path, int32_t* next_token,
                                 uint8_t* near_tie, int32_t* status) {
    return accept_sampling(logits, dprobs, tokens, parent, n_nodes, tau, 0, 1.0, uniforms, B, T, V, max_depth,
                           accept_len, path, next_token, near_tie, status);
}

int s4c_oracle_accept_filtered(const float* logits, const float* dprobs, const int32_t* tokens,
                               const int32_t* parent, const int32_t* n_nodes, double tau, int top_k, double top_p,
                               const float* uniforms, int B, int T, int V, int max_depth,
                               int32_t* accept_len, int32_t* path, int32_t* next_token,
                               uint8_t* near_tie, int32_t* status) {
    if (top_k < 1) return 2;
    return accept_sampling(logits, dprobs, tokens, parent, n_nodes, tau, top_k, top_p, uniforms, B, T, V, max_depth,
                           accept_len, path, next_token, near_tie, status);
}

/* ------------------------------------------------------------------------- */
/* Compaction of the accepted path (Section 3.2, last paragraph: accepted     */
/* tokens and their features are kept for the next drafting phase).            */
/*                                                                           */
/* Every cache is [B,Hkv,C,d] with elem_bytes per element.  For j = 0..a:     */
/* slot L_b + j  <-  old slot L_b + path[j]  (copied from a snapshot of the   */
/* T tree slots, so the order of the copies cannot matter);                   */
/* feat_out[b,j,:] = feat_in[b,path[j],:]; cache_len[b] = L_b + a + 1.        */
/* A sequence with accept_len < 0 is skipped.                                 */
/* ------------------------------------------------------------------------- */
int s4c_oracle_kv_compact(uint8_t* const* k_caches, uint8_t* const* v_caches, int n_layers,
                          int32_t* cache_len, const int32_t* path, const int32_t* accept_len,
                          int max_depth, const uint8_t* feat_in, uint8_t* feat_out, int B, int T,
                          int Hkv, int d, int C, int hid, int elem_bytes, int32_t* status) {
    if (!cache_len || !path || !accept_len) return 1;
    if (n_layers > 0 && (!k_caches || !v_caches)) return 1;
    if (B < 0 || T < 1 || Hkv < 1 || d < 1 || C < 1 || max_depth < 0 || elem_bytes < 1) return 2;
    const size_t row = (size_t)d * elem_bytes;
    const size_t frow = (size_t)hid * elem_bytes;
    uint8_t* snap = (uint8_t*)malloc(row * (size_t)T);
    for (int b = 0; b < B; ++b) {
        const int a = accept_len[b];
        const int L = cache_len[b];
        const int32_t* pth = path + (size_t)b * (max_depth + 1);
        int st = ORC_SEQ_OK;
        if (a < 0) {
            if (status) status[b] = st;
            continue;
        }
        if (a > max_depth) st |= ORC_SEQ_DEPTH;
        if (L < 0 || (long)L + T > (long)C) st |= ORC_SEQ_CAPACITY;
        if (!st) {
            for (int j = 0; j <= a; ++j) {
                if (pth[j] < j || pth[j] >= T) st |= ORC_SEQ_BAD_PATH;
                if (j > 0 && pth[j] <= pth[j - 1]) st |= ORC_SEQ_BAD_PATH;
            }
            if (pth[0] != 0) st |= ORC_SEQ_BAD_PATH;
        }
        if (status) status[b] = st;
        if (st) continue;
        for (int l = 0; l < n_layers; ++l)
            for (int kv = 0; kv < 2; ++kv) {
                uint8_t* cache = kv ? v_caches[l] : k_caches[l];
                for (int h = 0; h < Hkv; ++h) {
                    uint8_t* base = cache + (((size_t)b * Hkv + h) * C + L) * row;
                    memcpy(snap, base, row * (size_t)T);
                    for (int j = 0; j <= a; ++j)
                        memcpy(base + (size_t)j * row, snap + (size_t)pth[j] * row, row);
                }
            }
        if (feat_in && feat_out)
            for (int j = 0; j <= a; ++j)
                memcpy(feat_out + ((size_t)b * (max_depth + 1) + j) * frow,
                       feat_in + ((size_t)b * T + pth[j]) * frow, frow);
        cache_len[b] = L + a + 1;
    }
    free(snap);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Continuous verification tree (Section 3.2; Figure 3, left).                */
/*                                                                           */
/* The tree starts at the last committed token (the root).  Drafts are first  */
/* generated "vertically": a chain of top-1 choices, one per drafting depth.  */
/* Then the tree is extended "horizontally", depth by depth: every node at    */
/* depth l-1 receives the top-k alternatives at its position until it has     */
/* branching[l-1] children (its first child is the top-1 choice, the others   */
/* the 2nd, 3rd ... most probable tokens of the same distribution).  Growth   */
/* stops at T nodes.  Nodes are then numbered breadth-first, which makes      */
/* parent[i] < i, keeps siblings contiguous and in rank order.                */
/*                                                                           */
/* draft_probs [B,T,V] float32: row n (in the final numbering) is the         */
/*             distribution the children of node n are chosen from -- the     */
/*             same array s4c_oracle_accept_stochastic reads.                 */
/* branching   [D] children per node at depths 0..D-1 (>= 1 each)             */
/* root_token  [B]; cache_len [B] or NULL                                     */
/* tokens, parent, position [B,T]; n_nodes [B]                                */
/*   child j (j = 1..k) of node n carries the j-th most probable token of     */
/*   row n, ties going to the lower token index; position = cache_len + depth */
/*   (0-based depth; just the depth when cache_len is NULL).  Entries beyond  */
/*   n_nodes[b] are padding: parent -1, token 0, position 0.                  */
/* The shape depends on (branching, T) only, so it is the same for every      */
/* sequence of the batch; the tokens differ.                                  */
/* Readings: "top-k alternatives at the same position" are the siblings of    */
/* the top-1 token (children of the same parent), as the example of Figure 3  */
/* has it (two continuations of the root, each with a top-1 successor and two */
/* alternatives to that successor); nodes added horizontally are expanded at  */
/* the next depth like the vertical ones.                                     */
/* ------------------------------------------------------------------------- */
int s4c_oracle_build_tree(const float* draft_probs, const int32_t* branching, int D,
                          const int32_t* root_token, const int32_t* cache_len, int B, int T, int V,
                          int32_t* tokens, int32_t* parent, int32_t* position, int32_t* n_nodes) {
    if (!draft_probs || !branching || !root_token || !tokens || !parent || !position || !n_nodes) return 1;
    if (B < 0 || T < 1 || V < 1 || D < 0) return 2;
    for (int l = 0; l < D; ++l)
        if (branching[l] < 1 || branching[l] > V) return 2;
    /* ---- the shape, in creation order */
    int* cpar = (int*)malloc(sizeof(int) * (size_t)T);
    int* cdep = (int*)malloc(sizeof(int) * (size_t)T);
    int* nchild = (int*)calloc((size_t)T, sizeof(int));
    int n = 1;
    cpar[0] = -1, cdep[0] = 0;
    /* vertically: the chain of top-1 choices */
    for (int l = 0, tip = 0; l < D && n < T; ++l) {
        cpar[n] = tip, cdep[n] = l + 1, nchild[tip] += 1;
        tip = n++;
    }
    /* horizontally: depth by depth, alternatives at the same position */
    for (int l = 1; l <= D; ++l)
        for (int node = 0; node < n; ++node) {
            if (cdep[node] != l - 1) continue;
            while (nchild[node] < branching[l - 1] && n < T) {
                cpar[n] = node, cdep[n] = l, nchild[node] += 1;
                ++n;
            }
        }
    /* ---- breadth-first numbering: visit order = new index; children keep their creation order */
    int* order = (int*)malloc(sizeof(int) * (size_t)n);   /* order[new] = creation index */
    int* newid = (int*)malloc(sizeof(int) * (size_t)n);
    int head = 0, tail = 0;
    order[tail++] = 0;
    while (head < tail) {
        const int u = order[head++];
        for (int c = 0; c < n; ++c)
            if (cpar[c] == u) order[tail++] = c;
    }
    for (int i = 0; i < n; ++i) newid[order[i]] = i;
    int* par = (int*)malloc(sizeof(int) * (size_t)n);
    int* dep = (int*)malloc(sizeof(int) * (size_t)n);
    for (int i = 0; i < n; ++i) {
        par[i] = order[i] == 0 ? -1 : newid[cpar[order[i]]];
        dep[i] = cdep[order[i]];
    }
    /* ---- tokens: the children of a node, in index order, take the 1st, 2nd, ... most probable token of its row */
    unsigned char* taken = (unsigned char*)malloc((size_t)V);
    for (int b = 0; b < B; ++b) {
        int32_t* tok = tokens + (size_t)b * T;
        int32_t* pr = parent + (size_t)b * T;
        int32_t* pos = position + (size_t)b * T;
        const int base = cache_len ? cache_len[b] : 0;
        for (int i = 0; i < T; ++i) {
            pr[i] = i < n ? par[i] : -1;
            pos[i] = i < n ? base + dep[i] : 0;
            tok[i] = 0;
        }
        tok[0] = root_token[b];
        n_nodes[b] = n;
        for (int u = 0; u < n; ++u) {
            const float* row = draft_probs + ((size_t)b * T + u) * V;
            memset(taken, 0, (size_t)V);
            for (int c = u + 1; c < n; ++c) {
                if (par[c] != u) continue;
                int best = -1;  /* most probable token not taken yet; the lowest index among equals */
                for (int v = 0; v < V; ++v)
                    if (!taken[v] && (best < 0 || row[v] > row[best])) best = v;
                taken[best] = 1;
                tok[c] = best;
            }
        }
    }
    free(taken), free(par), free(dep), free(order), free(newid), free(cpar), free(cdep), free(nchild);
    return 0;
}
