/*
 * s4c.h -- C ABI of libs4c.so: the verify step of S4C speculative decoding
 * (arXiv 2506.14158) as hand-written CUDA kernels for NVIDIA B200 (sm_100a).
 *
 * One verify step of the target model over the continuous verification tree
 * (Section 3.2) is three calls, all asynchronous on one CUDA stream:
 *
 *   per decoder layer:  s4c_tree_attention   tree-masked attention of the T tree tokens
 *   once per step:      s4c_tree_accept      greedy / speculative-sampling acceptance + path walk
 *   once per step:      s4c_kv_compact       keep the accepted path's K/V (all layers) and features
 * and, before them, optionally
 *   once per step:      s4c_tree_build       the tree itself, from the drafter's distributions
 *
 * Around them, the rest of the target's pass and the drafter's head (Section 3.1, Eq. 3-6), so
 * that a whole greedy round runs from these calls alone:
 *   per decoder layer:  s4c_qkv_rope (_same_tree, _at)  q/k/v projections + rotary embedding into the
 *                                                   attention layout and the cache's tree slots
 *                       s4c_linear, s4c_linear_rmsnorm, s4c_rmsnorm   projections, gated MLP, norms
 *   once per step:      s4c_embed_gather            Eq. 6
 *                       s4c_lm_head_greedy / s4c_lm_head_topk   LM head with the greedy choice /
 *                                                   the k ranked choices kept in the epilogue
 *                       s4c_tree_accept_tokens      the greedy walk on the choices
 *                       s4c_tree_build_topk         the tree from ranked choices
 * Variants: s4c_tree_attention_rows (output as the rows the next projection reads), s4c_lm_head_logits
 * (float32 logits for speculative sampling), s4c_tree_attention_paged / s4c_kv_compact_paged (paged caches),
 * s4c_tree_accept_filtered (top-k / nucleus filtered sampling), s4c_tree_accept_noalloc.
 *
 * Conventions for every entry point
 *   - Every pointer is a DEVICE pointer owned by the caller unless its comment says "host".
 *     The library allocates nothing; scratch memory comes from the caller, sized by the
 *     matching *_workspace_bytes query (a host function, no CUDA call).
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and return without
 *     synchronising.  Results are never read on the host by the library.
 *   - The return value reports host-side argument validation and launch errors only.
 *     Data-dependent problems (a malformed tree, a token outside the vocabulary, a cache
 *     that is too short) are reported per sequence in the caller's device array
 *     `status[B]` (S4C_SEQ_* bit flags, 0 = fine; may be NULL): the kernels skip such a
 *     sequence, mark its outputs (accept_len = -1) and never trap or assert.
 *   - Base pointers of tensors must be 16-byte aligned.  All tensors are dense, row-major,
 *     innermost dimension last.
 *   - Tree order: node 0 is the root, i.e. the last committed token of the prefix (Section 3.2,
 *     Figure 3), parent[0] = -1 and 0 <= parent[i] < i.  A batch may pad trees to T nodes;
 *     n_nodes[b] gives the real count (NULL = T everywhere).
 *   - Limits: 1 <= T <= 128, d in {64, 128}, Hq % Hkv == 0.
 */
#ifndef S4C_H_
#define S4C_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    S4C_OK = 0,
    S4C_ERR_NULL = 1,        /* a required pointer is NULL */
    S4C_ERR_SHAPE = 2,       /* a size is out of range or inconsistent */
    S4C_ERR_DTYPE = 3,       /* unknown s4c_dtype */
    S4C_ERR_ALIGN = 4,       /* a tensor base pointer is not 16-byte aligned */
    S4C_ERR_WORKSPACE = 5,   /* workspace missing or smaller than the query says */
    S4C_ERR_UNSUPPORTED = 6, /* valid request the library has no kernel for */
    S4C_ERR_CUDA = 7         /* a CUDA runtime call (launch, attribute) failed */
} s4c_status;

typedef enum { S4C_F32 = 0, S4C_BF16 = 1 } s4c_dtype;

/* per-sequence flags written to status[b] */
#define S4C_SEQ_OK 0
#define S4C_SEQ_BAD_PARENT 1  /* n_nodes out of 1..T, parent[0] != -1 or parent[i] outside [0, i) */
#define S4C_SEQ_TOKEN_RANGE 2 /* a draft token outside [0, V) */
#define S4C_SEQ_CAPACITY 4    /* cache_len < 0 or cache_len + tree slots > C */
#define S4C_SEQ_DEPTH 8       /* a node deeper than max_depth / accept_len > max_depth */
#define S4C_SEQ_BAD_PATH 16   /* path not of the form 0 = path[0] < path[1] < ... < T */
#define S4C_SEQ_TIMEOUT 32    /* a bounded in-kernel wait expired (OR-ed in; results of that sequence are invalid) */
#define S4C_SEQ_NONFINITE 64  /* a target-logit row of a real node holds a NaN or +Inf, or nothing but -Inf */
#define S4C_SEQ_BAD_PAGE 128  /* a block-table entry in use names a page outside the pool */

typedef void* s4c_stream_t; /* a cudaStream_t */

/* Library version (major * 100 + minor) and a static, NUL-terminated name for a return code (host). */
int s4c_version(void);
const char* s4c_status_string(s4c_status code);

/* ------------------------------------------------------------------------------------------
 * s4c_tree_attention -- the tree-masked attention of the verification pass (Section 3.2; the
 * mask is drawn in Figure 3): one target forward pass verifies all drafts at once (Sections 1, 2).
 *
 * For sequence b, query head h and tree node i the output is softmax attention of q[b,h,i,:]
 * over the cache slots 0..L_b-1 (the committed prefix, fully visible) and the slots L_b+t of the
 * nodes t on the path root..i (i itself included); every other tree slot is masked.  KV head of
 * query head h is h / (Hq/Hkv).  Scores are scale * <q,k>; softmax statistics and accumulation
 * are fp32; for S4C_BF16 the probabilities are rounded to bf16 before the PV product, and partial
 * results of the splits of a long cache are exchanged as normalised fp16 rows: output entries
 * beyond +-65504 (possible only with V entries of that size) are clamped there.
 *
 *   q          [B,Hq,T,d]   dt     queries of the tree tokens (after positional encoding)
 *   k_cache    [B,Hkv,C,d]  dt     keys; the tree tokens' own keys already sit at slots L_b..L_b+T-1
 *   v_cache    [B,Hkv,C,d]  dt     values, same layout
 *   cache_len  [B]          int32  L_b, the committed length (tree slots not counted)
 *   parent     [B,T]        int32
 *   n_nodes    [B] or NULL  int32
 *   out        [B,Hq,T,d]   dt     rows of padding nodes (i >= n_nodes[b]) are written as zeros;
 *                                  rows of a flagged sequence are left untouched
 *   C          capacity of the caches in slots (what the tensors are laid out for)
 *   max_cache_len  what the host knows about the live lengths: an upper bound on cache_len[b] over
 *              the batch, or 0 if it knows nothing (the capacity then stands in).  A serving cache has
 *              C = the longest context it may ever hold while the sequences are far shorter; the host
 *              cannot read cache_len (device memory, no synchronisation), so the split of the cache
 *              over CTAs, the kernel variant and the grid are chosen for min(C, max_cache_len + T)
 *              slots.  The value steers the launch shape only: results are the same for any value,
 *              and a sequence longer than the bound is still handled correctly (only slower).
 *              Negative: S4C_ERR_SHAPE.
 *   scale      0 selects 1/sqrt(d)
 *   status     [B] or NULL  int32  S4C_SEQ_BAD_PARENT, S4C_SEQ_CAPACITY
 *   workspace  at least s4c_tree_attention_workspace_bytes(...) bytes, 256-byte aligned; holds the
 *              split-KV partial results; contents are scratch, nothing needs clearing.  The query
 *              takes the capacity C and covers every max_cache_len.
 * Calls sharing a workspace must be ordered on the stream.
 * ------------------------------------------------------------------------------------------ */
size_t s4c_tree_attention_workspace_bytes(int B, int T, int Hq, int Hkv, int d, int C, s4c_dtype dt);

s4c_status s4c_tree_attention(const void* q, const void* k_cache, const void* v_cache,
                              const int32_t* cache_len, const int32_t* parent, const int32_t* n_nodes,
                              void* out, int B, int T, int Hq, int Hkv, int d, int C, int max_cache_len,
                              s4c_dtype dt, float scale, int32_t* status, void* workspace,
                              size_t workspace_bytes, s4c_stream_t stream);

/* s4c_tree_attention_rows -- the same attention, written as the rows the layer's output projection
 * reads: out_rows [B, T, Hq, d] = [B*T rows, Hq*d] instead of [B, Hq, T, d] (no transposing copy
 * between the two).  Same arguments, workspace and status; S4C_BF16 only (S4C_ERR_UNSUPPORTED
 * otherwise).  Every element equals, bit for bit, the one s4c_tree_attention writes. */
s4c_status s4c_tree_attention_rows(const void* q, const void* k_cache, const void* v_cache,
                                   const int32_t* cache_len, const int32_t* parent, const int32_t* n_nodes,
                                   void* out_rows, int B, int T, int Hq, int Hkv, int d, int C, int max_cache_len,
                                   s4c_dtype dt, float scale, int32_t* status, void* workspace,
                                   size_t workspace_bytes, s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_tree_accept -- the accept / resample rule of Section 2 ("Speculative Sampling"): a draft token
 * passes with probability min(1, p/q), a rejected position is resampled from norm(max(0, p - q));
 * Eq. 11 and Eq. 12 of Section 3.2 apply it along the tree, whose longest accepted path is kept
 * (Section 3.2); greedy decoding is what Section 4.1.2 uses.
 *
 * temperature == 0: greedy.  g[n] = argmax_v target_logits[b,n,v] (lowest v on ties); node i is
 *   accepted iff its parent is and tokens[b,i] == g[parent]; the deepest accepted node e (lowest
 *   index among equals) ends the path and next_token = g[e].
 * temperature > 0: speculative sampling along the tree.  At the current node (root first) with
 *   p = softmax(target_logits[b,cur,:]/temperature) and q = draft_probs[b,cur,:], the children are
 *   tried in index order: child c with token x is accepted iff uniforms[b,c] < min(1, p(x)/q(x))
 *   (strict; q(x) = 0 counts as +inf when p(x) > 0, else 0).  After a rejection p becomes
 *   norm(max(p - q, 0)) (kept if that mass is 0) and q loses x and is renormalised.  When no child
 *   is accepted, next_token is the smallest v whose running sum of p exceeds uniforms[b,0] * sum(p).
 *   Sums and ratios are evaluated in float64.
 *
 *   target_logits [B,T,V] f32   row n: the target's logits for the token that follows node n
 *   draft_probs   [B,T,V] f32   row n: the distribution the children of n were proposed from, at this
 *                               temperature; may be NULL iff temperature == 0
 *   tokens        [B,T]   int32 tokens[b,0] is the root's token (committed, never tested)
 *   uniforms      [B,T]   f32   in [0,1); entry i >= 1: acceptance draw of node i; entry 0: final-token
 *                               draw; may be NULL iff temperature == 0
 *   max_depth     path buffers hold max_depth+1 entries; a deeper tree is flagged S4C_SEQ_DEPTH
 *   accept_len    [B]   int32  out: a = number of accepted draft tokens (-1 for a flagged sequence)
 *   path          [B,max_depth+1] int32 out: node indices root..e, path[b,0] = 0, -1 beyond a
 *   next_token    [B]   int32  out: the bonus / resampled token (-1 for a flagged sequence)
 *   near_tie      [B,T] uint8  out or NULL: 1 where node i was tested with |p/q - u| < 1e-6
 *   status        [B] or NULL  S4C_SEQ_BAD_PARENT, S4C_SEQ_TOKEN_RANGE, S4C_SEQ_DEPTH, S4C_SEQ_NONFINITE
 *   workspace     at least s4c_tree_accept_workspace_bytes(B,T,V) bytes, 256-byte aligned, scratch.
 * Non-finite logits.  A -Inf logit beside finite ones is legal (that token has probability 0, as after a
 * vocabulary mask).  A NaN or +Inf anywhere in the rows of the real nodes (i < n_nodes[b]), or a row holding
 * nothing but -Inf, makes the softmax undefined: the sequence is flagged S4C_SEQ_NONFINITE and skipped
 * (accept_len = next_token = -1), the other sequences of the batch are unaffected.  The check rides on the
 * maximum reduction that reads every logit anyway.  draft_probs are taken as given (finite, >= 0): they are
 * only read on the walked rows, so they are not screened.
 * Any finite temperature > 0 is served; rows whose float spacing at the maximum exceeds 172 temperatures are
 * summed as a count of their maxima (every other term is below e^-172 of the sum).
 * Returns S4C_ERR_SHAPE for temperature < 0 or NaN.
 * ------------------------------------------------------------------------------------------ */
size_t s4c_tree_accept_workspace_bytes(int B, int T, int V);

s4c_status s4c_tree_accept(const float* target_logits, const float* draft_probs, const int32_t* tokens,
                           const int32_t* parent, const int32_t* n_nodes, float temperature,
                           const float* uniforms, int B, int T, int V, int max_depth,
                           int32_t* accept_len, int32_t* path, int32_t* next_token, uint8_t* near_tie,
                           int32_t* status, void* workspace, size_t workspace_bytes, s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_tree_accept_noalloc -- the paper has no counterpart; this is a packaging variant of
 * s4c_tree_accept for callers that cannot provide scratch memory.
 *
 * Some hosts of this library may not call cudaMalloc at the point where they verify a tree: a
 * serving loop that has handed all device memory to its own pool, a plug-in running inside
 * another framework's allocator, code on a latency path where an allocation could block or
 * synchronise.  For them this entry point takes the same inputs and outputs as s4c_tree_accept
 * but no workspace: its scratch is a fixed array of S4C_NOALLOC_SCRATCH_BYTES bytes compiled into
 * the library (so every GPU that loads the library gives up that much memory until the process
 * exits).  The call itself allocates and frees nothing, directly or through any library.
 *
 *   - Size limit: s4c_tree_accept_workspace_bytes(B,T,V) must not exceed
 *     S4C_NOALLOC_SCRATCH_BYTES (about B*T*(16*ceil(V/4096) + 40) bytes); a larger problem is
 *     refused with S4C_ERR_WORKSPACE and nothing is launched.
 *   - The first call on each device looks up the array's device address (a host-side runtime
 *     query, made with that device current).  Make that first call outside any stream capture.
 *   - All calls in the process share the one array per device, and it keeps whatever the last
 *     call left in it.  Nothing in it needs to start at zero (every value is written before it is
 *     read), but two calls whose kernels overlap on the GPU -- different streams, or one stream per
 *     thread -- race on it: order such calls on one stream or with events.
 *   - Results are identical to s4c_tree_accept on the same inputs.
 * All other arguments, outputs, status flags and return codes are those of s4c_tree_accept.
 * ------------------------------------------------------------------------------------------ */
#define S4C_NOALLOC_SCRATCH_BYTES (1 << 20)

s4c_status s4c_tree_accept_noalloc(const float* target_logits, const float* draft_probs, const int32_t* tokens,
                                   const int32_t* parent, const int32_t* n_nodes, float temperature,
                                   const float* uniforms, int B, int T, int V, int max_depth,
                                   int32_t* accept_len, int32_t* path, int32_t* next_token, uint8_t* near_tie,
                                   int32_t* status, s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_kv_compact -- Section 3.2, last paragraph: accepted tokens and their features are kept for
 * the following drafting phase (feature reuse, Section 1; "feature" = hidden state before the
 * LM head, Section 2 Notations).
 *
 * For every layer, KV head and j = 0..a (a = accept_len[b]): cache slot L_b + j receives the old
 * contents of slot L_b + path[b,j], for K and V, in place; feat_out[b,j,:] = feat_in[b,path[b,j],:];
 * finally cache_len[b] = L_b + a + 1.  Slots >= the new length are unspecified afterwards; slots
 * < L_b and other sequences' rows are never written.  A sequence with accept_len[b] < 0 is skipped.
 *
 *   k_caches, v_caches  device arrays of n_layers device pointers, each cache [B,Hkv,C,d] dt
 *                       (n_layers may be 0, the arrays then may be NULL)
 *   cache_len   [B] int32  in: L_b   out: L_b + a + 1
 *   path        [B,max_depth+1] int32, accept_len [B] int32: as written by s4c_tree_accept
 *   feat_in     [B,T,hid] dt or NULL;  feat_out [B,max_depth+1,hid] dt or NULL (rows > a untouched)
 *   status      [B] or NULL  S4C_SEQ_CAPACITY (L_b + T > C), S4C_SEQ_DEPTH, S4C_SEQ_BAD_PATH
 * d * sizeof(dt) and hid * sizeof(dt) must be multiples of 16 bytes (rows move as 16-byte words).
 * ------------------------------------------------------------------------------------------ */
s4c_status s4c_kv_compact(void* const* k_caches, void* const* v_caches, int n_layers, int32_t* cache_len,
                          const int32_t* path, const int32_t* accept_len, int max_depth,
                          const void* feat_in, void* feat_out, int B, int T, int Hkv, int d, int C, int hid,
                          s4c_dtype dt, int32_t* status, s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_tree_accept_filtered -- s4c_tree_accept's speculative-sampling walk (Section 2; Eq. 11, Eq. 12;
 * longest accepted path, Section 3.2) against a FILTERED target distribution: the sampling regime of
 * the temperature study (Section 4, RQ5) as samplers usually run it.  The paper does not define a
 * filter; this one is the usual chain of logit warpers:
 *   temperature, then top-k, then nucleus.  At every node the tokens are ranked by target logit
 *   (higher first, equal logits by lower token); the first top_k are kept and p = softmax(logit /
 *   temperature) is renormalised over them; if top_p < 1 the shortest prefix in rank order whose
 *   cumulative (renormalised) probability reaches top_p is kept and renormalised again.  Every
 *   other token has target probability 0: it is never accepted and never emitted.
 * The accept / reject / resample rules, uniforms, outputs, status flags and the NONFINITE rule are
 * those of s4c_tree_accept with this p; the draft distribution is taken as given (a drafter that was
 * filtered the same way passes its filtered probabilities).  top_k = 1 is greedy verification.
 *   temperature > 0;  1 <= top_k <= 64 (values above V act as V);  0 < top_p <= 1.
 *   workspace: at least s4c_tree_accept_filtered_workspace_bytes(B, T, V, top_k) bytes, 256-byte aligned.
 * Cost: every logits row is read once and no exponential is taken over the vocabulary (the kept
 * tokens are found by selection); draft rows are read only where a sibling is rejected.
 * ------------------------------------------------------------------------------------------ */
size_t s4c_tree_accept_filtered_workspace_bytes(int B, int T, int V, int top_k);

s4c_status s4c_tree_accept_filtered(const float* target_logits, const float* draft_probs, const int32_t* tokens,
                                    const int32_t* parent, const int32_t* n_nodes, float temperature, int top_k,
                                    float top_p, const float* uniforms, int B, int T, int V, int max_depth,
                                    int32_t* accept_len, int32_t* path, int32_t* next_token, uint8_t* near_tie,
                                    int32_t* status, void* workspace, size_t workspace_bytes, s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_lm_head_greedy -- the LM head of the verify pass fused with the greedy choice (Eq. 6:
 * t = Argmax(LM_head(f)); Section 3.2: the target's logits at every tree node; Section 4.1: greedy
 * decoding in all experiments): for every row r of the hidden states
 *     logits[r, v] = sum_h hidden[r, h] * weight[v, h]      (bf16 inputs, float32 accumulation)
 *     token[r]     = the first v that reaches max_v logits[r, v];   max_logit[r] = that maximum
 * The [R, V] logits are not written anywhere.
 *   hidden [R, H] bf16 (device), weight [V, H] bf16 (device, the LM head's rows), both row-major and
 *   16-byte aligned; H a multiple of 64; any R (rows are served in groups of 256, each group reads
 *   the weights once); token [R] int32 (device); max_logit [R] float (device) or NULL;
 *   status: one int32 (device) or NULL, set to 0 and OR-ed with S4C_SEQ_TIMEOUT if a wait inside
 *   the kernel was given up (results are then undefined); workspace: at least
 *   s4c_lm_head_greedy_workspace_bytes(R, V, H) bytes, 256-byte aligned, caller-owned.
 * Equal logits (as float32 sums in the tensor cores' order) go to the lower token; a row without any
 * comparable logit (NaN everywhere) gets token -1.  Launches are asynchronous on `stream`.
 *
 * s4c_tree_accept_tokens -- greedy verification (Section 4.1; longest accepted path, Section 3.2)
 * from the target's choice per node instead of its logits: a node is accepted when its parent is and
 * its token equals target_token[parent]; the path ends at the accepted node of greatest depth
 * (lowest index among equals); next_token = target_token at that node.  Arguments, outputs and
 * status flags as s4c_tree_accept with temperature 0 (target_token [B, T] int32 replaces the logits).
 * ------------------------------------------------------------------------------------------ */
size_t s4c_lm_head_greedy_workspace_bytes(int R, int V, int H);

/* s4c_lm_head_topk -- the same contraction with the k best tokens per row instead of the best one: the
 * drafter's LM head and its ranked choices (Section 3.1: the heads' Argmax / top-2 candidates; Section
 * 3.2: the top-k alternatives of the verification tree).  token [R, k] int32 and logit [R, k] float
 * (or NULL), best first, equal logits by lower token; entries beyond the vocabulary (k > V) or without
 * a comparable logit are token -1, logit -inf.  1 <= k <= 8 (S4C_ERR_UNSUPPORTED above);
 * s4c_lm_head_greedy is the case k = 1.  Workspace: s4c_lm_head_topk_workspace_bytes(R, V, H, k).
 *
 * s4c_tree_build_topk -- s4c_tree_build from ranked choices instead of distributions: the tree of
 * Section 3.2 with the same shape and numbering; child j of node n carries topk[b, n, j]
 * (topk [B, T, k] int32, device; k >= every branching factor).  No workspace.  With s4c_lm_head_topk
 * in front, a drafting round needs no [B, T, V] array of probabilities at all. */
size_t s4c_lm_head_topk_workspace_bytes(int R, int V, int H, int k);

s4c_status s4c_lm_head_topk(const void* hidden, const void* weight, int R, int V, int H, int k, int32_t* token,
                            float* logit, int32_t* status, void* workspace, size_t workspace_bytes,
                            s4c_stream_t stream);

s4c_status s4c_tree_build_topk(const int32_t* topk, int k, const int32_t* branching, int depth,
                               const int32_t* root_token, const int32_t* cache_len, int B, int T, int32_t* tokens,
                               int32_t* parent, int32_t* position, int32_t* n_nodes, s4c_stream_t stream);

s4c_status s4c_lm_head_greedy(const void* hidden, const void* weight, int R, int V, int H, int32_t* token,
                              float* max_logit, int32_t* status, void* workspace, size_t workspace_bytes,
                              s4c_stream_t stream);

s4c_status s4c_tree_accept_tokens(const int32_t* target_token, const int32_t* tokens, const int32_t* parent,
                                  const int32_t* n_nodes, int B, int T, int V, int max_depth, int32_t* accept_len,
                                  int32_t* path, int32_t* next_token, int32_t* status, s4c_stream_t stream);

/* s4c_lm_head_logits -- the LM head when the logits themselves are wanted: verification by speculative
 * sampling (Eq. 11-12, temperature > 0) needs the target's distribution at the walked nodes, so
 * logits[r, v] = sum_h hidden[r, h] * weight[v, h] are written out as float32 [R, V] (the float32 sums
 * of the bf16 products, unrounded) in the layout s4c_tree_accept reads.  hidden [R, H], weight [V, H]
 * bf16; H a multiple of 64, V a multiple of 8; status and workspace as s4c_linear
 * (s4c_lm_head_logits_workspace_bytes(R, V, H) bytes).  Greedy verification does not need this call:
 * s4c_lm_head_greedy keeps the choice and writes no logits. */
size_t s4c_lm_head_logits_workspace_bytes(int R, int V, int H);

s4c_status s4c_lm_head_logits(const void* hidden, const void* weight, int R, int V, int H, float* logits,
                              int32_t* status, void* workspace, size_t workspace_bytes, s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_qkv_rope -- the input side of a decoder layer in the verify pass (Section 3.2: the target's
 * forward pass over the T tree tokens; the paper's targets are LLaMA-family models): for every tree
 * token the q, k, v projections of its hidden state (no bias), rotary embedding (rotate-half form)
 * of q and k at position cache_len[b] + depth(node), q stored where s4c_tree_attention reads it and
 * k, v stored straight into the caches' tree slots cache_len[b] + node:
 *     [q | k | v](b, t) = x[b, t, :] . w_qkv^T          (bf16 inputs, float32 accumulation)
 *     rot(u, p)[i]       = u[i] cos(p f_i) - u[i + d/2] sin(p f_i),
 *     rot(u, p)[i + d/2] = u[i + d/2] cos(p f_i) + u[i] sin(p f_i),   f_i = rope_theta^(-2i/d), i < d/2
 *     q_out[b, h, t, :] = rot(q_h, p);  k_cache[b, h, L_b + t, :] = rot(k_h, p);  v_cache[b, h, L_b + t, :] = v_h
 *   x [B, T, H] bf16 (device); w_qkv [(Hq + 2 Hkv) d, H] bf16 (device): the q heads' rows, then the
 *   k heads', then the v heads'; cache_len, parent, n_nodes as for s4c_tree_attention (node 0 is the
 *   root, depth 0); q_out [B, Hq, T, d] bf16; k_cache, v_cache [B, Hkv, C, d] bf16 (only the tree
 *   slots of the first n_nodes[b] nodes are written; everything else is left as it is);
 *   d in {64, 128}; H a multiple of 64; rope_theta > 1 (10000 for the paper's models);
 *   status [B] int32 (device) or NULL: S4C_SEQ_BAD_PARENT, S4C_SEQ_CAPACITY (L_b + T > C) -- such a
 *   sequence is skipped (nothing of it is written) --, S4C_SEQ_TIMEOUT; workspace: at least
 *   s4c_qkv_rope_workspace_bytes(B, T, d) bytes, 256-byte aligned.  All pointers 16-byte aligned.
 * cos / sin are evaluated in float64 and applied in float32; results are rounded to bf16 once.
 * ------------------------------------------------------------------------------------------ */
size_t s4c_qkv_rope_workspace_bytes(int B, int T, int d);

s4c_status s4c_qkv_rope(const void* x, const void* w_qkv, const int32_t* cache_len, const int32_t* parent,
                        const int32_t* n_nodes, void* q_out, void* k_cache, void* v_cache, int B, int T, int H,
                        int Hq, int Hkv, int d, int C, float rope_theta, int32_t* status, void* workspace,
                        size_t workspace_bytes, s4c_stream_t stream);

/* s4c_qkv_rope_at -- the same with the root's position given apart from the cache length: a node's
 * position is position_base[b] + depth, its slot stays cache_len[b] + node.  For a drafter head
 * (Section 3.1.1) whose own cache holds fewer entries than the text has tokens.  position_base [B]
 * int32 (device); a negative entry flags the sequence S4C_SEQ_CAPACITY.  Everything else as s4c_qkv_rope
 * (which is the case position_base = cache_len). */
s4c_status s4c_qkv_rope_at(const void* x, const void* w_qkv, const int32_t* cache_len, const int32_t* position_base,
                           const int32_t* parent, const int32_t* n_nodes, void* q_out, void* k_cache, void* v_cache,
                           int B, int T, int H, int Hq, int Hkv, int d, int C, float rope_theta, int32_t* status,
                           void* workspace, size_t workspace_bytes, s4c_stream_t stream);

/* s4c_qkv_rope_same_tree -- another layer of the same verify pass (Section 3.2: one forward pass over
 * one tree): the tree checks, the rows' cache positions and the rotary table depend on cache_len,
 * parent, n_nodes, T, d and rope_theta alone, so the layers after the first reuse what s4c_qkv_rope
 * left in `workspace` (same B, T, d, C; cache_len unchanged since; the workspace untouched since)
 * and skip that kernel.  Arguments as s4c_qkv_rope.  status [B] or NULL is NOT rewritten: it keeps
 * what it holds (the first call's flags, when the same array is passed) and gets S4C_SEQ_TIMEOUT
 * OR-ed in; sequences the first call flagged are skipped here too. */
s4c_status s4c_qkv_rope_same_tree(const void* x, const void* w_qkv, void* q_out, void* k_cache, void* v_cache, int B,
                                  int T, int H, int Hq, int Hkv, int d, int C, int32_t* status, void* workspace,
                                  size_t workspace_bytes, s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_linear, s4c_rmsnorm, s4c_embed_gather -- the pieces of the drafter's head (Section 3.1, Eq. 3-6)
 * and of a LLaMA-family decoder layer that are not attention:
 *   s4c_linear      out[r, n] = sum_k x1[r, k] w[n, k] + sum_k x2[r, k] w[n, K1 + k]  (+ bias[n])
 *                   Eq. 3, h = Linear(concat[e, f]), is x1 = e, x2 = f: the concatenation is never
 *                   formed.  gate != 0: w holds 2N rows (the gate projection's N rows, then the up
 *                   projection's; bias likewise 2N) and out[r, n] = silu(gate_n) * up_n with
 *                   silu(z) = z / (1 + exp(-z)).  residual [R, N] (or NULL) is added last.
 *                   x1 [R, K1], x2 [R, K2] (NULL when K2 = 0), w [N or 2N, K1 + K2], bias, residual,
 *                   out [R, N]: bf16, device, row-major, 16-byte aligned; K1, K2 multiples of 64,
 *                   N a multiple of 8.  float32 accumulation, one rounding to bf16.  status: one
 *                   int32 (device) or NULL, zeroed and OR-ed with S4C_SEQ_TIMEOUT if a wait inside
 *                   the kernel was given up.  A product with few output tiles shares each tile's
 *                   K range out over several CTAs, whose float32 partial sums pass through
 *                   workspace and are added in a fixed order (the result does not depend on
 *                   timing): workspace must hold s4c_linear_workspace_bytes(R, K1, K2, N, gate)
 *                   bytes (0 for shapes that need none; then NULL is accepted), 256-byte aligned;
 *                   S4C_ERR_WORKSPACE otherwise.  Stream order: the kernels are launched programmatically
 *                   dependent; inputs, bias, residual and outputs are touched only after the kernel
 *                   in front has completed, but tiles of w are requested earlier -- w must not be
 *                   the output of the kernel enqueued directly in front on the same stream (a
 *                   weight written earlier than that, or by a copy, is fine).
 *   s4c_linear_rmsnorm  the ungated s4c_linear followed by norm_out[r, :] = rmsnorm(out[r, :]) with
 *                   norm_weight [N] and eps >= 0 (norm_out [R, N] bf16, 16-byte aligned): the decoder
 *                   layer's "projection + residual, then the next block's normalisation".  Both out
 *                   and norm_out are written; the results equal, bit for bit, s4c_linear followed by
 *                   s4c_rmsnorm on out.  Where the K range is shared out the finishing kernel, which
 *                   holds whole rows, normalises them (no extra launch); otherwise the
 *                   normalisation kernel is launched behind the product.
 *   s4c_rmsnorm     out[r, :] = x[r, :] / sqrt(mean(x[r, :]^2) + eps) * weight   (bf16 in / out,
 *                   float32 arithmetic; H a multiple of 8)
 *   s4c_embed_gather out[r, :] = table[tokens[r], :]  (Eq. 6; bf16 table [V, H]; a token outside
 *                   [0, V) yields zeros)
 * ------------------------------------------------------------------------------------------ */
size_t s4c_linear_workspace_bytes(int R, int K1, int K2, int N, int gate);

s4c_status s4c_linear(const void* x1, const void* x2, const void* w, const void* bias, const void* residual,
                      void* out, int R, int K1, int K2, int N, int gate, int32_t* status, void* workspace,
                      size_t workspace_bytes, s4c_stream_t stream);

s4c_status s4c_linear_rmsnorm(const void* x1, const void* x2, const void* w, const void* bias, const void* residual,
                              void* out, int R, int K1, int K2, int N, const void* norm_weight, float eps,
                              void* norm_out, int32_t* status, void* workspace, size_t workspace_bytes,
                              s4c_stream_t stream);

s4c_status s4c_rmsnorm(const void* x, const void* weight, float eps, int R, int H, void* out, s4c_stream_t stream);

s4c_status s4c_embed_gather(const void* table, const int32_t* tokens, int R, int V, int H, void* out,
                            s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_tree_attention_paged, s4c_kv_compact_paged -- the same two operations (Section 3.2: tree-masked
 * attention of the verification pass; keeping the accepted tokens' K/V) on PAGED caches, the layout
 * serving systems keep their caches in.  The paper does not discuss cache layouts.
 *
 * A cache is a pool of pages [n_pages, Hkv, page_size, d] (page_size a multiple of 64 slots; K and V
 * pools of the same shape); block_table [B, max_blocks] int32 (device) names the page that holds
 * slots i*page_size .. (i+1)*page_size-1 of sequence b.  Every block that holds a slot below
 * cache_len[b] + T must be listed (the tree slots L_b..L_b+T-1 are ordinary slots of the sequence);
 * other entries are never read.  A sequence can hold max_blocks*page_size slots (the capacity C of
 * the contiguous calls).  A listed page outside [0, n_pages) flags the sequence S4C_SEQ_BAD_PAGE (its
 * results are invalid; no access leaves the pool).  Results equal those of the contiguous calls on the
 * cache the block table spells out.  s4c_tree_attention_paged serves S4C_BF16 (S4C_F32:
 * S4C_ERR_UNSUPPORTED); its workspace is sized by s4c_tree_attention_workspace_bytes with
 * C = max_blocks*page_size.  n_pages*Hkv*page_size must stay below 2^31.  All other arguments as in
 * s4c_tree_attention / s4c_kv_compact (k_pages / v_pages of s4c_kv_compact_paged: device arrays of
 * n_layers pool pointers; one block table serves all layers).
 * ------------------------------------------------------------------------------------------ */
s4c_status s4c_tree_attention_paged(const void* q, const void* k_pages, const void* v_pages,
                                    const int32_t* block_table, const int32_t* cache_len, const int32_t* parent,
                                    const int32_t* n_nodes, void* out, int B, int T, int Hq, int Hkv, int d,
                                    int n_pages, int page_size, int max_blocks, int max_cache_len, s4c_dtype dt,
                                    float scale, int32_t* status, void* workspace, size_t workspace_bytes,
                                    s4c_stream_t stream);

s4c_status s4c_kv_compact_paged(void* const* k_pages, void* const* v_pages, int n_layers, const int32_t* block_table,
                                int32_t* cache_len, const int32_t* path, const int32_t* accept_len, int max_depth,
                                const void* feat_in, void* feat_out, int B, int T, int Hkv, int d, int n_pages,
                                int page_size, int max_blocks, int hid, s4c_dtype dt, int32_t* status,
                                s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_tree_build -- the continuous verification tree of Section 3.2 (drawn in Figure 3, left),
 * built on the device from the drafter's distributions, in the layout the three calls above consume.
 *
 * Shape.  The root (node 0) is the last committed token.  Drafts are generated vertically first: a
 * chain of top-1 choices, one per drafting depth (`depth` levels).  Then the tree is extended
 * horizontally, depth by depth: every node at depth l (vertical or horizontal) gets the top-k
 * alternatives at its position until it has branching[l] children -- its first child is the top-1
 * choice, the others the 2nd, 3rd, ... most probable tokens of the same distribution.  Growth stops
 * at T nodes.  Nodes are numbered breadth-first, so parent[i] < i, siblings are contiguous and in
 * rank order.  The shape depends on (branching, T) only and is the same for every sequence.
 * Tokens.  Child j (j = 1..k) of node n carries the j-th most probable token of draft_probs[b,n,:],
 * ties going to the lower token index.
 *
 *   draft_probs [B,T,V] f32   row n: the drafter's distribution for the token after node n (the array
 *                             s4c_tree_accept takes); rows of nodes without children are not read.
 *                             Entries must not be NaN.
 *   branching   [depth] int32, HOST memory: children per node at depths 0..depth-1, each 1..16 and <= V
 *   root_token  [B] int32     the last committed token of each sequence
 *   cache_len   [B] int32 or NULL
 *   tokens, parent, position [B,T] int32  out: position[b,i] = cache_len[b] + depth of node i (the
 *                             position id of the node's K/V slot content; just the depth if cache_len is
 *                             NULL); entries of unused nodes (i >= n_nodes[b]): parent -1, token 0, position 0
 *   n_nodes     [B] int32     out: nodes in use, min(T, size of the full tree)
 *   workspace   at least s4c_tree_build_workspace_bytes(B, T, V, max over branching) bytes, 256-byte
 *               aligned, scratch (per-segment candidates of the top-k selection)
 * Asynchronous on `stream`; the host never reads the tree: tokens / parent / n_nodes go straight to
 * s4c_tree_attention, s4c_tree_accept and s4c_kv_compact on the same stream.
 * ------------------------------------------------------------------------------------------ */
size_t s4c_tree_build_workspace_bytes(int B, int T, int V, int max_branch);

s4c_status s4c_tree_build(const float* draft_probs, const int32_t* branching, int depth, const int32_t* root_token,
                          const int32_t* cache_len, int B, int T, int V, int32_t* tokens, int32_t* parent,
                          int32_t* position, int32_t* n_nodes, void* workspace, size_t workspace_bytes,
                          s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_launch_floor -- a measurement aid; the paper has no counterpart.
 *
 * Enqueues an EMPTY kernel with the launch shape of an attention launch: `ctas` blocks of `threads`
 * threads in clusters of `cluster`, `smem_bytes` of dynamic shared memory, `tmem_cols` tensor-memory
 * columns allocated and freed (0, 32, ..., 512), `cluster_syncs` cluster barriers, the programmatic
 * dependent-launch attribute if `dependent_launch` != 0, and one dependent read of `word` (device, may
 * be NULL) after the wait for the previous launch.  Timed in a CUDA graph of n_layers such launches it
 * gives the floor under one per-layer launch of a verify step (bench.py --workload launch-floor).
 * `sink` (device, may be NULL) is never written in practice.  Shapes whose co-resident blocks would
 * need more than 512 tensor-memory columns per SM are refused with S4C_ERR_UNSUPPORTED.
 * ------------------------------------------------------------------------------------------ */
s4c_status s4c_launch_floor(int ctas, int cluster, int threads, int smem_bytes, int tmem_cols, int cluster_syncs,
                            int dependent_launch, const int32_t* word, int32_t* sink, s4c_stream_t stream);

/* ------------------------------------------------------------------------------------------
 * s4c_selftest_attention_timeout -- checks the failure path of s4c_tree_attention; the paper has no
 * counterpart.
 *
 * Every wait inside the bf16 attention kernel is bounded: when one runs out of time the CTA stops
 * issuing copies and products, parks, merges and stores nothing, still meets its cluster's barriers,
 * sees its own copies and products complete, frees its tensor memory and returns; status[b] gets
 * S4C_SEQ_TIMEOUT and the context stays usable.  This call makes that happen without any fault: it is
 * the launch of s4c_tree_attention (bf16, scale 1/sqrt(d), all trees of T nodes) in which no CTA ever
 * requests cache tile `withhold_tile` (0-based, 64 slots each) of its own range and a wait gives up
 * after `limit_us` microseconds (1..100000).  Afterwards status[b] holds S4C_SEQ_TIMEOUT for every
 * sequence whose CTAs own such a tile, `out` is untouched for them, and the next call on the stream
 * works normally.  Shapes that would merge through a workspace are refused (S4C_ERR_UNSUPPORTED).
 * ------------------------------------------------------------------------------------------ */
s4c_status s4c_selftest_attention_timeout(const void* q, const void* k_cache, const void* v_cache,
                                          const int32_t* cache_len, const int32_t* parent, void* out, int B, int T,
                                          int Hq, int Hkv, int d, int C, int max_cache_len, int withhold_tile,
                                          int limit_us, int32_t* status, s4c_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* S4C_H_ */
