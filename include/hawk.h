/*
 * hawk.h - C ABI of the B200 (sm_100a) verify step of speculative decoding for autoregressive
 * image generation (Hawk).
 *
 * The verify step takes a block of K drafted image tokens per sequence and decides how many of
 * them the target model accepts.  It has three parts, one entry point each:
 *   hawk_verify_attn  block-causal attention of the K draft queries over the cached context, for
 *                     the conditional and the unconditional guidance stream;
 *   hawk_head_proj    projection of the K hidden states onto the image-token codebook;
 *   hawk_cfg_accept   guidance combine, temperature, top-k, softmax and speculative rejection
 *                     sampling, returning the accepted length and the correction token;
 *   hawk_tree_accept  the same for a candidate tree with several candidates per depth.
 *   hawk_spec_cache_*, hawk_pool_*  the cache of vertical predictions and the sampling pool that feed it;
 *   hawk_head_proj_cfg, hawk_*_accept_guided  the head with the guidance combine in its epilogue.
 *
 * Conventions common to all entry points
 *   - Every pointer is a DEVICE pointer owned by the caller unless the comment says "host".  The
 *     library allocates no device memory, frees nothing, never synchronises and keeps no pointer
 *     after the call returns.  All work is queued on `stream`.  (Two calls keep state of their own and
 *     say so in their comments: hawk_verify_step_host owns one stream and two events per device,
 *     hawk_cfg_accept_noalloc a fixed array in the library's device image.)
 *   - Tensors are dense, row-major in the index order written in brackets, base address aligned
 *     to 16 bytes.  bf16 is the 16 high bits of an IEEE fp32.
 *   - The return value is the only error channel.  On any error nothing is launched and the
 *     outputs are untouched.  Conditions that only the device can see (a draft id out of range,
 *     a NaN logit, a wait that ran out) are OR-ed into *dev_status (HAWK_DEV_* bits) when that
 *     pointer is not NULL; the caller clears the word.  No kernel traps or asserts.
 *   - B sequences, S = 2B guidance streams: stream b is the conditional one of sequence b,
 *     stream B+b its unconditional one.  K drafts per sequence.
 */
#ifndef HAWK_H
#define HAWK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st *hawk_stream_t; /* a cudaStream_t / CUstream; 0 = the default stream */

typedef enum {
    HAWK_OK = 0,
    HAWK_ERR_NULL = 1,        /* a required pointer is NULL                                     */
    HAWK_ERR_SHAPE = 2,       /* a size is negative or sizes contradict each other              */
    HAWK_ERR_ALIGN = 3,       /* a tensor base is not 16-byte aligned                           */
    HAWK_ERR_UNSUPPORTED = 4, /* a value outside what the kernels are built for (see each call) */
    HAWK_ERR_WORKSPACE = 5,   /* workspace missing or smaller than *_workspace_bytes says       */
    HAWK_ERR_PARAM = 6,       /* a scalar parameter is not a usable number                      */
    HAWK_ERR_CUDA = 7         /* the CUDA runtime or driver refused a call (launch, tensor map) */
} hawk_status;

/* bits of *dev_status */
#define HAWK_DEV_TIMEOUT 1    /* a bounded wait inside a kernel ran out; outputs are not valid  */
#define HAWK_DEV_BAD_DRAFT 2  /* a draft id lay outside [v_begin, v_end) and was clamped into it */
#define HAWK_DEV_NONFINITE 4  /* a NaN or +inf logit was treated as -inf                        */
#define HAWK_DEV_BAD_PREFIX 8 /* a prefix length lay outside [0, L_cap - K] and was clamped     */
#define HAWK_DEV_BAD_TREE 16  /* a child range or draft-row index of the tree was out of range    */
#define HAWK_DEV_BOUNDS 32    /* libraries built with -DHAWK_DEBUG only: an index lay outside its array, the access was skipped */

const char *hawk_status_string(hawk_status status);
int hawk_version(void); /* major*10000 + minor*100 + patch */

/* ------------------------------------------------------------------------------------------------
 * hawk_verify_attn - attention of the K draft queries against the cached prefix.
 *
 * Operation (Sec. 3, "Speculative Sampling": one forward pass of the target model verifies the
 * drafted tokens in parallel; the KV cache is the one App. C mentions).  For stream s, query head
 * h and draft position i, with n = prefix_len[s] + i + 1 visible keys and kv head g = h / (H/H_kv):
 *     e_j = sm_scale * <q[s,i,h,:], k_cache[s,g,j,:]>,  j < n
 *     out[s,i,h*D:(h+1)*D] = sum_j softmax(e)_j * v_cache[s,g,j,:]
 * The block's own K rows must already be stored in the caches at rows prefix_len[s] .. +K-1; rows
 * past that are never used (they may hold anything).  Scores and sums are fp32.
 *
 *   q            bf16 [S][K][H][D]
 *   k_cache      bf16 [S][H_kv][L_cap][D]
 *   v_cache      bf16 [S][H_kv][L_cap][D]
 *   prefix_len   int32 [S], each in [0, L_cap - K]
 *   out          bf16 [S][K][H*D]
 *   max_prefix_len  upper bound of prefix_len[] known on the host (sizes the launch only)
 *   sm_scale     score scale, > 0, normally 1/sqrt(D)
 *   workspace    scratch of at least hawk_verify_attn_workspace_bytes(...) bytes, 16-byte aligned;
 *                may be NULL when that function returns 0.  Contents need no initialisation and
 *                are garbage afterwards.
 * Supported: D in {64, 128}; 1 <= K <= 64; H a multiple of H_kv; S*H_kv*L_cap < 2^31.
 * Errors: NULL, SHAPE (negative sizes, max_prefix_len + K > L_cap), ALIGN, UNSUPPORTED, WORKSPACE,
 * PARAM (sm_scale not a positive finite number), CUDA.  S == 0 returns HAWK_OK without a launch.
 * ---------------------------------------------------------------------------------------------- */
size_t hawk_verify_attn_workspace_bytes(int S, int K, int H, int H_kv, int D, int max_prefix_len);

hawk_status hawk_verify_attn(const void *q, const void *k_cache, const void *v_cache,
                             const int32_t *prefix_len, void *out, int S, int K, int H, int H_kv,
                             int D, int L_cap, int max_prefix_len, float sm_scale, void *workspace,
                             size_t workspace_bytes, int32_t *dev_status, hawk_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * hawk_verify_attn_tree - the same attention for a candidate tree.
 *
 * Operation (Sec. 4.2: all candidates of the tree are verified in one forward pass of the target
 * model): the N tree nodes of a stream are N queries; node i attends to the whole
 * cached prefix and, inside the block, only to the nodes on its own path from the root:
 *     key j <  prefix_len[s]                  visible to every node
 *     key j == prefix_len[s] + m, 0 <= m < N  visible to node i iff bit m of anc_mask[i] is set
 * Node i's own key/value row is cache row prefix_len[s] + i, so anc_mask[i] has bit i set.
 * hawk_verify_attn is the special case anc_mask[i] = 2^(i+1) - 1.
 *
 *   q         bf16 [S][N][H][D]
 *   anc_mask  uint64 [N], device memory, shared by all streams
 *   out       bf16 [S][N][H*D]
 * Everything else, the workspace (hawk_verify_attn_workspace_bytes with K = N) and the errors are
 * those of hawk_verify_attn; 1 <= N <= 64.
 * ---------------------------------------------------------------------------------------------- */
hawk_status hawk_verify_attn_tree(const void *q, const void *k_cache, const void *v_cache,
                                  const int32_t *prefix_len, const uint64_t *anc_mask, void *out, int S,
                                  int N, int H, int H_kv, int D, int L_cap, int max_prefix_len,
                                  float sm_scale, void *workspace, size_t workspace_bytes,
                                  int32_t *dev_status, hawk_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * hawk_head_proj - output head: hidden states onto the token codebook.
 *
 * Operation (Sec. 3: the decoding head after the final hidden layer maps a hidden state to
 * logits over the codebook of image tokens):
 *     logits[m][v] = sum_c x[m][c] * w[v][c]      for v_begin <= v < v_end
 * bf16 operands, fp32 accumulation on the tensor cores, fp32 result.  Columns outside
 * [v_begin, v_end) are not written.
 *
 *   x       bf16 [M][hidden]   one row per (stream, draft position): M = 2*B*K
 *   w       bf16 [V][hidden]   one row per token id
 *   logits  fp32 [M][V]
 * Supported: hidden a multiple of 64 (and >= 64).
 * Errors: NULL, SHAPE (negative sizes, range outside [0, V]), ALIGN, UNSUPPORTED, CUDA.
 * M == 0 or an empty range returns HAWK_OK without a launch.
 * ---------------------------------------------------------------------------------------------- */
hawk_status hawk_head_proj(const void *x, const void *w, float *logits, int M, int hidden, int V,
                           int v_begin, int v_end, int32_t *dev_status, hawk_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * hawk_cfg_accept - target distribution and speculative rejection sampling of a draft chain.
 *
 * Operation, per sequence b and draft position i = 0, 1, ... (Sec. 3: accept draft x with
 * probability min(1, p(x)/q(x)), otherwise resample from norm(max(0, p - q)); Sec. 4.2, Eq.
 * "recur": a pass moves one position deeper, the first rejection ends the chain; generation
 * settings of Sec. 5: guidance scale, temperature, top-k):
 *   1. l[v] = lu[v] + cfg_scale*(lc[v] - lu[v]) over the valid ids, lc/lu the conditional and
 *      unconditional logit rows; -inf in either gives -inf.  Evaluated in fp32 as subtract, fused
 *      multiply-add, then divide by temperature.
 *   2. With 0 < top_k < number of finite l: keep every l >= the top_k-th largest (ties at the
 *      threshold are all kept); the rest become -inf.
 *   3. p = softmax(l); ids outside [v_begin, v_end) have p = 0.
 *   4. x = draft[b][i]; accept iff u_accept[b][i] * q[b][i][x] < p[x]; on a pass go to i+1.
 *   5. On the first rejection: r = max(0, p - q[b][i][:]); if r has no mass, r = p;
 *      out_token[b] = the smallest id whose running sum of r (ascending id) exceeds
 *      u_resample[b][i] * sum(r); accept_len[b] = i.
 *   6. All K accepted: accept_len[b] = K; out_token[b] = -1, or with has_bonus_row the same draw
 *      from p of row K with u_resample[b][K].
 * The paper's "accept length" counts the correction token: it equals accept_len + 1.
 *
 *   logits      fp32 [2B][K + has_bonus_row][V]
 *   q_probs     fp32 [B][K][V]   draft probabilities, used as given
 *   draft       int32 [B][K]
 *   u_accept    fp32 [B][K]      uniforms in [0,1)
 *   u_resample  fp32 [B][K+1]    uniforms in [0,1)
 *   accept_len  int32 [B]  (out)
 *   out_token   int32 [B]  (out)
 *   p_debug     optional fp32 [B][K + has_bonus_row][V]: receives p over the valid ids; NULL in
 *               normal use (p never leaves the chip)
 *   workspace   at least hawk_cfg_accept_workspace_bytes(...) bytes, 16-byte aligned; needs no
 *               initialisation
 * Every row is judged by a thread block of its own.  A call with more rows than the GPU runs at once
 * lets the blocks of later positions look at the verdicts their sequence already has, and a row
 * behind a rejection (step 5 never reads it) does no work; the results do not depend on it, and with
 * p_debug every row is computed.
 * Supported: 1 <= K <= 16; 1 <= v_end - v_begin <= 32768 (one row is held in one
 * thread block's registers); temperature > 0.
 * Errors: NULL, SHAPE, ALIGN, UNSUPPORTED, WORKSPACE, PARAM (cfg_scale or temperature not finite,
 * temperature <= 0), CUDA.  B == 0 returns HAWK_OK without a launch.
 * ---------------------------------------------------------------------------------------------- */
size_t hawk_cfg_accept_workspace_bytes(int B, int K, int V);

hawk_status hawk_cfg_accept(const float *logits, const float *q_probs, const int32_t *draft,
                            const float *u_accept, const float *u_resample, int B, int K, int V,
                            int v_begin, int v_end, float cfg_scale, float temperature, int top_k,
                            int has_bonus_row, int32_t *accept_len, int32_t *out_token,
                            float *p_debug, void *workspace, size_t workspace_bytes,
                            int32_t *dev_status, hawk_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * hawk_tree_accept - verification of a candidate tree: several candidates per depth, each with its
 * own draft distribution.
 *
 * Operation (Sec. 4.2, "Sampling and Verification", Eq. "recur"; distribution preservation: App. A).
 * The tree is shared by the batch: node 0 is the root (the last committed token), the children of
 * node n are the nodes child_begin[n] .. child_begin[n+1]-1 (all ids > n), verified in that order.
 * Per sequence b, starting at the root with depth 0:
 *   1. p = target distribution of the node's logit rows (steps 1-3 of hawk_cfg_accept).
 *   2. For each child c in order, with x = node_token[b][c], q = q_probs[b][node_q[c]]:
 *      accept iff u_accept[b][c] * q[x] < p[x]; on a pass move to node c, one level deeper, step 1.
 *      On a rejection p <- norm(max(0, p - q)); a residual without mass leaves p as it is.
 *   3. Every child rejected, or the node has none: out_token[b] = inverse-CDF draw (ascending id)
 *      from p as refined so far with u_resample[b][node]; accept_len[b] = depth; stop.
 * q may come from a different draft head for every candidate (horizontal or vertical), which is what
 * shrinks the probability that all candidates of a level are rejected.
 * A chain of K drafts is the tree with N = K + 1 nodes and child_begin[n] = n + 1.
 *
 *   logits      fp32 [2B][N][V]  row n: logits for the token that follows node n (b conditional, B+b not)
 *   q_probs     fp32 [B][NQ][V]  draft probabilities, used as given
 *   node_token  int32 [B][N]     candidate token of node n (entry 0 unused)
 *   node_q      int32 [N]        row of q_probs the token of node n was drawn from (entry 0 unused)
 *   child_begin int32 [N+1]      device memory, like everything else
 *   u_accept    fp32 [B][N]      uniforms in [0,1), one per candidate node (entry 0 unused)
 *   u_resample  fp32 [B][N]      uniforms in [0,1), entry n used if the walk stops at node n
 *   accept_len  int32 [B] (out)  number of accepted candidates
 *   out_token   int32 [B] (out)  correction token; -1 if the refined target has no mass at all
 *   path        optional int32 [B][max_depth] (out): accepted nodes in order, -1 beyond accept_len
 *   workspace   at least hawk_tree_accept_workspace_bytes(B, N) bytes, 16-byte aligned, no initialisation
 * Every node is judged by its own thread block, so the cost is at most B*N rows; in a call with more
 * rows than the GPU runs at once, a node whose parent is already known not to have picked it does no
 * work (the walk cannot reach it; the results do not depend on this).  Supported: 1 <= N <= 65536; at most 16 children per node; valid ids as hawk_cfg_accept.
 * A child range that breaks these rules is clamped and flagged HAWK_DEV_BAD_TREE; the walk always ends.
 * Errors: NULL, SHAPE, ALIGN, UNSUPPORTED, WORKSPACE, PARAM, CUDA.  B == 0 returns HAWK_OK.
 * ---------------------------------------------------------------------------------------------- */
size_t hawk_tree_accept_workspace_bytes(int B, int N);

hawk_status hawk_tree_accept(const float *logits, const float *q_probs, const int32_t *node_token,
                             const int32_t *node_q, const int32_t *child_begin, const float *u_accept,
                             const float *u_resample, int B, int N, int NQ, int V, int v_begin, int v_end,
                             float cfg_scale, float temperature, int top_k, int max_depth,
                             int32_t *accept_len, int32_t *out_token, int32_t *path, void *workspace,
                             size_t workspace_bytes, int32_t *dev_status, hawk_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * Guidance fused into the output head (generation settings of Sec. 5: guidance scale and temperature
 * applied to the target's logits before top-k and sampling).  The paper does not separate these
 * steps; the three calls below are the two-call form of hawk_head_proj + hawk_cfg_accept /
 * hawk_tree_accept in which the conditional and the unconditional logit rows never reach memory.
 *
 * hawk_head_proj_cfg: guided[b*rows + i][v] = (lu + cfg_scale * (lc - lu)) / temperature, with
 *     lc = sum_c x[b*rows + i][c] * w[v][c],   lu = sum_c x[(B + b)*rows + i][c] * w[v][c]
 * for v_begin <= v < v_end: the accumulators of hawk_head_proj combined in fp32 by subtract, fused
 * multiply-add, divide (step 1 of hawk_cfg_accept, on the same numbers), so the two-call form decides
 * exactly as the three-call form does.  (Where a call has few tiles and a long hidden dimension, both
 * hawk_head_proj and this call sum each logit as two halves of the hidden dimension, in the same way.)
 *   x       bf16 [2B][rows][hidden]   conditional streams first, as everywhere
 *   w       bf16 [V][hidden]
 *   guided  fp32 [B][rows][V]         columns outside [v_begin, v_end) are not written
 * Supported: hidden a multiple of 64.  Errors as hawk_head_proj, plus PARAM (temperature <= 0, NaN, inf).
 *
 * hawk_cfg_accept_guided / hawk_tree_accept_guided: hawk_cfg_accept / hawk_tree_accept from step 2 on,
 * reading `guided` fp32 [B][K(+1)][V] / [B][N][V] instead of the two logit rows (no guidance scale,
 * no temperature: both are already applied).  NaN or +inf in `guided` is treated as -inf and flagged
 * HAWK_DEV_NONFINITE.  All other arguments, limits, workspaces and errors as the calls they mirror.
 * ---------------------------------------------------------------------------------------------- */
hawk_status hawk_head_proj_cfg(const void *x, const void *w, float *guided, int B, int rows, int hidden, int V,
                               int v_begin, int v_end, float cfg_scale, float temperature, int32_t *dev_status,
                               hawk_stream_t stream);

hawk_status hawk_cfg_accept_guided(const float *guided, const float *q_probs, const int32_t *draft,
                                   const float *u_accept, const float *u_resample, int B, int K, int V, int v_begin,
                                   int v_end, int top_k, int has_bonus_row, int32_t *accept_len, int32_t *out_token,
                                   float *p_debug, void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                   hawk_stream_t stream);

hawk_status hawk_tree_accept_guided(const float *guided, const float *q_probs, const int32_t *node_token,
                                    const int32_t *node_q, const int32_t *child_begin, const float *u_accept,
                                    const float *u_resample, int B, int N, int NQ, int V, int v_begin, int v_end,
                                    int top_k, int max_depth, int32_t *accept_len, int32_t *out_token, int32_t *path,
                                    void *workspace, size_t workspace_bytes, int32_t *dev_status,
                                    hawk_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * Speculation cache and spatial sampling pool (Sec. 4.2, "Dual Direction Drafting Heads" and "Spatial
 * Sampling Pool", Eqs. 1-5): the step that hands hawk_tree_accept its draft distributions and tokens.
 *
 * Eq. 1: the vertical draft head of depth d (1 <= d <= VSD), run at raster position T of an image IW
 * tokens wide, predicts the token at T + IW * d.  Eq. 2: those predictions wait in a cache of
 * IW * VSD * (VSD + 1) / 2 rows per sequence until decoding reaches their target.  Eqs. 3-5: the pool
 * of speculation point T + n is the horizontal head's distribution for T + n followed, for
 * dv = 1 .. VSD, by the cached depth-dv prediction made at T + n - IW * dv.
 *
 * Device layout, owned by the caller, B sequences:
 *   cache_rows  fp32  [B][slots][V]   slots = hawk_spec_cache_slots(IW, VSD)
 *   cache_tags  int32 [B][slots]      raster position that wrote the slot, -1 = never written
 * hawk_spec_cache_slot gives the slot of the depth-d prediction made at `position`: predictions of one
 * image column and depth that are alive at the same time come from d consecutive rows, so the row
 * modulo d tells them apart.  Positions of a sequence must not decrease between calls (a new image
 * starts with hawk_spec_cache_clear).  A lookup whose slot carries another position finds nothing: no
 * forward pass started there (the position was accepted inside a step) or it lies above the image.
 *
 * hawk_spec_cache_slots    slots per sequence (Eq. 2); 0 if IW < 1 or VSD < 1.  Host only.
 * hawk_spec_cache_slot     slot index as above, -1 for arguments out of range.  Host only.
 * hawk_spec_cache_clear    marks every slot of B sequences unwritten.
 * hawk_spec_cache_put      stores q_vert fp32 [B][VSD][V] (row d-1 = depth d) made at position[b]
 *                          (int32 [B], device; a negative position stores nothing for that sequence).
 * hawk_pool_build          q_horiz fp32 [B][K][V] (row n-1 = the horizontal distribution for T + n),
 *                          position int32 [B] (T of every sequence) ->
 *                          pool_q fp32 [B][K*(1+VSD)][V], row (n-1)*(1+VSD) + j: j = 0 horizontal,
 *                          j = dv >= 1 the cached vertical prediction, or a copy of the horizontal row
 *                          where none is cached; pool_source int32 [B][K*(1+VSD)] (may be NULL): 0, dv,
 *                          or -dv for the stand-in.  pool_q is laid out as hawk_tree_accept's q_probs
 *                          with NQ = K*(1+VSD).
 * hawk_pool_sample         draws one token per pool row by inverse CDF in ascending id over
 *                          [v_begin, v_end) with u fp32 [B][NQ] in [0,1) (negative weights count as
 *                          zero; a row without mass gives -1), then fills
 *                          node_token int32 [B][N]: node_token[b][i] = draw of row node_q[i]
 *                          (node_q int32 [N], device, as in hawk_tree_accept; the root, i = 0, gets 0).
 *                          The candidate tree is the Cartesian product of the per-position draws, so
 *                          all nodes that stand for one pool row carry the same token.  A node_q entry
 *                          outside [0, NQ) is clamped and flagged HAWK_DEV_BAD_TREE in *dev_status.
 *                          workspace: hawk_pool_sample_workspace_bytes(B, NQ) bytes, 16-byte aligned.
 * All pointers are device pointers unless stated; rows are copied with 16-byte accesses when V % 4 == 0
 * and the buffers are 16-byte aligned, element by element otherwise.  Limits: VSD <= 8; the valid id
 * range of hawk_pool_sample at most 32768 wide.  Launches are asynchronous on `stream`.
 * Errors: NULL, SHAPE, ALIGN, UNSUPPORTED, WORKSPACE, CUDA.  B == 0 (or K == 0) returns HAWK_OK.
 * ---------------------------------------------------------------------------------------------- */
int hawk_spec_cache_slots(int IW, int VSD);

int hawk_spec_cache_slot(int IW, int VSD, int position, int depth);

hawk_status hawk_spec_cache_clear(int32_t *cache_tags, int B, int IW, int VSD, hawk_stream_t stream);

hawk_status hawk_spec_cache_put(const float *q_vert, const int32_t *position, float *cache_rows,
                                int32_t *cache_tags, int B, int IW, int VSD, int V, hawk_stream_t stream);

hawk_status hawk_pool_build(const float *q_horiz, const float *cache_rows, const int32_t *cache_tags,
                            const int32_t *position, float *pool_q, int32_t *pool_source, int B, int K, int IW,
                            int VSD, int V, hawk_stream_t stream);

size_t hawk_pool_sample_workspace_bytes(int B, int NQ);

hawk_status hawk_pool_sample(const float *pool_q, const float *u, const int32_t *node_q, int32_t *node_token,
                             int B, int NQ, int N, int V, int v_begin, int v_end, void *workspace,
                             size_t workspace_bytes, int32_t *dev_status, hawk_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * hawk_cfg_accept_noalloc - hawk_cfg_accept without a caller-provided workspace.
 *
 * The paper has no counterpart of this call; it exists for the way the library gets embedded.
 * Some callers cannot obtain device memory at the moment they need a verdict: a decode loop running
 * inside a serving engine whose memory manager took the whole device at start-up (a fresh
 * allocation there fails, or stalls every stream while the driver serves it), or a plug-in that is
 * handed its input and output buffers by a host application and owns nothing else.  For them the
 * per-row verdicts go to a fixed 64 KiB array that is part of the library's device image; every GPU
 * that loads the library carries that array until the process exits.
 *
 * Same operation, arguments and results as hawk_cfg_accept, minus p_debug, workspace and
 * workspace_bytes.  Limit: B * (K + 1) <= hawk_cfg_accept_noalloc_max_rows() (16384); a larger step
 * returns HAWK_ERR_WORKSPACE and launches nothing.  The call allocates and frees nothing.
 *
 * The first call on each device looks up the array's device address (one runtime query, made with
 * that device current); make that first call outside any stream capture.
 * All calls on a device share the one array, and it keeps the previous call's contents.  Nothing in
 * it has to start at zero (each row's slot is rewritten before it is read), but two calls whose
 * kernels overlap on the GPU - different streams without an ordering between them - race on it:
 * order such calls, or give the concurrent ones their own workspace through hawk_cfg_accept.
 * ---------------------------------------------------------------------------------------------- */
size_t hawk_cfg_accept_noalloc_max_rows(void);

hawk_status hawk_cfg_accept_noalloc(const float *logits, const float *q_probs, const int32_t *draft,
                                    const float *u_accept, const float *u_resample, int B, int K, int V,
                                    int v_begin, int v_end, float cfg_scale, float temperature,
                                    int top_k, int has_bonus_row, int32_t *accept_len,
                                    int32_t *out_token, int32_t *dev_status, hawk_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * hawk_verify_step_host - one whole verify step with the per-step inputs in HOST memory.
 *
 * Runs, on `stream`: host->device copies of the step's inputs into the caller's device staging,
 * hawk_verify_attn, hawk_head_proj, hawk_cfg_accept (contracts above, no bonus row), and
 * device->host copies of accept_len and out_token.  The attention output and the head input are
 * separate tensors: the layers between them (output projection, MLP, norm) are not part of this
 * library, so x is an input of the step like q.  The inputs that only the accept stage reads are
 * copied on a second stream that the library owns (created by the first call on a device: make that
 * call outside stream capture), forked from and joined back into `stream` by events, so they travel
 * while attention and the head projection run.  The call returns once everything is queued; the
 * results are valid after the stream has been synchronised.  Use pinned host memory for the copies
 * to be asynchronous.  The KV cache, the head weight and the prefix lengths are resident device
 * state; all d_* staging and workspaces are device memory owned by the caller.
 * State kept by this call: the first call on a device creates one non-blocking stream and two events
 * for that device and keeps them until the process exits (no device memory).  Every call on the device
 * uses them, so the queuing part of a call runs under a per-device mutex: calls from several host
 * threads are queued one after the other, each correctly ordered against its own `stream`, and the
 * late copies of steps that are in flight together share the one side stream.
 * Errors: the argument checks of all three stage calls run before anything is queued, on the staging
 * pointers and sizes the stages will be given, so a call refused for its arguments (any code but
 * HAWK_ERR_CUDA) has queued no copy and no kernel.  HAWK_ERR_CUDA means the runtime refused a copy,
 * an event or a launch after the call had started to queue work.
 * ---------------------------------------------------------------------------------------------- */
typedef struct {
    /* sizes and sampling parameters */
    int B, K, H, H_kv, D, L_cap, max_prefix_len, V, v_begin, v_end, top_k;
    float sm_scale, cfg_scale, temperature;
    /* per-step inputs, host */
    const void *h_q;            /* bf16 [2B][K][H][D]      */
    const void *h_x;            /* bf16 [2B*K][H*D]        */
    const float *h_q_probs;     /* fp32 [B][K][V]          */
    const int32_t *h_draft;     /* [B][K]                  */
    const float *h_u_accept;    /* [B][K]                  */
    const float *h_u_resample;  /* [B][K+1]                */
    /* per-step results, host */
    int32_t *h_accept_len;      /* [B] */
    int32_t *h_out_token;       /* [B] */
    /* resident device state */
    const void *d_k_cache, *d_v_cache;   /* bf16 [2B][H_kv][L_cap][D] */
    const int32_t *d_prefix_len;         /* [2B] */
    const void *d_w;                     /* bf16 [V][H*D] */
    /* device staging for the inputs, intermediates and results (same shapes as above) */
    void *d_q, *d_x;
    float *d_q_probs;
    int32_t *d_draft;
    float *d_u_accept, *d_u_resample;
    void *d_attn_out;           /* bf16 [2B][K][H*D] */
    float *d_logits;            /* fp32 [2B*K][V]    */
    int32_t *d_accept_len, *d_out_token;
    void *d_attn_workspace;
    size_t attn_workspace_bytes;
    void *d_accept_workspace;
    size_t accept_workspace_bytes;
    int32_t *d_status;          /* optional */
} hawk_step_host_args;

hawk_status hawk_verify_step_host(const hawk_step_host_args *args, hawk_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* HAWK_H */
