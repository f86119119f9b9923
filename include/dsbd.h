/*
 * dsbd.h -- C ABI of the B200 (sm_100a) hot path of dynamic-width speculative beam decoding:
 * the per-step parallel verification of a forest of draft trees, one tree per input beam.
 *
 * Conventions for every entry point
 *   - Pointers are DEVICE pointers unless a comment says "host".  The structs themselves
 *     (dsbd_forest_t, ...) live in host memory and are read during the call only.
 *   - The library never allocates, frees or synchronises: the caller owns every buffer,
 *     passes a workspace of at least the size the matching *_workspace() query returns, and
 *     every call is asynchronous on `stream`.  Workspaces may be reused by the next call on
 *     the same stream; their contents are undefined afterwards.
 *   - Return value: DSBD_OK, or a negative DSBD_ERR_* found by host-side checks (nothing was
 *     launched).  Problems only the device can see (a draft token outside the vocabulary, a
 *     distribution without mass, a bounded wait that ran out) are written to `*status`
 *     (device int32, must be zero before the call, first error wins) and, per request, to
 *     `req_error`; kernels never trap.
 *   - There is no CPU fallback and no global state (dsbd_node_stats_static, which says so, is
 *     the one exception); the same inputs and (seed, step) give the same outputs whatever the
 *     launch shape.
 */
#ifndef DSBD_H
#define DSBD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st *dsbd_stream_t;   /* a cudaStream_t */

enum {
    DSBD_OK = 0,
    DSBD_ERR_INVALID_ARG = -1,
    DSBD_ERR_UNSUPPORTED = -2,
    DSBD_ERR_WORKSPACE_TOO_SMALL = -3,
    DSBD_ERR_CUDA = -4
};

/* device-side codes written to *status / req_error */
enum {
    DSBD_DEV_BAD_TOKEN = 1,      /* draft token outside [0, V)                               */
    DSBD_DEV_EXHAUSTED = 2,      /* a draw from a distribution without mass                  */
    DSBD_DEV_CAPACITY = 3,       /* a range the caller sized is too small: output slots of a
                                    request, cache tokens, page-table entries, free pages    */
    DSBD_DEV_BAD_FOREST = 4,     /* an index that contradicts the forest: parent outside its
                                    tree, beam outside its request, too many live beams      */
    DSBD_DEV_TIMEOUT = 5,        /* a bounded wait gave up                                   */
    DSBD_DEV_BAD_PARAM = 6       /* a per-request width (W_min_r, W_max_r, W_nom_r) below 1, or
                                    W_max_r below W_min_r                                    */
};

/* limits of this build */
#define DSBD_MAX_TREE_NODES 64   /* nodes per draft tree (forest attention)                  */
#define DSBD_MAX_TREE_NODES_TC 128 /* the same on the tensor-core path (bf16, d = 128, up to
                                      1024 query rows per tree and KV head)                  */
#define DSBD_MAX_LIVE 64         /* beams of a request / live drafts of a layer (verify)     */

/* The draft forest of one decode step (Section "Draft and Verification Scheme", Overview):
 * B trees, one per input beam, grouped by request; tree b owns the nodes
 * [beam_node_off[b], beam_node_off[b+1]), its root (the input beam itself) first, and every
 * other node n has beam_node_off[b] <= parent[n] < n.  Depth d nodes are the drafts of
 * draft layer d; max_depth is gamma, the number of draft layers. */
typedef struct {
    int32_t R, B, N, max_depth;
    const int32_t *req_beam_off;   /* [R+1] trees of request r                               */
    const int32_t *beam_node_off;  /* [B+1]                                                  */
    const int32_t *parent;         /* [N]   global node id, -1 for a root                    */
    const int32_t *token;          /* [N]   draft token id (ignored for roots)               */
    const int32_t *draft_rank;     /* [N] or NULL: position of the node in the order in which
                                      the small model drew the drafts of its layer; the accept
                                      loop walks a layer by (draft_rank, node id).  The drafts
                                      must be tested in an order that does not depend on their
                                      values, so a forest whose node numbering is not the draw
                                      order has to pass it.  NULL = ascending node id.       */
    /* host-side facts about the arrays above; they size launches and are trusted */
    int32_t max_tree_nodes;        /* max_b nodes of tree b (an upper bound will do), <=
                                      DSBD_MAX_TREE_NODES(_TC) for dsbd_forest_attention     */
    int32_t max_req_beams;         /* max_r trees of request r, <= DSBD_MAX_LIVE             */
    int32_t max_layer_nodes;       /* max over (request, depth >= 1) of the nodes at that
                                      depth, <= DSBD_MAX_LIVE                                */
} dsbd_forest_t;

enum { DSBD_DTYPE_BF16 = 0, DSBD_DTYPE_F32 = 1 };

/* Shapes of the forest attention (Section "Forest-based Parallel Decoding").
 * Layouts, all contiguous:  q, out [N, Hq, d];  k_new, v_new [N, Hkv, d] (keys/values of the
 * forest nodes themselves);  k_prefix, v_prefix: the KV cache of each input beam packed
 * beam after beam, beam b as [Hkv, L_b, d] starting at element prefix_off[b]*Hkv*d, where
 * L_b = prefix_off[b+1]-prefix_off[b] tokens (the cache excludes the root token).  Query
 * head h uses KV head h / (Hq/Hkv).  All tensors share `dtype`; accumulation is fp32. */
typedef struct {
    int32_t Hq, Hkv, d;            /* d in {64, 128}; Hq % Hkv == 0                          */
    int32_t dtype;                 /* DSBD_DTYPE_*                                           */
    float scale;                   /* softmax scale, usually 1/sqrt(d)                       */
    int64_t total_prefix;          /* host copy of prefix_off[B]                             */
    int64_t max_prefix;            /* host: max_b L_b                                        */
} dsbd_attn_desc_t;

/* Forest-masked attention: for every node n and query head h,
 *   out[n,h] = sum_j softmax_j(scale * q[n,h] . K_j) V_j
 * over j in (KV prefix of n's beam) U (ancestors of n in its own tree) U {n}; nothing of any
 * other tree or beam is visible ("topology-aware mask" extended from one tree to a forest,
 * with a separate KV cache per input beam).  prefix_off: [B+1] int64, tokens.
 * Errors: INVALID_ARG (null pointer, Hq % Hkv), UNSUPPORTED (d, dtype, tree larger than
 * DSBD_MAX_TREE_NODES, pointers not 16-byte aligned), WORKSPACE_TOO_SMALL. */
int dsbd_forest_attention(const dsbd_forest_t *forest, const dsbd_attn_desc_t *desc,
                          const void *q, const void *k_new, const void *v_new,
                          const void *k_prefix, const void *v_prefix, const int64_t *prefix_off,
                          void *out, void *workspace, size_t workspace_bytes, int32_t *status,
                          dsbd_stream_t stream);

size_t dsbd_forest_attention_workspace(const dsbd_forest_t *forest, const dsbd_attn_desc_t *desc);

/* How many kernels dsbd_forest_attention launches for this shape (1: the attention kernel; 2:
 * plus a work plan that orders ragged units; 3: plus the merge of split units), 0 for invalid
 * arguments.  For launch accounting; host-only. */
int dsbd_forest_attention_launches(const dsbd_forest_t *forest, const dsbd_attn_desc_t *desc);

/* The same attention over PAGED caches.  The paper keeps one key-value cache per input beam and
 * does not say how it is stored; here a cache may be a list of pages of DSBD_PAGE_TOKENS tokens
 * in a pool, so that beams descending from one input beam share its pages and the cache update
 * (dsbd_kv_commit_paged) copies no prefix.  k_pool, v_pool: [n_pages, Hkv, DSBD_PAGE_TOKENS, d];
 * beam b owns the pages page_table[page_off[b] .. page_off[b+1]) in token order, ceil(L_b /
 * DSBD_PAGE_TOKENS) of them, L_b = prefix_off[b+1] - prefix_off[b] (prefix_off only carries the
 * lengths here; desc->total_prefix / max_prefix as before).  Rows of a last page past L_b are
 * never used but must hold finite values.  Supported: bf16, d = 128 (the tensor-core kernel);
 * otherwise UNSUPPORTED.  Workspace: dsbd_forest_attention_paged_workspace. */
enum { DSBD_PAGE_TOKENS = 64 };

typedef struct {
    const int32_t *page_table;     /* device                                                 */
    const int64_t *page_off;       /* device [B+1]                                           */
    int64_t n_pages;               /* host: pages in the pool                                */
    /* dsbd_forest_attention_paged only: the attention of several transformer layers in one call
     * (Section "Forest-based Parallel Decoding": the large model's forward runs the whole forest
     * through every layer, each layer attending over its own key-value cache).  All layers share
     * the forest, the page tables and the work plan; layer l reads its pools at k_pool / v_pool +
     * l * pool_layer_stride, its new keys/values at k_new / v_new + l * new_layer_stride and its
     * queries at q + l * q_layer_stride, and writes out + l * q_layer_stride (strides in
     * elements).  pool_layer_stride must be a multiple of DSBD_PAGE_TOKENS * d and at least one
     * pool, new_layer_stride a multiple of Hkv * d and at least N * Hkv * d, q_layer_stride a
     * multiple of 8 and at least N * Hq * d; otherwise INVALID_ARG.  n_layers 0 or 1: one layer,
     * strides ignored.  (In a model the layers run one after the other, each on the previous
     * layer's output; a caller that has the queries of several layers at hand -- a benchmark, a
     * pipeline stage replaying a step -- gets them in one launch with one plan.) */
    int32_t n_layers;
    int64_t pool_layer_stride, new_layer_stride, q_layer_stride;
} dsbd_kv_pages_t;

int dsbd_forest_attention_paged(const dsbd_forest_t *forest, const dsbd_attn_desc_t *desc,
                                const void *q, const void *k_new, const void *v_new,
                                const void *k_pool, const void *v_pool, const dsbd_kv_pages_t *pages,
                                const int64_t *prefix_off, void *out, void *workspace,
                                size_t workspace_bytes, int32_t *status, dsbd_stream_t stream);

/* Workspace of dsbd_forest_attention_paged for these page tables and layer count (for one layer
 * the same as dsbd_forest_attention_workspace); 0 for arguments the call would refuse. */
size_t dsbd_forest_attention_paged_workspace(const dsbd_forest_t *forest, const dsbd_attn_desc_t *desc,
                                             const dsbd_kv_pages_t *pages);

/* Parameters of the verification (Section "Details", Algorithm 1, and Section
 * "Dynamic-Width Speculative Beam Decoding"). */
typedef struct {
    int32_t V;                     /* vocabulary size                                        */
    float temperature;             /* tau > 0: both models' logits are divided by it before
                                      the per-node softmax                                   */
    float thresh;                  /* threshold t of the width rule                          */
    int32_t W_min, W_max, W_nom;   /* W_L^(l) = min(W_max, max(W_min, W~_L^(l)(t)));  W_nom is
                                      the width of the extra layer sampled when all gamma
                                      layers pass.  W_max = number of drafts gives the
                                      paper's uncapped rule.                                 */
    const int32_t *W_min_r;        /* optional per-request overrides, [R] each, or NULL      */
    const int32_t *W_max_r;
    const int32_t *W_nom_r;
    uint64_t seed;                 /* Philox4x32-10 key                                      */
    uint64_t step;                 /* decode-step counter, mixed into the Philox counter     */
    /* Warping T of the joint distributions p_beam, q_beam (Section "Decodings of LLMs" and the
     * definitions of p_beam, q_beam in Section "Details"; the paper's experiments use top-k 10,
     * top-p 0.8): keep the top_k most probable cells of the joint over (live parents x V) and
     * renormalise, then keep the shortest most-probable prefix whose mass reaches top_p and
     * renormalise; ties go to the lower (parent, token).  top_k = 0: no warping (then top_p must
     * be 0 or >= 1).  This build supports 1 <= top_k <= 64; top_p outside (0,1) is "off". */
    int32_t top_k;
    float top_p;
} dsbd_verify_params_t;

#define DSBD_REQ_STATS 8

/* node_status */
enum { DSBD_NODE_UNREACHED = 0, DSBD_NODE_ACCEPTED = 1, DSBD_NODE_REJECTED = 2,
       DSBD_NODE_CUT = 3, DSBD_NODE_PRUNED = 4 };
/* out_source */
enum { DSBD_SRC_DRAFT = 0, DSBD_SRC_RESIDUAL = 1, DSBD_SRC_FILL = 2, DSBD_SRC_EXTRA = 3 };

/* Results of dsbd_verify_step.  Request r writes its output beams to the slots
 * [out_off[r], out_off[r] + out_width[r]); the range must hold
 * max(W_nom, W_min, min(W_max, nodes of the request)) slots. */
typedef struct {
    int32_t *l_last;        /* [R]  layer whose beams are returned: the first short layer, or
                                    gamma+1 when every layer passed                          */
    int32_t *out_width;     /* [R]  number of output beams                                   */
    const int32_t *out_off; /* [R+1]                                                         */
    int32_t *out_parent;    /* node the output beam extends                                  */
    int32_t *out_node;      /* the draft node it is, or -1 if it was sampled                 */
    int32_t *out_root_beam; /* input beam (tree) it descends from -> which KV cache to keep  */
    int32_t *out_token;
    float   *out_logp;      /* cumulative log-prob of the new beam under p and under q       */
    float   *out_logq;
    int32_t *out_source;    /* DSBD_SRC_*                                                    */
    int8_t  *node_status;   /* [N]  DSBD_NODE_*                                              */
    int32_t *layer_width;   /* [R*(gamma+1)] width chosen per layer, -1 where not run        */
    float   *node_logp;     /* [N]  cumulative log-prob of every node under p and q          */
    float   *node_logq;
    float   *lse_p;         /* [N]  log-sum-exp of each tempered logits row                  */
    float   *lse_q;
    int32_t *req_error;     /* [R]  0 or a DSBD_DEV_* code                                   */
    int32_t *req_stats;     /* [R*DSBD_REQ_STATS] or NULL, per request: 0 layers verified, 1 accept
                                    tests made, 2 residual masses recomputed exactly by a pass over
                                    the rows, 3 extra passes made for completion draws, 4 accept
                                    tests with |u - ratio| < 1e-5 (near ties), 5 logits row pairs
                                    consulted after the dense pass (live parents summed over the
                                    verified layers), 6 layers whose histogram overflowed a word and
                                    fell back to exact passes, 7 reserved (0)                     */
} dsbd_verify_out_t;

/* One verification step (Algorithm 1 with the dynamic width of Eqs. for P, P~, alpha_j, W_L):
 *   1. for every node and both models: log-sum-exp of the tempered logits row, the log-prob
 *      of each draft token given its parent, cumulative beam scores (roots: root_logp/q);
 *   2. per request, layer by layer: live drafts = depth-l nodes whose parent was accepted;
 *      p_beam, q_beam = joint over (accepted parents x V), Eq. 1; width W_L^(l) from the
 *      acceptance-count recursion; drafts accepted with probability min(1, p'/q_beam) (the
 *      direction the proof of Theorem 1 and the alpha_j formula use), p' reset to p_beam on an
 *      accept and replaced by norm(max(0, p' - q_beam)) on a reject; stop at W_L^(l) accepts;
 *   3. a layer with fewer accepts is completed by one draw from p' and draws from p_beam and
 *      ends the step; if all gamma layers pass, W_nom beams are drawn from p_beam^(gamma+1).
 * logits_p, logits_q: [N, row_stride] fp32, row n = next-token logits after node n of the
 * large / small model (row_stride >= V, in elements; rows 16-byte aligned run fastest).
 * root_logp, root_logq: [B] cumulative log-probs of the input beams.
 * Randomness: Philox4x32-10, key (seed lo, seed hi ^ step hi), counter (index, layer*4+purpose,
 * request, step lo), purpose 0 accept test of the index-th live draft, 1 residual draw,
 * 2 index-th p_beam fill, 3 index-th extra-layer draw; u = ((word0 >> 8) + 0.5) * 2^-24.
 * Draws are inverse-CDF over (live parent ascending, token ascending). */
int dsbd_verify_step(const dsbd_forest_t *forest, const dsbd_verify_params_t *params,
                     const float *logits_p, const float *logits_q, int64_t row_stride,
                     const float *root_logp, const float *root_logq,
                     const dsbd_verify_out_t *out, void *workspace, size_t workspace_bytes,
                     int32_t *status, dsbd_stream_t stream);

size_t dsbd_verify_workspace(const dsbd_forest_t *forest, const dsbd_verify_params_t *params);

/* Step 1 of dsbd_verify_step on its own: the large and the small model's next-token
 * distribution of every node (Overview: "predict the distribution for the next token of each
 * node in parallel"), returned as the log-sum-exp of each tempered logits row,
 * lse_p[n] = log sum_v exp(logits_p[n,v]/tau), lse_q likewise ([N] each).  One dense pass over
 * both logits tensors; workspace as for dsbd_verify_step. */
int dsbd_node_stats(const dsbd_forest_t *forest, const dsbd_verify_params_t *params,
                    const float *logits_p, const float *logits_q, int64_t row_stride,
                    float *lse_p, float *lse_q, void *workspace, size_t workspace_bytes,
                    dsbd_stream_t stream);

/* dsbd_node_stats for callers that cannot allocate device memory.  (The paper has no
 * counterpart; this is a property of the library, not of the method.)  Some callers have no
 * way to hand over a workspace: a plug-in that runs after its host process has given every
 * byte of device memory to the host's own pool, or a latency-critical section that must not
 * call cudaMalloc because cudaMalloc synchronises the whole device.  For them the scratch of
 * the two kernels lives in a fixed array of DSBD_STATIC_SCRATCH_BYTES inside the library
 * image; every GPU that loads the library holds that array until the process exits.
 *   - Same inputs, outputs and results as dsbd_node_stats; the call allocates and frees
 *     nothing and calls no routine that does.
 *   - Limit: 8*2*N*ceil(V/1024) bytes (rounded up to 256) + 16*N bytes must fit into
 *     DSBD_STATIC_SCRATCH_BYTES, e.g. about 4100 rows of a 128256-token vocabulary; larger problems
 *     are refused with DSBD_ERR_WORKSPACE_TOO_SMALL and nothing is launched.
 *   - The first call on a device looks up the device address of the array (once per device,
 *     with that device current).  Make that first call outside any stream capture.
 *   - All calls share the one array, which still holds what the last call left in it.  The
 *     kernels overwrite every entry before they read it, so nothing needs clearing, but two
 *     calls that overlap on the GPU (different streams, or several host threads) race on it:
 *     serialise them. */
#define DSBD_STATIC_SCRATCH_BYTES (8u << 20)
int dsbd_node_stats_static(const dsbd_forest_t *forest, const dsbd_verify_params_t *params,
                           const float *logits_p, const float *logits_q, int64_t row_stride,
                           float *lse_p, float *lse_q, dsbd_stream_t stream);

/* The context-dependent width of ONE layer (Eqs. for P(m,k), P~(m,i), alpha_j and
 * W_L^(l) = max(W_min, W~_L^(l)(t)), capped by W_max) for a given live set: request r's live
 * parents are live_nodes[live_off[r] .. live_off[r+1]) (ascending node ids) with cumulative
 * scores node_logp/node_logq (indexed by node id), and m[r] live drafts follow them.
 * Outputs: width[r]; optionally alpha[r*out_stride + j] = alpha_{j+1} (j < m[r]) and
 * tail[r*out_stride + K] = P(at least K accepts), K <= m[r]; out_stride >= max m + 1. */
int dsbd_select_width(const dsbd_forest_t *forest, const dsbd_verify_params_t *params,
                      const float *logits_p, const float *logits_q, int64_t row_stride,
                      const float *node_logp, const float *node_logq,
                      const int32_t *live_off, const int32_t *live_nodes, const int32_t *m,
                      int32_t *width, float *alpha, float *tail, int32_t out_stride,
                      void *workspace, size_t workspace_bytes, int32_t *status,
                      dsbd_stream_t stream);

/* One step of the draft stage (Section "Overview": the small model performs beam sampling of
 * width W_S for gamma steps; Section "Details": every draft beam is a sample of
 * q_beam = T o (q / Q) over (current beams x V)).  Request r owns the current beams
 * req_beam_off[r] .. req_beam_off[r+1]) -- the input beams for the first draft layer, the W_S
 * beams of the previous layer afterwards -- with cumulative scores beam_logq [n_beams] and
 * next-token logits logits_q [n_beams rows, row_stride].  It draws W_S (W_S_r[r] when given) iid
 * cells by inverse CDF in canonical order (beam ascending, token ascending); draw k uses the
 * Philox uniform of (request r, layer number 2^29 + layer, purpose 3, index k), so the stream is
 * disjoint from the verification's.  Draw k lands in slot out_off[r] + k: out_parent (global
 * index of the beam it extends), out_token, out_logq (new cumulative score); k is the node's
 * draft_rank.  temperature, top_k and top_p act as in dsbd_verify_params_t.
 * All pointers device except params; req_error [R] optional.  Host facts: n_slots = out_off[R],
 * max_req_beams <= DSBD_MAX_LIVE.  *status / req_error: DSBD_DEV_CAPACITY when a slot range is
 * shorter than W_S, DSBD_DEV_EXHAUSTED for a request without beams. */
typedef struct {
    int32_t V;
    float temperature;
    int32_t W_S;
    const int32_t *W_S_r;          /* optional [R], device                                   */
    uint64_t seed, step;
    int32_t layer;                 /* draft layer 1..gamma this call samples                  */
    int32_t top_k;
    float top_p;
    int32_t n_slots;
    int32_t max_req_beams;
} dsbd_draft_params_t;

int dsbd_draft_layer(int32_t R, int32_t n_beams, const int32_t *req_beam_off,
                     const dsbd_draft_params_t *params, const float *logits_q, int64_t row_stride,
                     const float *beam_logq, const int32_t *out_off, int32_t *out_parent,
                     int32_t *out_token, float *out_logq, int32_t *req_error, void *workspace,
                     size_t workspace_bytes, int32_t *status, dsbd_stream_t stream);

size_t dsbd_draft_workspace(int32_t R, int32_t n_beams, const dsbd_draft_params_t *params);

/* The draft forest from the draft stage's draws (Section "Overview": the small model's beam
 * sampling of width W_S over gamma steps traces a forest of W_L trees, one per input beam, every
 * later layer holding W_S nodes).  draw_parent / draw_token: [gamma][R * W_S], layer l (1-based)
 * at offset (l-1)*R*W_S, request r's draws at r*W_S .. as dsbd_draft_layer wrote them with
 * out_off[r] = r*W_S: for l = 1 the parent is a global input-beam index, for l > 1 the index
 * r*W_S + k' of a draw of layer l-1.  Output (device arrays sized for N = B + gamma*R*W_S nodes):
 * the forest in the layout dsbd_forest_t describes -- trees beam-major, a tree's nodes contiguous,
 * the root first and then its draws in (layer, draw) order, so parent[n] < n -- with
 * draft_rank[n] = the draw index k, beam_node_off [B+1], and node_of_draw [gamma][R * W_S]: the node
 * each draw became (to place the models' rows).  Node numbering inside a tree is a convention of
 * this library; any topological order would do.  gamma * W_S <= 1024, beams per request <=
 * DSBD_MAX_LIVE.  max_tree_nodes (optional device int32, set it to 0 before the call) is raised
 * to the size of the largest tree: dsbd_forest_t.max_tree_nodes may be the bound 1 + gamma*W_S,
 * but the attention picks a faster kernel shape when it is given the true, usually much smaller
 * value.  *status: DSBD_DEV_BAD_FOREST when a draw names a beam of another request. */
int dsbd_forest_build(int32_t R, int32_t gamma, int32_t W_S, const int32_t *req_beam_off,
                      const int32_t *draw_parent, const int32_t *draw_token,
                      int32_t *beam_node_off, int32_t *parent, int32_t *token, int32_t *draft_rank,
                      int32_t *node_of_draw, int32_t *max_tree_nodes, int32_t *status,
                      dsbd_stream_t stream);

/* KV-cache update at the end of a decode step (Section "Forest-based Parallel Decoding": after
 * the iteration the key-value caches are updated according to the output beams, an output beam
 * keeping the cache of the input beam it descends from; Section "Reducing Memory Cost": keeping
 * only the output beam of lowest perplexity leaves one cache per request).
 *
 * An output beam in slot s (parent node n = out_parent[s], input beam b = out_root_beam[s])
 * gets the cache  [cache of b] ++ [keys/values of the nodes on the path root(b) .. n], which is
 * exactly what n attended to; its new token becomes the root of the next draft tree.  Kept
 * beams are numbered request by request, inside a request in slot order, and their caches are
 * written packed in the layout dsbd_forest_attention reads: new beam j as [Hkv, L'_j, d]
 * starting at element new_prefix_off[j]*Hkv*d of k_dst / v_dst, L'_j = L_b + depth(n) + 1.
 * keep_best: per request only the slot of lowest perplexity exp(-out_logp/(L'+1)) is kept (the
 * lower slot on a tie).
 *
 * Device inputs: the forest; out_off [R+1], out_width [R], out_parent, out_root_beam, out_logp
 * as dsbd_verify_step wrote them (out_logp is read only with keep_best); k_new, v_new, k_prefix,
 * v_prefix, prefix_off as given to dsbd_forest_attention (desc gives Hkv, d, dtype).
 * Device outputs: k_dst, v_dst (dst_capacity tokens each, 16-byte aligned, must not overlap the
 * inputs); new_req_beam_off [R+1]; new_prefix_off [n_slots+1] (entries past the number of kept
 * beams repeat the total); new_beam_slot [n_slots] (the output slot each new beam came from, -1
 * past the end).  n_slots is the host's copy of out_off[R].
 * *status: DSBD_DEV_CAPACITY when the kept caches need more than dst_capacity tokens,
 * DSBD_DEV_BAD_FOREST when a slot names a beam outside its request or a node outside that
 * beam's tree; nothing is copied then. */
typedef struct {
    int32_t n_slots;
    int32_t keep_best;
    int64_t dst_capacity;
    /* dsbd_kv_commit_paged only: the caches of all transformer layers in one call.  Every layer
     * has its own pools and its own k_new / v_new, at the same address offsets from layer to
     * layer, and all layers share the page tables (a page id means the same slot in every
     * layer's pool), so the plan, the tables and the allocator update are made once.
     * n_layers 0 or 1: a single layer. */
    int32_t n_layers;
    int64_t pool_layer_stride;     /* elements between consecutive layers' pools            */
    int64_t new_layer_stride;      /* elements between consecutive layers' k_new / v_new    */
} dsbd_commit_params_t;

int dsbd_kv_commit(const dsbd_forest_t *forest, const dsbd_attn_desc_t *desc,
                   const dsbd_commit_params_t *params,
                   const int32_t *out_off, const int32_t *out_width, const int32_t *out_parent,
                   const int32_t *out_root_beam, const float *out_logp,
                   const void *k_new, const void *v_new, const void *k_prefix, const void *v_prefix,
                   const int64_t *prefix_off, void *k_dst, void *v_dst,
                   int32_t *new_req_beam_off, int64_t *new_prefix_off, int32_t *new_beam_slot,
                   void *workspace, size_t workspace_bytes, int32_t *status, dsbd_stream_t stream);

size_t dsbd_kv_commit_workspace(const dsbd_forest_t *forest, const dsbd_commit_params_t *params);

/* The same update for PAGED caches (see dsbd_forest_attention_paged): nothing of a prefix is
 * copied.  New beam j keeps the first L_b / DSBD_PAGE_TOKENS pages of its input beam b (shared),
 * and gets ceil((L_b % DSBD_PAGE_TOKENS + path length) / DSBD_PAGE_TOKENS) fresh pages that
 * receive b's partly filled last page, then the path's keys/values, then zeros.  Selection,
 * numbering and keep_best as in dsbd_kv_commit.
 * Allocator state (device, updated in place): free_stack [n_pages] and free_count [1]; the k-th
 * fresh page of the call is free_stack[free_count - 1 - k], beams in order; afterwards the
 * stack is rebuilt as every page that no new table names, ascending.  The pools are written
 * only at fresh pages.  The old page_table / page_off / prefix_off are not modified.
 * Outputs: new_req_beam_off [R+1], new_prefix_off [n_slots+1] (cumulative lengths), new_page_off
 * [n_slots+1], new_page_table [params->dst_capacity entries], new_beam_slot [n_slots].
 * *status: DSBD_DEV_CAPACITY when the tables need more than dst_capacity entries or the stack has
 * too few free pages, DSBD_DEV_BAD_FOREST as in dsbd_kv_commit; then pools, tables and allocator
 * stay as they were. */
int dsbd_kv_commit_paged(const dsbd_forest_t *forest, const dsbd_attn_desc_t *desc,
                         const dsbd_commit_params_t *params,
                         const int32_t *out_off, const int32_t *out_width, const int32_t *out_parent,
                         const int32_t *out_root_beam, const float *out_logp,
                         const void *k_new, const void *v_new, void *k_pool, void *v_pool,
                         const dsbd_kv_pages_t *pages, const int64_t *prefix_off,
                         int32_t *free_stack, int32_t *free_count,
                         int32_t *new_req_beam_off, int64_t *new_prefix_off, int64_t *new_page_off,
                         int32_t *new_page_table, int32_t *new_beam_slot,
                         void *workspace, size_t workspace_bytes, int32_t *status, dsbd_stream_t stream);

size_t dsbd_kv_commit_paged_workspace(const dsbd_forest_t *forest, const dsbd_commit_params_t *params,
                                      int64_t n_pages);

const char *dsbd_status_string(int code);

#ifdef __cplusplus
}
#endif
#endif
