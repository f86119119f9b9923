/*
 * DSBD oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, double-precision CPU statement of what one decode step of dynamic-width
 * speculative beam decoding computes: forest-masked attention, and the layer-by-layer
 * verification of a draft forest (beam-sampling distributions, accept / residual-resample
 * rule, dynamic layer width).  It is written from the paper's definitions and Algorithm 1 and
 * shares no code, header, table or constant generator with the CUDA library.  Only tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it.
 *
 * Parity status: the *distribution* of the outputs is pinned by the paper (Theorem 1, exact
 * enumeration and chi-square tests).  The per-seed outputs (which token a given Philox
 * stream yields) depend on conventions the paper does not fix -- the counter layout, the
 * inverse-CDF cell order -- and are therefore "parity unpinned": nothing outside this file
 * can confirm those conventions; the CUDA path has to match them.
 */
#ifndef DSBD_ORACLE_H
#define DSBD_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Draft forest: R requests, B trees (one per input beam), N nodes.
 * Trees are stored beam-major, the root of tree b is node beam_node_off[b], and every
 * non-root node has parent[n] < n inside the same tree (Section "Draft and Verification
 * Scheme", Overview: W_L trees whose roots are the input beams). */
typedef struct {
    int32_t R, B, N, max_depth;      /* max_depth = gamma, the number of draft layers        */
    const int32_t *req_beam_off;     /* [R+1] trees of request r                             */
    const int32_t *beam_node_off;    /* [B+1] nodes of tree b, root first                    */
    const int32_t *parent;           /* [N]   global node id of the parent, -1 for a root    */
    const int32_t *token;            /* [N]   draft token of the node (ignored for roots)    */
    const int32_t *draft_rank;       /* [N] or NULL: position of the node in the order in    */
                                     /* which the small model drew the drafts of its layer;  */
                                     /* NULL = ascending node id                             */
} dsbd_oracle_forest;

typedef struct {
    int32_t V;
    double temperature;              /* divides the logits of both models                    */
    double thresh;                   /* threshold t of the width rule                        */
    int32_t W_min, W_max, W_nom;     /* minimum width, cap, width of the extra layer         */
    const int32_t *W_min_r;          /* optional per-request overrides ([R] or NULL)         */
    const int32_t *W_max_r;
    const int32_t *W_nom_r;
    uint64_t seed, step;             /* Philox key and decode-step counter                   */
    const int32_t *req_id;           /* optional [R]: request number used in the Philox      */
                                     /* counter (NULL = 0..R-1); lets a test verify a subset */
    int32_t top_k;                   /* warping T of the joint distributions: keep the top_k  */
    double top_p;                    /* cells (0 = off), then the smallest set of the largest */
                                     /* cells whose mass reaches top_p (<= 0 or >= 1 = off)   */
} dsbd_oracle_params;

/* node_status values */
enum {
    DSBD_O_NODE_UNREACHED = 0,       /* layer never verified                                 */
    DSBD_O_NODE_ACCEPTED  = 1,       /* roots, and drafts that passed the accept test        */
    DSBD_O_NODE_REJECTED  = 2,       /* failed the accept test                               */
    DSBD_O_NODE_CUT       = 3,       /* not tested: the layer already had its width          */
    DSBD_O_NODE_PRUNED    = 4        /* parent was not accepted                              */
};

/* out_source values */
enum {
    DSBD_O_SRC_DRAFT = 0, DSBD_O_SRC_RESIDUAL = 1, DSBD_O_SRC_FILL = 2, DSBD_O_SRC_EXTRA = 3
};

/* trace kinds */
enum {
    DSBD_O_TR_ACCEPT = 0, DSBD_O_TR_RESIDUAL = 1, DSBD_O_TR_FILL = 2, DSBD_O_TR_EXTRA = 3,
    DSBD_O_TR_WIDTH = 4,
    DSBD_O_TR_WARP = 5      /* one per warped distribution: a = relative gap between the last
                               kept and the first dropped cell of the top-k cut, b = distance
                               of the kept mass from top_p at the top-p cut; index 0 = p, 1 = q */
};

typedef struct {
    /* per request */
    int32_t *l_last;        /* [R]  layer that produced the outputs (1..gamma+1)             */
    int32_t *out_width;     /* [R]  number of output beams                                   */
    const int32_t *out_off; /* [R+1] slot range of request r in the out_* arrays (capacity)  */
    /* per output slot */
    int32_t *out_parent;    /* node the beam extends                                         */
    int32_t *out_node;      /* draft node it is, or -1 when sampled                          */
    int32_t *out_root_beam; /* tree (input beam) it descends from                            */
    int32_t *out_token;
    double  *out_logp;      /* new cumulative log-prob under p and q                         */
    double  *out_logq;
    int32_t *out_source;
    /* per node / per layer */
    int8_t  *node_status;   /* [N]                                                           */
    int32_t *layer_width;   /* [R*(gamma+1)] chosen width, -1 where the layer was not run    */
    double  *node_logp;     /* [N] cumulative log-prob S_p, S_q of every node                */
    double  *node_logq;
    double  *lse_p;         /* [N] log-sum-exp of the tempered logits row, both models       */
    double  *lse_q;
    int32_t *error;         /* [R] 0, or a DSBD_O_ERR_* code                                 */
    /* optional decision trace (all NULL or all valid); one record per random decision or
     * width choice, in the order they happen inside a request, requests in order            */
    int64_t  trace_cap;
    int64_t *trace_len;     /* [1]  records written (may exceed cap: then truncated)         */
    int32_t *trace_req, *trace_layer, *trace_kind, *trace_index, *trace_near;
    double  *trace_u;       /* uniform used (0 for width records)                            */
    double  *trace_a;       /* accept: ratio;  sample: cdf below cell / Z;  width: G(W~)     */
    double  *trace_b;       /* accept: unused; sample: cdf through cell / Z; width: G(W~+1)  */
    /* optional dump of the normalised mass vector behind every sample record, small cases   */
    int64_t  dist_cap;      /* capacity in doubles                                           */
    int64_t *dist_len;      /* [1]                                                           */
    double  *dist;          /* consecutive vectors of length |A|*V, in trace order           */
} dsbd_oracle_verify_out;

enum { DSBD_O_ERR_BAD_TOKEN = 1, DSBD_O_ERR_EXHAUSTED = 2, DSBD_O_ERR_CAPACITY = 3,
       DSBD_O_ERR_BAD_FOREST = 4 };

/* Philox4x32-10 block function (Salmon et al., SC'11). */
void dsbd_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/* The uniform in (0,1) a decision uses: word 0 of the Philox block whose counter is
 * (index, layer*4 + purpose, request, low 32 bits of step) and whose key is
 * (seed low, seed high xor step high); u = ((x >> 8) + 0.5) * 2^-24. */
double dsbd_oracle_uniform(uint64_t seed, uint64_t step, uint32_t request, uint32_t layer,
                           uint32_t purpose, uint32_t index);

/* Forest attention by definition (Section "Forest-based Parallel Decoding"):
 * O[n,h] = softmax_j(scale * Q[n,h].K_j) V_j over the prefix of n's beam and the
 * ancestors-or-self of n.  Inputs are float (exact images of the bf16/fp32 device data),
 * arithmetic is double.  q/out: [N,Hq,d]; k_new/v_new: [N,Hkv,d]; prefixes packed per beam
 * as [Hkv, L_b, d], beam b starting at element prefix_off[b]*Hkv*d. Returns 0 or an error. */
int dsbd_oracle_forest_attention(const dsbd_oracle_forest *f, int32_t Hq, int32_t Hkv,
                                 int32_t d, double scale, const float *q, const float *k_new,
                                 const float *v_new, const float *k_prefix,
                                 const float *v_prefix, const int64_t *prefix_off,
                                 double *out, int32_t threads);

/* alpha_j of the width rule by the paper's own recursion: p_1 = p_beam,
 * p_{k+1} = norm(max(p_k - q_beam, 0)), alpha_k = sum min(p_k, q_beam).  n = |A|*V. */
void dsbd_oracle_alpha_chain(const double *p_beam, const double *q_beam, int64_t n, int32_t m,
                             double *alpha);

/* Acceptance-count recursion: fills P as a (m+1)x(m+1) row-major table P[n][k] and G[K],
 * K = 0..m+1 (G[m+1] = 0); returns W~ = max{K in 0..m : G(K) >= thresh}. */
int32_t dsbd_oracle_width_dp(const double *alpha, int32_t m, double thresh, double *P,
                             double *G);

/* The warping T applied to a joint distribution w over n cells, in place (Section "Decodings of
 * LLMs": top-k keeps the k most probable entries, top-p the smallest set of most probable
 * entries whose mass reaches p; both renormalise).  Ties are broken towards the lower cell
 * index.  gap_k / gap_p (optional) receive the quantities of the DSBD_O_TR_WARP record. */
void dsbd_oracle_warp(double *w, int64_t n, int32_t top_k, double top_p, double *gap_k, double *gap_p);

/* One verification step (Algorithm 1 with the dynamic width) for every request.
 * inject_u: NULL, or [R*inject_stride] uniforms consumed in order by the random decisions of
 * request r in place of the Philox stream (tests only). */
int dsbd_oracle_verify_step(const dsbd_oracle_forest *f, const dsbd_oracle_params *prm,
                            const float *logits_p, const float *logits_q, int64_t row_stride,
                            const double *root_logp, const double *root_logq,
                            const double *inject_u, int64_t inject_stride,
                            dsbd_oracle_verify_out *out, int32_t threads);

/* Width of one layer for a given live set: live parents live_nodes[live_off[r]..live_off[r+1])
 * with cumulative scores node_logp/node_logq (indexed by node id), m[r] live drafts.
 * alpha/tail are optional, laid out [R*alpha_stride]; tail holds G(0..m). */
int dsbd_oracle_select_width(const dsbd_oracle_forest *f, const dsbd_oracle_params *prm,
                             const float *logits_p, const float *logits_q, int64_t row_stride,
                             const double *node_logp, const double *node_logq,
                             const int32_t *live_off, const int32_t *live_nodes,
                             const int32_t *m, int32_t *width, double *alpha, double *tail,
                             int32_t alpha_stride);

/* One step of the small model's beam sampling (Sections "Overview" and "Details"): request r
 * draws W_S (W_S_r[r] when given) iid cells from q_beam = T o (q / Q) over its current beams
 * req_beam_off[r] .. req_beam_off[r+1]) x V, draw k with the uniform of (request, layer
 * 2^29 + layer, purpose 3, index k) or inject_u[r*inject_stride + k].  Per draw, in slot
 * out_off[r] + k: the beam it extends (global index), the token, the new cumulative score, and
 * optionally the cell's CDF interval.  error: [R]. */
int dsbd_oracle_draft_layer(int32_t R, const int32_t *req_beam_off, const dsbd_oracle_params *prm,
                            int32_t layer, const int32_t *W_S_r, int32_t W_S,
                            const float *logits_q, int64_t row_stride, const double *beam_logq,
                            const double *inject_u, int64_t inject_stride,
                            const int32_t *out_off, int32_t *out_parent, int32_t *out_token,
                            double *out_logq, double *cdf_lo, double *cdf_hi, int32_t *error);

#ifdef __cplusplus
}
#endif
#endif
