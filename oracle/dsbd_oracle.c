/*
 * DSBD oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE (see dsbd_oracle.h).
 *
 * Everything here follows the paper's statements in their own order and in double
 * precision; there is no blocking, fusion or reordering.  Parity of per-seed token ids is
 * "parity unpinned" (conventions of this file); the output law is pinned by Theorem 1.
 * With warped joints (top-k / top-p) the law is pinned at every layer for drafts drawn from the
 * q_beam this file verifies against (the warp of the joint over the ACCEPTED beams); for drafts
 * that a drafter drew from the warp of the joint over all its beams, layers >= 2 carry
 * "parity unpinned: distribution under warping at l >= 2" -- pruning and warping do not
 * commute, and the size of the difference is recorded in the tests.
 */
#include "dsbd_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define NEAR_TIE 1e-5

/* ------------------------------------------------------------------ Philox4x32-10 ---- */
/* Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3" (SC'11):
 * ten rounds of  (c0,c1,c2,c3) <- (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)),
 * the key bumped by the Weyl constants between rounds. */
void dsbd_oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = M0 * (uint64_t)c0;
        uint64_t p1 = M1 * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

double dsbd_oracle_uniform(uint64_t seed, uint64_t step, uint32_t request, uint32_t layer,
                           uint32_t purpose, uint32_t index)
{
    uint32_t ctr[4] = { index, layer * 4u + purpose, request, (uint32_t)step };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) ^ (uint32_t)(step >> 32) };
    uint32_t x[4];
    dsbd_oracle_philox4x32_10(ctr, key, x);
    return ((double)(x[0] >> 8) + 0.5) * (1.0 / 16777216.0);
}

/* ------------------------------------------------------------------ forest helpers ---- */
static int forest_depths(const dsbd_oracle_forest *f, int32_t *depth, int32_t *tree_of)
{
    for (int32_t b = 0; b < f->B; ++b) {
        int32_t lo = f->beam_node_off[b], hi = f->beam_node_off[b + 1];
        if (hi <= lo) return DSBD_O_ERR_BAD_FOREST;
        for (int32_t n = lo; n < hi; ++n) {
            tree_of[n] = b;
            int32_t par = f->parent[n];
            if (n == lo) {
                if (par != -1) return DSBD_O_ERR_BAD_FOREST;
                depth[n] = 0;
            } else {
                if (par < lo || par >= n) return DSBD_O_ERR_BAD_FOREST;
                depth[n] = depth[par] + 1;
                if (depth[n] > f->max_depth) return DSBD_O_ERR_BAD_FOREST;
            }
        }
    }
    return 0;
}

/* ------------------------------------------------------------------ attention --------- */
/* Section "Forest-based Parallel Decoding": one KV cache per input beam; inside a tree a
 * node sees its ancestors and itself (topology-aware mask), nothing of any other tree. */
int dsbd_oracle_forest_attention(const dsbd_oracle_forest *f, int32_t Hq, int32_t Hkv,
                                 int32_t d, double scale, const float *q, const float *k_new,
                                 const float *v_new, const float *k_prefix,
                                 const float *v_prefix, const int64_t *prefix_off,
                                 double *out, int32_t threads)
{
    if (Hq <= 0 || Hkv <= 0 || d <= 0 || Hq % Hkv) return DSBD_O_ERR_BAD_FOREST;
    int32_t *depth = (int32_t *)malloc(sizeof(int32_t) * (size_t)f->N);
    int32_t *tree_of = (int32_t *)malloc(sizeof(int32_t) * (size_t)f->N);
    int rc = forest_depths(f, depth, tree_of);
    if (rc) { free(depth); free(tree_of); return rc; }
    const int32_t group = Hq / Hkv;
    (void)threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads > 0 ? threads : 1)
#endif
    for (int32_t n = 0; n < f->N; ++n) {
        const int32_t b = tree_of[n];
        const int64_t L = prefix_off[b + 1] - prefix_off[b];
        /* the keys node n may see: prefix tokens, then its ancestors root-first, then n */
        int32_t anc[4096];
        int32_t na = 0;
        for (int32_t a = n; a != -1 && na < 4096; a = f->parent[a]) anc[na++] = a;
        const int64_t nk = L + na;
        double *score = (double *)malloc(sizeof(double) * (size_t)nk);
        for (int32_t h = 0; h < Hq; ++h) {
            const int32_t g = h / group;
            const float *qv = q + ((int64_t)n * Hq + h) * d;
            const float *kp = k_prefix + (prefix_off[b] * Hkv + (int64_t)g * L) * d;
            const float *vp = v_prefix + (prefix_off[b] * Hkv + (int64_t)g * L) * d;
            double mx = -INFINITY;
            for (int64_t j = 0; j < nk; ++j) {
                const float *kv = (j < L) ? kp + j * d
                                          : k_new + ((int64_t)anc[na - 1 - (j - L)] * Hkv + g) * d;
                double s = 0.0;
                for (int32_t c = 0; c < d; ++c) s += (double)qv[c] * (double)kv[c];
                score[j] = s * scale;
                if (score[j] > mx) mx = score[j];
            }
            double denom = 0.0;
            for (int64_t j = 0; j < nk; ++j) { score[j] = exp(score[j] - mx); denom += score[j]; }
            double *o = out + ((int64_t)n * Hq + h) * d;
            for (int32_t c = 0; c < d; ++c) o[c] = 0.0;
            for (int64_t j = 0; j < nk; ++j) {
                const float *vv = (j < L) ? vp + j * d
                                          : v_new + ((int64_t)anc[na - 1 - (j - L)] * Hkv + g) * d;
                const double w = score[j] / denom;
                for (int32_t c = 0; c < d; ++c) o[c] += w * (double)vv[c];
            }
        }
        free(score);
    }
    free(depth); free(tree_of);
    return 0;
}

/* ------------------------------------------------------------------ width rule -------- */
/* alpha_j = sum q_beam * min(p_j / q_beam, 1) = sum min(p_j, q_beam), with p_1 = p_beam and
 * p_{k+1} = norm(max(p_k - q_beam, 0))  (Section "Dynamic-Width Speculative Beam Decoding").
 * If the residual has no mass (p_k == q_beam, alpha_k = 1) no rejection can follow: the
 * remaining alphas are set to 1. */
void dsbd_oracle_alpha_chain(const double *p_beam, const double *q_beam, int64_t n, int32_t m,
                             double *alpha)
{
    double *pk = (double *)malloc(sizeof(double) * (size_t)n);
    memcpy(pk, p_beam, sizeof(double) * (size_t)n);
    for (int32_t k = 0; k < m; ++k) {
        double a = 0.0, z = 0.0;
        for (int64_t i = 0; i < n; ++i) a += fmin(pk[i], q_beam[i]);
        alpha[k] = a;
        for (int64_t i = 0; i < n; ++i) {
            double r = pk[i] - q_beam[i];
            pk[i] = r > 0.0 ? r : 0.0;
            z += pk[i];
        }
        if (!(z > 0.0)) {
            alpha[k] = 1.0;
            for (int32_t j = k + 1; j < m; ++j) alpha[j] = 1.0;
            break;
        }
        for (int64_t i = 0; i < n; ++i) pk[i] /= z;
    }
    free(pk);
}

/* P(0,0) = 1; P(n,0) = prod_{j<=n}(1-alpha_j); P(n,k) = 0 for k > n;
 * P(n,k) = sum_{i=1..n} alpha_i prod_{j<i}(1-alpha_j) P(n-i, k-1)   (Eqs. for P and P~);
 * G(K) = 1 - sum_{k<K} P(m,k) is the probability of at least K accepts;
 * W~ = max{K : G(K) >= thresh}. */
int32_t dsbd_oracle_width_dp(const double *alpha, int32_t m, double thresh, double *P,
                             double *G)
{
    const int32_t s = m + 1;
    for (int32_t i = 0; i < s * s; ++i) P[i] = 0.0;
    P[0] = 1.0;
    for (int32_t n = 1; n <= m; ++n) {
        double none = 1.0;
        for (int32_t j = 1; j <= n; ++j) none *= (1.0 - alpha[j - 1]);
        P[n * s + 0] = none;
        for (int32_t k = 1; k <= n; ++k) {
            double acc = 0.0, first_rej = 1.0;   /* prod_{j<i}(1-alpha_j) */
            for (int32_t i = 1; i <= n; ++i) {
                acc += alpha[i - 1] * first_rej * P[(n - i) * s + (k - 1)];
                first_rej *= (1.0 - alpha[i - 1]);
            }
            P[n * s + k] = acc;
        }
    }
    double below = 0.0;
    int32_t wt = 0;
    for (int32_t K = 0; K <= m; ++K) {
        G[K] = 1.0 - below;
        if (G[K] >= thresh) wt = K;
        below += P[m * s + K];
    }
    G[m + 1] = 0.0;
    if (G[0] < thresh) wt = 0;    /* thresh > 1: nothing qualifies, keep 0 */
    return wt;
}

/* ------------------------------------------------------------------ verification ------ */
typedef struct {
    const dsbd_oracle_forest *f;
    const dsbd_oracle_params *prm;
    const float *zp, *zq;
    int64_t stride;
    dsbd_oracle_verify_out *out;
    /* trace staging for one request */
    int64_t tcap, tlen;
    int32_t *t_layer, *t_kind, *t_index, *t_near;
    double *t_u, *t_a, *t_b;
    int64_t dcap, dlen;
    double *dbuf;
} req_ctx;

static void trace_push(req_ctx *c, int32_t layer, int32_t kind, int32_t index, double u,
                       double a, double b, int32_t near)
{
    if (!c->t_layer) return;
    if (c->tlen == c->tcap) {
        c->tcap = c->tcap ? c->tcap * 2 : 64;
        c->t_layer = (int32_t *)realloc(c->t_layer, sizeof(int32_t) * (size_t)c->tcap);
        c->t_kind = (int32_t *)realloc(c->t_kind, sizeof(int32_t) * (size_t)c->tcap);
        c->t_index = (int32_t *)realloc(c->t_index, sizeof(int32_t) * (size_t)c->tcap);
        c->t_near = (int32_t *)realloc(c->t_near, sizeof(int32_t) * (size_t)c->tcap);
        c->t_u = (double *)realloc(c->t_u, sizeof(double) * (size_t)c->tcap);
        c->t_a = (double *)realloc(c->t_a, sizeof(double) * (size_t)c->tcap);
        c->t_b = (double *)realloc(c->t_b, sizeof(double) * (size_t)c->tcap);
    }
    c->t_layer[c->tlen] = layer; c->t_kind[c->tlen] = kind; c->t_index[c->tlen] = index;
    c->t_near[c->tlen] = near; c->t_u[c->tlen] = u; c->t_a[c->tlen] = a; c->t_b[c->tlen] = b;
    c->tlen++;
}

static void dist_push(req_ctx *c, const double *w, int64_t n, double z)
{
    if (!c->dbuf) return;
    if (c->dlen + n > c->dcap) {
        while (c->dlen + n > c->dcap) c->dcap = c->dcap ? c->dcap * 2 : 1024;
        c->dbuf = (double *)realloc(c->dbuf, sizeof(double) * (size_t)c->dcap);
    }
    for (int64_t i = 0; i < n; ++i) c->dbuf[c->dlen + i] = w[i] / z;
    c->dlen += n;
}

/* log-sum-exp of the tempered row z/tau */
static double row_lse(const float *z, int32_t V, double tau)
{
    double mx = -INFINITY;
    for (int32_t v = 0; v < V; ++v) { double x = (double)z[v] / tau; if (x > mx) mx = x; }
    double s = 0.0;
    for (int32_t v = 0; v < V; ++v) s += exp((double)z[v] / tau - mx);
    return mx + log(s);
}

/* Inverse-CDF draw from the (unnormalised) mass vector w over A x V, cells in canonical
 * order (live parent major, token minor): the first cell whose running sum reaches u*Z,
 * else the last cell with mass.  Returns the cell or -1 if the vector has no mass. */
static int64_t draw_cell(const double *w, int64_t n, double u, double *lo, double *hi,
                         double *z_out)
{
    double z = 0.0;
    for (int64_t i = 0; i < n; ++i) z += w[i];
    *z_out = z;
    if (!(z > 0.0)) return -1;
    const double target = u * z;
    double cum = 0.0, prev = 0.0;
    int64_t last = -1;
    double last_lo = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        prev = cum;
        cum += w[i];
        if (w[i] > 0.0) { last = i; last_lo = prev; }
        if (w[i] > 0.0 && cum >= target) { *lo = prev / z; *hi = cum / z; return i; }
    }
    *lo = last_lo / z; *hi = 1.0;
    return last;
}

static double next_uniform(const req_ctx *c, const double *inject, int64_t inject_stride,
                           int64_t *inject_pos, uint32_t req, uint32_t layer, uint32_t purpose,
                           uint32_t index)
{
    if (inject) {
        double u = (*inject_pos < inject_stride) ? inject[*inject_pos] : 0.5;
        (*inject_pos)++;
        return u;
    }
    return dsbd_oracle_uniform(c->prm->seed, c->prm->step, req, layer, purpose, index);
}

/* p_beam over A x V (Eq. 1): p_beam(a, v) = exp(S[a]) p(v | a) / sum_{a',v'} exp(S[a']) p(v'|a')
 * and, since every p(.|a) sums to one, = softmax_A(S)[a] * softmax(z[a]/tau)[v]. */
static void beam_distribution(const float *z, int64_t stride, int32_t V, double tau,
                              const int32_t *A, int32_t nA, const double *S, const double *lse,
                              double *dst)
{
    double mx = -INFINITY;
    for (int32_t i = 0; i < nA; ++i) if (S[A[i]] > mx) mx = S[A[i]];
    double tot = 0.0;
    for (int32_t i = 0; i < nA; ++i) tot += exp(S[A[i]] - mx);
    for (int32_t i = 0; i < nA; ++i) {
        const double w = exp(S[A[i]] - mx) / tot;
        const float *row = z + (int64_t)A[i] * stride;
        for (int32_t v = 0; v < V; ++v)
            dst[(int64_t)i * V + v] = w * exp((double)row[v] / tau - lse[A[i]]);
    }
}

/* ------------------------------------------------------------------ warping ---------- */
typedef struct { double v; int64_t i; } cell_t;
static int cmp_cell_desc(const void *x, const void *y)
{
    const cell_t *a = (const cell_t *)x, *b = (const cell_t *)y;
    if (a->v != b->v) return a->v > b->v ? -1 : 1;
    return a->i < b->i ? -1 : (a->i > b->i ? 1 : 0);
}

/* T o w: sort the cells by probability, keep the first top_k, renormalise, then keep the
 * shortest prefix whose mass reaches top_p, renormalise.  (The order top-k, then top-p on the
 * renormalised vector is the usual one for chained warpers.) */
void dsbd_oracle_warp(double *w, int64_t n, int32_t top_k, double top_p, double *gap_k, double *gap_p)
{
    if (gap_k) *gap_k = 1.0;
    if (gap_p) *gap_p = 1.0;
    const int use_k = top_k > 0 && top_k < n, use_p = top_p > 0.0 && top_p < 1.0;
    if (!use_k && !use_p) return;
    cell_t *c = (cell_t *)malloc(sizeof(cell_t) * (size_t)n);
    for (int64_t i = 0; i < n; ++i) { c[i].v = w[i]; c[i].i = i; }
    qsort(c, (size_t)n, sizeof(cell_t), cmp_cell_desc);
    int64_t keep = n;
    if (use_k) {
        keep = top_k;
        if (gap_k && c[keep - 1].v > 0.0) *gap_k = (c[keep - 1].v - c[keep].v) / c[keep - 1].v;
    }
    double z = 0.0;
    for (int64_t j = 0; j < keep; ++j) z += c[j].v;
    if (use_p && z > 0.0) {
        double cum = 0.0;
        int64_t j = 0;
        for (; j < keep; ++j) {
            cum += c[j].v / z;
            if (gap_p) { double g = fabs(cum - top_p); if (g < *gap_p) *gap_p = g; }
            if (cum >= top_p) { ++j; break; }
        }
        keep = j;
        z = 0.0;
        for (int64_t q = 0; q < keep; ++q) z += c[q].v;
    }
    for (int64_t i = 0; i < n; ++i) w[i] = 0.0;
    if (z > 0.0) for (int64_t j = 0; j < keep; ++j) w[c[j].i] = c[j].v / z;
    free(c);
}

static int cmp_rank(const void *x, const void *y)
{
    const int64_t *a = (const int64_t *)x, *b = (const int64_t *)y;
    if (a[0] != b[0]) return a[0] < b[0] ? -1 : 1;
    return a[1] < b[1] ? -1 : (a[1] > b[1] ? 1 : 0);
}

static void emit(req_ctx *c, int32_t r, int32_t *n_out, int32_t parent, int32_t node,
                 int32_t token, int32_t source, const int32_t *tree_of, int *err)
{
    const dsbd_oracle_verify_out *o = c->out;
    const int32_t cap = o->out_off[r + 1] - o->out_off[r];
    if (*n_out >= cap) { *err = DSBD_O_ERR_CAPACITY; return; }
    const int64_t s = o->out_off[r] + *n_out;
    const double tau = c->prm->temperature;
    o->out_parent[s] = parent;
    o->out_node[s] = node;
    o->out_root_beam[s] = tree_of[parent];
    o->out_token[s] = token;
    o->out_source[s] = source;
    o->out_logp[s] = o->node_logp[parent] +
        ((double)c->zp[(int64_t)parent * c->stride + token] / tau - o->lse_p[parent]);
    o->out_logq[s] = o->node_logq[parent] +
        ((double)c->zq[(int64_t)parent * c->stride + token] / tau - o->lse_q[parent]);
    (*n_out)++;
}

/* Algorithm 1 for one request. */
static void verify_request(req_ctx *c, int32_t r, const int32_t *depth, const int32_t *tree_of,
                           const double *root_logp, const double *root_logq,
                           const double *inject, int64_t inject_stride)
{
    const dsbd_oracle_forest *f = c->f;
    const dsbd_oracle_params *prm = c->prm;
    dsbd_oracle_verify_out *o = c->out;
    const int32_t V = prm->V, gamma = f->max_depth;
    const double tau = prm->temperature;
    const int32_t b_lo = f->req_beam_off[r], b_hi = f->req_beam_off[r + 1];
    const int32_t n_lo = f->beam_node_off[b_lo], n_hi = f->beam_node_off[b_hi];
    const int32_t W_min = prm->W_min_r ? prm->W_min_r[r] : prm->W_min;
    const int32_t W_max = prm->W_max_r ? prm->W_max_r[r] : prm->W_max;
    const int32_t W_nom = prm->W_nom_r ? prm->W_nom_r[r] : prm->W_nom;
    const uint32_t rid = prm->req_id ? (uint32_t)prm->req_id[r] : (uint32_t)r;
    int64_t inject_pos = 0;
    int err = 0;

    o->l_last[r] = gamma + 1;
    o->out_width[r] = 0;
    for (int32_t l = 0; l <= gamma; ++l) o->layer_width[(int64_t)r * (gamma + 1) + l] = -1;

    /* the large and the small model's next-token distribution of every node (Overview) */
    for (int32_t n = n_lo; n < n_hi; ++n) {
        o->lse_p[n] = row_lse(c->zp + (int64_t)n * c->stride, V, tau);
        o->lse_q[n] = row_lse(c->zq + (int64_t)n * c->stride, V, tau);
        o->node_status[n] = DSBD_O_NODE_UNREACHED;
    }
    /* cumulative sequence log-probs: log p(x_{1:t+1}) = log p(x_{1:t}) + log p(x_{t+1}|x_{1:t}) */
    for (int32_t n = n_lo; n < n_hi; ++n) {
        const int32_t par = f->parent[n];
        if (par < 0) {
            o->node_logp[n] = root_logp[tree_of[n]];
            o->node_logq[n] = root_logq[tree_of[n]];
            o->node_status[n] = DSBD_O_NODE_ACCEPTED;
        } else {
            const int32_t tok = f->token[n];
            if (tok < 0 || tok >= V) { err = DSBD_O_ERR_BAD_TOKEN; break; }
            o->node_logp[n] = o->node_logp[par] +
                ((double)c->zp[(int64_t)par * c->stride + tok] / tau - o->lse_p[par]);
            o->node_logq[n] = o->node_logq[par] +
                ((double)c->zq[(int64_t)par * c->stride + tok] / tau - o->lse_q[par]);
        }
    }
    if (err) { o->error[r] = err; return; }

    const int32_t max_nodes = n_hi - n_lo;
    int32_t *A = (int32_t *)malloc(sizeof(int32_t) * (size_t)(max_nodes + 1));
    int32_t *S = (int32_t *)malloc(sizeof(int32_t) * (size_t)(max_nodes + 1));
    int64_t *keys = (int64_t *)malloc(sizeof(int64_t) * 2 * (size_t)(max_nodes + 1));
    int32_t *acc = (int32_t *)malloc(sizeof(int32_t) * (size_t)(max_nodes + 1));
    int32_t nA = 0;
    for (int32_t b = b_lo; b < b_hi; ++b) A[nA++] = f->beam_node_off[b];   /* input beams */

    int32_t n_out = 0;
    int finished = 0;
    for (int32_t l = 1; l <= gamma && !finished; ++l) {
        /* drafts of layer l whose parent was accepted, in the order they were drawn */
        int32_t m = 0;
        for (int32_t n = n_lo; n < n_hi; ++n) {
            if (depth[n] != l) continue;
            if (o->node_status[f->parent[n]] == DSBD_O_NODE_ACCEPTED) {
                keys[2 * m] = f->draft_rank ? f->draft_rank[n] : n;
                keys[2 * m + 1] = n;
                m++;
            } else {
                o->node_status[n] = DSBD_O_NODE_PRUNED;
            }
        }
        qsort(keys, (size_t)m, 2 * sizeof(int64_t), cmp_rank);
        for (int32_t i = 0; i < m; ++i) S[i] = (int32_t)keys[2 * i + 1];

        const int64_t cells = (int64_t)nA * V;
        double *p_beam = (double *)malloc(sizeof(double) * (size_t)cells);
        double *q_beam = (double *)malloc(sizeof(double) * (size_t)cells);
        double *p_cur = (double *)malloc(sizeof(double) * (size_t)cells);
        beam_distribution(c->zp, c->stride, V, tau, A, nA, o->node_logp, o->lse_p, p_beam);
        beam_distribution(c->zq, c->stride, V, tau, A, nA, o->node_logq, o->lse_q, q_beam);
        if (prm->top_k > 0 || (prm->top_p > 0.0 && prm->top_p < 1.0)) {
            /* p_beam = T o (p / P), q_beam = T o (q / Q)  (Section "Details") */
            double gk, gp;
            dsbd_oracle_warp(p_beam, cells, prm->top_k, prm->top_p, &gk, &gp);
            trace_push(c, l, DSBD_O_TR_WARP, 0, 0.0, gk, gp, gk < NEAR_TIE || gp < NEAR_TIE);
            dsbd_oracle_warp(q_beam, cells, prm->top_k, prm->top_p, &gk, &gp);
            trace_push(c, l, DSBD_O_TR_WARP, 1, 0.0, gk, gp, gk < NEAR_TIE || gp < NEAR_TIE);
        }

        /* width of this layer */
        double *alpha = (double *)malloc(sizeof(double) * (size_t)(m + 1));
        double *P = (double *)malloc(sizeof(double) * (size_t)(m + 1) * (size_t)(m + 1));
        double *G = (double *)malloc(sizeof(double) * (size_t)(m + 2));
        dsbd_oracle_alpha_chain(p_beam, q_beam, cells, m, alpha);
        const int32_t wt = dsbd_oracle_width_dp(alpha, m, prm->thresh, P, G);
        int32_t W = wt > W_min ? wt : W_min;
        if (W > W_max) W = W_max;
        o->layer_width[(int64_t)r * (gamma + 1) + (l - 1)] = W;
        {
            int near = fabs(G[wt] - prm->thresh) < NEAR_TIE;
            if (wt + 1 <= m && fabs(G[wt + 1] - prm->thresh) < NEAR_TIE) near = 1;
            trace_push(c, l, DSBD_O_TR_WIDTH, wt, 0.0, G[wt], G[wt + 1], near);
        }

        /* the accept / residual loop */
        memcpy(p_cur, p_beam, sizeof(double) * (size_t)cells);
        int32_t count = 0;
        for (int32_t i = 0; i < m && count < W; ++i) {
            const int32_t n = S[i];
            int32_t ai = 0;
            while (A[ai] != f->parent[n]) ai++;
            const int64_t x = (int64_t)ai * V + f->token[n];
            const double u = next_uniform(c, inject, inject_stride, &inject_pos, rid,
                                          (uint32_t)l, 0u, (uint32_t)i);
            double ratio;
            if (q_beam[x] > 0.0) ratio = p_cur[x] / q_beam[x];
            else ratio = p_cur[x] > 0.0 ? INFINITY : 0.0;
            if (ratio > 1.0) ratio = 1.0;
            trace_push(c, l, DSBD_O_TR_ACCEPT, i, u, ratio, 0.0, fabs(u - ratio) < NEAR_TIE);
            if (u <= ratio) {
                o->node_status[n] = DSBD_O_NODE_ACCEPTED;
                acc[count++] = n;
                memcpy(p_cur, p_beam, sizeof(double) * (size_t)cells);
            } else {
                o->node_status[n] = DSBD_O_NODE_REJECTED;
                double z = 0.0;
                for (int64_t k = 0; k < cells; ++k) {
                    double d = p_cur[k] - q_beam[k];
                    z += d > 0.0 ? d : 0.0;
                }
                if (z > 0.0) {
                    for (int64_t k = 0; k < cells; ++k) {
                        double d = p_cur[k] - q_beam[k];
                        p_cur[k] = (d > 0.0 ? d : 0.0) / z;
                    }
                }
                /* else p' == q_beam: only a draft outside the support of q_beam can be rejected
                 * there (an event of probability zero when the drafts are samples of q_beam);
                 * it carries nothing to subtract and p' stays as it is */
            }
        }
        for (int32_t i = 0; i < m; ++i)
            if (o->node_status[S[i]] == DSBD_O_NODE_UNREACHED) o->node_status[S[i]] = DSBD_O_NODE_CUT;

        if (count < W) {
            /* short layer: keep the accepted drafts, one beam from p', the rest from p_beam */
            for (int32_t i = 0; i < count && !err; ++i)
                emit(c, r, &n_out, f->parent[acc[i]], acc[i], f->token[acc[i]],
                     DSBD_O_SRC_DRAFT, tree_of, &err);
            int32_t fill = 0;
            for (int32_t k = count; k < W && !err; ++k) {
                const int residual = (k == count);
                const double *w = residual ? p_cur : p_beam;
                const double u = next_uniform(c, inject, inject_stride, &inject_pos, rid,
                                              (uint32_t)l, residual ? 1u : 2u,
                                              residual ? 0u : (uint32_t)fill);
                double lo = 0, hi = 0, z = 0;
                const int64_t cell = draw_cell(w, cells, u, &lo, &hi, &z);
                if (cell < 0) { err = DSBD_O_ERR_EXHAUSTED; break; }
                trace_push(c, l, residual ? DSBD_O_TR_RESIDUAL : DSBD_O_TR_FILL,
                           residual ? 0 : fill, u, lo, hi,
                           (u - lo < NEAR_TIE) || (hi - u < NEAR_TIE));
                dist_push(c, w, cells, z);
                emit(c, r, &n_out, A[cell / V], -1, (int32_t)(cell % V),
                     residual ? DSBD_O_SRC_RESIDUAL : DSBD_O_SRC_FILL, tree_of, &err);
                if (!residual) fill++;
            }
            o->l_last[r] = l;
            finished = 1;
        } else {
            /* every beam of the next layer's input is an accepted draft, ascending id */
            nA = 0;
            for (int32_t n = n_lo; n < n_hi; ++n)
                if (depth[n] == l && o->node_status[n] == DSBD_O_NODE_ACCEPTED) A[nA++] = n;
        }
        free(p_beam); free(q_beam); free(p_cur); free(alpha); free(P); free(G);
    }

    if (!finished && !err) {
        /* all gamma layers passed: W_nom beams straight from p_beam^(gamma+1) */
        const int64_t cells = (int64_t)nA * V;
        double *p_beam = (double *)malloc(sizeof(double) * (size_t)cells);
        beam_distribution(c->zp, c->stride, V, tau, A, nA, o->node_logp, o->lse_p, p_beam);
        if (prm->top_k > 0 || (prm->top_p > 0.0 && prm->top_p < 1.0)) {
            double gk, gp;
            dsbd_oracle_warp(p_beam, cells, prm->top_k, prm->top_p, &gk, &gp);
            trace_push(c, gamma + 1, DSBD_O_TR_WARP, 0, 0.0, gk, gp, gk < NEAR_TIE || gp < NEAR_TIE);
        }
        o->layer_width[(int64_t)r * (gamma + 1) + gamma] = W_nom;
        for (int32_t k = 0; k < W_nom && !err; ++k) {
            const double u = next_uniform(c, inject, inject_stride, &inject_pos, rid,
                                          (uint32_t)(gamma + 1), 3u, (uint32_t)k);
            double lo = 0, hi = 0, z = 0;
            const int64_t cell = draw_cell(p_beam, cells, u, &lo, &hi, &z);
            if (cell < 0) { err = DSBD_O_ERR_EXHAUSTED; break; }
            trace_push(c, gamma + 1, DSBD_O_TR_EXTRA, k, u, lo, hi,
                       (u - lo < NEAR_TIE) || (hi - u < NEAR_TIE));
            dist_push(c, p_beam, cells, z);
            emit(c, r, &n_out, A[cell / V], -1, (int32_t)(cell % V), DSBD_O_SRC_EXTRA,
                 tree_of, &err);
        }
        o->l_last[r] = gamma + 1;
        free(p_beam);
    }
    o->out_width[r] = n_out;
    o->error[r] = err;
    free(A); free(S); free(keys); free(acc);
}

int dsbd_oracle_verify_step(const dsbd_oracle_forest *f, const dsbd_oracle_params *prm,
                            const float *logits_p, const float *logits_q, int64_t row_stride,
                            const double *root_logp, const double *root_logq,
                            const double *inject_u, int64_t inject_stride,
                            dsbd_oracle_verify_out *out, int32_t threads)
{
    if (prm->V <= 0 || !(prm->temperature > 0.0) || row_stride < prm->V)
        return DSBD_O_ERR_BAD_FOREST;
    int32_t *depth = (int32_t *)malloc(sizeof(int32_t) * (size_t)(f->N + 1));
    int32_t *tree_of = (int32_t *)malloc(sizeof(int32_t) * (size_t)(f->N + 1));
    int rc = forest_depths(f, depth, tree_of);
    if (rc) { free(depth); free(tree_of); return rc; }

    const int want_trace = out->trace_req != NULL;
    const int want_dist = out->dist != NULL;
    req_ctx *ctx = (req_ctx *)calloc((size_t)f->R, sizeof(req_ctx));
    (void)threads;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) num_threads(threads > 0 ? threads : 1)
#endif
    for (int32_t r = 0; r < f->R; ++r) {
        req_ctx *c = &ctx[r];
        c->f = f; c->prm = prm; c->zp = logits_p; c->zq = logits_q; c->stride = row_stride;
        c->out = out;
        if (want_trace) {
            c->tcap = 64;
            c->t_layer = (int32_t *)malloc(sizeof(int32_t) * 64);
            c->t_kind = (int32_t *)malloc(sizeof(int32_t) * 64);
            c->t_index = (int32_t *)malloc(sizeof(int32_t) * 64);
            c->t_near = (int32_t *)malloc(sizeof(int32_t) * 64);
            c->t_u = (double *)malloc(sizeof(double) * 64);
            c->t_a = (double *)malloc(sizeof(double) * 64);
            c->t_b = (double *)malloc(sizeof(double) * 64);
        }
        if (want_dist) { c->dcap = 1024; c->dbuf = (double *)malloc(sizeof(double) * 1024); }
        verify_request(c, r, depth, tree_of, root_logp, root_logq,
                       inject_u ? inject_u + (int64_t)r * inject_stride : NULL, inject_stride);
    }
    /* gather the per-request traces in request order */
    int64_t tl = 0, dl = 0;
    for (int32_t r = 0; r < f->R; ++r) {
        req_ctx *c = &ctx[r];
        if (want_trace) {
            for (int64_t i = 0; i < c->tlen; ++i, ++tl) {
                if (tl >= out->trace_cap) continue;
                out->trace_req[tl] = r; out->trace_layer[tl] = c->t_layer[i];
                out->trace_kind[tl] = c->t_kind[i]; out->trace_index[tl] = c->t_index[i];
                out->trace_near[tl] = c->t_near[i]; out->trace_u[tl] = c->t_u[i];
                out->trace_a[tl] = c->t_a[i]; out->trace_b[tl] = c->t_b[i];
            }
            free(c->t_layer); free(c->t_kind); free(c->t_index); free(c->t_near);
            free(c->t_u); free(c->t_a); free(c->t_b);
        }
        if (want_dist) {
            for (int64_t i = 0; i < c->dlen; ++i, ++dl)
                if (dl < out->dist_cap) out->dist[dl] = c->dbuf[i];
            free(c->dbuf);
        }
    }
    if (want_trace) *out->trace_len = tl;
    if (want_dist) *out->dist_len = dl;
    free(ctx); free(depth); free(tree_of);
    return 0;
}

int dsbd_oracle_select_width(const dsbd_oracle_forest *f, const dsbd_oracle_params *prm,
                             const float *logits_p, const float *logits_q, int64_t row_stride,
                             const double *node_logp, const double *node_logq,
                             const int32_t *live_off, const int32_t *live_nodes,
                             const int32_t *m, int32_t *width, double *alpha, double *tail,
                             int32_t alpha_stride)
{
    const int32_t V = prm->V;
    const double tau = prm->temperature;
    double *lse_p = (double *)calloc((size_t)f->N, sizeof(double));
    double *lse_q = (double *)calloc((size_t)f->N, sizeof(double));
    for (int32_t r = 0; r < f->R; ++r) {
        const int32_t *A = live_nodes + live_off[r];
        const int32_t nA = live_off[r + 1] - live_off[r];
        const int32_t mr = m[r];
        const int32_t W_min = prm->W_min_r ? prm->W_min_r[r] : prm->W_min;
        const int32_t W_max = prm->W_max_r ? prm->W_max_r[r] : prm->W_max;
        for (int32_t i = 0; i < nA; ++i) {
            lse_p[A[i]] = row_lse(logits_p + (int64_t)A[i] * row_stride, V, tau);
            lse_q[A[i]] = row_lse(logits_q + (int64_t)A[i] * row_stride, V, tau);
        }
        const int64_t cells = (int64_t)nA * V;
        double *p_beam = (double *)malloc(sizeof(double) * (size_t)(cells + 1));
        double *q_beam = (double *)malloc(sizeof(double) * (size_t)(cells + 1));
        beam_distribution(logits_p, row_stride, V, tau, A, nA, node_logp, lse_p, p_beam);
        beam_distribution(logits_q, row_stride, V, tau, A, nA, node_logq, lse_q, q_beam);
        dsbd_oracle_warp(p_beam, cells, prm->top_k, prm->top_p, NULL, NULL);
        dsbd_oracle_warp(q_beam, cells, prm->top_k, prm->top_p, NULL, NULL);
        double *al = (double *)malloc(sizeof(double) * (size_t)(mr + 1));
        double *P = (double *)malloc(sizeof(double) * (size_t)(mr + 1) * (size_t)(mr + 1));
        double *G = (double *)malloc(sizeof(double) * (size_t)(mr + 2));
        dsbd_oracle_alpha_chain(p_beam, q_beam, cells, mr, al);
        const int32_t wt = dsbd_oracle_width_dp(al, mr, prm->thresh, P, G);
        int32_t W = wt > W_min ? wt : W_min;
        if (W > W_max) W = W_max;
        width[r] = W;
        if (alpha) for (int32_t j = 0; j < mr && j < alpha_stride; ++j)
            alpha[(int64_t)r * alpha_stride + j] = al[j];
        if (tail) for (int32_t j = 0; j <= mr && j < alpha_stride; ++j)
            tail[(int64_t)r * alpha_stride + j] = G[j];
        free(p_beam); free(q_beam); free(al); free(P); free(G);
    }
    free(lse_p); free(lse_q);
    return 0;
}

/* ------------------------------------------------------------------ draft stage ------ */
/* One step of the small model's beam sampling (Section "Overview": beam sampling of width W_S
 * for gamma steps; Section "Details": every draft beam is a sample of
 * q_beam = T o (q / Q) over (current beams x V)).  Request r owns the current beams
 * req_beam_off[r] .. req_beam_off[r+1]) with cumulative scores beam_logq and logits rows
 * logits_q; it draws W_S iid cells by inverse CDF in canonical order, draw k with the uniform
 * of (request, layer 2^29 + layer, purpose 3, index k).  Outputs per draw: the beam it extends
 * (global index), the token, the new cumulative score; optional cdf_lo / cdf_hi (the cell's CDF
 * interval, for near-tie accounting). */
int dsbd_oracle_draft_layer(int32_t R, const int32_t *req_beam_off, const dsbd_oracle_params *prm,
                            int32_t layer, const int32_t *W_S_r, int32_t W_S,
                            const float *logits_q, int64_t row_stride, const double *beam_logq,
                            const double *inject_u, int64_t inject_stride,
                            const int32_t *out_off, int32_t *out_parent, int32_t *out_token,
                            double *out_logq, double *cdf_lo, double *cdf_hi, int32_t *error)
{
    if (prm->V <= 0 || !(prm->temperature > 0.0) || row_stride < prm->V) return DSBD_O_ERR_BAD_FOREST;
    const int32_t V = prm->V;
    const double tau = prm->temperature;
    for (int32_t r = 0; r < R; ++r) {
        const int32_t b0 = req_beam_off[r], nA = req_beam_off[r + 1] - b0;
        const int32_t W = W_S_r ? W_S_r[r] : W_S;
        const uint32_t rid = prm->req_id ? (uint32_t)prm->req_id[r] : (uint32_t)r;
        error[r] = 0;
        if (nA <= 0) { if (W > 0) error[r] = DSBD_O_ERR_EXHAUSTED; continue; }
        if (out_off[r + 1] - out_off[r] < W) { error[r] = DSBD_O_ERR_CAPACITY; continue; }
        const int64_t cells = (int64_t)nA * V;
        int32_t *A = (int32_t *)malloc(sizeof(int32_t) * (size_t)nA);
        double *lse = (double *)malloc(sizeof(double) * (size_t)(b0 + nA));
        double *q_beam = (double *)malloc(sizeof(double) * (size_t)cells);
        for (int32_t i = 0; i < nA; ++i) {
            A[i] = b0 + i;
            lse[b0 + i] = row_lse(logits_q + (int64_t)(b0 + i) * row_stride, V, tau);
        }
        beam_distribution(logits_q, row_stride, V, tau, A, nA, beam_logq, lse, q_beam);
        if (prm->top_k > 0 || (prm->top_p > 0.0 && prm->top_p < 1.0))
            dsbd_oracle_warp(q_beam, cells, prm->top_k, prm->top_p, NULL, NULL);
        for (int32_t k = 0; k < W; ++k) {
            double u;
            if (inject_u) u = k < inject_stride ? inject_u[(int64_t)r * inject_stride + k] : 0.5;
            else u = dsbd_oracle_uniform(prm->seed, prm->step, rid, (1u << 29) + (uint32_t)layer, 3u, (uint32_t)k);
            double lo = 0, hi = 0, z = 0;
            const int64_t cell = draw_cell(q_beam, cells, u, &lo, &hi, &z);
            if (cell < 0) { error[r] = DSBD_O_ERR_EXHAUSTED; break; }
            const int32_t a = A[cell / V], tok = (int32_t)(cell % V);
            const int64_t s = out_off[r] + k;
            out_parent[s] = a;
            out_token[s] = tok;
            out_logq[s] = beam_logq[a] + ((double)logits_q[(int64_t)a * row_stride + tok] / tau - lse[a]);
            if (cdf_lo) cdf_lo[s] = lo;
            if (cdf_hi) cdf_hi[s] = hi;
        }
        free(A); free(lse); free(q_beam);
    }
    return 0;
}
