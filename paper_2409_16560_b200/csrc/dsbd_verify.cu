// dsbd_verify_step / dsbd_select_width: the verification step of speculative beam decoding
// (Algorithm 1 with the dynamic layer width) for sm_100a.
//
// Kernels
//   k_tile_stats   one dense streaming pass over every logits row of both models: per
//                  1024-token tile the row maximum and sum of exponentials (warp-autonomous,
//                  128-bit loads, warp-shuffle reductions).  HBM-bound; this is the pass the
//                  algorithmic bytes 8*N*V belong to.
//   k_row_finish   per row: log-sum-exp from the tile statistics (dsbd_node_stats and
//                  dsbd_select_width; dsbd_verify_step does this inside k_verify).
//   k_verify       one thread-block cluster per request.  Prologue: log-sum-exp of the request's
//                  rows, log-prob of every draft token, cumulative beam scores.  Then layer by
//                  layer: live set and beam weights; ONE pass over the live rows that builds a
//                  fixed-point histogram of the cells' ratios p_beam/q_beam, from which all the
//                  residual masses c_{j+1} = F(s_j) of the layer follow without touching the
//                  rows again; the acceptance-count recursion; the accept loop; the
//                  inverse-CDF completion draws.
//
// The residual chain uses the closed form of the paper's recursion p_{k+1} = norm(max(p_k -
// q_beam, 0)):  with F(s) = sum max(p_beam - s q_beam, 0), c_1 = 1, s_0 = 0, s_j = s_{j-1} + c_j
// and c_{j+1} = F(s_j) one has p_j = max(p_beam - s_{j-1} q_beam, 0) / c_j, hence
// alpha_j = 1 - c_{j+1}/c_j and the accept ratio of a draft x at run position j is
// max(rho(x) - s_{j-1}, 0) / c_j with rho = p_beam(x)/q_beam(x).  F(s) = P(rho > s) - s Q(rho > s)
// only needs the p and q mass above a ratio threshold, which is what the histogram holds; the
// one bin that s falls into is bracketed from its two sums and its edges, and when half the
// bracket plus the bound on the histogram's fixed-point error exceeds 2.5e-7 that F(s_j) is
// recomputed exactly by a pass over the rows.
//
// Building with -DDSBD_PHASE_TIMING makes k_verify record %globaltimer stamps of its phases at
// the end of the workspace (a tuning aid; off in normal builds).
#include <cooperative_groups.h>
#include <math.h>

#include "dsbd_common.cuh"

namespace cg = cooperative_groups;
using namespace dsbd;

namespace {

constexpr int kTile = 1024;          // tokens per tile: 32 lanes x 8 x float4
constexpr int kThreads = 256;        // streaming kernels
constexpr int kWarps = kThreads / 32;
constexpr int kVThreads = 512;       // the per-request kernel: two CTAs of 16 warps per SM
constexpr int kVWarps = kVThreads / 32;
constexpr int kMaxLive = DSBD_MAX_LIVE;
constexpr float kLog2e = 1.4426950408889634f;
constexpr double kLn2 = 0.6931471805599453;

struct TileStat { float mx; float sum; };   // max of the raw logits, sum exp((z-mx)/tau)

__device__ __forceinline__ void load_tile(const float *__restrict__ row, int e0, int V, bool aligned,
                                          int lane, float4 (&v)[8]) {
    const float ninf = -INFINITY;
#pragma unroll
    for (int it = 0; it < 8; ++it) {
        const int e = e0 + it * 128 + lane * 4;
        if (aligned && e + 3 < V) {
            v[it] = ldg_stream(reinterpret_cast<const float4 *>(row + e));
        } else {
            v[it].x = e < V ? __ldg(row + e) : ninf;
            v[it].y = e + 1 < V ? __ldg(row + e + 1) : ninf;
            v[it].z = e + 2 < V ? __ldg(row + e + 2) : ninf;
            v[it].w = e + 3 < V ? __ldg(row + e + 3) : ninf;
        }
    }
}

__device__ __forceinline__ void load_half_tile(const float *__restrict__ row, int e0, int V, bool aligned,
                                               int lane, float4 (&v)[4]) {
    const float ninf = -INFINITY;
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const int e = e0 + it * 128 + lane * 4;
        if (aligned && e + 3 < V) {
            v[it] = ldg_stream(reinterpret_cast<const float4 *>(row + e));
        } else {
            v[it].x = e < V ? __ldg(row + e) : ninf;
            v[it].y = e + 1 < V ? __ldg(row + e + 1) : ninf;
            v[it].z = e + 2 < V ? __ldg(row + e + 2) : ninf;
            v[it].w = e + 3 < V ? __ldg(row + e + 3) : ninf;
        }
    }
}

// ---------------------------------------------------------------------------------------
// Dense pass: tile statistics of every (model, row).  Item = (model, row, tile), tile fastest,
// one warp per item.  rows == nullptr: all n_rows rows; else the listed rows (n_rows read
// from *n_rows_dev when it is given, never more than the n_rows the launch was sized for; a
// listed row outside [0, N) is skipped -- the kernel that consumes the list reports it).
// ---------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
k_tile_stats(const float *__restrict__ zp, const float *__restrict__ zq, int64_t stride, int V,
             int T, int N, int n_rows, const int32_t *__restrict__ rows,
             const int32_t *__restrict__ n_rows_dev, float k2, TileStat *__restrict__ stats,
             int one_model = 0) {
    // one_model: zq is the same tensor as zp; read it once and store the statistics for both
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    if (n_rows_dev) n_rows = min(max(*n_rows_dev, 0), n_rows);
    const int64_t total = (int64_t)(one_model ? 1 : 2) * n_rows * T;
    for (int64_t item = warp; item < total; item += nwarps) {
        const int t = (int)(item % T);
        const int64_t rm = item / T;
        const int model = (int)(rm / n_rows);
        const int ri = (int)(rm % n_rows);
        const int row = rows ? rows[ri] : ri;
        if (row < 0 || row >= N) continue;
        const float *z = (model ? zq : zp) + (int64_t)row * stride;
        const bool aligned = (reinterpret_cast<uintptr_t>(z) & 15) == 0;
        float4 v[8];
        load_tile(z, t * kTile, V, aligned, lane, v);
        float mx = -INFINITY;
#pragma unroll
        for (int it = 0; it < 8; ++it)
            mx = fmaxf(mx, fmaxf(fmaxf(v[it].x, v[it].y), fmaxf(v[it].z, v[it].w)));
        mx = warp_max(mx);
        float sum = 0.f;
        if (mx > -INFINITY) {
            const float b = -mx * k2;
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                sum += exp2f(fmaf(v[it].x, k2, b)) + exp2f(fmaf(v[it].y, k2, b)) +
                       exp2f(fmaf(v[it].z, k2, b)) + exp2f(fmaf(v[it].w, k2, b));
            }
        }
        sum = warp_sum(sum);
        if (lane == 0) {
            TileStat s; s.mx = mx; s.sum = sum;
            stats[((int64_t)model * N + row) * T + t] = s;
            if (one_model) stats[((int64_t)N + row) * T + t] = s;
        }
    }
}

// log-sum-exp of a tempered row from its tile statistics, by one warp (same value on every lane;
// the order of the sums depends on T only).
__device__ __forceinline__ double row_lse(const TileStat *s, int T, double inv_tau, int lane) {
    double mx = -INFINITY;
    for (int t = lane; t < T; t += 32) mx = fmax(mx, (double)s[t].mx);
    mx = warp_max(mx);
    double acc = 0.0;
    if (mx > -INFINITY)
        for (int t = lane; t < T; t += 32)
            if (s[t].sum > 0.f) acc += (double)s[t].sum * exp(((double)s[t].mx - mx) * inv_tau);
    acc = warp_sum(acc);
    return (mx > -INFINITY) ? mx * inv_tau + log(acc) : -INFINITY;
}

// log-sum-exp of the tempered row from its tile statistics; one warp per (model, row).
__global__ void k_row_finish(const TileStat *__restrict__ stats, int T, int N, int n_rows,
                             const int32_t *__restrict__ rows, const int32_t *__restrict__ n_rows_dev,
                             double inv_tau, double *__restrict__ lse /*[2][N]*/,
                             float *__restrict__ lse_p_out, float *__restrict__ lse_q_out) {
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (n_rows_dev) n_rows = min(max(*n_rows_dev, 0), n_rows);
    if (warp >= (int64_t)2 * n_rows) return;
    const int model = (int)(warp / n_rows);
    const int ri = (int)(warp % n_rows);
    const int row = rows ? rows[ri] : ri;
    if (row < 0 || row >= N) return;
    const double v = row_lse(stats + ((int64_t)model * N + row) * T, T, inv_tau, lane);
    if (lane == 0) {
        lse[(int64_t)model * N + row] = v;
        if (model == 0 && lse_p_out) lse_p_out[row] = (float)v;
        if (model == 1 && lse_q_out) lse_q_out[row] = (float)v;
    }
}

// ---------------------------------------------------------------------------------------
// The per-request kernel.
// ---------------------------------------------------------------------------------------
struct VerifyArgs {
    // forest
    int R, N, gamma;
    const int32_t *req_beam_off, *beam_node_off, *parent, *token, *draft_rank;
    // parameters
    int V, T;
    float k2;                 // log2(e)/tau
    double inv_tau, thresh;
    int W_min, W_max, W_nom;
    const int32_t *W_min_r, *W_max_r, *W_nom_r;
    uint64_t seed, step;
    int top_k;                // 0: unwarped joints
    double top_p;             // outside (0,1): off
    // inputs
    const float *zp, *zq;
    int64_t stride;
    // workspace
    const TileStat *stats;    // [2][N][T]
    const double *lse;        // [2][N]
    const double *score;      // [2][N]
    const int32_t *depth;     // [N]
    double *tile_sums;        // [R][2][max_m][max_live*T]
    unsigned long long *hist; // [R][2 banks][kBins+1] fixed-point ratio histograms (p<<32 | q)
    unsigned long long *dbg;  // phase time stamps (DSBD_PHASE_TIMING builds only)
    // verify mode computes the row and tree statistics of its own request first
    double *lse_w, *score_w;
    int32_t *depth_w;
    const float *root_logp, *root_logq;
    int max_m, max_live;
    int check_widths;            // verification / width selection: per-request widths are validated
    uint32_t extra_layer_bias;   // added to the layer number in the Philox counter of the extra layer
    // outputs
    dsbd_verify_out_t out;
    int32_t *status;
    // select-width mode
    int select_mode;
    const float *sel_logp, *sel_logq;
    const int32_t *live_off, *live_nodes, *m_in;
    int sel_rows;             // list entries the dense pass was sized for
    int32_t *width_out;
    float *alpha_out, *tail_out;
    int out_stride;
};

struct Shared {
    int nA, m, W, count, done, chain_len, err;
    int A[kMaxLive];
    int S[kMaxLive];
    int S_parent_idx[kMaxLive];
    int acc[kMaxLive];
    // log2 of (beam weight / sum of the row's exponentials), split so that the cell masses do not
    // inherit the rounding of one large float: bp/bq hold the nearest integer (exact in fp32), cp/cq
    // the factor 2^(remainder) in [2^-0.5, 2^0.5], dc = log2(cp/cq)
    float bp[kMaxLive], bq[kMaxLive], cp[kMaxLive], cq[kMaxLive], dc[kMaxLive];
    double lwp[kMaxLive], lwq[kMaxLive];    // natural log of the beam weights
    double wp[kMaxLive];
    double s_arr[kMaxLive + 2];             // s_0 .. s_m
    double c_arr[kMaxLive + 2];             // c_1 .. c_{m+1} (index j)
    double alpha[kMaxLive + 1];
    double first[kMaxLive + 1];             // alpha_i prod_{j<i}(1-alpha_j)
    double col_a[kMaxLive + 1], col_b[kMaxLive + 1];
    double tail[kMaxLive + 2];
    int bank, need_exact, res_j, run_j, chain_pos;
    int n_out, n_fill;                      // output beams so far; p_beam fills left to the whole CTA
    int n_layers, n_tests, n_exact, n_respass;
    int n_near, n_rows;                     // accept tests inside the 1e-5 tie band; live rows consulted
    unsigned long long wtot_p[kVWarps], wtot_q[kVWarps];
    double n_cells;                         // cells that entered the layer's histogram
    unsigned long long w_tot[10];           // sums of one histogram pass: see histogram_pass / hist_merge
    int wrapped, n_wrapped;                 // a w word of the layer's histogram wrapped; layers where that happened
    double rho[kMaxLive], uu[kMaxLive];     // per live draft: p_beam/q_beam and its uniform
};

// mass of one cell of the residual max(p_beam - s q_beam, 0); s == 0 gives p_beam
struct RowOff { float bp, bq, cp, cq, dc; };
__device__ __forceinline__ float cell_mass(float zp, float zq, float k2, const RowOff &o, float s) {
    const float a = exp2f(fmaf(zp, k2, o.bp)) * o.cp;
    const float b = exp2f(fmaf(zq, k2, o.bq)) * o.cq;
    return fmaxf(fmaf(-s, b, a), 0.f);
}
// Splits b = log2(weight) - lse*log2(e) (double) into its nearest integer and the factor 2^(rest).
__device__ __forceinline__ void split_offset(double b, float *bi, float *c, double *rest) {
    if (b == b && fabs(b) < 1e30) {
        const double r = rint(b);
        *bi = (float)r; *c = (float)exp2(b - r); *rest = b - r;
    } else {
        *bi = (float)b; *c = 1.f; *rest = 0.0;
    }
}

// One cluster-wide pass: tile sums of max(p_beam - s q_beam, 0) over the live rows.
__device__ void residual_pass(const VerifyArgs &a, const Shared &sh, float s, double *sums,
                              int cta_rank, int n_cta) {
    const int lane = threadIdx.x & 31;
    const int warp = cta_rank * kVWarps + (threadIdx.x >> 5);
    const int nwarps = n_cta * kVWarps;
    const int items = sh.nA * a.T;
    for (int item = warp; item < items; item += nwarps) {
        const int i = item / a.T, t = item - i * a.T;
        const int row = sh.A[i];
        const float *rp = a.zp + (int64_t)row * a.stride;
        const float *rq = a.zq + (int64_t)row * a.stride;
        const bool al = ((reinterpret_cast<uintptr_t>(rp) | reinterpret_cast<uintptr_t>(rq)) & 15) == 0;
        const RowOff ro = {sh.bp[i], sh.bq[i], sh.cp[i], sh.cq[i], sh.dc[i]};
        float acc = 0.f;
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            float4 vp[4], vq[4];
            load_half_tile(rp, t * kTile + half * (kTile / 2), a.V, al, lane, vp);
            load_half_tile(rq, t * kTile + half * (kTile / 2), a.V, al, lane, vq);
#pragma unroll
            for (int it = 0; it < 4; ++it) {
                acc += cell_mass(vp[it].x, vq[it].x, a.k2, ro, s);
                acc += cell_mass(vp[it].y, vq[it].y, a.k2, ro, s);
                acc += cell_mass(vp[it].z, vq[it].z, a.k2, ro, s);
                acc += cell_mass(vp[it].w, vq[it].w, a.k2, ro, s);
            }
        }
        const double tot = warp_sum((double)acc);
        if (lane == 0) sums[item] = tot;
    }
}

// Ordered sum of n doubles by one warp: lane-strided partial sums, then a butterfly.  The
// order depends on n only, never on the launch shape.
__device__ double ordered_sum(const double *v, int n, int lane) {
    double acc = 0.0;
    for (int i = lane; i < n; i += 32) acc += __ldcg(v + i);
    return warp_sum(acc);
}

// Inverse-CDF search over tile masses (canonical order).  mass(i) must be the same on every
// lane.  Returns the tile holding the first cell whose running sum reaches target, and the
// mass before that tile; if rounding leaves the target beyond the total, the last tile with
// mass.  -1 if there is no mass at all.
template <class F>
__device__ int locate_tile(F mass, int n, double target, int lane, double *before) {
    double running = 0.0, last_before = 0.0;
    int last = -1;
    for (int base = 0; base < n; base += 32) {
        const int i = base + lane;
        const double v = i < n ? mass(i) : 0.0;
        const double incl = warp_scan(v, lane);
        const bool hit = v > 0.0 && running + incl >= target;
        const unsigned hits = __ballot_sync(kFull, hit);
        if (hits) {
            const int l = __ffs(hits) - 1;
            *before = running + __shfl_sync(kFull, incl - v, l);
            return base + l;
        }
        const unsigned pos = __ballot_sync(kFull, v > 0.0);
        if (pos) {
            const int l = 31 - __clz(pos);
            last = base + l;
            last_before = running + __shfl_sync(kFull, incl - v, l);
        }
        running += __shfl_sync(kFull, incl, 31);
    }
    *before = last_before;
    return last;
}

// Inverse-CDF search inside one tile of row `row` (and its q row when s > 0): the first
// token whose running mass reaches `target`, else the last token with mass.  -1: no mass.
__device__ int locate_token(const VerifyArgs &a, int row, int t, const RowOff &ro, float s,
                            double target, int lane) {
    const float *rp = a.zp + (int64_t)row * a.stride;
    const float *rq = a.zq + (int64_t)row * a.stride;
    double running = 0.0;
    int last = -1;
    for (int it = 0; it < 8; ++it) {
        const int e = t * kTile + it * 128 + lane * 4;
        float mss[4];
        double loc = 0.0;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            float mv = 0.f;
            if (e + c < a.V) {
                const float zpv = __ldg(rp + e + c);
                mv = (s > 0.f) ? cell_mass(zpv, __ldg(rq + e + c), a.k2, ro, s)
                               : exp2f(fmaf(zpv, a.k2, ro.bp)) * ro.cp;
            }
            mss[c] = mv;
            loc += (double)mv;
        }
        const double incl = warp_scan(loc, lane);
        const bool hit = loc > 0.0 && running + incl >= target;
        const unsigned hits = __ballot_sync(kFull, hit);
        if (hits) {
            const int l = __ffs(hits) - 1;
            int tok = -1;
            if (lane == l) {
                double cum = running + incl - loc;
                int lastpos = -1;
                for (int c = 0; c < 4; ++c) {
                    cum += (double)mss[c];
                    if (mss[c] > 0.f) {
                        lastpos = c;
                        if (cum >= target) { tok = e + c; break; }
                    }
                }
                if (tok < 0) tok = e + lastpos;
            }
            return __shfl_sync(kFull, tok, l);
        }
        const unsigned pos = __ballot_sync(kFull, loc > 0.0);
        if (pos) {
            const int l = 31 - __clz(pos);
            int lp = -1;
            if (lane == l)
                for (int c = 0; c < 4; ++c) if (mss[c] > 0.f) lp = e + c;
            last = __shfl_sync(kFull, lp, l);
        }
        running += __shfl_sync(kFull, incl, 31);
    }
    return last;
}

// Writes output beam number `index` of request r (the caller has checked the slot range).
__device__ void emit_at(const VerifyArgs &a, int r, int index, int parent, int node, int tok, int source) {
    {
        const int s = a.out.out_off[r] + index;
        // the tree of a node: walk to the root, then find which beam starts there
        int root = parent;
        while (a.parent[root] >= 0) root = a.parent[root];
        int lo = a.req_beam_off[r], hi = a.req_beam_off[r + 1];
        int beam = lo;
        for (int b = lo; b < hi; ++b) if (a.beam_node_off[b] == root) beam = b;
        a.out.out_parent[s] = parent;
        a.out.out_node[s] = node;
        a.out.out_root_beam[s] = beam;
        a.out.out_token[s] = tok;
        a.out.out_source[s] = source;
        const double lp = (double)a.zp[(int64_t)parent * a.stride + tok] * a.inv_tau - a.lse[parent];
        const double lq = (double)a.zq[(int64_t)parent * a.stride + tok] * a.inv_tau - a.lse[a.N + parent];
        a.out.out_logp[s] = (float)(a.score[parent] + lp);
        a.out.out_logq[s] = (float)(a.score[a.N + parent] + lq);
    }
}

__device__ void emit_output(const VerifyArgs &a, int r, int *n_out, int parent, int node, int tok,
                            int source, bool writer, int *err) {
    const int cap = a.out.out_off[r + 1] - a.out.out_off[r];
    if (*n_out >= cap) { *err = DSBD_DEV_CAPACITY; return; }
    if (writer) emit_at(a, r, *n_out, parent, node, tok, source);
    (*n_out)++;
}

// Beam weights of the live set: softmax of the cumulative scores over A (Eq. 1 factorised).
// Called by all lanes of one warp; beam i is handled by lane i % 32.
// Per-node data of the request that every layer's set-up reads, kept in shared memory when the
// request is small enough (otherwise the set-up reads the global arrays).
constexpr int kCacheNodes = 256;
struct NodeCache {
    double score_p[kCacheNodes], score_q[kCacheNodes], lse_p[kCacheNodes], lse_q[kCacheNodes];
    int16_t parent[kCacheNodes];          // local index of the parent, -1 for a root
    uint8_t depth[kCacheNodes];
    int on;
};

// Natural log of the softmax of n scores, by one warp (lanes over the scores).
__device__ __forceinline__ void log_softmax_warp(const double *s, int n, int lane, double *out) {
    double mx = -INFINITY;
    for (int i = lane; i < n; i += 32) mx = fmax(mx, s[i]);
    mx = warp_max(mx);
    double t = 0.0;
    for (int i = lane; i < n; i += 32) t += exp(s[i] - mx);
    t = warp_sum(t);
    const double lt = log(t);
    for (int i = lane; i < n; i += 32) out[i] = (s[i] - mx) - lt;
    __syncwarp();
}

// nc: the request's node cache or nullptr; n_lo: first node of the request.
__device__ void live_weights(const VerifyArgs &a, Shared &sh, const double *sp, const double *sq, int lane,
                             const NodeCache *nc = nullptr, int n_lo = 0) {
    log_softmax_warp(sp, sh.nA, lane, sh.lwp);
    log_softmax_warp(sq, sh.nA, lane, sh.lwq);
    for (int i = lane; i < sh.nA; i += 32) {
        const double lwp = sh.lwp[i], lwq = sh.lwq[i];
        sh.wp[i] = exp(lwp);
        const int row = sh.A[i];
        double rest_p, rest_q;
        const double lse_p = nc ? nc->lse_p[row - n_lo] : a.lse[row];
        const double lse_q = nc ? nc->lse_q[row - n_lo] : a.lse[a.N + row];
        split_offset((lwp - lse_p) / kLn2, &sh.bp[i], &sh.cp[i], &rest_p);
        split_offset((lwq - lse_q) / kLn2, &sh.bq[i], &sh.cq[i], &rest_q);
        sh.dc[i] = (float)(rest_p - rest_q);
    }
    __syncwarp();
}

// Acceptance-count recursion by one warp (lanes over n): tail[K] = P(at least K accepts),
// returns W~ = max{K : tail[K] >= thresh}.
// k_stop >= 0: stop once W = min(W_max = k_stop, max(W_min, W~)) is decided; -1: the whole tail
__device__ int width_rule(Shared &sh, int m, double thresh, int lane, int k_stop) {
    if (lane == 0) {
        double none = 1.0;
        for (int i = 1; i <= m; ++i) {
            sh.first[i] = sh.alpha[i] * none;
            none *= (1.0 - sh.alpha[i]);
            sh.col_a[i] = none;                    // P(n, 0) = prod_{j<=n}(1 - alpha_j)
        }
        sh.col_a[0] = 1.0;
        sh.tail[0] = 1.0;
    }
    __syncwarp();
    double *prev = sh.col_a, *cur = sh.col_b;
    double below = 0.0;
    for (int k = 0; k <= m; ++k) {
        // prev = P(., k); record tail
        below += prev[m];
        if (lane == 0) sh.tail[k + 1] = 1.0 - below;
        if (k == m) break;
        // tails only fall: past the first one below the threshold, or past the cap, nothing changes W
        if (k_stop >= 0 && (1.0 - below < thresh || k + 1 >= k_stop)) {
            for (int K = k + 2 + lane; K <= m + 1; K += 32) sh.tail[K] = 0.0;
            break;
        }
        for (int n = lane; n <= m; n += 32) {
            double acc = 0.0;
            if (n >= k + 1)
                for (int i = 1; i <= n; ++i) acc += sh.first[i] * prev[n - i];
            cur[n] = acc;                          // P(n, k+1), zero for n < k+1
        }
        __syncwarp();
        double *tmp = prev; prev = cur; cur = tmp;
    }
    __syncwarp();
    int wt = 0;
    for (int K = 0; K <= m; ++K) if (sh.tail[K] >= thresh) wt = K;
    if (lane == 0) sh.tail[m + 1] = 0.0;
    return wt;
}

// ---------------------------------------------------------------------------------------
// Ratio histogram of one layer.  Every cell with rho = p_beam/q_beam > 1 adds its p and q mass to
// the bin of log2(rho); bin kBins collects rho beyond the last edge.  F(s) for any s in [1, top]
// is then (sum of the bins above s) plus the straddled bin, whose contribution is bracketed from
// its two sums and its edges.
//
// Masses are summed as integers in units of 2^-44, so the sums do not depend on the order in which
// warps and CTAs add, and a cell of mass >= 2^-20 enters without any rounding (its 24-bit
// mantissa is a whole number of units); a smaller cell is rounded by at most 2^-45.  With n cells
// the fixed-point error of any partial sum is therefore at most n 2^-45 (2.8e-8 for a million
// cells), which the chain adds to its bracket.
// In shared memory a bin has two 32-bit words per model, fed by plain (non-returning) atomic adds:
//   w: units of 2^-44.  A cell below 2^-16 adds all of itself here (less than 2^28 units); a larger
//      cell only its remainder below 2^-28 (less than 2^16 units).
//   b: units of 2^-28, the whole multiples of 2^-28 of the cells of at least 2^-16; it cannot
//      overflow because a joint distribution sums to one.
// A w word wraps once the small cells of ONE bin that ONE CTA added reach 2^-12 of the mass --
// twenty times what a bin holds in ordinary data, but possible when the two models' rows are
// proportional and every cell lands in the same bin.  A wrap is detected exactly: every thread
// keeps the 64-bit total of what it added to the w words, and the CTA compares the sum of those
// totals with the sum of its w words; a difference marks the layer, whose residual masses are
// then all computed by exact passes over the rows.
// ---------------------------------------------------------------------------------------
constexpr int kBins = 4096;
constexpr int kOverSlots = 256;                   // copies of the last bin (rho beyond the last edge): one per
                                                  // warp and half-warp lane, so that none collects enough to wrap
constexpr int kHistWords = kBins + kOverSlots + 16;  // bins 0..kBins-1, the copies of bin kBins, spare words
static_assert(kHistWords % 4 == 0, "the arrays that share this memory need 16-byte alignment");
constexpr float kFix = 17592186044416.f;          // 2^44
constexpr double kUnfix = 1.0 / 17592186044416.0;
constexpr float kBigCell = 1.f / 65536.f;         // 2^-16: cells from here on put their top part into the b word
constexpr float kBigFix = 268435456.f;            // 2^28, the unit of the b word is 2^-28
constexpr double kErrTol = 2.5e-7;                // error bound of F(s) above which it is recomputed exactly
// global image of one histogram: P and Q of bin i at 2i, 2i+1 (units of 2^-44), two spare words
constexpr int kHistLen = 2 * (kBins + 1) + 2;

constexpr int kHistArrays = 4;
struct HistSmem { uint32_t *wp, *wq, *bp, *bq; };

__device__ __forceinline__ HistSmem hist_arrays(uint32_t *base) {
    return HistSmem{base, base + kHistWords, base + 2 * kHistWords, base + 3 * kHistWords};
}

__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Per-thread sums of one histogram pass.
struct PassSums {
    unsigned long long tot;               // what went into the w words (p and q together)
};

// The cells of one half tile (4 x float4 per lane and model) into the histogram; adds their
// (p - q)+, in units of 2^-44, to res1u.
// The work per cell decides the speed of this pass (it is bound by instruction issue, not by
// memory), so the common case is straight-line code: masses are computed directly in units
// (the row's factor 2^rest carries the 2^44), the bin comes from an fma onto 1.5 * 2^23 whose
// low mantissa bits are then the integer (no conversion instruction), the two atomic adds, the
// residual sum and the check sum are predicated on p_beam > q_beam inside one asm block, and only a
// cell of at least 2^-16 (rare) takes a branch.
// wbase: shared-memory byte address of wp[0] minus 4 * (the bits of the fma's constant), so that
// the address of a bin's word is wbase + 4 * (bits of the fma's result); the q array follows the p
// array at kHistWords words, the b arrays at twice that.
// (ex2.approx flushes results below 2^-126 to zero; a cell enters the sums from 2^-45 on.)
constexpr float kBinMagic = 12582912.f;                         // 1.5 * 2^23
constexpr float kBigUnits = 268435456.f;                        // 2^28 units = a cell of 2^-16
__device__ __forceinline__ void hist_half_tile(const float4 (&vp)[4], const float4 (&vq)[4], float k2,
                                               const RowOff &o, float binscale, float half_bin, float top, uint32_t wbase,
                                               float &res1u, PassSums &ps, uint32_t over_bits) {
    // dl = log2(rho) - half: the half bin (in log2 units) that turns the fma's round-to-nearest into
    // the bin's floor is part of the row offset, so p_beam > q_beam reads dl > -half
    const float bd = ((o.bp - o.bq) + o.dc) - half_bin;
    const float pass_thr = -half_bin;
    const float cpu = o.cp * kFix, cqu = o.cq * kFix;           // exact: powers of two
    uint32_t t0 = 0u, t1 = 0u;                                  // each below 2^32: 8 cells x 2 x less than 2^28 units
#pragma unroll
    for (int it = 0; it < 4; ++it) {
        const float zp4[4] = {vp[it].x, vp[it].y, vp[it].z, vp[it].w};
        const float zq4[4] = {vq[it].x, vq[it].y, vq[it].z, vq[it].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const float dl = fmaf(zp4[c] - zq4[c], k2, bd);     // NaN compares false
            float pmu = ex2_approx(fmaf(zp4[c], k2, o.bp)) * cpu;
            float qmu = ex2_approx(fmaf(zq4[c], k2, o.bq)) * cqu;
            const float diff = fmaxf(pmu - qmu, 0.f);
            // floor(log2(rho) * binscale) in the low bits (round to nearest of x - 0.5; an x that is a
            // whole number may fall to either side, both within the bins' edge tolerance)
            const float tb = fmaf(dl, binscale, kBinMagic);
            // (all cells beyond the last edge in one word would wrap it: every warp and half-warp
            // lane has its own copy of that bin)
            const uint32_t bits = dl < top ? __float_as_uint(tb) : over_bits;
            const uint32_t addr = wbase + (bits << 2);
            if (pmu >= kBigUnits && dl > pass_thr) {
                // whole multiples of 2^-28 of a big cell go to the b word (units of 2^-28), the
                // remainder (below 2^16 units) stays for the w word
                const float hp = floorf(pmu * (1.f / 65536.f));
                pmu = fmaf(-hp, 65536.f, pmu);
                asm volatile("red.shared.add.u32 [%0+%1], %2;" ::"r"(addr), "n"(2 * kHistWords * 4), "r"((uint32_t)hp) : "memory");
                if (qmu >= kBigUnits) {
                    const float hq = floorf(qmu * (1.f / 65536.f));
                    qmu = fmaf(-hq, 65536.f, qmu);
                    asm volatile("red.shared.add.u32 [%0+%1], %2;" ::"r"(addr), "n"(3 * kHistWords * 4), "r"((uint32_t)hq) : "memory");
                }
            }
            const uint32_t ap = __float2uint_rn(pmu), aq = __float2uint_rn(qmu);
            uint32_t &tacc = (it < 2) ? t0 : t1;
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "setp.gt.f32 p, %2, %8;\n\t"
                "@p red.shared.add.u32 [%3], %4;\n\t"
                "@p red.shared.add.u32 [%3+%6], %5;\n\t"
                "@p add.f32 %0, %0, %7;\n\t"
                "@p add.u32 %1, %1, %4;\n\t"
                "@p add.u32 %1, %1, %5;\n\t}"
                : "+f"(res1u), "+r"(tacc)
                : "f"(dl), "r"(addr), "r"(ap), "r"(aq), "n"(kHistWords * 4), "f"(diff), "f"(pass_thr)
                : "memory");
        }
    }
    ps.tot += (unsigned long long)t0 + t1;
}

// One cluster-wide pass over the live rows; every CTA fills its own shared-memory histogram.
// tot (shared memory, zero before the call): [0] what the CTA added to its w words (p and q).
__device__ void histogram_pass(const VerifyArgs &a, const Shared &sh, float binscale, const HistSmem &h,
                               double *sums1, int cta_rank, int n_cta, unsigned long long *tot) {
    const int lane = threadIdx.x & 31;
    const int warp = cta_rank * kVWarps + (threadIdx.x >> 5);
    const int nwarps = n_cta * kVWarps;
    const int items = sh.nA * a.T;
    PassSums ps = {0ull};
    const uint32_t magic_bits = __float_as_uint(kBinMagic);
    const uint32_t wbase = (uint32_t)__cvta_generic_to_shared(h.wp) - (magic_bits << 2);
    const uint32_t over_bits = magic_bits + (uint32_t)(kBins + ((threadIdx.x >> 5) & 15) * 16 + (threadIdx.x & 15));
    const float half_bin = 0.5f / binscale;                      // half a bin in log2 units
    const float top = (float)kBins / binscale - half_bin;        // log2 of the last edge (minus the half), as the bins see it
    for (int item = warp; item < items; item += nwarps) {
        const int i = item / a.T, t = item - i * a.T;
        const int row = sh.A[i];
        const float *rp = a.zp + (int64_t)row * a.stride;
        const float *rq = a.zq + (int64_t)row * a.stride;
        const bool al = ((reinterpret_cast<uintptr_t>(rp) | reinterpret_cast<uintptr_t>(rq)) & 15) == 0;
        const RowOff ro = {sh.bp[i], sh.bq[i], sh.cp[i], sh.cq[i], sh.dc[i]};
        float res1u = 0.f;                               // sum of (p - q)+ over the tile in units: residual mass at s = 1
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            float4 vp[4], vq[4];
            const int e0 = t * kTile + half * (kTile / 2);
            load_half_tile(rp, e0, a.V, al, lane, vp);
            load_half_tile(rq, e0, a.V, al, lane, vq);
            hist_half_tile(vp, vq, a.k2, ro, binscale, half_bin, top, wbase, res1u, ps, over_bits);
        }
        // tile sums of the residual after ONE rejection (s_1 = 1): what a completion draw at run
        // position 2 searches, so that this common case needs no second pass over the rows
        const double tot1 = warp_sum((double)res1u) * kUnfix;
        if (lane == 0) sums1[item] = tot1;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) ps.tot += __shfl_xor_sync(kFull, ps.tot, o);
    if (lane == 0 && ps.tot) atomicAdd(tot, ps.tot);
}

// Merge of the cluster's histograms, after a cluster barrier that follows the pass: every CTA sums
// one slice of the bins over all CTAs' shared memory (distributed shared memory loads, no atomics)
// and stores the 64-bit sums, in units of 2^-44, to the global image, which therefore needs no
// clearing; the last CTA also folds the copies of the last bin.  Returns through tot[9] whether
// any CTA's w words wrapped (each CTA checks its own words against what its threads added, tot[0]).
// The caller puts a cluster barrier behind this before anyone reads the image or reuses the arrays.
__device__ void hist_check_local(const HistSmem &h, unsigned long long *tot, unsigned long long *warp_p,
                                 unsigned long long *warp_q) {
    unsigned long long sp = 0ull, sq = 0ull;
    for (int i = threadIdx.x; i < kBins + kOverSlots; i += blockDim.x) { sp += h.wp[i]; sq += h.wq[i]; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        sp += __shfl_xor_sync(kFull, sp, o);
        sq += __shfl_xor_sync(kFull, sq, o);
    }
    if ((threadIdx.x & 31) == 0) { warp_p[threadIdx.x >> 5] = sp; warp_q[threadIdx.x >> 5] = sq; }
    __syncthreads();
    if (threadIdx.x == 0) {
        sp = sq = 0ull;
        for (int w = 0; w < (int)(blockDim.x >> 5); ++w) { sp += warp_p[w]; sq += warp_q[w]; }
        tot[6] = (tot[0] != sp + sq) ? 1ull : 0ull;               // a wrapped word lowers sp + sq by 2^32
    }
}

__device__ void hist_merge(cg::cluster_group &cluster, const HistSmem &h, unsigned long long *gh,
                           unsigned long long *tot, int cta_rank, int n_cta) {
    const int per = (kBins + n_cta - 1) / n_cta;
    const int lo = cta_rank * per, hi = min(lo + per, kBins);
    for (int i = lo + (int)threadIdx.x; i < hi; i += blockDim.x) {
        unsigned long long P = 0ull, Q = 0ull;
        for (int c = 0; c < n_cta; ++c) {
            const uint32_t *wp = cluster.map_shared_rank(h.wp, c), *wq = cluster.map_shared_rank(h.wq, c);
            const uint32_t *bp = cluster.map_shared_rank(h.bp, c), *bq = cluster.map_shared_rank(h.bq, c);
            P += ((unsigned long long)bp[i] << 16) + wp[i];
            Q += ((unsigned long long)bq[i] << 16) + wq[i];
        }
        gh[2 * i] = P;
        gh[2 * i + 1] = Q;
    }
    if (cta_rank == n_cta - 1) {
        // the copies of the last bin (one per warp and half-warp lane, in every CTA) are one bin again
        unsigned long long P = 0ull, Q = 0ull;
        for (int i = kBins + (int)threadIdx.x; i < kBins + kOverSlots; i += blockDim.x)
            for (int c = 0; c < n_cta; ++c) {
                const uint32_t *wp = cluster.map_shared_rank(h.wp, c), *wq = cluster.map_shared_rank(h.wq, c);
                const uint32_t *bp = cluster.map_shared_rank(h.bp, c), *bq = cluster.map_shared_rank(h.bq, c);
                P += ((unsigned long long)bp[i] << 16) + wp[i];
                Q += ((unsigned long long)bq[i] << 16) + wq[i];
            }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            P += __shfl_xor_sync(kFull, P, o);
            Q += __shfl_xor_sync(kFull, Q, o);
        }
        if ((threadIdx.x & 31) == 0 && threadIdx.x < kOverSlots) {
            if (P) atomicAdd(tot + 7, P);
            if (Q) atomicAdd(tot + 8, Q);
        }
        __syncthreads();
        if (threadIdx.x == 0) { gh[2 * kBins] = tot[7]; gh[2 * kBins + 1] = tot[8]; }
    }
    if (threadIdx.x == 0) {
        unsigned long long wrapped = 0ull;
        for (int c = 0; c < n_cta; ++c) wrapped |= cluster.map_shared_rank(tot, c)[6];
        tot[9] = wrapped;
    }
}

// One completion draw (residual if s_res > 0 else p_beam) by warp 0; returns the token or -1
// and the index of the live parent.
__device__ int draw_cell(const VerifyArgs &a, const Shared &sh, double u, bool use_res, float s_res,
                         double z_res, const double *res_sums, int lane, int *ia_out) {
    int tile = -1;
    double before = 0.0, target;
    if (use_res) {
        target = u * z_res;
        tile = locate_tile([&](int i) { return __ldcg(res_sums + i); }, sh.nA * a.T, target, lane, &before);
    } else {
        // p_beam: first the live parent (its row holds exactly its beam weight), then the tile
        double z = 0.0;
        for (int i = 0; i < sh.nA; ++i) z += sh.wp[i];
        target = u * z;
        double row_before = 0.0;
        const int ia = locate_tile([&](int i) { return sh.wp[i]; }, sh.nA, target, lane, &row_before);
        if (ia < 0) return -1;
        const int T = a.T, row = sh.A[ia];
        const double wpa = sh.wp[ia], lse_row = a.lse[row];
        double in_row = 0.0;
        const int t = locate_tile([&](int i) {
            const TileStat ts = a.stats[(int64_t)row * T + i];
            if (!(ts.sum > 0.f)) return 0.0;
            return wpa * (double)ts.sum * exp((double)ts.mx * a.inv_tau - lse_row);
        }, T, target - row_before, lane, &in_row);
        if (t < 0) return -1;
        tile = ia * T + t;
        before = row_before + in_row;
    }
    if (tile < 0) return -1;
    const int ia = tile / a.T;
    *ia_out = ia;
    const RowOff ro = {sh.bp[ia], sh.bq[ia], sh.cp[ia], sh.cq[ia], sh.dc[ia]};
    return locate_token(a, sh.A[ia], tile - ia * a.T, ro, use_res ? s_res : 0.f, target - before, lane);
}

// ---------------------------------------------------------------------------------------
// Warped joints (top-k / top-p).  The support of T o p_beam has at most top_k <= 64 cells, so
// once it is known everything else of the layer is scalar work.  Finding it needs no pass over
// the rows: the maximum of every 1024-token tile is known from the dense pass, the k largest
// tile maxima are k distinct cells, hence the k-th largest cell of the joint is at least the
// k-th largest tile bound and every cell of the top k lies in a tile whose bound reaches it.
// Only those (about k) tiles are read.
// ---------------------------------------------------------------------------------------
constexpr int kMaxTopK = 64;
constexpr int kMaxCand = 680;      // candidate cells per model (two lists overlay one histogram array)
constexpr int kHalf = 256;         // threads that build one model's support (the two models run side by side)
// scratch of one build_support instance
struct SupportTmp {
    float off[kMaxLive];          // log(beam weight) - lse of each live row
    int sel[256];                 // tiles whose bound reaches the threshold
    int rhist[256];               // radix select of the k-th largest tile bound
    int n_sel, n_cand, err, n_finite, rk;
    unsigned rprefix;
    float theta;
    double zsum;
};
struct WarpScratch {
    double prob[2][kMaxTopK];     // warped probabilities, most probable first (0: p, 1: q)
    double qat[kMaxTopK];         // q~ at the cells of the p support
    int cell[2][kMaxTopK];        // live parent index * V + token
    int order[kMaxTopK];          // the p support in canonical (cell-ascending) order
    int n[2];
    SupportTmp tmp[2];
};
constexpr int kBoundCache = 1152;  // tile bounds per model kept in shared memory behind the WarpScratch
static_assert(((sizeof(WarpScratch) + 15) & ~size_t(15)) + 2 * kBoundCache * sizeof(float) <=
                  (kBins + 2) * sizeof(uint32_t),
              "the support scratch and the two bound caches overlay one histogram array");
static_assert(2 * kMaxCand * (sizeof(double) + sizeof(int)) <= (kBins + 2) * sizeof(uint32_t),
              "the two candidate lists overlay the other histogram array");

// barrier of the kHalf threads that work on one model (ids 1 and 2; 0 is __syncthreads)
__device__ __forceinline__ void half_sync(int half) {
    asm volatile("bar.sync %0, %1;" ::"r"(half + 1), "r"(kHalf) : "memory");
}

// Support of the warped joint of one model; called by the kHalf threads of half `model` of the CTA
// (warps 0-7: p, warps 8-15: q), the two halves side by side on their own scratch.  hist_p / hist_q:
// the two idle histogram arrays.  Returns 0 or a DSBD_DEV_* code (the same on every thread of the
// half).
__device__ int build_support(const VerifyArgs &a, const Shared &sh, int model, uint32_t *hist_p, uint32_t *hist_q) {
    WarpScratch &ws = *reinterpret_cast<WarpScratch *>(hist_q);
    SupportTmp &tp = ws.tmp[model];
    double *cand_key = reinterpret_cast<double *>(hist_p) + model * kMaxCand;
    int *cand_cell = reinterpret_cast<int *>(reinterpret_cast<double *>(hist_p) + 2 * kMaxCand) + model * kMaxCand;
    const int tl = threadIdx.x & (kHalf - 1);                 // thread and warp inside the half
    const int lane = threadIdx.x & 31, warp = tl >> 5;
    constexpr int kHalfWarps = kHalf / 32;
    const int T = a.T, nt = sh.nA * T, k = a.top_k;
    const TileStat *stats = a.stats + (int64_t)model * a.N * T;
    const double *lw = model ? sh.lwq : sh.lwp;
    const double *lse = a.lse + (int64_t)model * a.N;
    const float *z = model ? a.zq : a.zp;
    const float inv_tau_f = (float)a.inv_tau;
    for (int i = tl; i < sh.nA; i += kHalf) tp.off[i] = (float)(lw[i] - lse[sh.A[i]]);
    if (tl == 0) { tp.n_sel = 0; tp.n_cand = 0; tp.err = 0; ws.n[model] = 0; }
    half_sync(model);
    // float upper bound of log(joint probability) over tile i
    auto bound = [&](int i) -> float {
        const int ia = i / T;
        return fmaf(stats[(int64_t)sh.A[ia] * T + (i - ia * T)].mx, inv_tau_f, tp.off[ia]);
    };
    // The k-th largest tile bound (with multiplicity: k tiles each hold a cell at least that
    // large); with fewer than k finite bounds every tile counts.
    float *bcache = reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(&ws) +
                                              ((sizeof(WarpScratch) + 15) & ~size_t(15))) + model * kBoundCache;
    const bool cached = nt <= kBoundCache;
    if (cached) {
        // all warps: bounds into shared memory, then a radix select over their order-preserving
        // integer images, one byte per pass from the top
        auto image = [](float v) -> unsigned {
            const unsigned b = __float_as_uint(v);
            return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
        };
        if (tl == 0) { tp.rprefix = 0u; tp.rk = k; tp.n_finite = 0; }
        half_sync(model);
        int finite = 0;
        for (int i = tl; i < nt; i += kHalf) {
            const float v = bound(i);
            bcache[i] = v;
            finite += v > -INFINITY;
        }
        if (finite) atomicAdd(&tp.n_finite, finite);
        for (int pass = 3; pass >= 0; --pass) {
            for (int i = tl; i < 256; i += kHalf) tp.rhist[i] = 0;
            half_sync(model);
            const unsigned prefix = tp.rprefix;
            for (int i = tl; i < nt; i += kHalf) {
                const unsigned u = image(bcache[i]);
                if (pass == 3 || (u >> (8 * (pass + 1))) == prefix) atomicAdd(&tp.rhist[(u >> (8 * pass)) & 255u], 1);
            }
            half_sync(model);
            if (warp == 0) {
                // the digit whose bin holds the rk-th largest: lane l owns bins 8l .. 8l+7; a suffix
                // sum over the lanes finds the owning lane, which then walks its own bins
                int mine = 0;
#pragma unroll
                for (int q = 0; q < 8; ++q) mine += tp.rhist[lane * 8 + q];
                int above = mine;                              // bins of this lane and of the lanes above
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_down_sync(kFull, above, o);
                    if (lane + o < 32) above += t;
                }
                const int need0 = tp.rk;
                const bool owner = above >= need0 && above - mine < need0;
                const unsigned who = __ballot_sync(kFull, owner);
                if (who == 0u) {
                    if (lane == 0) { tp.rprefix = prefix << 8; tp.rk = need0 - above; }   // fewer than rk values
                } else if (owner) {
                    int need = need0 - (above - mine), d = lane * 8 + 7;
                    for (; d > lane * 8; --d) {
                        if (tp.rhist[d] >= need) break;
                        need -= tp.rhist[d];
                    }
                    tp.rk = need;
                    tp.rprefix = (prefix << 8) | (unsigned)d;
                }
            }
            half_sync(model);
        }
    }
    if (warp == 0) {
        float thr = INFINITY;
        bool enough = true, any = false;
        if (cached) {
            const unsigned u = tp.rprefix;
            thr = __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
            enough = tp.n_finite >= k && thr > -INFINITY;
            any = tp.n_finite > 0;
        } else {
            // too many live rows x tiles for the cache: k rounds of arg-max over distinct bounds
            for (int kk = 0; kk < k; ++kk) {
                float best = -INFINITY;
                for (int i = lane; i < nt; i += 32) {
                    const float v = bound(i);
                    if (v < thr && v > best) best = v;
                }
                best = warp_max(best);
                if (!(best > -INFINITY)) { enough = false; break; }
                any = true;
                thr = best;
            }
        }
        // the float keys carry an error of about 1e-5; the slack keeps the selection conservative
        const float theta = enough ? thr - 5e-5f - 4e-6f * fabsf(thr) : -INFINITY;
        int n_sel = 0;
        if (any)
            for (int base = 0; base < nt; base += 32) {
                const int i = base + lane;
                const float bv = i < nt ? (cached ? bcache[i] : bound(i)) : -INFINITY;
                const bool hit = i < nt && bv >= theta && bv > -INFINITY;
                const unsigned mask = __ballot_sync(kFull, hit);
                if (hit) {
                    const int pos = n_sel + __popc(mask & ((1u << lane) - 1));
                    if (pos < 256) tp.sel[pos] = i;
                }
                n_sel += __popc(mask);
            }
        if (lane == 0) {
            tp.theta = theta;
            tp.n_sel = n_sel;
            if (n_sel > 256) tp.err = DSBD_DEV_CAPACITY;       // hundreds of tiles tie at the cut
        }
    }
    half_sync(model);
    if (tp.err) return tp.err;
    float theta = tp.theta;
    const int n_sel = tp.n_sel;
    // One sweep over the selected tiles by all warps: counts the cells whose key reaches th and,
    // when asked, appends them to the candidate list (order is irrelevant: the final choice is
    // by (key, cell)).
    auto sweep = [&](float th, bool collect) {
        if (tl == 0) tp.n_cand = 0;
        half_sync(model);
        // this warp's tiles into L2 first (a tile is 32 lines of 128 bytes: one per lane), so that
        // the dependent tile loads below do not each pay a trip to HBM
        for (int sidx = warp; sidx < n_sel; sidx += kHalfWarps) {
            const int ti = tp.sel[sidx], ia = ti / T, t = ti - ia * T;
            const int e = t * kTile + lane * 32;
            if (e < a.V) asm volatile("prefetch.global.L2 [%0];" ::"l"(z + (int64_t)sh.A[ia] * a.stride + e));
        }
        for (int sidx = warp; sidx < n_sel; sidx += kHalfWarps) {
            const int ti = tp.sel[sidx], ia = ti / T, t = ti - ia * T, row = sh.A[ia];
            const float *rowp = z + (int64_t)row * a.stride;
            const bool al = (reinterpret_cast<uintptr_t>(rowp) & 15) == 0;
            float4 v[8];
            load_tile(rowp, t * kTile, a.V, al, lane, v);
            const float off_f = tp.off[ia];
            const double off_d = lw[ia] - lse[row];
            unsigned hits = 0;                               // bit (it*4+c) of this lane's 32 cells
#pragma unroll
            for (int it = 0; it < 8; ++it) {
                const float zz[4] = {v[it].x, v[it].y, v[it].z, v[it].w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float kf = fmaf(zz[c], inv_tau_f, off_f);
                    if (kf >= th && kf > -INFINITY) hits |= 1u << (it * 4 + c);
                }
            }
            const int mine = __popc(hits);
            int incl = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int tmp = __shfl_up_sync(kFull, incl, o);
                if (lane >= o) incl += tmp;
            }
            const int total = __shfl_sync(kFull, incl, 31);
            int base_pos = 0;
            if (lane == 0 && total) base_pos = atomicAdd(&tp.n_cand, total);
            base_pos = __shfl_sync(kFull, base_pos, 0);
            if (collect && mine) {
                int pos = base_pos + incl - mine;
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const float zz[4] = {v[it].x, v[it].y, v[it].z, v[it].w};
#pragma unroll
                    for (int c = 0; c < 4; ++c)
                        if (hits & (1u << (it * 4 + c))) {
                            if (pos < kMaxCand) {
                                cand_key[pos] = off_d + (double)zz[c] * a.inv_tau;
                                cand_cell[pos] = ia * a.V + t * kTile + it * 128 + lane * 4 + c;
                            }
                            ++pos;
                        }
                }
            }
        }
        half_sync(model);
        return tp.n_cand;
    };
    int n_cand = sweep(theta, true);
    if (n_cand > kMaxCand) {
        // too many cells reach the conservative threshold (few tiles, large k, or near ties):
        // bisect for a threshold with between k and kMaxCand cells above it
        float lo_t = theta, hi_t = -INFINITY;
        for (int sidx = 0; sidx < n_sel; ++sidx) hi_t = fmaxf(hi_t, bound(tp.sel[sidx]));
        if (!(lo_t > -INFINITY)) lo_t = hi_t - 400.f;
        bool found = false;
        for (int itn = 0; itn < 60 && hi_t > lo_t; ++itn) {
            const float mid = 0.5f * (lo_t + hi_t);
            const int c = sweep(mid, false);
            if (c > kMaxCand) lo_t = mid;
            else if (c < k) hi_t = mid;
            else { theta = mid; found = true; break; }
        }
        if (!found) return DSBD_DEV_CAPACITY;              // a huge tie at the cut
        n_cand = sweep(theta, true);
    }
    // exact top k of the candidates: every candidate counts those that beat it (key descending,
    // cell ascending -- a total order, cells are unique) and, if fewer than k do, that count is its
    // place in the support
    if (n_cand > kMaxCand) n_cand = kMaxCand;
    for (int jc = tl; jc < n_cand; jc += kHalf) {
        const double key = cand_key[jc];
        const int cell = cand_cell[jc];
        int rank = 0;
        for (int i = 0; i < n_cand; ++i) {
            const double ki = cand_key[i];
            rank += (ki > key) || (ki == key && cand_cell[i] < cell);
        }
        if (rank < k) {
            ws.prob[model][rank] = exp(key);
            ws.cell[model][rank] = cell;
        }
    }
    half_sync(model);
    if (warp == 0) {
        const int n_sup = n_cand < k ? n_cand : k;
        // renormalise over the top k, then the top-p cut and its renormalisation (sorted order)
        if (lane == 0) {
            double zsum = 0.0;
            for (int j = 0; j < n_sup; ++j) zsum += ws.prob[model][j];
            int keep = n_sup;
            if (a.top_p > 0.0 && a.top_p < 1.0 && zsum > 0.0) {
                double cum = 0.0;
                int j = 0;
                for (; j < n_sup; ++j) {
                    cum += ws.prob[model][j] / zsum;
                    if (cum >= a.top_p) { ++j; break; }
                }
                keep = j;
                zsum = 0.0;
                for (int q = 0; q < keep; ++q) zsum += ws.prob[model][q];
            }
            ws.n[model] = keep;
            tp.zsum = zsum;
        }
        __syncwarp();
        const double inv = tp.zsum > 0.0 ? 1.0 / tp.zsum : 0.0;
        for (int j = lane; j < ws.n[model]; j += 32) ws.prob[model][j] *= inv;
    }
    half_sync(model);
    return 0;
}

__device__ __forceinline__ double support_lookup(const WarpScratch &ws, int model, int cell) {
    for (int j = 0; j < ws.n[model]; ++j)
        if (ws.cell[model][j] == cell) return ws.prob[model][j];
    return 0.0;
}

// Inverse-CDF draw over the p support in canonical order; mass max(p~ - s q~, 0) (s = 0: p~).
// By one thread.  Returns the index into the p support or -1.
__device__ int draw_support(const WarpScratch &ws, double u, double s) {
    const int n = ws.n[0];
    double zsum = 0.0;
    for (int o = 0; o < n; ++o) {
        const int i = ws.order[o];
        zsum += fmax(ws.prob[0][i] - s * ws.qat[i], 0.0);
    }
    if (!(zsum > 0.0)) return -1;
    const double target = u * zsum;
    double cum = 0.0;
    int last = -1;
    for (int o = 0; o < n; ++o) {
        const int i = ws.order[o];
        const double w = fmax(ws.prob[0][i] - s * ws.qat[i], 0.0);
        cum += w;
        if (w > 0.0) { last = i; if (cum >= target) return i; }
    }
    return last;
}

// After build_support(p) [and q]: q~ at the p cells and the canonical order of the p support.
__device__ void finish_supports(WarpScratch &ws, bool have_q, int lane) {
    for (int i = lane; i < ws.n[0]; i += 32) ws.qat[i] = have_q ? support_lookup(ws, 1, ws.cell[0][i]) : 0.0;
    // canonical order: the place of a cell is the number of support cells below it (cells are unique)
    const int n = ws.n[0];
    for (int i = lane; i < n; i += 32) {
        const int c = ws.cell[0][i];
        int place = 0;
        for (int j = 0; j < n; ++j) place += ws.cell[0][j] < c;
        ws.order[place] = i;
    }
    __syncwarp();
}

#ifdef DSBD_PHASE_TIMING
#define TS(slot) do { if (threadIdx.x == 0 && writer) { unsigned long long t_; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t_)); a.dbg[(int64_t)r * 256 + ts_n] = ((unsigned long long)(slot) << 48) | (t_ & 0xFFFFFFFFFFFFull); if (ts_n < 255) ++ts_n; } } while (0)
#else
#define TS(slot) do {} while (0)
#endif

// dynamic shared memory of k_verify: the histogram of a layer as four 32-bit arrays while it is
// being built, then (over the same bytes) the 64-bit suffix sums of its p and q mass
constexpr size_t kVerifyDynSmem = kHistArrays * sizeof(uint32_t) * kHistWords;
static_assert(2 * sizeof(unsigned long long) * kHistWords <= kVerifyDynSmem, "the suffix sums fit over the building arrays");

__global__ void __launch_bounds__(kVThreads, 2)
k_verify(VerifyArgs a) {
    cg::cluster_group cluster = cg::this_cluster();
    const int n_cta = (int)cluster.num_blocks();
    const int cta_rank = (int)cluster.block_rank();
    const int r = blockIdx.x / n_cta;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const bool writer = (cta_rank == 0);
    __shared__ Shared sh;
    __shared__ double sp_live[kMaxLive], sq_live[kMaxLive];
    __shared__ int8_t st[kMaxLive * kMaxLive];     // status of the request's nodes, local index
    __shared__ NodeCache nc;
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    uint32_t *hp = reinterpret_cast<uint32_t *>(dyn_smem), *hq = hp + kHistWords;     // first two digit arrays
    const HistSmem hs = hist_arrays(hp);
    unsigned long long *sufP = reinterpret_cast<unsigned long long *>(dyn_smem), *sufQ = sufP + kHistWords;

    // launched with programmatic stream serialization: everything before this line overlaps the
    // tail of the kernel ahead in the stream, nothing after it may run before that kernel is done
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int b_lo = a.req_beam_off[r], b_hi = a.req_beam_off[r + 1];
    const int n_lo = a.beam_node_off[b_lo], n_hi = a.beam_node_off[b_hi];
    int W_min = a.W_min_r ? a.W_min_r[r] : a.W_min;
    int W_max = a.W_max_r ? a.W_max_r[r] : a.W_max;
    int W_nom = a.W_nom_r ? a.W_nom_r[r] : a.W_nom;
    // per-request widths come from device memory: a width below 1 or a cap below the minimum is
    // reported (after the set-up below) and the request is not verified
    const bool bad_widths = a.check_widths && (W_min < 1 || W_max < W_min || W_nom < 1);
    if (bad_widths) { W_min = W_max = W_nom = 1; }
    double *sums_base = a.tile_sums + (int64_t)r * 2 * a.max_m * ((int64_t)a.max_live * a.T);
    const int64_t slot_stride = (int64_t)a.max_live * a.T;
    unsigned long long *ghist = a.hist + (int64_t)r * 2 * kHistLen;        // [2 banks][kHistLen]
    const int hist_len = kHistLen;
    int n_out = 0;
#ifdef DSBD_PHASE_TIMING
    int ts_n = 0;
#endif

    TS(1);
    if (!a.select_mode) {
        // ---- log-sum-exp of every row of the request from the dense pass's tile statistics ----
        const int n_req = n_hi - n_lo;
        const int cw = cta_rank * kVWarps + warp, ncw = n_cta * kVWarps;
        for (int task = cw; task < 2 * n_req; task += ncw) {
            const int model = task / n_req, row = n_lo + (task - model * n_req);
            const double v = row_lse(a.stats + ((int64_t)model * a.N + row) * a.T, a.T, a.inv_tau, lane);
            if (lane == 0) {
                a.lse_w[(int64_t)model * a.N + row] = v;
                float *o = model ? a.out.lse_q : a.out.lse_p;
                if (o) o[row] = (float)v;
            }
        }
        __threadfence();
        cluster.sync();
        // ---- log-prob of every draft token given its parent (all nodes at once) ----
        for (int i = cta_rank * kVThreads + threadIdx.x; i < n_req; i += n_cta * kVThreads) {
            const int n = n_lo + i, par = a.parent[n];
            double lp = 0.0, lq = 0.0;
            if (par >= 0) {
                const int tok = a.token[n];
                if (par < n_lo || par >= n) {
                    report(a.status, DSBD_DEV_BAD_FOREST);
                    lp = lq = -INFINITY;
                } else if (tok < 0 || tok >= a.V) {
                    report(a.status, DSBD_DEV_BAD_TOKEN);
                    lp = lq = -INFINITY;
                } else {
                    lp = (double)a.zp[(int64_t)par * a.stride + tok] * a.inv_tau - a.lse_w[par];
                    lq = (double)a.zq[(int64_t)par * a.stride + tok] * a.inv_tau - a.lse_w[a.N + par];
                }
            }
            a.score_w[n] = lp;
            a.score_w[a.N + n] = lq;
        }
        __threadfence();
        cluster.sync();
        // ---- cumulative beam scores and depths (rank 0 of the cluster) ----
        if (writer) {
            if (n_req <= 1024) {
                // stage the per-node log-probs in shared memory (the histogram arrays are idle
                // here), then every node sums its own path to the root
                double *slp = reinterpret_cast<double *>(hp), *slq = reinterpret_cast<double *>(hq);
                for (int i = threadIdx.x; i < n_req; i += kVThreads) {
                    slp[i] = a.score_w[n_lo + i];
                    slq[i] = a.score_w[a.N + n_lo + i];
                }
                __syncthreads();
                for (int b = b_lo + (int)threadIdx.x; b < b_hi; b += kVThreads) {
                    const int root = a.beam_node_off[b];
                    if (a.parent[root] != -1) report(a.status, DSBD_DEV_BAD_FOREST);
                    slp[root - n_lo] = (double)a.root_logp[b];
                    slq[root - n_lo] = (double)a.root_logq[b];
                }
                __syncthreads();
                for (int i = threadIdx.x; i < n_req; i += kVThreads) {
                    double sp = 0.0, sq = 0.0;
                    int dep = 0, cur = i;
                    while (true) {
                        sp += slp[cur];
                        sq += slq[cur];
                        const int par = a.parent[n_lo + cur];
                        if (par < n_lo || par >= n_lo + cur) break;      // root (-1) or malformed
                        cur = par - n_lo;
                        if (++dep > a.gamma) { report(a.status, DSBD_DEV_BAD_FOREST); break; }
                    }
                    a.score_w[n_lo + i] = sp;
                    a.score_w[a.N + n_lo + i] = sq;
                    a.depth_w[n_lo + i] = dep;
                    if (a.out.node_logp) a.out.node_logp[n_lo + i] = (float)sp;
                    if (a.out.node_logq) a.out.node_logq[n_lo + i] = (float)sq;
                }
                __syncthreads();
            } else {
                for (int b = b_lo + (int)threadIdx.x; b < b_hi; b += kVThreads) {
                    const int lo = a.beam_node_off[b], hi = a.beam_node_off[b + 1];
                    for (int n = lo; n < hi; ++n) {
                        const int par = a.parent[n];
                        double sp, sq;
                        int dep = 0;
                        if (n == lo) {
                            sp = (double)a.root_logp[b];
                            sq = (double)a.root_logq[b];
                            if (par != -1) report(a.status, DSBD_DEV_BAD_FOREST);
                        } else if (par < lo || par >= n) {
                            sp = sq = -INFINITY;
                            dep = a.gamma + 1;
                        } else {
                            sp = a.score_w[par] + a.score_w[n];
                            sq = a.score_w[a.N + par] + a.score_w[a.N + n];
                            dep = a.depth_w[par] + 1;
                            if (dep > a.gamma) report(a.status, DSBD_DEV_BAD_FOREST);
                        }
                        a.score_w[n] = sp;
                        a.score_w[a.N + n] = sq;
                        a.depth_w[n] = dep;
                        if (a.out.node_logp) a.out.node_logp[n] = (float)sp;
                        if (a.out.node_logq) a.out.node_logq[n] = (float)sq;
                    }
                }
            }
        }
        __threadfence();
        cluster.sync();
    }

    // ---- set-up ----
    if (warp == 0) {
        if (lane == 0) {
            sh.err = 0; sh.done = 0; sh.n_out = 0; sh.n_fill = 0;
            sh.n_layers = sh.n_tests = sh.n_exact = sh.n_respass = 0;
            sh.n_wrapped = 0; sh.n_near = 0; sh.n_rows = 0;
            if (a.select_mode) {
                const int lo = a.live_off[r], hi = a.live_off[r + 1];
                sh.nA = hi - lo;
                // the dense pass before this kernel covered the first sel_rows list entries only
                if (sh.nA > kMaxLive || sh.nA < 0 || lo < 0 || hi > a.sel_rows) {
                    sh.err = DSBD_DEV_BAD_FOREST;
                    sh.nA = 0;
                }
                for (int i = 0; i < sh.nA; ++i)
                    if (a.live_nodes[lo + i] < 0 || a.live_nodes[lo + i] >= a.N) sh.err = DSBD_DEV_BAD_FOREST;
                if (sh.err) sh.nA = 0;
                for (int i = 0; i < sh.nA; ++i) {
                    sh.A[i] = a.live_nodes[lo + i];
                    sp_live[i] = (double)a.sel_logp[sh.A[i]];
                    sq_live[i] = (double)a.sel_logq[sh.A[i]];
                }
            } else {
                sh.nA = b_hi - b_lo;
                if (sh.nA > kMaxLive) { sh.err = DSBD_DEV_BAD_FOREST; sh.nA = 0; }
                for (int i = 0; i < sh.nA; ++i) {
                    sh.A[i] = a.beam_node_off[b_lo + i];
                    sp_live[i] = a.score[sh.A[i]];
                    sq_live[i] = a.score[a.N + sh.A[i]];
                }
                if (writer) {
                    for (int l = 0; l <= a.gamma; ++l) a.out.layer_width[(int64_t)r * (a.gamma + 1) + l] = -1;
                    a.out.l_last[r] = a.gamma + 1;
                    a.out.out_width[r] = 0;
                }
            }
        }
        __syncwarp();
        if (!a.select_mode && writer)
            for (int n = n_lo + lane; n < n_hi; n += 32)
                a.out.node_status[n] = a.parent[n] < 0 ? DSBD_NODE_ACCEPTED : DSBD_NODE_UNREACHED;
    }
    // Every CTA of the cluster takes identical decisions from identical data, so each keeps its
    // own copy of the node statuses and only rank 0 writes results.
    const int n_layers = a.select_mode ? 1 : a.gamma;
    const int n_req_nodes = n_hi - n_lo;
    const bool st_ok = n_req_nodes <= kMaxLive * kMaxLive;
    if (!a.select_mode)
        for (int n = threadIdx.x; n < n_req_nodes && st_ok; n += blockDim.x)
            st[n] = a.parent[n_lo + n] < 0 ? DSBD_NODE_ACCEPTED : DSBD_NODE_UNREACHED;
    __threadfence();
    cluster.sync();
    if (!a.select_mode && !st_ok && threadIdx.x == 0) sh.err = DSBD_DEV_BAD_FOREST;
    if (bad_widths && threadIdx.x == 0) sh.err = DSBD_DEV_BAD_PARAM;
    const bool cached = !a.select_mode && n_req_nodes <= kCacheNodes && a.gamma < 256;
    if (threadIdx.x == 0) nc.on = cached ? 1 : 0;
    if (cached)
        for (int i = threadIdx.x; i < n_req_nodes; i += blockDim.x) {
            const int n = n_lo + i, par = a.parent[n];
            nc.score_p[i] = a.score[n];   nc.score_q[i] = a.score[a.N + n];
            nc.lse_p[i] = a.lse[n];       nc.lse_q[i] = a.lse[a.N + n];
            nc.parent[i] = (int16_t)((par >= n_lo && par < n) ? par - n_lo : -1);
            nc.depth[i] = (uint8_t)min(max(a.depth[n], 0), 255);
        }
    __syncthreads();
    // node data by local index, from the cache when there is one
    auto nd_depth = [&](int i) -> int { return cached ? (int)nc.depth[i] : a.depth[n_lo + i]; };
    auto nd_parent = [&](int i) -> int { return cached ? (int)nc.parent[i] : a.parent[n_lo + i] - n_lo; };
    auto nd_score = [&](int model, int i) -> double {
        return cached ? (model ? nc.score_q[i] : nc.score_p[i]) : a.score[(int64_t)model * a.N + n_lo + i];
    };

    for (int l = 1; l <= n_layers && !sh.done && !sh.err; ++l) {
        // ---- live drafts of layer l, in draw order; beam weights ----
        TS(2);
        if (warp == 0) {
            int m = 0;
            if (a.select_mode) {
                m = a.m_in[r];
                if (m < 0 || m > kMaxLive) { if (lane == 0) sh.err = DSBD_DEV_BAD_FOREST; m = 0; }
            } else {
                for (int base = 0; base < n_req_nodes; base += 32) {
                    const int n = base + lane;
                    bool live = false;
                    if (n < n_req_nodes && nd_depth(n) == l) {
                        const int pl = nd_parent(n);
                        live = pl >= 0 && st[pl] == DSBD_NODE_ACCEPTED;
                        if (!live) {
                            st[n] = DSBD_NODE_PRUNED;
                            if (writer) a.out.node_status[n_lo + n] = DSBD_NODE_PRUNED;
                        }
                    }
                    const unsigned mask = __ballot_sync(kFull, live);
                    const int pos = m + __popc(mask & ((1u << lane) - 1));
                    if (live && pos < kMaxLive) sh.S[pos] = n_lo + n;
                    m += __popc(mask);
                }
                if (m > kMaxLive) { if (lane == 0) sh.err = DSBD_DEV_BAD_FOREST; m = 0; }
                __syncwarp();
                if (lane == 0 && a.draft_rank) {
                    // insertion sort by (draft_rank, node id); ids are already ascending
                    for (int i = 1; i < m; ++i) {
                        const int n = sh.S[i];
                        const int key = a.draft_rank[n];
                        int j = i - 1;
                        while (j >= 0 && a.draft_rank[sh.S[j]] > key) { sh.S[j + 1] = sh.S[j]; --j; }
                        sh.S[j + 1] = n;
                    }
                }
            }
            __syncwarp();
            live_weights(a, sh, sp_live, sq_live, lane, cached ? &nc : nullptr, n_lo);
            if (lane == 0) {
                sh.m = m;
                sh.s_arr[0] = 0.0;
                sh.c_arr[1] = 1.0;
                sh.chain_len = 0;          // c_{j+1} is known for j = 1..chain_len
                sh.bank = l & 1;
            }
            // per live draft: index of its parent in A, rho = p_beam/q_beam of its cell, its uniform
            if (!a.select_mode)
                for (int i = lane; i < m; i += 32) {
                    const int n = sh.S[i];
                    const int pl = nd_parent(n - n_lo), par = n_lo + pl;
                    int ai = 0;
                    while (ai < sh.nA && sh.A[ai] != par) ++ai;
                    sh.S_parent_idx[i] = ai;
                    const double lp = nd_score(0, n - n_lo) - nd_score(0, pl);
                    const double lq = nd_score(1, n - n_lo) - nd_score(1, pl);
                    double rho;
                    if (lq == -INFINITY || sh.lwq[ai] == -INFINITY)
                        rho = (lp > -INFINITY && sh.lwp[ai] > -INFINITY) ? INFINITY : 0.0;
                    else
                        rho = exp((sh.lwp[ai] - sh.lwq[ai]) + (lp - lq));
                    sh.rho[i] = rho;
                    sh.uu[i] = decision_uniform(a.seed, a.step, (uint32_t)r, (uint32_t)l, 0u, (uint32_t)i);
                }
        }
        for (int i = threadIdx.x; i < kHistArrays * kHistWords; i += blockDim.x) hp[i] = 0u;
        if (threadIdx.x < 10) sh.w_tot[threadIdx.x] = 0ull;
        if (threadIdx.x == 0) sh.wrapped = 0;
        __syncthreads();
        const int m = sh.m;
        TS(3);

        const bool warped = a.top_k > 0;
        WarpScratch &wsup = *reinterpret_cast<WarpScratch *>(hq);       // the histogram arrays are idle when warped
        if (warped) {
            // ---- supports of T o p_beam and T o q_beam, then the whole chain on <= 64 cells ----
            if (!sh.err) {
                // the first half of the warps builds the support of p, the second that of q, side by side
                const int half = warp / (kHalf / 32);
                const int e_half = build_support(a, sh, half, hp, hq);
                if (e_half && (threadIdx.x & (kHalf - 1)) == 0) wsup.tmp[half].err = e_half;
                __syncthreads();
                const int e = wsup.tmp[0].err ? wsup.tmp[0].err : wsup.tmp[1].err;
                if (e) { if (threadIdx.x == 0) sh.err = e; }
                else if (warp == 0) {
                    finish_supports(wsup, true, lane);
                    // rho of every live draft from the warped joints
                    if (!a.select_mode)
                        for (int i = lane; i < m; i += 32) {
                            const int cell = sh.S_parent_idx[i] * a.V + a.token[sh.S[i]];
                            const double pw = support_lookup(wsup, 0, cell), qw = support_lookup(wsup, 1, cell);
                            sh.rho[i] = qw > 0.0 ? pw / qw : (pw > 0.0 ? INFINITY : 0.0);
                        }
                    // c_{j+1} = F(s_j) over the p support, lanes over cells
                    // (every lane keeps its at most two cells and the running s, c in registers)
                    const int ns = wsup.n[0];
                    const double p0 = lane < ns ? wsup.prob[0][lane] : 0.0, q0 = lane < ns ? wsup.qat[lane] : 0.0;
                    const double p1 = lane + 32 < ns ? wsup.prob[0][lane + 32] : 0.0;
                    const double q1 = lane + 32 < ns ? wsup.qat[lane + 32] : 0.0;
                    double s_prev = 0.0, c_cur = 1.0;
                    for (int j = 1; j <= m; ++j) {
                        const double s_j = s_prev + c_cur;
                        double acc = fmax(p0 - s_j * q0, 0.0);
                        if (lane + 32 < ns) acc += fmax(p1 - s_j * q1, 0.0);
                        acc = warp_sum(acc);
                        if (lane == 0) { sh.s_arr[j] = s_j; sh.c_arr[j + 1] = acc; sh.chain_len = j; }
                        s_prev = s_j;
                        c_cur = acc;
                        if (!(acc > 0.0)) break;
                    }
                    __syncwarp();
                }
            }
            __syncthreads();
        } else if (m >= 1 && !sh.err) {
            // ---- one pass: ratio histogram of the layer over the live rows ----
            const double top = log2((double)(m > 2 ? m : 2));          // s_j <= j <= m
            const float binscale = (float)((double)kBins / top);
            unsigned long long *gh = ghist + sh.bank * hist_len;
            histogram_pass(a, sh, binscale, hs, sums_base + ((int64_t)sh.bank * a.max_m) * slot_stride, cta_rank,
                           n_cta, sh.w_tot);
            __syncthreads();
            hist_check_local(hs, sh.w_tot, sh.wtot_p, sh.wtot_q);
            TS(4);
            cluster.sync();                            // every CTA's histogram is complete
            hist_merge(cluster, hs, gh, sh.w_tot, cta_rank, n_cta);
            cluster.sync();                            // the image is whole (the barrier orders the stores for
                                                       // the cluster); nobody reads the arrays any more
            TS(5);
            // the merged histogram into shared memory (over the building arrays)
            for (int i = threadIdx.x; i <= kBins; i += blockDim.x) {
                sufP[i] = __ldcg(gh + 2 * i);
                sufQ[i] = __ldcg(gh + 2 * i + 1);
            }
            if (threadIdx.x == 0) {
                sh.n_cells = (double)sh.nA * (double)a.V;      // every cell of the live rows, at most
                sh.wrapped = sh.w_tot[9] != 0ull;
                if (sh.wrapped) ++sh.n_wrapped;
            }
            __syncthreads();
            TS(6);
            // in-place suffix sums: sufP[k] = p mass of the bins >= k (17 bins per thread)
            {
                constexpr int per = (kBins + 1 + kVThreads - 1) / kVThreads;
                const int lo = min((int)threadIdx.x * per, kBins + 1), hi = min(lo + per, kBins + 1);
                unsigned long long mp_ = 0ull, mq_ = 0ull;
                for (int i = lo; i < hi; ++i) { mp_ += sufP[i]; mq_ += sufQ[i]; }
                unsigned long long ap = mp_, aq = mq_;    // suffix scan inside the warp, top lane down
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const unsigned long long tp = __shfl_down_sync(kFull, ap, o), tq = __shfl_down_sync(kFull, aq, o);
                    if (lane + o < 32) { ap += tp; aq += tq; }
                }
                if (lane == 0) { sh.wtot_p[warp] = ap; sh.wtot_q[warp] = aq; }
                __syncthreads();
                unsigned long long rp_ = ap - mp_, rq_ = aq - mq_;  // mass of the lanes above in this warp
                for (int w = warp + 1; w < kVWarps; ++w) { rp_ += sh.wtot_p[w]; rq_ += sh.wtot_q[w]; }
                for (int i = hi - 1; i >= lo; --i) {
                    rp_ += sufP[i]; rq_ += sufQ[i];
                    sufP[i] = rp_; sufQ[i] = rq_;
                }
                if (threadIdx.x == 0) { sufP[kBins + 1] = 0ull; sufQ[kBins + 1] = 0ull; }
            }
            __syncthreads();

            TS(7);
            int j0 = 1;
            while (j0 <= m) {
                if (threadIdx.x == 0) {
                    int j = j0;
                    int need = 0;
                    for (; j <= m; ++j) {
                        const double s_j = sh.s_arr[j - 1] + sh.c_arr[j];
                        sh.s_arr[j] = s_j;
                        sh.chain_len = j;
                        double c_next;
                        // every partial sum of the histogram is off by at most half a unit per cell
                        const double fix_err = sh.n_cells * (0.5 * kUnfix) * (1.0 + s_j);
                        if (sh.wrapped) { need = 1; break; }             // a wrapped word: exact passes only
                        if (j == 1) {
                            c_next = ((double)sufP[0] - (double)sufQ[0]) * kUnfix;
                            if (fix_err > kErrTol) { need = 1; break; }
                        } else {
                            int k = (int)(log2(s_j) * (double)binscale);
                            if (k < 0) k = 0;
                            if (k >= kBins) { need = 1; break; }      // cannot happen for s_j <= m
                            const double Pa = (double)sufP[k + 1] * kUnfix, Qa = (double)sufQ[k + 1] * kUnfix;
                            const double Pk = (double)(sufP[k] - sufP[k + 1]) * kUnfix;
                            const double Qk = (double)(sufQ[k] - sufQ[k + 1]) * kUnfix;
                            const double r_lo = (double)exp2f((float)k / binscale) * (1.0 - 2e-6);
                            const double r_hi = (double)exp2f((float)(k + 1) / binscale) * (1.0 + 2e-6);
                            const double lo_b = fmax(Pk - s_j * Qk, 0.0);
                            double q_hi = (Pk - r_lo * Qk) / (r_hi - r_lo);
                            q_hi = fmin(fmax(q_hi, 0.0), Qk);
                            const double hi_b = fmax(q_hi * (r_hi - s_j), lo_b);
                            // the midpoint of the bracket is used: half its width plus the fixed-point term
                            if (0.5 * (hi_b - lo_b) + fix_err > kErrTol) { need = 1; break; }
                            c_next = fmax(Pa - s_j * Qa, 0.0) + 0.5 * (lo_b + hi_b);
                        }
                        sh.c_arr[j + 1] = c_next;
                        if (!(c_next > 0.0)) { j = m; }               // chain exhausted: stop walking
                    }
                    sh.need_exact = need;
                    sh.chain_pos = need ? j : m + 1;
                }
                __syncthreads();
                if (!sh.need_exact) break;
                const int j = sh.chain_pos;
                if (threadIdx.x == 0) ++sh.n_exact;
                double *sums = sums_base + ((int64_t)sh.bank * a.max_m + (j - 1)) * slot_stride;
                residual_pass(a, sh, (float)sh.s_arr[j], sums, cta_rank, n_cta);
                __threadfence();
                cluster.sync();
                if (warp == 0) {
                    const double c_next = ordered_sum(sums, sh.nA * a.T, lane);
                    if (lane == 0) sh.c_arr[j + 1] = c_next;
                }
                __syncthreads();
                if (!(sh.c_arr[j + 1] > 0.0)) break;
                j0 = j + 1;
            }
        }
        __syncthreads();

        TS(8);
        // ---- width and accept loop (warp 0) ----
        if (warp == 0 && !sh.err) {
            // alpha_j = 1 - c_{j+1}/c_j; once a residual has no mass every later alpha is 1
            for (int j = 1 + lane; j <= m; j += 32) {
                double al = 1.0;
                if (j <= sh.chain_len && sh.c_arr[j] > 0.0 && sh.c_arr[j + 1] > 0.0)
                    al = fmin(fmax(1.0 - sh.c_arr[j + 1] / sh.c_arr[j], 0.0), 1.0);
                sh.alpha[j] = al;
            }
            if (lane == 0) sh.res_j = 0;
            __syncwarp();
            // (the verification only needs W~ up to W_max and can stop at the first tail below the
            // threshold; dsbd_select_width returns the whole tail)
            const int wt = width_rule(sh, m, a.thresh, lane, a.select_mode ? -1 : W_max);
            int W = wt > W_min ? wt : W_min;
            if (W > W_max) W = W_max;
            if (a.select_mode) {
                if (writer && lane == 0) {
                    a.width_out[r] = W;
                    if (a.alpha_out)
                        for (int j = 0; j < m && j < a.out_stride; ++j)
                            a.alpha_out[(int64_t)r * a.out_stride + j] = (float)sh.alpha[j + 1];
                    if (a.tail_out)
                        for (int K = 0; K <= m && K < a.out_stride; ++K)
                            a.tail_out[(int64_t)r * a.out_stride + K] = (float)sh.tail[K];
                }
                if (lane == 0) sh.done = 1;
            } else if (lane == 0) {
                if (writer) a.out.layer_width[(int64_t)r * (a.gamma + 1) + (l - 1)] = W;
                int count = 0, j = 1, err = 0, tests = 0, near = 0;
                for (int i = 0; i < m && count < W; ++i) {
                    const int n = sh.S[i];
                    const double rho = sh.rho[i];
                    double ratio;
                    if (j == 1) ratio = rho;
                    else ratio = fmax(rho - sh.s_arr[j - 1], 0.0) / sh.c_arr[j];
                    if (ratio > 1.0) ratio = 1.0;
                    const double u = sh.uu[i];
                    ++tests;
                    near += fabs(u - ratio) < 1e-5;
                    if (u <= ratio) {
                        st[n - n_lo] = DSBD_NODE_ACCEPTED;
                        if (writer) a.out.node_status[n] = DSBD_NODE_ACCEPTED;
                        sh.acc[count++] = n;
                        j = 1;
                    } else {
                        st[n - n_lo] = DSBD_NODE_REJECTED;
                        if (writer) a.out.node_status[n] = DSBD_NODE_REJECTED;
                        // an empty residual means p' == q_beam: the rejected draft lay outside the
                        // support of q_beam, there is nothing to subtract and p' stays
                        if (j <= sh.chain_len && sh.c_arr[j + 1] > 0.0) ++j;
                    }
                }
                for (int i = 0; i < m; ++i)
                    if (st[sh.S[i] - n_lo] == DSBD_NODE_UNREACHED) {
                        st[sh.S[i] - n_lo] = DSBD_NODE_CUT;
                        if (writer) a.out.node_status[sh.S[i]] = DSBD_NODE_CUT;
                    }
                sh.W = W;
                sh.count = count;
                sh.n_tests += tests;
                sh.n_near += near;
                sh.n_rows += sh.nA;
                ++sh.n_layers;
                sh.res_j = (count < W && j > 1) ? j : 0;   // residual draw at run position j needs tile sums
                sh.run_j = j;
                if (err) sh.err = err;
            }
        }
        __syncthreads();

        TS(9);
        // ---- a residual draw locates its tile through tile sums of max(p_beam - s_{j-1} q_beam, 0) ----
        double *res_sums = sums_base + ((int64_t)sh.bank * a.max_m) * slot_stride;   // slot 0 of the bank
        if (!a.select_mode && !sh.err && !warped && sh.res_j > 2) {   // run position 2 is served by the histogram pass
            if (threadIdx.x == 0) ++sh.n_respass;
            residual_pass(a, sh, (float)sh.s_arr[sh.res_j - 1], res_sums, cta_rank, n_cta);
            __threadfence();
            cluster.sync();
        }

        TS(10);
        // ---- completion of a short layer, or the next layer's input beams (warp 0) ----
        if (warp == 0 && !a.select_mode && !sh.err) {
            const int W = sh.W, count = sh.count, j = sh.run_j;
            int err = 0;
            if (count < W) {
                if (lane == 0)
                    for (int i = 0; i < count && !err; ++i)
                        emit_output(a, r, &n_out, a.parent[sh.acc[i]], sh.acc[i], a.token[sh.acc[i]],
                                    DSBD_SRC_DRAFT, writer, &err);
                n_out = __shfl_sync(kFull, n_out, 0);
                err = __shfl_sync(kFull, err, 0);
                int fill = 0;
                // unwarped: warp 0 makes the residual draw, the p_beam fills (independent draws)
                // are then spread over the warps of the CTA
                const int kk_end = warped ? W : count + 1;
                for (int kk = count; kk < kk_end && !err; ++kk) {
                    const bool residual = (kk == count);
                    const bool use_res = residual && j > 1;
                    const double u = decision_uniform(a.seed, a.step, (uint32_t)r, (uint32_t)l,
                                                      residual ? 1u : 2u, residual ? 0u : (uint32_t)fill);
                    int ia = 0, tok;
                    if (warped) {
                        int pick = -1;
                        if (lane == 0) pick = draw_support(wsup, u, use_res ? sh.s_arr[j - 1] : 0.0);
                        pick = __shfl_sync(kFull, pick, 0);
                        tok = -1;
                        if (pick >= 0) { ia = wsup.cell[0][pick] / a.V; tok = wsup.cell[0][pick] - ia * a.V; }
                    } else {
                        double z_res = 0.0;
                        if (use_res) z_res = ordered_sum(res_sums, sh.nA * a.T, lane);
                        tok = draw_cell(a, sh, u, use_res, use_res ? (float)sh.s_arr[j - 1] : 0.f, z_res, res_sums,
                                        lane, &ia);
                    }
                    if (tok < 0) { err = DSBD_DEV_EXHAUSTED; break; }
                    if (lane == 0)
                        emit_output(a, r, &n_out, sh.A[ia], -1, tok, residual ? DSBD_SRC_RESIDUAL : DSBD_SRC_FILL,
                                    writer, &err);
                    n_out = __shfl_sync(kFull, n_out, 0);
                    err = __shfl_sync(kFull, err, 0);
                    if (!residual) ++fill;
                }
                if (lane == 0) {
                    sh.done = 1;
                    if (writer) a.out.l_last[r] = l;
                    sh.n_out = n_out;
                    sh.n_fill = (!warped && !err) ? W - count - 1 : 0;
                }
            } else {
                // the accepted drafts, ascending node id, are the next layer's input beams
                int nA = 0;
                for (int base = 0; base < n_req_nodes; base += 32) {
                    const int n = base + lane;
                    const bool in = n < n_req_nodes && nd_depth(n) == l && st[n] == DSBD_NODE_ACCEPTED;
                    const unsigned mask = __ballot_sync(kFull, in);
                    const int pos = nA + __popc(mask & ((1u << lane) - 1));
                    if (in && pos < kMaxLive) {
                        sh.A[pos] = n_lo + n;
                        sp_live[pos] = nd_score(0, n);
                        sq_live[pos] = nd_score(1, n);
                    }
                    nA += __popc(mask);
                }
                if (lane == 0) sh.nA = nA;
            }
            if (lane == 0 && err) sh.err = err;
        }
        __syncthreads();
        if (!a.select_mode && sh.done && sh.n_fill > 0 && !sh.err) {
            // fill f is output beam n_out + f, drawn from p_beam with its own uniform
            const int cap = a.out.out_off[r + 1] - a.out.out_off[r];
            const int base = sh.n_out, want = sh.n_fill;
            const int n_draw = min(want, max(cap - base, 0));
            __syncthreads();
            for (int f = warp; f < n_draw; f += kVWarps) {
                const double u = decision_uniform(a.seed, a.step, (uint32_t)r, (uint32_t)l, 2u, (uint32_t)f);
                int ia = 0;
                const int tok = draw_cell(a, sh, u, false, 0.f, 0.0, nullptr, lane, &ia);
                if (tok < 0) { if (lane == 0) sh.err = DSBD_DEV_EXHAUSTED; }
                else if (lane == 0 && writer) emit_at(a, r, base + f, sh.A[ia], -1, tok, DSBD_SRC_FILL);
            }
            __syncthreads();
            if (threadIdx.x == 0) {
                if (!sh.err) { sh.n_out = base + n_draw; if (want > n_draw) sh.err = DSBD_DEV_CAPACITY; }
                sh.n_fill = 0;
            }
            __syncthreads();
            n_out = sh.n_out;
        }
    }

    TS(11);
    // ---- every layer passed: W_nom beams from p_beam^(gamma+1) ----
    const bool extra = !a.select_mode && !sh.done && !sh.err;
    WarpScratch &wsx = *reinterpret_cast<WarpScratch *>(hq);
    int extra_err = 0;
    if (extra) {
        if (warp == 0) live_weights(a, sh, sp_live, sq_live, lane);
        __syncthreads();
        if (a.top_k > 0) {
            if (warp < kHalf / 32) {                            // one model only: the first half builds it
                const int e_half = build_support(a, sh, 0, hp, hq);
                if (e_half && threadIdx.x == 0) wsx.tmp[0].err = e_half;
            }
            __syncthreads();
            extra_err = wsx.tmp[0].err;
            if (!extra_err && warp == 0) finish_supports(wsx, false, lane);
        }
    }
    if (extra && a.top_k == 0) {
        // W_nom independent draws from p_beam, one warp each
        const int cap = a.out.out_off[r + 1] - a.out.out_off[r];
        const int n_draw = min(W_nom, max(cap - n_out, 0));
        if (writer && threadIdx.x == 0) a.out.layer_width[(int64_t)r * (a.gamma + 1) + a.gamma] = W_nom;
        for (int kk = warp; kk < n_draw; kk += kVWarps) {
            const double u = decision_uniform(a.seed, a.step, (uint32_t)r, (uint32_t)(a.gamma + 1) + a.extra_layer_bias, 3u,
                                              (uint32_t)kk);
            int ia = 0;
            const int tok = draw_cell(a, sh, u, false, 0.f, 0.0, nullptr, lane, &ia);
            if (tok < 0) { if (lane == 0) sh.err = DSBD_DEV_EXHAUSTED; }
            else if (lane == 0 && writer) emit_at(a, r, n_out + kk, sh.A[ia], -1, tok, DSBD_SRC_EXTRA);
        }
        __syncthreads();
        if (!sh.err) {
            n_out += n_draw;
            if (W_nom > n_draw && threadIdx.x == 0) sh.err = DSBD_DEV_CAPACITY;
        }
    } else if (extra && warp == 0) {
        int err = extra_err;
        if (writer && lane == 0) a.out.layer_width[(int64_t)r * (a.gamma + 1) + a.gamma] = W_nom;
        for (int kk = 0; kk < W_nom && !err; ++kk) {
            const double u = decision_uniform(a.seed, a.step, (uint32_t)r, (uint32_t)(a.gamma + 1) + a.extra_layer_bias, 3u,
                                              (uint32_t)kk);
            int ia = 0, tok;
            if (a.top_k > 0) {
                int pick = -1;
                if (lane == 0) pick = draw_support(wsx, u, 0.0);
                pick = __shfl_sync(kFull, pick, 0);
                tok = -1;
                if (pick >= 0) { ia = wsx.cell[0][pick] / a.V; tok = wsx.cell[0][pick] - ia * a.V; }
            } else {
                tok = draw_cell(a, sh, u, false, 0.f, 0.0, nullptr, lane, &ia);
            }
            if (tok < 0) { err = DSBD_DEV_EXHAUSTED; break; }
            if (lane == 0) emit_output(a, r, &n_out, sh.A[ia], -1, tok, DSBD_SRC_EXTRA, writer, &err);
            n_out = __shfl_sync(kFull, n_out, 0);
            err = __shfl_sync(kFull, err, 0);
        }
        if (lane == 0 && err) sh.err = err;
    }
    __syncthreads();
    TS(12);
    if (threadIdx.x == 0 && writer) {
        if (!a.select_mode) {
            a.out.out_width[r] = n_out;
            if (a.out.req_error) a.out.req_error[r] = sh.err;
            if (a.out.req_stats) {
                int32_t *rs = a.out.req_stats + (int64_t)DSBD_REQ_STATS * r;
                rs[0] = sh.n_layers; rs[1] = sh.n_tests; rs[2] = sh.n_exact; rs[3] = sh.n_respass;
                rs[4] = sh.n_near; rs[5] = sh.n_rows; rs[6] = sh.n_wrapped; rs[7] = 0;
            }
        }
        if (sh.err) report(a.status, sh.err);
    }
}

// ------------------------------------------------------------------------------ host side
struct Layout {
    size_t stats, lse, score, depth, sums, hist, total;
    int T, max_m, max_live;
};

Layout make_layout(const dsbd_forest_t *f, int V) {
    Layout L;
    L.T = (V + kTile - 1) / kTile;
    L.max_live = f->max_req_beams > f->max_layer_nodes ? f->max_req_beams : f->max_layer_nodes;
    if (L.max_live < 1) L.max_live = 1;
    L.max_m = f->max_layer_nodes > 1 ? f->max_layer_nodes : 1;
    size_t off = 0;
    L.stats = off; off = align_up(off + sizeof(TileStat) * 2 * (size_t)f->N * L.T, 256);
    L.lse = off;   off = align_up(off + sizeof(double) * 2 * (size_t)f->N, 256);
    L.score = off; off = align_up(off + sizeof(double) * 2 * (size_t)f->N, 256);
    L.depth = off; off = align_up(off + sizeof(int32_t) * (size_t)f->N, 256);
    L.sums = off;
    off = align_up(off + sizeof(double) * (size_t)f->R * 2 * L.max_m * (size_t)L.max_live * L.T, 256);
    L.hist = off;
    off = align_up(off + sizeof(unsigned long long) * (size_t)f->R * 2 * kHistLen, 256);
#ifdef DSBD_PHASE_TIMING
    off = align_up(off + sizeof(unsigned long long) * (size_t)f->R * 256, 256);
#endif
    L.total = off;
    return L;
}

int check_forest(const dsbd_forest_t *f) {
    if (!f || f->R <= 0 || f->B <= 0 || f->N <= 0 || f->max_depth < 0) return DSBD_ERR_INVALID_ARG;
    if (!f->req_beam_off || !f->beam_node_off || !f->parent || !f->token) return DSBD_ERR_INVALID_ARG;
    if (f->max_req_beams <= 0 || f->max_layer_nodes < 0) return DSBD_ERR_INVALID_ARG;
    if (f->max_req_beams > DSBD_MAX_LIVE || f->max_layer_nodes > DSBD_MAX_LIVE) return DSBD_ERR_UNSUPPORTED;
    return DSBD_OK;
}

// The widths of the width rule W_L^(l) = min(W_max, max(W_min, W~)): without per-request
// overrides a zero width or a cap below the minimum is a caller's mistake (a zero-initialised
// struct), not a setting.
int check_widths(const dsbd_verify_params_t *p) {
    if (!p->W_min_r && p->W_min < 1) return DSBD_ERR_INVALID_ARG;
    if (!p->W_max_r && p->W_max < 1) return DSBD_ERR_INVALID_ARG;
    if (!p->W_nom_r && p->W_nom < 1) return DSBD_ERR_INVALID_ARG;
    if (!p->W_min_r && !p->W_max_r && p->W_max < p->W_min) return DSBD_ERR_INVALID_ARG;
    return DSBD_OK;
}

int check_params(const dsbd_verify_params_t *p) {
    if (!p || p->V <= 0 || !(p->temperature > 0.f)) return DSBD_ERR_INVALID_ARG;
    if (p->W_min < 1 && !p->W_min_r) return DSBD_ERR_INVALID_ARG;
    if (p->top_k < 0) return DSBD_ERR_INVALID_ARG;
    if (p->top_k > 64) return DSBD_ERR_UNSUPPORTED;
    if (p->top_k == 0 && p->top_p > 0.f && p->top_p < 1.f) return DSBD_ERR_UNSUPPORTED;   // top-p needs a top-k bound
    return DSBD_OK;
}

// Cluster size: as many CTAs per request as its tile count can use, but few enough that all
// requests are resident at once (two CTAs per SM fit).
int cluster_size_for(int tiles, int R) {
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    int cs = 1;
    if (tiles >= 256) cs = 16;
    else if (tiles >= 64) cs = 8;
    else if (tiles >= 32) cs = 4;
    else if (tiles >= 16) cs = 2;
    while (cs > 1 && (long long)R * cs > 2ll * sms) cs >>= 1;
    return cs;
}

int launch_verify(const VerifyArgs &args, int R, int tiles, cudaStream_t stream) {
    const int cs = cluster_size_for(tiles, R);
    if (cs > 8 && cudaFuncSetAttribute(k_verify, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)
        return DSBD_ERR_CUDA;
    if (cudaFuncSetAttribute(k_verify, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kVerifyDynSmem) != cudaSuccess)
        return DSBD_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(R * cs));
    cfg.blockDim = dim3(kVThreads);
    cfg.dynamicSmemBytes = kVerifyDynSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)cs;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // the clusters may be set up while the dense pass before them drains; the kernel waits for
    // that grid's results (griddepcontrol.wait) before it reads anything
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, k_verify, args) == cudaSuccess ? DSBD_OK : DSBD_ERR_CUDA;
}

int stats_grid(int64_t items) {
    // enough warps to cover the items, capped at a few waves of a 148-SM part
    int64_t blocks = (items + kWarps - 1) / kWarps;
    const int64_t cap = 148 * 8 * 4;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

}  // namespace

extern "C" size_t dsbd_verify_workspace(const dsbd_forest_t *forest, const dsbd_verify_params_t *params) {
    if (check_forest(forest) != DSBD_OK || check_params(params) != DSBD_OK) return 0;
    return make_layout(forest, params->V).total;
}

extern "C" int dsbd_verify_step(const dsbd_forest_t *f, const dsbd_verify_params_t *p,
                                const float *logits_p, const float *logits_q, int64_t row_stride,
                                const float *root_logp, const float *root_logq,
                                const dsbd_verify_out_t *out, void *workspace, size_t workspace_bytes,
                                int32_t *status, dsbd_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    int rc = check_forest(f);
    if (rc) return rc;
    rc = check_params(p);
    if (rc) return rc;
    rc = check_widths(p);
    if (rc) return rc;
    if (!logits_p || !logits_q || !root_logp || !root_logq || !out || !workspace || !status)
        return DSBD_ERR_INVALID_ARG;
    if (row_stride < p->V) return DSBD_ERR_INVALID_ARG;
    if (!out->l_last || !out->out_width || !out->out_off || !out->out_parent || !out->out_node ||
        !out->out_root_beam || !out->out_token || !out->out_logp || !out->out_logq ||
        !out->out_source || !out->node_status || !out->layer_width)
        return DSBD_ERR_INVALID_ARG;
    const Layout L = make_layout(f, p->V);
    if (workspace_bytes < L.total) return DSBD_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return DSBD_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    TileStat *stats = reinterpret_cast<TileStat *>(ws + L.stats);
    double *lse = reinterpret_cast<double *>(ws + L.lse);
    double *score = reinterpret_cast<double *>(ws + L.score);
    int32_t *depth = reinterpret_cast<int32_t *>(ws + L.depth);
    const double inv_tau = 1.0 / (double)p->temperature;
    const float k2 = (float)((double)kLog2e * inv_tau);

    const int64_t items = (int64_t)2 * f->N * L.T;
    k_tile_stats<<<stats_grid(items), kThreads, 0, stream>>>(logits_p, logits_q, row_stride, p->V, L.T,
                                                            f->N, f->N, nullptr, nullptr, k2, stats);
    if (cudaGetLastError() != cudaSuccess) return DSBD_ERR_CUDA;

    VerifyArgs a = {};
    a.R = f->R; a.N = f->N; a.gamma = f->max_depth;
    a.req_beam_off = f->req_beam_off; a.beam_node_off = f->beam_node_off;
    a.parent = f->parent; a.token = f->token; a.draft_rank = f->draft_rank;
    a.V = p->V; a.T = L.T; a.k2 = k2; a.inv_tau = inv_tau; a.thresh = (double)p->thresh;
    a.W_min = p->W_min; a.W_max = p->W_max; a.W_nom = p->W_nom;
    a.W_min_r = p->W_min_r; a.W_max_r = p->W_max_r; a.W_nom_r = p->W_nom_r;
    a.seed = p->seed; a.step = p->step;
    a.top_k = p->top_k; a.top_p = (double)p->top_p;
    a.zp = logits_p; a.zq = logits_q; a.stride = row_stride;
    a.stats = stats; a.lse = lse; a.score = score; a.depth = depth;
    a.tile_sums = reinterpret_cast<double *>(ws + L.sums);
    a.max_m = L.max_m; a.max_live = L.max_live;
    a.hist = reinterpret_cast<unsigned long long *>(ws + L.hist);
#ifdef DSBD_PHASE_TIMING
    a.dbg = reinterpret_cast<unsigned long long *>(ws + L.total) - (size_t)f->R * 256;
#endif
    a.out = *out; a.status = status; a.select_mode = 0; a.check_widths = 1;
    a.lse_w = lse; a.score_w = score; a.depth_w = depth;
    a.root_logp = root_logp; a.root_logq = root_logq;
    return launch_verify(a, f->R, L.max_live * L.T, stream);
}

extern "C" int dsbd_node_stats(const dsbd_forest_t *f, const dsbd_verify_params_t *p,
                               const float *logits_p, const float *logits_q, int64_t row_stride,
                               float *lse_p, float *lse_q, void *workspace, size_t workspace_bytes,
                               dsbd_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    int rc = check_forest(f);
    if (rc) return rc;
    rc = check_params(p);
    if (rc) return rc;
    if (!logits_p || !logits_q || !lse_p || !lse_q || !workspace || row_stride < p->V)
        return DSBD_ERR_INVALID_ARG;
    const Layout L = make_layout(f, p->V);
    if (workspace_bytes < L.total) return DSBD_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return DSBD_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    TileStat *stats = reinterpret_cast<TileStat *>(ws + L.stats);
    double *lse = reinterpret_cast<double *>(ws + L.lse);
    const double inv_tau = 1.0 / (double)p->temperature;
    const float k2 = (float)((double)kLog2e * inv_tau);
    const int64_t items = (int64_t)2 * f->N * L.T;
    k_tile_stats<<<stats_grid(items), kThreads, 0, stream>>>(logits_p, logits_q, row_stride, p->V, L.T,
                                                            f->N, f->N, nullptr, nullptr, k2, stats);
    const int64_t warps = (int64_t)2 * f->N;
    k_row_finish<<<(unsigned)((warps + kWarps - 1) / kWarps), kThreads, 0, stream>>>(
        stats, L.T, f->N, f->N, nullptr, nullptr, inv_tau, lse, lse_p, lse_q);
    return cudaGetLastError() == cudaSuccess ? DSBD_OK : DSBD_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------
// dsbd_draft_layer: a beam-sampling step of the small model is the "extra layer" of the
// verification kernel on a forest that has only roots (the current beams), with the small
// model's logits standing for both models: W_S inverse-CDF draws from T o q_beam.
// ---------------------------------------------------------------------------------------
namespace {
__global__ void k_draft_init(int n_beams, int32_t *beam_node_off, int32_t *parent) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i <= n_beams) beam_node_off[i] = i;
    if (i < n_beams) parent[i] = -1;
}

struct DraftLayout {
    Layout v;
    size_t beam_node_off, parent, l_last, out_width, layer_width, node_status, out_node, out_root_beam,
        out_source, out_logp, total;
};

dsbd_forest_t draft_forest(int R, int n_beams, const dsbd_draft_params_t *p) {
    dsbd_forest_t f = {};
    f.R = R; f.B = n_beams; f.N = n_beams; f.max_depth = 0;
    f.max_tree_nodes = 1; f.max_req_beams = p->max_req_beams; f.max_layer_nodes = 0;
    return f;
}

bool draft_args_ok(int R, int n_beams, const dsbd_draft_params_t *p) {
    return p && R > 0 && n_beams > 0 && p->V > 0 && p->temperature > 0.f && p->n_slots > 0 &&
           p->max_req_beams > 0 && (p->W_S >= 0 || p->W_S_r) && p->layer >= 0 && p->top_k >= 0;
}

DraftLayout make_draft_layout(int R, int n_beams, const dsbd_draft_params_t *p) {
    DraftLayout D;
    const dsbd_forest_t f = draft_forest(R, n_beams, p);
    D.v = make_layout(&f, p->V);
    size_t off = D.v.total;
    auto take = [&](size_t bytes) { const size_t at = off; off = align_up(off + bytes, 256); return at; };
    D.beam_node_off = take(sizeof(int32_t) * ((size_t)n_beams + 1));
    D.parent = take(sizeof(int32_t) * (size_t)n_beams);
    D.l_last = take(sizeof(int32_t) * (size_t)R);
    D.out_width = take(sizeof(int32_t) * (size_t)R);
    D.layer_width = take(sizeof(int32_t) * (size_t)R);
    D.node_status = take((size_t)n_beams);
    D.out_node = take(sizeof(int32_t) * (size_t)p->n_slots);
    D.out_root_beam = take(sizeof(int32_t) * (size_t)p->n_slots);
    D.out_source = take(sizeof(int32_t) * (size_t)p->n_slots);
    D.out_logp = take(sizeof(float) * (size_t)p->n_slots);
    D.total = off;
    return D;
}
}  // namespace

extern "C" size_t dsbd_draft_workspace(int32_t R, int32_t n_beams, const dsbd_draft_params_t *p) {
    if (!draft_args_ok(R, n_beams, p)) return 0;
    return make_draft_layout(R, n_beams, p).total;
}

extern "C" int dsbd_draft_layer(int32_t R, int32_t n_beams, const int32_t *req_beam_off,
                                const dsbd_draft_params_t *p, const float *logits_q, int64_t row_stride,
                                const float *beam_logq, const int32_t *out_off, int32_t *out_parent,
                                int32_t *out_token, float *out_logq, int32_t *req_error, void *workspace,
                                size_t workspace_bytes, int32_t *status, dsbd_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    if (!draft_args_ok(R, n_beams, p)) return DSBD_ERR_INVALID_ARG;
    if (!req_beam_off || !logits_q || !beam_logq || !out_off || !out_parent || !out_token || !out_logq ||
        !workspace || !status || row_stride < p->V)
        return DSBD_ERR_INVALID_ARG;
    if (p->max_req_beams > DSBD_MAX_LIVE || p->top_k > 64) return DSBD_ERR_UNSUPPORTED;
    if (p->top_k == 0 && p->top_p > 0.f && p->top_p < 1.f) return DSBD_ERR_UNSUPPORTED;
    const DraftLayout D = make_draft_layout(R, n_beams, p);
    if (workspace_bytes < D.total) return DSBD_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return DSBD_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    const Layout &L = D.v;
    TileStat *stats = reinterpret_cast<TileStat *>(ws + L.stats);
    double *lse = reinterpret_cast<double *>(ws + L.lse);
    double *score = reinterpret_cast<double *>(ws + L.score);
    int32_t *depth = reinterpret_cast<int32_t *>(ws + L.depth);
    int32_t *beam_node_off = reinterpret_cast<int32_t *>(ws + D.beam_node_off);
    int32_t *parent = reinterpret_cast<int32_t *>(ws + D.parent);
    const double inv_tau = 1.0 / (double)p->temperature;
    const float k2 = (float)((double)kLog2e * inv_tau);

    k_draft_init<<<(n_beams + 1 + 255) / 256, 256, 0, stream>>>(n_beams, beam_node_off, parent);
    const int64_t items = (int64_t)n_beams * L.T;
    k_tile_stats<<<stats_grid(items), kThreads, 0, stream>>>(logits_q, logits_q, row_stride, p->V, L.T, n_beams,
                                                            n_beams, nullptr, nullptr, k2, stats, 1);
    if (cudaGetLastError() != cudaSuccess) return DSBD_ERR_CUDA;

    VerifyArgs a = {};
    a.R = R; a.N = n_beams; a.gamma = 0;
    a.req_beam_off = req_beam_off; a.beam_node_off = beam_node_off; a.parent = parent;
    a.token = nullptr; a.draft_rank = nullptr;
    a.V = p->V; a.T = L.T; a.k2 = k2; a.inv_tau = inv_tau; a.thresh = 0.5;
    a.W_min = 1; a.W_max = 1; a.W_nom = p->W_S; a.W_nom_r = p->W_S_r;
    a.seed = p->seed; a.step = p->step;
    a.top_k = p->top_k; a.top_p = (double)p->top_p;
    a.zp = logits_q; a.zq = logits_q; a.stride = row_stride;
    a.stats = stats; a.lse = lse; a.score = score; a.depth = depth;
    a.tile_sums = reinterpret_cast<double *>(ws + L.sums);
    a.max_m = L.max_m; a.max_live = L.max_live;
    a.hist = reinterpret_cast<unsigned long long *>(ws + L.hist);
#ifdef DSBD_PHASE_TIMING
    a.dbg = reinterpret_cast<unsigned long long *>(ws + L.total) - (size_t)R * 256;
#endif
    a.extra_layer_bias = (1u << 29) + (uint32_t)p->layer - 1u;     // layer number 2^29 + layer
    a.out = dsbd_verify_out_t{};
    a.out.l_last = reinterpret_cast<int32_t *>(ws + D.l_last);
    a.out.out_width = reinterpret_cast<int32_t *>(ws + D.out_width);
    a.out.out_off = out_off;
    a.out.out_parent = out_parent;
    a.out.out_node = reinterpret_cast<int32_t *>(ws + D.out_node);
    a.out.out_root_beam = reinterpret_cast<int32_t *>(ws + D.out_root_beam);
    a.out.out_token = out_token;
    a.out.out_logp = reinterpret_cast<float *>(ws + D.out_logp);
    a.out.out_logq = out_logq;
    a.out.out_source = reinterpret_cast<int32_t *>(ws + D.out_source);
    a.out.node_status = reinterpret_cast<int8_t *>(ws + D.node_status);
    a.out.layer_width = reinterpret_cast<int32_t *>(ws + D.layer_width);
    a.out.req_error = req_error;
    a.status = status; a.select_mode = 0;
    a.lse_w = lse; a.score_w = score; a.depth_w = depth;
    a.root_logp = beam_logq; a.root_logq = beam_logq;
    return launch_verify(a, R, L.max_live * L.T, stream);
}

// ---------------------------------------------------------------------------------------
// dsbd_node_stats_static: the same two kernels as dsbd_node_stats, with their scratch (tile
// statistics and double-precision row sums) in a fixed array that is part of the library image
// instead of a caller-supplied workspace.
// ---------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[DSBD_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
unsigned char *g_static_scratch_ptr[kMaxDevices];   // device address of the array, per device

// The array's name is only a host-side handle; the device address a kernel can use has to be
// asked for, once per device, while that device is current.
int static_scratch_address(unsigned char **ptr) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DSBD_ERR_CUDA;
    unsigned char *p = __atomic_load_n(&g_static_scratch_ptr[dev], __ATOMIC_ACQUIRE);
    if (!p) {
        void *addr = nullptr;
        if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || !addr) return DSBD_ERR_CUDA;
        p = static_cast<unsigned char *>(addr);
        __atomic_store_n(&g_static_scratch_ptr[dev], p, __ATOMIC_RELEASE);
    }
    *ptr = p;
    return DSBD_OK;
}
}  // namespace

extern "C" int dsbd_node_stats_static(const dsbd_forest_t *f, const dsbd_verify_params_t *p,
                                      const float *logits_p, const float *logits_q, int64_t row_stride,
                                      float *lse_p, float *lse_q, dsbd_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    int rc = check_forest(f);
    if (rc) return rc;
    rc = check_params(p);
    if (rc) return rc;
    if (!logits_p || !logits_q || !lse_p || !lse_q || row_stride < p->V) return DSBD_ERR_INVALID_ARG;
    // scratch this call needs: tile statistics of both models, then the double row sums
    const int T = (p->V + kTile - 1) / kTile;
    const size_t stats_bytes = align_up(sizeof(TileStat) * 2 * (size_t)f->N * T, 256);
    const size_t need = stats_bytes + sizeof(double) * 2 * (size_t)f->N;
    if (need > (size_t)DSBD_STATIC_SCRATCH_BYTES) return DSBD_ERR_WORKSPACE_TOO_SMALL;
    unsigned char *scratch = nullptr;
    rc = static_scratch_address(&scratch);
    if (rc) return rc;
    // Nothing here has to start from zero: both kernels overwrite every entry they later read.
    TileStat *stats = reinterpret_cast<TileStat *>(scratch);
    double *lse = reinterpret_cast<double *>(scratch + stats_bytes);
    const double inv_tau = 1.0 / (double)p->temperature;
    const float k2 = (float)((double)kLog2e * inv_tau);
    const int64_t items = (int64_t)2 * f->N * T;
    k_tile_stats<<<stats_grid(items), kThreads, 0, stream>>>(logits_p, logits_q, row_stride, p->V, T,
                                                            f->N, f->N, nullptr, nullptr, k2, stats);
    const int64_t warps = (int64_t)2 * f->N;
    k_row_finish<<<(unsigned)((warps + kWarps - 1) / kWarps), kThreads, 0, stream>>>(
        stats, T, f->N, f->N, nullptr, nullptr, inv_tau, lse, lse_p, lse_q);
    return cudaGetLastError() == cudaSuccess ? DSBD_OK : DSBD_ERR_CUDA;
}

extern "C" int dsbd_select_width(const dsbd_forest_t *f, const dsbd_verify_params_t *p,
                                 const float *logits_p, const float *logits_q, int64_t row_stride,
                                 const float *node_logp, const float *node_logq,
                                 const int32_t *live_off, const int32_t *live_nodes, const int32_t *m,
                                 int32_t *width, float *alpha, float *tail, int32_t out_stride,
                                 void *workspace, size_t workspace_bytes, int32_t *status,
                                 dsbd_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    int rc = check_forest(f);
    if (rc) return rc;
    rc = check_params(p);
    if (rc) return rc;
    rc = check_widths(p);
    if (rc) return rc;
    if (!logits_p || !logits_q || !node_logp || !node_logq || !live_off || !live_nodes || !m ||
        !width || !workspace || !status)
        return DSBD_ERR_INVALID_ARG;
    if (row_stride < p->V || ((alpha || tail) && out_stride < 1)) return DSBD_ERR_INVALID_ARG;
    const Layout L = make_layout(f, p->V);
    if (workspace_bytes < L.total) return DSBD_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return DSBD_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);
    TileStat *stats = reinterpret_cast<TileStat *>(ws + L.stats);
    double *lse = reinterpret_cast<double *>(ws + L.lse);
    const double inv_tau = 1.0 / (double)p->temperature;
    const float k2 = (float)((double)kLog2e * inv_tau);

    // statistics of the live rows only; their number is live_off[R], known on the device
    const int max_rows = f->R * L.max_live < f->N ? f->R * L.max_live : f->N;
    const int64_t items = (int64_t)2 * max_rows * L.T;
    k_tile_stats<<<stats_grid(items), kThreads, 0, stream>>>(logits_p, logits_q, row_stride, p->V, L.T,
                                                            f->N, max_rows, live_nodes, live_off + f->R, k2, stats);
    {
        const int64_t warps = (int64_t)2 * max_rows;
        k_row_finish<<<(unsigned)((warps + kWarps - 1) / kWarps), kThreads, 0, stream>>>(
            stats, L.T, f->N, max_rows, live_nodes, live_off + f->R, inv_tau, lse, nullptr, nullptr);
    }
    if (cudaGetLastError() != cudaSuccess) return DSBD_ERR_CUDA;

    VerifyArgs a = {};
    a.R = f->R; a.N = f->N; a.gamma = f->max_depth;
    a.req_beam_off = f->req_beam_off; a.beam_node_off = f->beam_node_off;
    a.parent = f->parent; a.token = f->token; a.draft_rank = f->draft_rank;
    a.V = p->V; a.T = L.T; a.k2 = k2; a.inv_tau = inv_tau; a.thresh = (double)p->thresh;
    a.W_min = p->W_min; a.W_max = p->W_max; a.W_nom = p->W_nom;
    a.W_min_r = p->W_min_r; a.W_max_r = p->W_max_r; a.W_nom_r = p->W_nom_r;
    a.seed = p->seed; a.step = p->step;
    a.top_k = p->top_k; a.top_p = (double)p->top_p;
    a.zp = logits_p; a.zq = logits_q; a.stride = row_stride;
    a.stats = stats; a.lse = lse; a.score = nullptr; a.depth = nullptr;
    a.tile_sums = reinterpret_cast<double *>(ws + L.sums);
    a.max_m = L.max_m; a.max_live = L.max_live;
    a.hist = reinterpret_cast<unsigned long long *>(ws + L.hist);
#ifdef DSBD_PHASE_TIMING
    a.dbg = reinterpret_cast<unsigned long long *>(ws + L.total) - (size_t)f->R * 256;
#endif
    a.status = status; a.select_mode = 1; a.check_widths = 1;
    a.sel_logp = node_logp; a.sel_logq = node_logq;
    a.live_off = live_off; a.live_nodes = live_nodes; a.m_in = m; a.sel_rows = max_rows;
    a.width_out = width; a.alpha_out = alpha; a.tail_out = tail; a.out_stride = out_stride;
    return launch_verify(a, f->R, L.max_live * L.T, stream);
}
