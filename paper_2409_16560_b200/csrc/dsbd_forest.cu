// Draft forest from the draft stage's draws (Section "Overview": the trajectory of the small
// model's beam sampling is a forest of W_L trees, one per input beam; from the second layer on
// every layer holds W_S nodes).  The draws arrive layer by layer; the attention and the
// verification want the nodes tree by tree, a tree's nodes contiguous with parents first.
//
//   k_forest_build   one CTA per request: which tree every draw belongs to (layer by layer),
//                    tree sizes, and each draw's place inside its tree in (layer, draw) order.
#include <cuda_runtime.h>
#include <stdint.h>

#include "dsbd_common.cuh"

namespace {
using namespace dsbd;

constexpr int kThreads = 256;
constexpr int kMaxDraws = 1024;          // gamma * W_S per request
constexpr int kMaxBeams = DSBD_MAX_LIVE;

struct BuildArgs {
    int R, gamma, W_S;
    const int32_t *req_beam_off;
    const int32_t *draw_parent, *draw_token;      // [gamma][R * W_S]
    int32_t *beam_node_off, *parent, *token, *draft_rank, *node_of_draw;
    int32_t *max_tree_nodes;                      // optional: raised to the largest tree (atomicMax)
    int32_t *status;
};

__global__ void __launch_bounds__(kThreads)
k_forest_build(BuildArgs a) {
    __shared__ int tree_of[kMaxDraws];            // tree (local beam index) of draw (l, k) at [(l-1) * W_S + k]
    __shared__ int place[kMaxDraws];              // position among the draws of its tree
    __shared__ int tree_size[kMaxBeams + 1];
    __shared__ int bad;
    const int r = blockIdx.x;
    const int b0 = a.req_beam_off[r], nb = a.req_beam_off[r + 1] - b0;
    const int W = a.W_S, n = a.gamma * W;
    const int64_t layer_stride = (int64_t)a.R * W;
    const int node0 = b0 + r * n;                 // every request before this one has gamma * W_S drafts
    if (threadIdx.x == 0) bad = 0;
    for (int i = threadIdx.x; i <= nb && i <= kMaxBeams; i += blockDim.x) tree_size[i] = 0;
    __syncthreads();
    if (nb <= 0 || nb > kMaxBeams || n > kMaxDraws) {
        if (threadIdx.x == 0) report(a.status, DSBD_DEV_BAD_FOREST);
        return;
    }
    // the tree of every draw: layer 1 names an input beam, layer l > 1 a draw of layer l - 1
    for (int l = 1; l <= a.gamma; ++l) {
        for (int k = threadIdx.x; k < W; k += blockDim.x) {
            const int p = a.draw_parent[(l - 1) * layer_stride + (int64_t)r * W + k];
            int t = -1;
            if (l == 1) { if (p >= b0 && p < b0 + nb) t = p - b0; }
            else if (p >= r * W && p < (r + 1) * W) t = tree_of[(l - 2) * W + (p - r * W)];
            if (t < 0) { bad = 1; t = 0; }
            tree_of[(l - 1) * W + k] = t;
        }
        __syncthreads();
    }
    if (bad) {
        if (threadIdx.x == 0) report(a.status, DSBD_DEV_BAD_FOREST);
        return;
    }
    // place of a draw inside its tree: draws of the same tree that come before it in (layer, draw) order
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int t = tree_of[i];
        int c = 0;
        for (int j = 0; j < i; ++j) c += tree_of[j] == t;
        place[i] = c;
        atomicAdd(&tree_size[t + 1], 1);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;                                           // first node of each tree, relative to node0
        for (int t = 0; t < nb; ++t) { const int c = tree_size[t + 1]; tree_size[t] = run; run += 1 + c; }
        tree_size[nb] = run;
    }
    __syncthreads();
    for (int t = threadIdx.x; t < nb; t += blockDim.x) {
        if (a.max_tree_nodes) atomicMax(a.max_tree_nodes, tree_size[t + 1] - tree_size[t]);
        const int root = node0 + tree_size[t];
        a.beam_node_off[b0 + t] = root;
        a.parent[root] = -1;
        a.token[root] = 0;
        a.draft_rank[root] = 0;
    }
    if (r == a.R - 1 && threadIdx.x == 0) a.beam_node_off[b0 + nb] = node0 + tree_size[nb];
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int l = i / W + 1, k = i - (l - 1) * W;
        const int t = tree_of[i];
        const int node = node0 + tree_size[t] + 1 + place[i];
        const int p = a.draw_parent[(l - 1) * layer_stride + (int64_t)r * W + k];
        int pnode;
        if (l == 1) pnode = node0 + tree_size[t];
        else {
            const int pi = (l - 2) * W + (p - r * W);
            pnode = node0 + tree_size[t] + 1 + place[pi];
        }
        a.parent[node] = pnode;
        a.token[node] = a.draw_token[(l - 1) * layer_stride + (int64_t)r * W + k];
        a.draft_rank[node] = k;
        a.node_of_draw[(l - 1) * layer_stride + (int64_t)r * W + k] = node;
    }
}

}  // namespace

extern "C" int dsbd_forest_build(int32_t R, int32_t gamma, int32_t W_S, const int32_t *req_beam_off,
                                 const int32_t *draw_parent, const int32_t *draw_token, int32_t *beam_node_off,
                                 int32_t *parent, int32_t *token, int32_t *draft_rank, int32_t *node_of_draw,
                                 int32_t *max_tree_nodes, int32_t *status, dsbd_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    if (R <= 0 || gamma <= 0 || W_S <= 0 || !req_beam_off || !draw_parent || !draw_token || !beam_node_off ||
        !parent || !token || !draft_rank || !node_of_draw || !status)
        return DSBD_ERR_INVALID_ARG;
    if ((int64_t)gamma * W_S > kMaxDraws) return DSBD_ERR_UNSUPPORTED;
    BuildArgs a = {};
    a.R = R; a.gamma = gamma; a.W_S = W_S;
    a.req_beam_off = req_beam_off; a.draw_parent = draw_parent; a.draw_token = draw_token;
    a.beam_node_off = beam_node_off; a.parent = parent; a.token = token; a.draft_rank = draft_rank;
    a.node_of_draw = node_of_draw; a.max_tree_nodes = max_tree_nodes; a.status = status;
    k_forest_build<<<R, kThreads, 0, stream>>>(a);
    return cudaGetLastError() == cudaSuccess ? DSBD_OK : DSBD_ERR_CUDA;
}
