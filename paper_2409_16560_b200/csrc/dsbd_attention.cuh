// Internal interface between the attention entry point and its tensor-core kernel.
#pragma once

#include "dsbd_common.cuh"

namespace dsbd {

// True when the tcgen05 kernel covers this problem (bf16, d = 128, at most DSBD_MAX_TREE_NODES_TC
// nodes and 1024 query rows per tree and KV head, a non-empty KV prefix).  n_pages > 0: the caches
// are paged (k_prefix / v_prefix are then the page pools).
bool attention_tc_supported(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, int64_t n_pages = 0);

// Workspace bytes of the tensor-core path (work plan and partial results of split units; the
// partial results once per transformer layer of the call).
size_t attention_tc_workspace(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, int n_layers = 1);

// True when the layer count and layer strides of a paged call can be served (strides are whole
// rows of the operands' tensor maps and the row coordinates stay below 2^31).
bool attention_tc_layers_ok(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, const dsbd_kv_pages_t *pages);

// Kernels one call launches: the attention kernel, plus the plan and the combine kernel when used.
int attention_tc_launches(const dsbd_forest_t *f, const dsbd_attn_desc_t *d);

int launch_attention_tc(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, const void *q, const void *k_new,
                        const void *v_new, const void *k_prefix, const void *v_prefix, const int64_t *prefix_off,
                        void *out, void *workspace, size_t workspace_bytes, int32_t *status, cudaStream_t stream,
                        const dsbd_kv_pages_t *pages = nullptr);

}  // namespace dsbd
