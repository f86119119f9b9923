// dsbd_forest_attention: forest-masked attention for sm_100a.
//
// Every draft node attends to the KV prefix of its own beam plus its ancestors-or-self inside
// its own tree (the topology-aware tree mask, one KV cache per input beam).  A work unit is
// one (beam, KV head): its prefix is a contiguous [L_b, d] matrix for K and for V, and all
// query rows of the tree that map to this KV head (n_tree * Hq/Hkv of them) share it, so the
// prefix is streamed once per unit.
//
// k_forest_attn_simt  fp32-accumulating CUDA-core kernel for any dtype: K/V tiles are staged
//                     in shared memory with 128-bit loads, one thread pair per query row.
#include <cuda_bf16.h>
#include <math.h>


#include "dsbd_attention.cuh"

using namespace dsbd;

namespace {

constexpr int kRowsPerBlock = 64;     // query rows per CTA (two threads each)
constexpr int kTok = 32;              // tokens per staged tile

template <class T> struct Elem;
template <> struct Elem<float> {
    static constexpr int kPerVec = 4;
    __device__ static void load(const float *p, float *dst) {
        const float4 v = *reinterpret_cast<const float4 *>(p);
        dst[0] = v.x; dst[1] = v.y; dst[2] = v.z; dst[3] = v.w;
    }
    __device__ static float to_float(float v) { return v; }
    __device__ static float from_float(float v) { return v; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int kPerVec = 8;
    __device__ static void load(const __nv_bfloat16 *p, float *dst) {
        const uint4 v = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            dst[2 * i] = __uint_as_float(w[i] << 16);
            dst[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    __device__ static float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
    __device__ static __nv_bfloat16 from_float(float v) { return __float2bfloat16_rn(v); }
};

struct AttnArgs {
    int B, N, Hq, Hkv, group;
    float scale_log2;              // scale * log2(e)
    const int32_t *beam_node_off, *parent;
    const int64_t *prefix_off;
    const void *q, *k_new, *v_new, *k_prefix, *v_prefix;
    void *out;
    int32_t *status;
    int row_blocks;
};

// Stage `cnt` (<= kTok) rows of d elements, row i at src + i*row_stride, into fp32 smem.
template <class T, int D>
__device__ void stage_rows(const T *src, int64_t row_stride, int cnt, float *dst, int tid, int nthreads) {
    constexpr int PV = Elem<T>::kPerVec;
    constexpr int VPR = D / PV;           // vectors per row
    for (int i = tid; i < kTok * VPR; i += nthreads) {
        const int row = i / VPR, c = (i - row * VPR) * PV;
        float tmp[PV];
        if (row < cnt) {
            Elem<T>::load(src + (int64_t)row * row_stride + c, tmp);
        } else {
#pragma unroll
            for (int e = 0; e < PV; ++e) tmp[e] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < PV; ++e) dst[row * D + c + e] = tmp[e];
    }
}

template <class T, int D>
__global__ void __launch_bounds__(2 * kRowsPerBlock)
k_forest_attn_simt(AttnArgs a) {
    constexpr int H = D / 2;              // elements per thread of the pair
    extern __shared__ float smem[];
    float *ks = smem;                     // [kTok][D]
    float *vs = smem + kTok * D;          // [kTok][D]
    __shared__ unsigned long long anc[DSBD_MAX_TREE_NODES];

    int unit = blockIdx.x;
    const int rb = unit % a.row_blocks; unit /= a.row_blocks;
    const int g = unit % a.Hkv;
    const int b = unit / a.Hkv;
    const int n_lo = a.beam_node_off[b];
    const int n_tree = a.beam_node_off[b + 1] - n_lo;
    const int M = n_tree * a.group;
    if (rb * kRowsPerBlock >= M) return;
    const int tid = threadIdx.x, nthreads = blockDim.x;

    // ancestor-or-self bitmasks of the tree: anc[i] = anc[parent(i)] | bit(i)
    if (tid == 0) {
        for (int i = 0; i < n_tree; ++i) {
            const int par = a.parent[n_lo + i];
            unsigned long long m = 1ull << i;
            if (par >= n_lo && par < n_lo + i) m |= anc[par - n_lo];
            else if (par != -1 || i != 0) report(a.status, DSBD_DEV_BAD_FOREST);
            anc[i] = m;
        }
    }

    const int row = rb * kRowsPerBlock + (tid >> 1);     // query row inside the unit
    const int half = tid & 1;
    const bool active = row < M;
    const int node = active ? row / a.group : 0;          // tree-local node
    const int hq = g * a.group + (active ? row % a.group : 0);
    const T *Q = static_cast<const T *>(a.q);
    float qv[H], o[H];
#pragma unroll
    for (int c = 0; c < H; ++c) {
        qv[c] = active ? Elem<T>::to_float(Q[((int64_t)(n_lo + node) * a.Hq + hq) * D + half * H + c]) *
                             a.scale_log2
                       : 0.f;
        o[c] = 0.f;
    }
    float mrun = -INFINITY, lrun = 0.f;
    __syncthreads();
    const unsigned long long my_anc = anc[node];

    const int64_t L = a.prefix_off[b + 1] - a.prefix_off[b];
    const T *kp = static_cast<const T *>(a.k_prefix) + (a.prefix_off[b] * a.Hkv + (int64_t)g * L) * D;
    const T *vp = static_cast<const T *>(a.v_prefix) + (a.prefix_off[b] * a.Hkv + (int64_t)g * L) * D;
    const T *kn = static_cast<const T *>(a.k_new) + ((int64_t)n_lo * a.Hkv + g) * D;
    const T *vn = static_cast<const T *>(a.v_new) + ((int64_t)n_lo * a.Hkv + g) * D;

    const int64_t total = L + n_tree;
    for (int64_t t0 = 0; t0 < total; t0 += kTok) {
        // a tile never straddles the prefix / tree boundary
        const bool in_tree = t0 >= L;
        int cnt;
        if (!in_tree) {
            cnt = (int)((L - t0) < kTok ? (L - t0) : kTok);
            stage_rows<T, D>(kp + t0 * D, D, cnt, ks, tid, nthreads);
            stage_rows<T, D>(vp + t0 * D, D, cnt, vs, tid, nthreads);
        } else {
            const int j0 = (int)(t0 - L);
            cnt = (n_tree - j0) < kTok ? (n_tree - j0) : kTok;
            stage_rows<T, D>(kn + (int64_t)j0 * a.Hkv * D, (int64_t)a.Hkv * D, cnt, ks, tid, nthreads);
            stage_rows<T, D>(vn + (int64_t)j0 * a.Hkv * D, (int64_t)a.Hkv * D, cnt, vs, tid, nthreads);
        }
        __syncthreads();
        float s[kTok];
        float tmax = -INFINITY;
#pragma unroll 4
        for (int j = 0; j < kTok; ++j) {
            const float4 *kr = reinterpret_cast<const float4 *>(ks + j * D + half * H);
            float acc = 0.f;
#pragma unroll
            for (int c = 0; c < H / 4; ++c) {
                const float4 kv = kr[c];
                acc = fmaf(qv[4 * c], kv.x, acc);
                acc = fmaf(qv[4 * c + 1], kv.y, acc);
                acc = fmaf(qv[4 * c + 2], kv.z, acc);
                acc = fmaf(qv[4 * c + 3], kv.w, acc);
            }
            acc += __shfl_xor_sync(kFull, acc, 1);
            bool vis = j < cnt;
            if (in_tree) vis = vis && ((my_anc >> ((int)(t0 - L) + j)) & 1ull);
            s[j] = vis ? acc : -INFINITY;
            tmax = fmaxf(tmax, s[j]);
        }
        if (tmax > -INFINITY) {
            const float mnew = fmaxf(mrun, tmax);
            const float corr = exp2f(mrun - mnew);      // 0 when mrun == -inf
            lrun *= corr;
#pragma unroll
            for (int c = 0; c < H; ++c) o[c] *= corr;
#pragma unroll 4
            for (int j = 0; j < kTok; ++j) {
                const float p = exp2f(s[j] - mnew);      // 0 for masked entries
                lrun += p;
                const float4 *vr = reinterpret_cast<const float4 *>(vs + j * D + half * H);
#pragma unroll
                for (int c = 0; c < H / 4; ++c) {
                    const float4 vv = vr[c];
                    o[4 * c] = fmaf(p, vv.x, o[4 * c]);
                    o[4 * c + 1] = fmaf(p, vv.y, o[4 * c + 1]);
                    o[4 * c + 2] = fmaf(p, vv.z, o[4 * c + 2]);
                    o[4 * c + 3] = fmaf(p, vv.w, o[4 * c + 3]);
                }
            }
            mrun = mnew;
        }
        __syncthreads();
        if (!in_tree && t0 + kTok > L) t0 = L - kTok;   // next tile starts the tree part
    }
    if (active) {
        T *O = static_cast<T *>(a.out);
        const float inv = 1.f / lrun;
#pragma unroll
        for (int c = 0; c < H; ++c)
            O[((int64_t)(n_lo + node) * a.Hq + hq) * D + half * H + c] = Elem<T>::from_float(o[c] * inv);
    }
}

template <class T, int D>
int launch_simt(const AttnArgs &a, int units, cudaStream_t stream) {
    const size_t smem = sizeof(float) * 2 * kTok * D;
    k_forest_attn_simt<T, D><<<units, 2 * kRowsPerBlock, smem, stream>>>(a);
    return cudaGetLastError() == cudaSuccess ? DSBD_OK : DSBD_ERR_CUDA;
}

int check(const dsbd_forest_t *f, const dsbd_attn_desc_t *d) {
    if (!f || !d || f->B <= 0 || f->N <= 0 || !f->beam_node_off || !f->parent) return DSBD_ERR_INVALID_ARG;
    if (d->Hq <= 0 || d->Hkv <= 0 || d->Hq % d->Hkv) return DSBD_ERR_INVALID_ARG;
    if (d->d != 64 && d->d != 128) return DSBD_ERR_UNSUPPORTED;
    if (d->dtype != DSBD_DTYPE_BF16 && d->dtype != DSBD_DTYPE_F32) return DSBD_ERR_UNSUPPORTED;
    if (f->max_tree_nodes <= 0) return DSBD_ERR_INVALID_ARG;
    if (f->max_tree_nodes > DSBD_MAX_TREE_NODES_TC) return DSBD_ERR_UNSUPPORTED;
    return DSBD_OK;
}

}  // namespace

extern "C" size_t dsbd_forest_attention_workspace(const dsbd_forest_t *f, const dsbd_attn_desc_t *d) {
    if (check(f, d) != DSBD_OK) return 0;
    return attention_tc_supported(f, d) ? attention_tc_workspace(f, d) : 256;
}

extern "C" int dsbd_forest_attention_launches(const dsbd_forest_t *f, const dsbd_attn_desc_t *d) {
    if (check(f, d) != DSBD_OK) return 0;
    return attention_tc_supported(f, d) ? attention_tc_launches(f, d) : 1;
}

extern "C" int dsbd_forest_attention(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, const void *q,
                                     const void *k_new, const void *v_new, const void *k_prefix,
                                     const void *v_prefix, const int64_t *prefix_off, void *out,
                                     void *workspace, size_t workspace_bytes, int32_t *status,
                                     dsbd_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    const int rc = check(f, d);
    if (rc) return rc;
    if (!q || !k_new || !v_new || !prefix_off || !out || !status) return DSBD_ERR_INVALID_ARG;
    if (d->total_prefix > 0 && (!k_prefix || !v_prefix)) return DSBD_ERR_INVALID_ARG;
    if (workspace_bytes < dsbd_forest_attention_workspace(f, d) || !workspace) return DSBD_ERR_WORKSPACE_TOO_SMALL;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_new) |
                           reinterpret_cast<uintptr_t>(v_new) | reinterpret_cast<uintptr_t>(k_prefix) |
                           reinterpret_cast<uintptr_t>(v_prefix) | reinterpret_cast<uintptr_t>(out);
    if (bits & 15) return DSBD_ERR_UNSUPPORTED;

    if (attention_tc_supported(f, d))
        return launch_attention_tc(f, d, q, k_new, v_new, k_prefix, v_prefix, prefix_off, out, workspace,
                                   workspace_bytes, status, stream);

    if (f->max_tree_nodes > DSBD_MAX_TREE_NODES) return DSBD_ERR_UNSUPPORTED;      // CUDA-core kernel: 64-bit masks
    AttnArgs a = {};
    a.B = f->B; a.N = f->N; a.Hq = d->Hq; a.Hkv = d->Hkv; a.group = d->Hq / d->Hkv;
    a.scale_log2 = d->scale * 1.4426950408889634f;
    a.beam_node_off = f->beam_node_off; a.parent = f->parent; a.prefix_off = prefix_off;
    a.q = q; a.k_new = k_new; a.v_new = v_new; a.k_prefix = k_prefix; a.v_prefix = v_prefix;
    a.out = out; a.status = status;
    const int max_rows = f->max_tree_nodes * a.group;
    a.row_blocks = (max_rows + kRowsPerBlock - 1) / kRowsPerBlock;
    const int units = f->B * d->Hkv * a.row_blocks;
    if (d->dtype == DSBD_DTYPE_F32)
        return d->d == 64 ? launch_simt<float, 64>(a, units, stream) : launch_simt<float, 128>(a, units, stream);
    return d->d == 64 ? launch_simt<__nv_bfloat16, 64>(a, units, stream)
                      : launch_simt<__nv_bfloat16, 128>(a, units, stream);
}

extern "C" size_t dsbd_forest_attention_paged_workspace(const dsbd_forest_t *f, const dsbd_attn_desc_t *d,
                                                        const dsbd_kv_pages_t *pages) {
    if (check(f, d) != DSBD_OK || !pages || pages->n_pages <= 0 || pages->n_layers < 0) return 0;
    if (!attention_tc_supported(f, d, pages->n_pages) || !attention_tc_layers_ok(f, d, pages)) return 0;
    return attention_tc_workspace(f, d, pages->n_layers);
}

extern "C" int dsbd_forest_attention_paged(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, const void *q,
                                           const void *k_new, const void *v_new, const void *k_pool,
                                           const void *v_pool, const dsbd_kv_pages_t *pages,
                                           const int64_t *prefix_off, void *out, void *workspace,
                                           size_t workspace_bytes, int32_t *status, dsbd_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    const int rc = check(f, d);
    if (rc) return rc;
    if (!q || !k_new || !v_new || !k_pool || !v_pool || !pages || !pages->page_table || !pages->page_off ||
        pages->n_pages <= 0 || !prefix_off || !out || !status)
        return DSBD_ERR_INVALID_ARG;
    if (!attention_tc_supported(f, d, pages->n_pages)) return DSBD_ERR_UNSUPPORTED;
    if (pages->n_layers < 0 || !attention_tc_layers_ok(f, d, pages)) return DSBD_ERR_INVALID_ARG;
    if (workspace_bytes < attention_tc_workspace(f, d, pages->n_layers) || !workspace)
        return DSBD_ERR_WORKSPACE_TOO_SMALL;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k_new) |
                           reinterpret_cast<uintptr_t>(v_new) | reinterpret_cast<uintptr_t>(k_pool) |
                           reinterpret_cast<uintptr_t>(v_pool) | reinterpret_cast<uintptr_t>(out);
    if (bits & 15) return DSBD_ERR_UNSUPPORTED;
    return launch_attention_tc(f, d, q, k_new, v_new, k_pool, v_pool, prefix_off, out, workspace, workspace_bytes,
                               status, stream, pages);
}
