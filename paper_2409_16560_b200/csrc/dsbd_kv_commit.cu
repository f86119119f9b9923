// KV-cache update at the end of a decode step (Section "Forest-based Parallel Decoding": the
// caches are updated according to the output beams; Section "Reducing Memory Cost": keep only
// the output beam of lowest perplexity).
//
//   k_commit_plan   one CTA: which output slots survive, their new cache lengths, the packed
//                   offsets of the new caches, the nodes on each kept beam's path, and the list
//                   of copy chunks.
//   k_commit_copy   a streaming copy: every (new beam, kv head, K|V) is a byte stream -- the
//                   input beam's cache, then one row per path node -- cut into 128 KB chunks;
//                   CTAs walk the chunk list with 128-bit loads kept out of L1 and streaming
//                   stores.  HBM-bound: read + write of every kept cache once.
//
// Paged caches (pages of 64 tokens in a pool, see dsbd_forest_attention_paged) make the update
// O(path) instead of O(prefix): a kept beam shares the full pages of its input beam and gets
// fresh pages only for the input beam's last, partly filled page plus its path.
//   k_commit_plan   (paged mode) also sizes the new page tables and the fresh pages
//   k_commit_pages  writes the tables and fills the fresh pages
//   k_commit_free   one CTA: rebuilds the free stack (every page no new table names)
#include <cuda_runtime.h>
#include <stdint.h>

#include "dsbd_common.cuh"

namespace {
using namespace dsbd;

constexpr int kPlanThreads = 1024;
constexpr int kPage = DSBD_PAGE_TOKENS;
constexpr int kCopyThreads = 256;
constexpr int kRoundBytes = 32768;                  // 8 x 16 B per thread in flight
constexpr int kRounds = 4;
constexpr int kChunkBytes = kRoundBytes * kRounds;  // one work item
constexpr int kUnits = kRoundBytes / 16 / kCopyThreads;

struct Plan {
    int32_t n_beams;          // kept output beams
    int32_t error;
    int64_t n_chunks;         // chunks of one (kv head, K|V) stream summed over the beams
    int64_t total_tokens;
};

struct CommitArgs {
    int R, B, N, gamma, Hkv, n_slots, keep_best;
    int row_bytes;                                  // d * element size
    int64_t capacity;
    const int32_t *req_beam_off, *beam_node_off, *parent;
    const int32_t *out_off, *out_width, *out_parent, *out_root_beam;
    const float *out_logp;
    const int64_t *prefix_off;
    const unsigned char *k_new, *v_new, *k_prefix, *v_prefix;
    unsigned char *k_dst, *v_dst;
    int32_t *new_req_beam_off, *new_beam_slot;
    int64_t *new_prefix_off;
    // paged mode: k_prefix / v_prefix and k_dst / v_dst are the pools [n_pages, Hkv, 64, d]
    int paged;
    int64_t n_pages;
    const int32_t *page_table;
    const int64_t *page_off;
    int32_t *new_page_table;
    int64_t *new_page_off;
    int32_t *free_stack, *free_count;
    int32_t *used;            // [n_pages + 1] workspace
    int64_t pool_layer_bytes, new_layer_bytes;   // several layers: blockIdx.y is the layer
    // workspace
    Plan *plan;
    int32_t *req_count;       // [R]     kept beams of the request, then its first new beam
    int32_t *src_beam;        // [n_slots]
    int32_t *path;            // [n_slots][gamma+1] nodes root .. parent
    int32_t *path_len;        // [n_slots]
    int64_t *chunk_off;       // [n_slots+1] copy chunks before each beam; paged: fresh pages before it
    int32_t *slot_req, *slot_depth, *req_best;   // [n_slots], [n_slots], [R]
    double *slot_key;         // [n_slots]
    int32_t *status;
};

// exclusive scan of v[0..n) in place by one CTA; returns the total in every thread
template <typename T>
__device__ T block_exclusive_scan(T *v, int n, T *warp_tot /*[32]*/) {
    const int per = (n + blockDim.x - 1) / blockDim.x;
    const int lo = min((int)threadIdx.x * per, n), hi = min(lo + per, n);
    T local = 0;
    for (int i = lo; i < hi; ++i) local += v[i];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    T incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const T t = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    T base = 0, total = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); ++w) {
        if (w < warp) base += warp_tot[w];
        total += warp_tot[w];
    }
    T run = base + incl - local;
    for (int i = lo; i < hi; ++i) { const T x = v[i]; v[i] = run; run += x; }
    __syncthreads();
    return total;
}

__global__ void __launch_bounds__(kPlanThreads)
k_commit_plan(CommitArgs a) {
    __shared__ int64_t tot64[32];
    __shared__ int32_t tot32[32];
    __shared__ int bad;
    if (threadIdx.x == 0) bad = 0;
    __syncthreads();
    // every slot on its own thread: which request it belongs to, whether it is in use, the depth
    // of its parent node (the walk to the root is a chain of dependent loads, so slots run in
    // parallel), and its perplexity key
    for (int s = threadIdx.x; s < a.n_slots; s += blockDim.x) {
        int lo = 0, hi = a.R - 1;                       // last request whose range starts at or before s
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (a.out_off[mid] <= s) lo = mid; else hi = mid - 1;
        }
        const int r = lo;
        int depth = -1;                                  // -1: slot not in use
        double key = 0.0;
        if (s >= a.out_off[r] && s < a.out_off[r] + a.out_width[r] && s < a.out_off[r + 1]) {
            const int b = a.out_root_beam[s];
            const int n = a.out_parent[s];
            if (b < a.req_beam_off[r] || b >= a.req_beam_off[r + 1] || n < a.beam_node_off[b] ||
                n >= a.beam_node_off[b + 1]) {
                bad = DSBD_DEV_BAD_FOREST;
            } else {
                depth = 0;
                for (int c = n; a.parent[c] >= 0 && depth <= a.gamma; c = a.parent[c]) ++depth;
                if (depth > a.gamma) { bad = DSBD_DEV_BAD_FOREST; depth = -1; }
                else if (a.keep_best)
                    key = -(double)a.out_logp[s] / ((double)(a.prefix_off[b + 1] - a.prefix_off[b]) + depth + 2);
            }
        }
        a.slot_req[s] = r;
        a.slot_depth[s] = depth;
        a.slot_key[s] = key;
    }
    __syncthreads();
    // kept slots per request; with keep_best the slot of lowest perplexity exp(-logp / length),
    // i.e. of lowest -logp / length, the first one on a tie
    for (int r = threadIdx.x; r < a.R; r += blockDim.x) {
        const int w = a.out_width[r];
        a.req_count[r] = w <= 0 ? 0 : (a.keep_best ? 1 : w);
        int best = -1;
        if (a.keep_best && w > 0) {
            const int s0 = a.out_off[r];
            double best_key = 0.0;
            for (int s = s0; s < s0 + w && s < a.n_slots; ++s)
                if (a.slot_depth[s] >= 0 && (best < 0 || a.slot_key[s] < best_key)) { best = s; best_key = a.slot_key[s]; }
        }
        a.req_best[r] = best;
    }
    __syncthreads();
    const int n_beams = block_exclusive_scan<int32_t>(a.req_count, a.R, tot32);
    if (n_beams > a.n_slots) { if (threadIdx.x == 0) bad = DSBD_DEV_CAPACITY; }
    __syncthreads();
    const bool fits = !bad;
    for (int r = threadIdx.x; r < a.R && fits; r += blockDim.x) a.new_req_beam_off[r] = a.req_count[r];
    // every kept slot: its new beam number, source beam, path and new length
    for (int s = threadIdx.x; s < a.n_slots && fits; s += blockDim.x) {
        const int depth = a.slot_depth[s];
        if (depth < 0) continue;
        const int r = a.slot_req[s];
        if (a.keep_best && a.req_best[r] != s) continue;
        const int j = a.req_count[r] + (a.keep_best ? 0 : s - a.out_off[r]);
        const int b = a.out_root_beam[s];
        int32_t *pj = a.path + (int64_t)j * (a.gamma + 1);
        for (int c = a.out_parent[s], i = depth; i >= 0; --i, c = a.parent[c]) pj[i] = c;
        a.path_len[j] = depth + 1;
        a.src_beam[j] = b;
        a.new_beam_slot[j] = s;
        const int64_t len = (a.prefix_off[b + 1] - a.prefix_off[b]) + depth + 1;
        a.new_prefix_off[j] = len;
        if (a.paged) {
            const int64_t L_old = len - depth - 1;
            const int64_t fresh = (L_old % kPage + depth + 1 + kPage - 1) / kPage;
            a.chunk_off[j] = fresh;
            a.new_page_off[j] = L_old / kPage + fresh;
        } else {
            a.chunk_off[j] = (len * a.row_bytes + kChunkBytes - 1) / kChunkBytes;
        }
    }
    __syncthreads();
    const bool ok = !bad;
    const int nb = ok ? n_beams : 0;
    if (threadIdx.x == 0) a.new_req_beam_off[a.R] = nb;
    for (int r = threadIdx.x; r < a.R && !ok; r += blockDim.x) a.new_req_beam_off[r] = 0;
    for (int j = nb + threadIdx.x; j < a.n_slots; j += blockDim.x) {
        a.new_beam_slot[j] = -1;
        a.new_prefix_off[j] = 0;
        a.chunk_off[j] = 0;
        if (a.paged) a.new_page_off[j] = 0;
    }
    __syncthreads();
    const int64_t total = block_exclusive_scan<int64_t>(a.new_prefix_off, a.n_slots, tot64);
    const int64_t chunks = block_exclusive_scan<int64_t>(a.chunk_off, a.n_slots, tot64);
    int64_t table_len = 0;
    if (a.paged) table_len = block_exclusive_scan<int64_t>(a.new_page_off, a.n_slots, tot64);
    if (threadIdx.x == 0) {
        a.new_prefix_off[a.n_slots] = total;
        a.chunk_off[a.n_slots] = chunks;
        int err = bad;
        if (a.paged) {
            a.new_page_off[a.n_slots] = table_len;
            if (!err && (table_len > a.capacity || chunks > (int64_t)*a.free_count)) err = DSBD_DEV_CAPACITY;
        } else if (!err && total > a.capacity) {
            err = DSBD_DEV_CAPACITY;
        }
        a.plan->n_beams = nb;
        a.plan->error = err;
        a.plan->total_tokens = total;
        a.plan->n_chunks = err ? 0 : chunks;
        if (err) report(a.status, err);
    }
}

__device__ __forceinline__ uint4 ld_stream16(const unsigned char *p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ void st_stream16(unsigned char *p, const uint4 &v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" :: "l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// Item = (chunk of the per-beam chunk list, kv head, K|V).  All offsets are multiples of 16
// bytes because a row (d elements) is.
__global__ void __launch_bounds__(kCopyThreads)
k_commit_copy(CommitArgs a) {
    __shared__ int s_j;
    const int64_t n_chunks = a.plan->n_chunks;
    const int n_beams = a.plan->n_beams;
    const int64_t items = n_chunks * a.Hkv * 2;
    const int rb = a.row_bytes;
    for (int64_t item = blockIdx.x; item < items; item += gridDim.x) {
        const int kv = (int)(item & 1);
        const int64_t rest = item >> 1;
        const int g = (int)(rest % a.Hkv);
        const int64_t c = rest / a.Hkv;
        if (threadIdx.x == 0) {
            int lo = 0, hi = n_beams - 1;              // last j with chunk_off[j] <= c
            while (lo < hi) {
                const int mid = (lo + hi + 1) >> 1;
                if (a.chunk_off[mid] <= c) lo = mid; else hi = mid - 1;
            }
            s_j = lo;
        }
        __syncthreads();
        const int j = s_j;
        const int b = a.src_beam[j];
        const int64_t L_old = a.prefix_off[b + 1] - a.prefix_off[b];
        const int plen = a.path_len[j];
        const int64_t L_new = L_old + plen;
        const int64_t stream_bytes = L_new * rb, old_bytes = L_old * rb;
        const int64_t start = (c - a.chunk_off[j]) * (int64_t)kChunkBytes;
        const unsigned char *src_old = (kv ? a.v_prefix : a.k_prefix) + (a.prefix_off[b] * a.Hkv + (int64_t)g * L_old) * rb;
        const unsigned char *src_new = kv ? a.v_new : a.k_new;
        unsigned char *dst = (kv ? a.v_dst : a.k_dst) + ((a.new_prefix_off[j]) * a.Hkv + (int64_t)g * L_new) * rb;
        const int32_t *path = a.path + (int64_t)j * (a.gamma + 1);
        for (int round = 0; round < kRounds; ++round) {
            const int64_t r0 = start + (int64_t)round * kRoundBytes;
            if (r0 >= stream_bytes) break;
            uint4 v[kUnits];
            int64_t off[kUnits];
#pragma unroll
            for (int u = 0; u < kUnits; ++u) {
                off[u] = r0 + ((int64_t)u * kCopyThreads + threadIdx.x) * 16;
                if (off[u] < old_bytes) {
                    v[u] = ld_stream16(src_old + off[u]);
                } else if (off[u] < stream_bytes) {
                    const int64_t o = off[u] - old_bytes;
                    const int t = (int)(o / rb);
                    const int within = (int)(o - (int64_t)t * rb);
                    v[u] = ld_stream16(src_new + ((int64_t)path[t] * a.Hkv + g) * rb + within);
                }
            }
#pragma unroll
            for (int u = 0; u < kUnits; ++u)
                if (off[u] < stream_bytes) st_stream16(dst + off[u], v[u]);
        }
        __syncthreads();
    }
}

// Paged update, CTA = (new beam j, kv head g, K|V): the (j, 0, K) CTA also writes the beam's page
// table; every CTA fills its head's rows of the beam's fresh pages -- the rows of the input
// beam's partial page, the path rows, then zeros (rows past a cache's length must stay finite
// because the attention multiplies them by zero weights).
__global__ void __launch_bounds__(kCopyThreads)
k_commit_pages(CommitArgs a) {
    if (a.plan->error) return;
    const int j = blockIdx.x / (a.Hkv * 2);
    if (j >= a.plan->n_beams) return;
    const int g = (blockIdx.x / 2) % a.Hkv, kv = blockIdx.x & 1;
    const int b = a.src_beam[j];
    const int64_t L_old = a.prefix_off[b + 1] - a.prefix_off[b];
    const int full = (int)(L_old / kPage), rem = (int)(L_old % kPage);
    const int plen = a.path_len[j];
    const int n_fresh = (int)(a.chunk_off[j + 1] - a.chunk_off[j]);
    const int32_t *old_pages = a.page_table + a.page_off[b];
    const int32_t *fresh = a.free_stack + (*a.free_count - 1 - a.chunk_off[j]);     // fresh page i = fresh[-i]
    int32_t *table = a.new_page_table + a.new_page_off[j];
    if (g == 0 && kv == 0 && blockIdx.y == 0) {
        for (int i = threadIdx.x; i < full; i += blockDim.x) table[i] = old_pages[i];
        for (int i = threadIdx.x; i < n_fresh; i += blockDim.x) table[full + i] = fresh[-i];
    }
    const int rb = a.row_bytes, upr = rb / 16;                   // 16-byte units per row
    const int64_t pool_shift = (int64_t)blockIdx.y * a.pool_layer_bytes;
    const unsigned char *pool_in = (kv ? a.v_prefix : a.k_prefix) + pool_shift;
    unsigned char *pool_out = (kv ? a.v_dst : a.k_dst) + pool_shift;
    const unsigned char *src_new = (kv ? a.v_new : a.k_new) + (int64_t)blockIdx.y * a.new_layer_bytes;
    const int32_t *path = a.path + (int64_t)j * (a.gamma + 1);
    const int64_t part_row0 = rem ? ((int64_t)old_pages[full] * a.Hkv + g) * kPage : 0;
    const int units = n_fresh * kPage * upr;
    for (int u = threadIdx.x; u < units; u += blockDim.x) {
        const int row = u / upr, within = (u - row * upr) * 16;  // row of the fresh pages' token range
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (row < rem) v = ld_stream16(pool_in + (part_row0 + row) * rb + within);
        else if (row < rem + plen) v = ld_stream16(src_new + ((int64_t)path[row - rem] * a.Hkv + g) * rb + within);
        const int pg = fresh[-(row / kPage)];
        st_stream16(pool_out + (((int64_t)pg * a.Hkv + g) * kPage + (row % kPage)) * rb + within, v);
    }
}

// The free stack after the update: every page that no new table names, ascending.  One CTA; a
// bitmap in shared memory for pools of up to 256 K pages, else flags in the workspace that the
// compaction walks in super-tiles of 16 per thread (four independent 128-bit loads), with a
// block scan of the per-thread counts either way.
__global__ void __launch_bounds__(kPlanThreads)
k_commit_free(CommitArgs a) {
    __shared__ int32_t warp_tot[32];
    __shared__ int32_t carry;
    if (a.plan->error) return;
    const int n = (int)a.n_pages;
    // Pools of up to 256 K pages: one bit per page in shared memory (1 = free), so that marking
    // and compaction never leave the SM; larger pools use the flag array in the workspace.
    constexpr int kBitWords = 8192;
    __shared__ uint32_t bits[kBitWords];
    if (n <= kBitWords * 32) {
        const int words = (n + 31) >> 5;
        for (int w = threadIdx.x; w < words; w += blockDim.x)
            bits[w] = (w + 1) * 32 <= n ? 0xffffffffu : ((1u << (n & 31)) - 1u);
        if (threadIdx.x == 0) carry = 0;
        __syncthreads();
        const int64_t entries = a.new_page_off[a.n_slots];
        for (int64_t i = threadIdx.x; i < entries; i += blockDim.x) {
            const int pg = a.new_page_table[i];
            if (pg >= 0 && pg < n) atomicAnd(&bits[pg >> 5], ~(1u << (pg & 31)));
        }
        __syncthreads();
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        for (int base = 0; base < words; base += kPlanThreads) {
            const int w = base + threadIdx.x;
            uint32_t m = w < words ? bits[w] : 0u;
            const int cnt = __popc(m);
            int incl = cnt;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(kFull, incl, o);
                if (lane >= o) incl += t;
            }
            if (lane == 31) warp_tot[warp] = incl;
            __syncthreads();
            int before = carry, tile_total = 0;
            for (int x = 0; x < kPlanThreads / 32; ++x) {
                if (x < warp) before += warp_tot[x];
                tile_total += warp_tot[x];
            }
            int pos = before + incl - cnt;
            while (m) {
                const int b = __ffs(m) - 1;
                a.free_stack[pos++] = w * 32 + b;
                m &= m - 1;
            }
            __syncthreads();
            if (threadIdx.x == 0) carry += tile_total;
            __syncthreads();
        }
        if (threadIdx.x == 0) *a.free_count = carry;
        return;
    }
    const int n_pad = (n + 15) & ~15;                                             // the array holds n + 1 <= n_pad + 16
    for (int i = threadIdx.x; i < n_pad; i += blockDim.x) a.used[i] = i < n ? 1 : 0;   // 1 = free
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    const int64_t entries = a.new_page_off[a.n_slots];
    for (int64_t i = threadIdx.x; i < entries; i += blockDim.x) {
        const int pg = a.new_page_table[i];
        if (pg >= 0 && pg < n) a.used[pg] = 0;
    }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int base = 0; base < n_pad; base += kPlanThreads * 16) {
        const int i0 = base + threadIdx.x * 16;
        int4 f[4];
#pragma unroll
        for (int q = 0; q < 4; ++q)
            f[q] = i0 + 4 * q < n_pad ? *reinterpret_cast<const int4 *>(a.used + i0 + 4 * q) : make_int4(0, 0, 0, 0);
        int cnt = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) cnt += f[q].x + f[q].y + f[q].z + f[q].w;
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        int before = carry, tile_total = 0;
        for (int w = 0; w < kPlanThreads / 32; ++w) {
            if (w < warp) before += warp_tot[w];
            tile_total += warp_tot[w];
        }
        int pos = before + incl - cnt;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int v[4] = {f[q].x, f[q].y, f[q].z, f[q].w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (v[e]) a.free_stack[pos++] = i0 + 4 * q + e;
        }
        __syncthreads();
        if (threadIdx.x == 0) carry += tile_total;
        __syncthreads();
    }
    if (threadIdx.x == 0) *a.free_count = carry;
}

struct Layout {
    size_t plan, req_count, src_beam, path, path_len, chunk_off, slot_req, slot_depth, req_best, slot_key, used, total;
};

Layout make_layout(const dsbd_forest_t *f, const dsbd_commit_params_t *p, int64_t n_pages = 0) {
    Layout L;
    size_t off = 0;
    L.plan = off;      off = align_up(off + sizeof(Plan), 256);
    L.req_count = off; off = align_up(off + sizeof(int32_t) * (size_t)f->R, 256);
    L.src_beam = off;  off = align_up(off + sizeof(int32_t) * (size_t)p->n_slots, 256);
    L.path = off;      off = align_up(off + sizeof(int32_t) * (size_t)p->n_slots * ((size_t)f->max_depth + 1), 256);
    L.path_len = off;  off = align_up(off + sizeof(int32_t) * (size_t)p->n_slots, 256);
    L.chunk_off = off; off = align_up(off + sizeof(int64_t) * ((size_t)p->n_slots + 1), 256);
    L.slot_req = off;  off = align_up(off + sizeof(int32_t) * (size_t)p->n_slots, 256);
    L.slot_depth = off; off = align_up(off + sizeof(int32_t) * (size_t)p->n_slots, 256);
    L.req_best = off;  off = align_up(off + sizeof(int32_t) * (size_t)f->R, 256);
    L.slot_key = off;  off = align_up(off + sizeof(double) * (size_t)p->n_slots, 256);
    L.used = off;      off = align_up(off + sizeof(int32_t) * ((size_t)n_pages + 32), 256);
    L.total = off;
    return L;
}

bool args_ok(const dsbd_forest_t *f, const dsbd_commit_params_t *p) {
    return f && p && f->R > 0 && f->B > 0 && f->N > 0 && f->max_depth >= 0 && f->req_beam_off &&
           f->beam_node_off && f->parent && p->n_slots > 0 && p->dst_capacity >= 0;
}

}  // namespace

extern "C" size_t dsbd_kv_commit_workspace(const dsbd_forest_t *forest, const dsbd_commit_params_t *params) {
    if (!args_ok(forest, params)) return 0;
    return make_layout(forest, params).total;
}

extern "C" int dsbd_kv_commit(const dsbd_forest_t *f, const dsbd_attn_desc_t *desc, const dsbd_commit_params_t *p,
                              const int32_t *out_off, const int32_t *out_width, const int32_t *out_parent,
                              const int32_t *out_root_beam, const float *out_logp, const void *k_new,
                              const void *v_new, const void *k_prefix, const void *v_prefix,
                              const int64_t *prefix_off, void *k_dst, void *v_dst, int32_t *new_req_beam_off,
                              int64_t *new_prefix_off, int32_t *new_beam_slot, void *workspace,
                              size_t workspace_bytes, int32_t *status, dsbd_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    if (!args_ok(f, p) || !desc) return DSBD_ERR_INVALID_ARG;
    if (!out_off || !out_width || !out_parent || !out_root_beam || !k_new || !v_new || !k_prefix || !v_prefix ||
        !prefix_off || !k_dst || !v_dst || !new_req_beam_off || !new_prefix_off || !new_beam_slot || !workspace ||
        !status)
        return DSBD_ERR_INVALID_ARG;
    if (p->keep_best && !out_logp) return DSBD_ERR_INVALID_ARG;
    if (desc->Hkv <= 0 || desc->d <= 0) return DSBD_ERR_INVALID_ARG;
    if (desc->dtype != DSBD_DTYPE_BF16 && desc->dtype != DSBD_DTYPE_F32) return DSBD_ERR_UNSUPPORTED;
    const int row_bytes = desc->d * (desc->dtype == DSBD_DTYPE_BF16 ? 2 : 4);
    if (row_bytes % 16) return DSBD_ERR_UNSUPPORTED;
    const uintptr_t ptrs = reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) |
                           reinterpret_cast<uintptr_t>(k_prefix) | reinterpret_cast<uintptr_t>(v_prefix) |
                           reinterpret_cast<uintptr_t>(k_dst) | reinterpret_cast<uintptr_t>(v_dst);
    if (ptrs & 15) return DSBD_ERR_UNSUPPORTED;
    const Layout L = make_layout(f, p);
    if (workspace_bytes < L.total) return DSBD_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return DSBD_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);

    CommitArgs a = {};
    a.R = f->R; a.B = f->B; a.N = f->N; a.gamma = f->max_depth; a.Hkv = desc->Hkv;
    a.n_slots = p->n_slots; a.keep_best = p->keep_best ? 1 : 0; a.row_bytes = row_bytes;
    a.capacity = p->dst_capacity;
    a.req_beam_off = f->req_beam_off; a.beam_node_off = f->beam_node_off; a.parent = f->parent;
    a.out_off = out_off; a.out_width = out_width; a.out_parent = out_parent; a.out_root_beam = out_root_beam;
    a.out_logp = out_logp; a.prefix_off = prefix_off;
    a.k_new = static_cast<const unsigned char *>(k_new); a.v_new = static_cast<const unsigned char *>(v_new);
    a.k_prefix = static_cast<const unsigned char *>(k_prefix);
    a.v_prefix = static_cast<const unsigned char *>(v_prefix);
    a.k_dst = static_cast<unsigned char *>(k_dst); a.v_dst = static_cast<unsigned char *>(v_dst);
    a.new_req_beam_off = new_req_beam_off; a.new_prefix_off = new_prefix_off; a.new_beam_slot = new_beam_slot;
    a.plan = reinterpret_cast<Plan *>(ws + L.plan);
    a.req_count = reinterpret_cast<int32_t *>(ws + L.req_count);
    a.src_beam = reinterpret_cast<int32_t *>(ws + L.src_beam);
    a.path = reinterpret_cast<int32_t *>(ws + L.path);
    a.path_len = reinterpret_cast<int32_t *>(ws + L.path_len);
    a.chunk_off = reinterpret_cast<int64_t *>(ws + L.chunk_off);
    a.slot_req = reinterpret_cast<int32_t *>(ws + L.slot_req);
    a.slot_depth = reinterpret_cast<int32_t *>(ws + L.slot_depth);
    a.req_best = reinterpret_cast<int32_t *>(ws + L.req_best);
    a.slot_key = reinterpret_cast<double *>(ws + L.slot_key);
    a.status = status;

    k_commit_plan<<<1, kPlanThreads, 0, stream>>>(a);
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    k_commit_copy<<<sms * 8, kCopyThreads, 0, stream>>>(a);
    return cudaGetLastError() == cudaSuccess ? DSBD_OK : DSBD_ERR_CUDA;
}

extern "C" size_t dsbd_kv_commit_paged_workspace(const dsbd_forest_t *forest, const dsbd_commit_params_t *params,
                                                 int64_t n_pages) {
    if (!args_ok(forest, params) || n_pages <= 0) return 0;
    return make_layout(forest, params, n_pages).total;
}

extern "C" int dsbd_kv_commit_paged(const dsbd_forest_t *f, const dsbd_attn_desc_t *desc,
                                    const dsbd_commit_params_t *p, const int32_t *out_off,
                                    const int32_t *out_width, const int32_t *out_parent,
                                    const int32_t *out_root_beam, const float *out_logp, const void *k_new,
                                    const void *v_new, void *k_pool, void *v_pool, const dsbd_kv_pages_t *pages,
                                    const int64_t *prefix_off, int32_t *free_stack, int32_t *free_count,
                                    int32_t *new_req_beam_off, int64_t *new_prefix_off, int64_t *new_page_off,
                                    int32_t *new_page_table, int32_t *new_beam_slot, void *workspace,
                                    size_t workspace_bytes, int32_t *status, dsbd_stream_t stream_) {
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_);
    if (!args_ok(f, p) || !desc || !pages) return DSBD_ERR_INVALID_ARG;
    if (!out_off || !out_width || !out_parent || !out_root_beam || !k_new || !v_new || !k_pool || !v_pool ||
        !pages->page_table || !pages->page_off || pages->n_pages <= 0 || !prefix_off || !free_stack || !free_count ||
        !new_req_beam_off || !new_prefix_off || !new_page_off || !new_page_table || !new_beam_slot || !workspace ||
        !status)
        return DSBD_ERR_INVALID_ARG;
    if (p->keep_best && !out_logp) return DSBD_ERR_INVALID_ARG;
    if (desc->Hkv <= 0 || desc->d <= 0) return DSBD_ERR_INVALID_ARG;
    if (desc->dtype != DSBD_DTYPE_BF16 && desc->dtype != DSBD_DTYPE_F32) return DSBD_ERR_UNSUPPORTED;
    if (pages->n_pages >= (int64_t)1 << 31) return DSBD_ERR_UNSUPPORTED;
    if (p->n_layers > 1 && (p->pool_layer_stride <= 0 || p->new_layer_stride <= 0 ||
                            (p->pool_layer_stride * (desc->dtype == DSBD_DTYPE_BF16 ? 2 : 4)) % 16 ||
                            (p->new_layer_stride * (desc->dtype == DSBD_DTYPE_BF16 ? 2 : 4)) % 16 ||
                            p->n_layers > 65535))
        return DSBD_ERR_INVALID_ARG;
    const int row_bytes = desc->d * (desc->dtype == DSBD_DTYPE_BF16 ? 2 : 4);
    if (row_bytes % 16) return DSBD_ERR_UNSUPPORTED;
    const uintptr_t ptrs = reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) |
                           reinterpret_cast<uintptr_t>(k_pool) | reinterpret_cast<uintptr_t>(v_pool);
    if (ptrs & 15) return DSBD_ERR_UNSUPPORTED;
    const Layout L = make_layout(f, p, pages->n_pages);
    if (workspace_bytes < L.total) return DSBD_ERR_WORKSPACE_TOO_SMALL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255) return DSBD_ERR_INVALID_ARG;
    char *ws = static_cast<char *>(workspace);

    CommitArgs a = {};
    a.R = f->R; a.B = f->B; a.N = f->N; a.gamma = f->max_depth; a.Hkv = desc->Hkv;
    a.n_slots = p->n_slots; a.keep_best = p->keep_best ? 1 : 0; a.row_bytes = row_bytes;
    a.capacity = p->dst_capacity;
    a.req_beam_off = f->req_beam_off; a.beam_node_off = f->beam_node_off; a.parent = f->parent;
    a.out_off = out_off; a.out_width = out_width; a.out_parent = out_parent; a.out_root_beam = out_root_beam;
    a.out_logp = out_logp; a.prefix_off = prefix_off;
    a.k_new = static_cast<const unsigned char *>(k_new); a.v_new = static_cast<const unsigned char *>(v_new);
    a.k_prefix = static_cast<const unsigned char *>(k_pool);
    a.v_prefix = static_cast<const unsigned char *>(v_pool);
    a.k_dst = static_cast<unsigned char *>(k_pool); a.v_dst = static_cast<unsigned char *>(v_pool);
    a.new_req_beam_off = new_req_beam_off; a.new_prefix_off = new_prefix_off; a.new_beam_slot = new_beam_slot;
    a.paged = 1; a.n_pages = pages->n_pages; a.page_table = pages->page_table; a.page_off = pages->page_off;
    a.new_page_table = new_page_table; a.new_page_off = new_page_off;
    a.free_stack = free_stack; a.free_count = free_count;
    a.plan = reinterpret_cast<Plan *>(ws + L.plan);
    a.req_count = reinterpret_cast<int32_t *>(ws + L.req_count);
    a.src_beam = reinterpret_cast<int32_t *>(ws + L.src_beam);
    a.path = reinterpret_cast<int32_t *>(ws + L.path);
    a.path_len = reinterpret_cast<int32_t *>(ws + L.path_len);
    a.chunk_off = reinterpret_cast<int64_t *>(ws + L.chunk_off);
    a.slot_req = reinterpret_cast<int32_t *>(ws + L.slot_req);
    a.slot_depth = reinterpret_cast<int32_t *>(ws + L.slot_depth);
    a.req_best = reinterpret_cast<int32_t *>(ws + L.req_best);
    a.slot_key = reinterpret_cast<double *>(ws + L.slot_key);
    a.used = reinterpret_cast<int32_t *>(ws + L.used);
    a.status = status;

    k_commit_plan<<<1, kPlanThreads, 0, stream>>>(a);
    const int n_layers = p->n_layers > 1 ? p->n_layers : 1;
    const int esz = desc->dtype == DSBD_DTYPE_BF16 ? 2 : 4;
    a.pool_layer_bytes = p->pool_layer_stride * esz;
    a.new_layer_bytes = p->new_layer_stride * esz;
    k_commit_pages<<<dim3((unsigned)(p->n_slots * desc->Hkv * 2), (unsigned)n_layers), kCopyThreads, 0, stream>>>(a);
    k_commit_free<<<1, kPlanThreads, 0, stream>>>(a);
    return cudaGetLastError() == cudaSuccess ? DSBD_OK : DSBD_ERR_CUDA;
}
