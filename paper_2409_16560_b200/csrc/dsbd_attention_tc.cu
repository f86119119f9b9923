// Forest attention on the 5th-generation tensor cores (tcgen05 + TMEM + TMA), bf16, d = 128.
//
// Work unit = (beam, KV head): all query rows of the beam's draft tree that map to this KV head
// (row = node * group + head, at most 128) against the beam's KV prefix, streamed once in
// 64-token tiles, followed by one tile holding the tree's own keys/values under the
// ancestor-or-self mask.
//
// CTA = 6 warps, two CTAs per SM:
//   warps 0-3  softmax: warp w owns TMEM lanes 32w..32w+31 = query rows 32w..32w+31, one row per
//              thread, so row max / row sum are thread-local.  They write O at a unit's end.
//   warp 4     TMA producer: K and V tiles (2 x 64x64 bf16 boxes each, 128-byte swizzle) into a
//              ring of shared-memory stages, completion on mbarriers; and the unit's query rows
//              (two boxes of 64 columns x group heads x nodes of a 3-D map over q), issued as soon
//              as the previous unit's last Q K^T product has completed, so that the copy runs
//              behind that unit's last softmax, P V product and output write.
//   warp 5     MMA issuer (one lane): S = Q K^T (M128 N64 K16 x 8, both operands K-major in
//              shared memory) into one of two S buffers in TMEM, one tile ahead, so that it runs
//              while the softmax warps work on the previous tile; after they have written P
//              (bf16, over the S buffer they just read), O += P V (A from TMEM, B = the V tile
//              as an MN-major shared-memory operand).
// O stays in TMEM for the whole unit; its rows are rescaled only when a row maximum grows by
// more than 2^8 (the rescale is a TMEM load/scale/store by the row's own thread).
// Every mbarrier wait is bounded; on a time-out the kernel records DSBD_DEV_TIMEOUT, lets its
// copies land, frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include <algorithm>

#include "dsbd_attention.cuh"

using namespace dsbd;

namespace {

constexpr int kD = 128;                 // head dim
constexpr int kBN = 64;                 // tokens per tile
constexpr int kMaxStages = 3;
constexpr int kRows = 128;              // UMMA M
constexpr int kThreadsTc = 192;
constexpr uint32_t kTileBytes = kBN * kD * 2;         // 16 KB per K or V tile (two 8 KB boxes)
constexpr uint32_t kStageBytes = 2 * kTileBytes;      // K then V
// Shared memory of one CTA: Q (QROWS rows x 256 B as two swizzled halves), the K/V stage ring,
// then the mbarriers.  With at most 64 query rows only 64 rows of Q are stored: the MMA still
// runs with M = 128, and the A-operand rows 64..127 then alias the bytes that follow Q.  Rows of
// an MMA are independent and rows >= M are never read back, so whatever those bytes hold is
// harmless; the 16 KB saved buy a third stage at two CTAs per SM.
constexpr uint32_t smem_bytes(int qrows, int stages) { return qrows * kD * 2 + stages * kStageBytes; }
constexpr uint32_t kTmemCols = 256;
// TMEM columns: two S buffers of 64 fp32 columns (P, bf16 pairs, overwrites the first 32 columns
// of its S buffer once S has been read), then O (128 fp32 columns).
constexpr uint32_t kColS = 0, kColO = 128;
#ifdef DSBD_TEST_WAIT_TIMEOUT
// Test build only (a second library that no product path loads): waits give up after about a
// millisecond and the producer leaves out one tile, so that a wait runs out without anything
// faulting or hanging.  The test checks the status, and that the next launch of the normal
// library on the same context is correct.
constexpr long long kWaitCycles = 2000000ll;
#else
constexpr long long kWaitCycles = 2000000000ll;   // about a second
#endif

// One work item: the query rows of unit (b, g) against the prefix tokens [t0, t1) of its beam,
// plus the tree tile when `last`.  A unit split into several items leaves partial results
// (reference maximum, row sum, unnormalised O) that a second kernel merges.
// Trees with more than 128 query rows (nodes x query heads per KV head) are cut into row blocks
// of 128 rows; every row block is an item of its own that streams the same keys and values.
struct AttnItem { int b, g, t0, t1, last, nparts, slot, rb; };

struct TcArgs {
    int B, N, Hq, Hkv, group, n_units;
    int max_rows;                     // max over trees of nodes * group
    int block_rows;                   // query rows per row block: whole nodes, at most the kernel's Q tile (64 or 128)
    int nodes_per_block;              // block_rows / group
    int row_blocks;                   // ceil(max_rows / block_rows)
    const AttnItem *items;            // nullptr: one item per unit, in unit order
    const int *n_items;               // device count of items (with items)
    float *partial;                   // [slot][max_rows][130]: m_ref, l, O[128]
    float scale_log2;
    const int32_t *beam_node_off, *parent;
    const int64_t *prefix_off;
    const int32_t *page_table;        // paged caches: page ids of beam b at page_off[b] ..; nullptr: packed
    const int64_t *page_off;
    const __nv_bfloat16 *q;
    __nv_bfloat16 *out;
    int32_t *status;
    // several transformer layers in one launch (paged caches): layer l uses the same plan, page
    // tables and forest; its pools, new keys/values, queries and outputs lie l strides further
    int n_layers;                     // >= 1
    int pool_layer_rows;              // rows of the pool map between consecutive layers
    int new_layer_rows;               // rows of the k_new / v_new maps between consecutive layers
    int64_t q_layer_stride;           // elements between consecutive layers' q (and out)
    int q_layer_nodes;                // the same in nodes (rows of the query map between consecutive layers)
    int slots_per_layer;              // partial-result slots of one layer
    // Tail split of a batch of equal-length units in unit order (no plan kernel): the units from
    // tail_first on -- those that would leave most CTAs idle in a last, partly filled round --
    // are cut into tail_k parts each, so that the last round has work for (nearly) every CTA.
    int tail_first, tail_k;           // tail_k == 0: off
    // Ragged batch of whole units without a plan kernel: every CTA ranks the units by tile count
    // itself (longest first, ties by unit number, rounds alternating in direction) and keeps the
    // entries of its own column.  rank_units = number of units, 0 = off.
    int rank_units;
};

constexpr int kMaxRanked = 8;             // items of one CTA when it ranks the units itself
struct Barriers {
    unsigned long long kv_full[kMaxStages], kv_empty[kMaxStages], s_full[2], p_full[2], pv_done, q_full, q_empty, o_full;
    uint32_t tmem_base;
    int abort;
    int my_units[kMaxRanked];             // rank mode: the unit of this CTA's k-th item, -1 for none
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(void *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(void *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(void *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try(void *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: false if it gave up (time-out here, or another role already aborted).
__device__ __forceinline__ bool mbar_wait(void *bar, uint32_t parity, Barriers *sb, int32_t *status) {
    if (mbar_try(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try(bar, parity)) return true;
        if (*reinterpret_cast<volatile int *>(&sb->abort)) return false;
        if (clock64() - t0 > kWaitCycles) break;
    }
    *reinterpret_cast<volatile int *>(&sb->abort) = 1;
    report(status, DSBD_DEV_TIMEOUT);
    return false;
}

__device__ __forceinline__ void tma_load_2d(void *dst, const CUtensorMap *map, int x, int y, void *bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tma_load_2d_hint(void *dst, const CUtensorMap *map, int x, int y, void *bar, uint64_t pol) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(pol) : "memory");
}

__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, int x, int y, int z, void *bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(void *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,"
        "%28,%29,%30,%31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,"
        "%29,%30,%31,%32};"
        ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
          "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]),
          "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]),
          "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptors (128-byte swizzle, 8-row groups 1024 bytes apart).
__device__ __forceinline__ uint64_t desc_k_major(uint32_t saddr) {
    // leading offset unused for swizzled K-major (1), stride offset 1024 B, version 1, SWIZZLE_128B
    return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ uint64_t desc_mn_major(uint32_t saddr, uint32_t lbo_bytes) {
    // leading offset = distance between 64-element groups along N, stride offset = 8 k-rows
    return (uint64_t)((saddr & 0x3FFFF) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) |
           ((uint64_t)(1024 >> 4) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(N >> 3) << 17) |
           ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ int item_count(const TcArgs &a) {
    if (a.items) return *a.n_items;
    if (a.rank_units) return (a.rank_units + (int)gridDim.x - 1) / (int)gridDim.x * (int)gridDim.x;
    if (a.tail_k) return a.tail_first + (a.n_units - a.tail_first) * a.tail_k;
    return a.n_units * a.row_blocks;
}
// The item, with b = -1 when there is nothing to do: a padding entry of the plan, or a row block
// beyond the rows of this tree.  All three roles of the CTA skip such items alike.
__device__ __forceinline__ AttnItem get_item(const TcArgs &a, int it, const Barriers &sb) {
    AttnItem x;
    if (a.items) {
        x = a.items[it];
    } else if (a.rank_units) {
        // (every item index a CTA asks for is in its own column: it % grid == blockIdx.x)
        const int u = sb.my_units[it / (int)gridDim.x];
        x.rb = 0; x.b = -1; x.g = 0; x.t0 = 0; x.t1 = 0; x.last = 1; x.nparts = 1; x.slot = 0;
        if (u >= 0) {
            x.b = u / a.Hkv; x.g = u - x.b * a.Hkv;
            x.t1 = (int)(a.prefix_off[x.b + 1] - a.prefix_off[x.b]);
        }
    } else if (a.tail_k && it >= a.tail_first) {
        // part p of tail unit u: equal parts of whole tiles, the tree tile with the last part
        const int r = it - a.tail_first, u = a.tail_first + r / a.tail_k, p = r - (r / a.tail_k) * a.tail_k;
        x.rb = 0;
        x.b = u / a.Hkv; x.g = u - x.b * a.Hkv;
        const int L = (int)(a.prefix_off[x.b + 1] - a.prefix_off[x.b]);
        const int plen = ((L + a.tail_k - 1) / a.tail_k + kBN - 1) / kBN * kBN;
        x.t0 = min(p * plen, L); x.t1 = min(x.t0 + plen, L);
        x.last = (p == a.tail_k - 1); x.nparts = a.tail_k; x.slot = r;
    } else {
        const int u = it / a.row_blocks;
        x.rb = it - u * a.row_blocks;
        x.b = u / a.Hkv; x.g = u - x.b * a.Hkv;
        x.t0 = 0; x.t1 = (int)(a.prefix_off[x.b + 1] - a.prefix_off[x.b]);
        x.last = 1; x.nparts = 1; x.slot = 0;
    }
    if (x.b >= 0 && x.rb > 0 &&
        x.rb * a.block_rows >= (a.beam_node_off[x.b + 1] - a.beam_node_off[x.b]) * a.group)
        x.b = -1;
    return x;
}

// Tiles of 64 tokens that hold the tree's own keys and values (trees of up to 128 nodes).
__device__ __forceinline__ int tree_tiles(const TcArgs &a, int b) {
    return (a.beam_node_off[b + 1] - a.beam_node_off[b] + kBN - 1) / kBN;
}

__device__ __forceinline__ float ex2_ftz(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t *>(&v);
}

template <int QROWS, int kStages>
__global__ void __launch_bounds__(kThreadsTc, 2)
k_forest_attn_tc(const __grid_constant__ CUtensorMap map_kp, const __grid_constant__ CUtensorMap map_vp,
                 const __grid_constant__ CUtensorMap map_kn, const __grid_constant__ CUtensorMap map_vn,
                 const __grid_constant__ CUtensorMap map_q, TcArgs a) {
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr uint32_t kQBytes = QROWS * kD * 2;
    unsigned char *q_s = smem;                               // [2 halves][QROWS rows][128 B], swizzled
    unsigned char *stage_s = smem + kQBytes;                 // [stages][K 16 KB | V 16 KB]
    __shared__ Barriers sb;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((smem_u32(smem) & 1023u) != 0u) {                    // the swizzled operands need 1024-byte alignment
        if (threadIdx.x == 0) report(a.status, DSBD_DEV_BAD_FOREST);
        return;
    }

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(&sb.kv_full[s], 1); mbar_init(&sb.kv_empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&sb.s_full[b], 1); mbar_init(&sb.p_full[b], 4); }
        mbar_init(&sb.pv_done, 1);
        mbar_init(&sb.q_full, 1);
        mbar_init(&sb.q_empty, 1);
        mbar_init(&sb.o_full, 1);
        sb.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sb.tmem_base)),
                     "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t *>(&sb.tmem_base);

    if (a.rank_units) {
        // A counting sort by tile count in the (still idle) stage ring: position of a unit = units
        // with more tiles + earlier units with as many.  Columns are mirrored in odd rounds so
        // that the CTA with the longest item of one round gets the shortest of the next.  Every
        // CTA computes the same order and keeps the entries of its own column.
        int *nt_s = reinterpret_cast<int *>(stage_s);            // [n] tile count of each unit
        int *start_s = nt_s + 2048;                              // [1024] first position of a tile count
        const int n = a.rank_units, grid = (int)gridDim.x;
        for (int i = threadIdx.x; i < 1024; i += kThreadsTc) start_s[i] = 0;
        if (threadIdx.x < kMaxRanked) sb.my_units[threadIdx.x] = -1;
        __syncthreads();
        for (int u = threadIdx.x; u < n; u += kThreadsTc) {
            const int b = u / a.Hkv;
            const int nt = min((int)((a.prefix_off[b + 1] - a.prefix_off[b] + kBN - 1) / kBN), 1023);
            nt_s[u] = nt;
            atomicAdd(&start_s[nt], 1);                          // counts first
        }
        __syncthreads();
        if (warp == 0) {
            // counts -> first positions, largest tile count first (lane l owns counts 32l .. 32l+31)
            int cnt[32], mine = 0;
#pragma unroll
            for (int i = 0; i < 32; ++i) { cnt[i] = start_s[1023 - (lane * 32 + i)]; mine += cnt[i]; }
            int before = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(kFull, before, o);
                if (lane >= o) before += t;
            }
            before -= mine;
#pragma unroll
            for (int i = 0; i < 32; ++i) { start_s[1023 - (lane * 32 + i)] = before; before += cnt[i]; }
            __syncwarp();
            // units in order, 32 at a time: equal counts inside a group keep their unit order
            for (int base = 0; base < n; base += 32) {
                const int u = base + lane;
                const int nt = u < n ? nt_s[u] : -1 - lane;                  // idle lanes match nobody
                const unsigned same = __match_any_sync(kFull, nt);
                if (u < n) {
                    const int pos = start_s[nt] + __popc(same & ((1u << lane) - 1));
                    const int round = pos / grid;
                    int col = pos - round * grid;
                    if (round & 1) col = grid - 1 - col;
                    if (col == (int)blockIdx.x && round < kMaxRanked) sb.my_units[round] = u;
                }
                __syncwarp();
                if (u < n && lane == 31 - __clz(same)) start_s[nt] += __popc(same);   // one lane per count
                __syncwarp();
            }
        }
        __syncthreads();
    }

    if (warp == 4) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            uint32_t tile = 0, unit = 0;
            bool ok = true;
            const int n_items = item_count(a);
            // a prefix that is read once: its lines are the first to leave L2 again, so that the queries,
            // the tree's keys and values and the metadata the units keep coming back to stay there
            // (with several row blocks per unit the blocks read the same prefix: ordinary policy)
            uint64_t pol_stream;
            if (a.row_blocks == 1) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol_stream));
            else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol_stream));
            for (int u = blockIdx.x; u < n_items * a.n_layers && ok; u += gridDim.x) {
                const int layer = u / n_items;
                const AttnItem item = get_item(a, u - layer * n_items, sb);
                if (item.b < 0) continue;
                const int b = item.b, g = item.g;
                const int64_t L = a.prefix_off[b + 1] - a.prefix_off[b];
                const int64_t row0 = a.prefix_off[b] * a.Hkv + (int64_t)g * L + item.t0;
                // paged: tile j of the item is page t0/64 + j of the beam, one 64-row box of the pool
                const int32_t *pages = a.page_table ? a.page_table + a.page_off[b] + item.t0 / kBN : nullptr;
                int page_next = (pages && item.t1 > item.t0) ? pages[0] : 0;
                const int nt_p = (item.t1 - item.t0 + kBN - 1) / kBN;
                const int n_lo = a.beam_node_off[b];
                const int nt = nt_p + (item.last ? tree_tiles(a, b) : 0);
                // The unit's query rows: one box per 64-column half, rows = (node, query head of this
                // KV head) in the order the MMA reads them.  The single Q buffer is free once the
                // previous unit's last Q K^T product has completed, which is while that unit's last
                // softmax, P V product and output write are still running: the copy hides behind them.
                if (unit > 0) ok = mbar_wait(&sb.q_empty, (unit - 1) & 1, &sb, a.status);
                if (!ok) break;
                {
                    const int z = n_lo + item.rb * a.nodes_per_block + layer * a.q_layer_nodes;
                    mbar_expect_tx(&sb.q_full, (uint32_t)a.block_rows * kD * 2);
                    tma_load_3d(q_s, &map_q, 0, g * a.group, z, &sb.q_full);
                    tma_load_3d(q_s + QROWS * 128, &map_q, 64, g * a.group, z, &sb.q_full);
                }
                ++unit;
                for (int j = 0; j < nt && ok; ++j, ++tile) {
                    const int s = tile % kStages;
                    const uint32_t par = (tile / kStages) & 1;
                    ok = mbar_wait(&sb.kv_empty[s], par ^ 1, &sb, a.status);
                    if (!ok) break;
                    unsigned char *ks = stage_s + s * kStageBytes, *vs = ks + kTileBytes;
                    mbar_expect_tx(&sb.kv_full[s], kStageBytes);
#ifdef DSBD_TEST_WAIT_TIMEOUT
                    if (tile == 1 && blockIdx.x == 0) continue;      // the bytes this barrier expects never come
#endif
                    if (j < nt_p) {
                        int y = (int)(row0 + (int64_t)j * kBN);
                        if (pages) {
                            y = (page_next * a.Hkv + g) * kBN + layer * a.pool_layer_rows;
                            if (j + 1 < nt_p) page_next = pages[j + 1];
                        }
                        tma_load_2d_hint(ks, &map_kp, 0, y, &sb.kv_full[s], pol_stream);
                        tma_load_2d_hint(ks + kTileBytes / 2, &map_kp, 64, y, &sb.kv_full[s], pol_stream);
                        tma_load_2d_hint(vs, &map_vp, 0, y, &sb.kv_full[s], pol_stream);
                        tma_load_2d_hint(vs + kTileBytes / 2, &map_vp, 64, y, &sb.kv_full[s], pol_stream);
                    } else {
                        const int x = g * kD;                                  // tree tile j - nt_p
                        const int y = n_lo + (j - nt_p) * kBN + layer * a.new_layer_rows;
                        tma_load_2d(ks, &map_kn, x, y, &sb.kv_full[s]);
                        tma_load_2d(ks + kTileBytes / 2, &map_kn, x + 64, y, &sb.kv_full[s]);
                        tma_load_2d(vs, &map_vn, x, y, &sb.kv_full[s]);
                        tma_load_2d(vs + kTileBytes / 2, &map_vn, x + 64, y, &sb.kv_full[s]);
                    }
                }
            }
            if (!ok) {
                // let the copies already issued land before the CTA goes away
                for (uint32_t k = 0; k < (uint32_t)kStages && k < tile; ++k) {
                    const uint32_t t = tile - 1 - k;
                    const long long t0 = clock64();
                    while (!mbar_try(&sb.kv_full[t % kStages], (t / kStages) & 1))
                        if (clock64() - t0 > kWaitCycles) break;
                }
            }
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc_s = instr_desc(kRows, kBN, 0);
            constexpr uint32_t idesc_o = instr_desc(kRows, kD, 1);
            uint32_t tile = 0, unit = 0;
            bool ok = true;
            const uint64_t qd = desc_k_major(smem_u32(q_s));
            const int n_items = item_count(a);
            for (int u = blockIdx.x; u < n_items * a.n_layers && ok; u += gridDim.x) {
                const AttnItem item = get_item(a, u % n_items, sb);
                if (item.b < 0) continue;
                const int nt = (item.t1 - item.t0 + kBN - 1) / kBN + (item.last ? tree_tiles(a, item.b) : 0);
                ok = mbar_wait(&sb.q_full, unit & 1, &sb, a.status);
                // S(t) = Q K(t)^T into S buffer t & 1; issued one tile ahead of the P V product so
                // that it runs while the softmax warps work on the previous tile
                auto issue_s = [&](uint32_t t) -> bool {
                    const int s = t % kStages;
                    if (!mbar_wait(&sb.kv_full[s], (t / kStages) & 1, &sb, a.status)) return false;
                    tc_fence_after();
                    const uint64_t kd = desc_k_major(smem_u32(stage_s + s * kStageBytes));
#pragma unroll
                    for (int ks = 0; ks < kD / 16; ++ks) {
                        const uint64_t ad = qd + (uint64_t)((ks / 4) * ((QROWS * 128) >> 4) + (ks % 4) * 2);
                        const uint64_t bd = kd + (uint64_t)((ks / 4) * ((kBN * 128) >> 4) + (ks % 4) * 2);
                        mma_ss(tmem + kColS + (t & 1) * 64, ad, bd, idesc_s, ks > 0);
                    }
                    tc_commit(&sb.s_full[t & 1]);
                    return true;
                };
                if (ok) ok = issue_s(tile);
                if (ok && nt == 1) tc_commit(&sb.q_empty);       // the unit's last (only) Q K^T product
                for (int j = 0; j < nt && ok; ++j, ++tile) {
                    if (j + 1 < nt) {
                        ok = issue_s(tile + 1);
                        if (!ok) break;
                        if (j + 2 == nt) tc_commit(&sb.q_empty);
                    }
                    const int s = tile % kStages;
                    ok = mbar_wait(&sb.p_full[tile & 1], (tile >> 1) & 1, &sb, a.status);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t vd = desc_mn_major(smem_u32(stage_s + s * kStageBytes) + kTileBytes, kBN * 128);
#pragma unroll
                    for (int ks = 0; ks < kBN / 16; ++ks)
                        mma_ts(tmem + kColO, tmem + kColS + (tile & 1) * 64 + ks * 8,
                               vd + (uint64_t)(ks * ((16 * 128) >> 4)), idesc_o, (j > 0 || ks > 0) ? 1u : 0u);
                    tc_commit(&sb.kv_empty[s]);
                    tc_commit(&sb.pv_done);
                }
                if (ok) tc_commit(&sb.o_full);
                ++unit;
            }
        }
    } else {
        // ------------------------------------------------------------ softmax warps
        const int row = warp * 32 + lane;
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        uint32_t tile = 0, unit = 0;
        bool ok = true;
        const int n_items = item_count(a);
        for (int u = blockIdx.x; u < n_items * a.n_layers && ok; u += gridDim.x) {
            const AttnItem item = get_item(a, u % n_items, sb);
            if (item.b < 0) continue;
            const int b = item.b, g = item.g;
            const int64_t L = item.t1;                         // tokens beyond t1 belong to other items
            const int nt_p = (item.t1 - item.t0 + kBN - 1) / kBN;
            const int n_lo = a.beam_node_off[b];
            const int n_tree = a.beam_node_off[b + 1] - n_lo;
            const int nt = nt_p + (item.last ? (n_tree + kBN - 1) / kBN : 0);
            const int M = n_tree * a.group;
            const int r0 = item.rb * a.block_rows;              // first row of this row block
            // (the MMA's rows from block_rows on hold no query of this block: never active)
            const bool warp_active = warp * 32 < a.block_rows && r0 + warp * 32 < M;
            const bool active = row < a.block_rows && r0 + row < M;
            const int node = active ? (r0 + row) / a.group : 0;
            const int hq = g * a.group + (active ? r0 + row - node * a.group : 0);
            // ancestor-or-self mask of this row's node: walk up the tree
            unsigned long long anc_lo = 0ull, anc_hi = 0ull;       // nodes 0..63, 64..127
            {
                int n = node;
                for (int hop = 0; hop < 2 * kBN && n >= 0 && n < n_tree; ++hop) {
                    if (n < 64) anc_lo |= 1ull << n; else anc_hi |= 1ull << (n - 64);
                    const int par = a.parent[n_lo + n];
                    if (par >= n_lo + n) { report(a.status, DSBD_DEV_BAD_FOREST); break; }
                    n = par < 0 ? -1 : par - n_lo;
                }
            }
            float m_ref = -INFINITY, l_run = 0.f;
            for (int j = 0; j < nt && ok; ++j, ++tile) {
                ok = mbar_wait(&sb.s_full[tile & 1], (tile >> 1) & 1, &sb, a.status);
                if (!ok) break;
                tc_fence_after();
                if (warp_active) {
                    uint32_t sv[2][32];
                    const uint32_t s_col = kColS + (tile & 1) * 64;
                    tmem_ld32(tmem + lane_base + s_col, sv[0]);
                    tmem_ld32(tmem + lane_base + s_col + 32, sv[1]);
                    tmem_wait_ld();
                    float mx = -INFINITY;
                    const bool tree = (j >= nt_p);
                    // visibility of the tile's 64 tokens for this row, as a bit mask
                    unsigned long long vis;
                    if (tree) {
                        const int jt = j - nt_p, left = n_tree - jt * kBN;
                        vis = (jt ? anc_hi : anc_lo) & (left >= 64 ? ~0ull : ((1ull << left) - 1));
                    }
                    else {
                        const int64_t left = L - item.t0 - (int64_t)j * kBN;
                        vis = left >= 64 ? ~0ull : ((1ull << left) - 1);
                    }
                    // The softmax warps set the pace of a unit (one row per thread, 64 columns in sequence),
                    // so the common tile -- every token visible -- does no masking, the scale is folded
                    // into the exponent's fma, and the exponential is the bare ex2.approx.
                    if (vis != ~0ull) {
#pragma unroll
                        for (int c = 0; c < 64; ++c)
                            if (!((vis >> c) & 1ull)) sv[c >> 5][c & 31] = 0xff800000u;      // -inf: weight 0
                    }
                    {   // four independent chains: this warp has its scheduler nearly to itself, so a
                        // 64-long dependent chain would be pure latency
                        float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                        for (int c = 0; c < 64; ++c) m4[c & 3] = fmaxf(m4[c & 3], __uint_as_float(sv[c >> 5][c & 31]));
                        mx = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
                    }
                    mx *= a.scale_log2;                                  // scale > 0 (checked by the host)
                    // lazy rescale: move the reference only when some row of the warp needs it
                    const bool need = mx > m_ref + 8.f;
                    if (__any_sync(kFull, need)) {
                        // O is about to be rescaled in place: the previous tile's P V must have landed
                        if (j > 0 && !mbar_wait(&sb.pv_done, (tile - 1) & 1, &sb, a.status)) { ok = false; }
                        tc_fence_after();
                        const float m_new = need ? mx : m_ref;
                        const float f = (m_ref == -INFINITY) ? 0.f : exp2f(m_ref - m_new);
                        l_run *= f;
                        if (j > 0) {
#pragma unroll
                            for (int cc = 0; cc < 4; ++cc) {
                                uint32_t ov[32];
                                tmem_ld32(tmem + lane_base + kColO + cc * 32, ov);
                                tmem_wait_ld();
#pragma unroll
                                for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * f);
                                tmem_st32(tmem + lane_base + kColO + cc * 32, ov);
                            }
                        }
                        m_ref = m_new;
                    }
                    uint32_t pv[32];
                    const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                    float l4[4] = {0.f, 0.f, 0.f, 0.f};                  // (independent chains again)
#pragma unroll
                    for (int c = 0; c < 32; ++c) {
                        const float p0 = ex2_ftz(fmaf(__uint_as_float(sv[(2 * c) >> 5][(2 * c) & 31]), a.scale_log2, -m_use));
                        const float p1 = ex2_ftz(fmaf(__uint_as_float(sv[(2 * c + 1) >> 5][(2 * c + 1) & 31]), a.scale_log2, -m_use));
                        const uint32_t pk = pack_bf16(p0, p1);
                        // the row sum must match what the tensor core will see: the rounded values
                        l4[c & 1] += __uint_as_float(pk << 16);
                        l4[2 + (c & 1)] += __uint_as_float(pk & 0xffff0000u);
                        pv[c] = pk;
                    }
                    l_run += (l4[0] + l4[1]) + (l4[2] + l4[3]);
                    tmem_st32(tmem + lane_base + s_col, pv);
                    tmem_wait_st();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&sb.p_full[tile & 1]);
            }
            if (!ok) break;
            // ---- unit done: O / l -> global
            ok = mbar_wait(&sb.o_full, unit & 1, &sb, a.status);
            if (!ok) break;
            tc_fence_after();
            if (warp_active) {
                const int layer = u / n_items;
                if (item.nparts == 1) {
                    const float inv = active ? 1.f / l_run : 0.f;
                    __nv_bfloat16 *dst = a.out + (int64_t)layer * a.q_layer_stride +
                                         ((int64_t)(n_lo + node) * a.Hq + hq) * kD;
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t ov[32];
                        tmem_ld32(tmem + lane_base + kColO + cc * 32, ov);
                        tmem_wait_ld();
                        if (active) {
#pragma unroll
                            for (int c = 0; c < 32; c += 8) {
                                uint4 w;
                                w.x = pack_bf16(__uint_as_float(ov[c]) * inv, __uint_as_float(ov[c + 1]) * inv);
                                w.y = pack_bf16(__uint_as_float(ov[c + 2]) * inv, __uint_as_float(ov[c + 3]) * inv);
                                w.z = pack_bf16(__uint_as_float(ov[c + 4]) * inv, __uint_as_float(ov[c + 5]) * inv);
                                w.w = pack_bf16(__uint_as_float(ov[c + 6]) * inv, __uint_as_float(ov[c + 7]) * inv);
                                *reinterpret_cast<uint4 *>(dst + cc * 32 + c) = w;
                            }
                        }
                    }
                } else {
                    // partial result of this part of the unit: reference maximum, row sum, raw O
                    float *dst = a.partial +
                                 (((int64_t)layer * a.slots_per_layer + item.slot) * a.max_rows + r0 + row) * 130;
                    if (active) { dst[0] = m_ref; dst[1] = l_run; }
#pragma unroll
                    for (int cc = 0; cc < 4; ++cc) {
                        uint32_t ov[32];
                        tmem_ld32(tmem + lane_base + kColO + cc * 32, ov);
                        tmem_wait_ld();
                        if (active) {
#pragma unroll
                            for (int c = 0; c < 32; c += 2)
                                *reinterpret_cast<float2 *>(dst + 2 + cc * 32 + c) =
                                    make_float2(__uint_as_float(ov[c]), __uint_as_float(ov[c + 1]));
                        }
                    }
                }
            }
            tc_fence_before();
            ++unit;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ---------------------------------------------------------------------------------------
// Work plan for ragged or small batches: every unit's prefix is cut into parts of at most
// `chunk` tokens (equal parts, multiples of 64), and the items are ordered by decreasing tile
// count, so that handing item i to CTA i mod grid spreads the work evenly.
// ---------------------------------------------------------------------------------------
struct UnitParts { int first_slot, nparts; };

__device__ __forceinline__ void unit_parts(int64_t L, int chunk, int *np, int *plen) {
    int n = (int)((L + chunk - 1) / chunk);
    if (n < 1) n = 1;
    const int64_t per = (L + n - 1) / n;
    *np = n;
    *plen = (int)((per + kBN - 1) / kBN) * kBN;
}

__global__ void __launch_bounds__(1024)
k_attn_plan(int B, int Hkv, const int64_t *__restrict__ prefix_off, const int32_t *__restrict__ beam_node_off,
            int group, int block_rows, int chunk, int grid, AttnItem *__restrict__ items,
            int *__restrict__ n_items, UnitParts *__restrict__ units) {
    __shared__ int bucket[1024];
    __shared__ int scan[1024];
    __shared__ int carry;
    const int tid = threadIdx.x, n_units = B * Hkv;
    // row blocks a tree really has: only those become items
    auto blocks_of = [&](int b) {
        const int rows = (beam_node_off[b + 1] - beam_node_off[b]) * group;
        return rows > block_rows ? (rows + block_rows - 1) / block_rows : 1;
    };
    bucket[tid] = 0;
    if (tid == 0) carry = 0;
    __syncthreads();
    // slots: exclusive scan of the part counts over the units, 1024 units at a time
    for (int base = 0; base < n_units; base += 1024) {
        const int u = base + tid;
        int np = 0, plen = 0;
        if (u < n_units) {
            const int b = u / Hkv;
            unit_parts(prefix_off[b + 1] - prefix_off[b], chunk, &np, &plen);
        }
        scan[tid] = np;
        __syncthreads();
        for (int o = 1; o < 1024; o <<= 1) {
            const int v = tid >= o ? scan[tid - o] : 0;
            __syncthreads();
            scan[tid] += v;
            __syncthreads();
        }
        if (u < n_units) {
            units[u].first_slot = carry + scan[tid] - np;
            units[u].nparts = np;
            const int b = u / Hkv;
            const int64_t L = prefix_off[b + 1] - prefix_off[b];
            for (int p = 0; p < np; ++p) {
                const int64_t t0 = (int64_t)p * plen;
                const int64_t t1 = t0 + plen < L ? t0 + plen : L;
                int nt = (int)((t1 - t0 + kBN - 1) / kBN) + (p == np - 1);
                atomicAdd(&bucket[nt < 1023 ? nt : 1023], blocks_of(b));
            }
        }
        __syncthreads();
        if (tid == 0) carry += scan[1023];
        __syncthreads();
    }
    // start of every bucket in the output, largest tile count first
    scan[tid] = bucket[1023 - tid];
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {
        const int v = tid >= o ? scan[tid - o] : 0;
        __syncthreads();
        scan[tid] += v;
        __syncthreads();
    }
    const int start = scan[tid] - bucket[1023 - tid];
    const int total_items = scan[1023];          // all buckets together
    __syncthreads();
    bucket[1023 - tid] = start;                 // bucket[k] becomes the cursor of tile count k
    // The list is read in rounds of `grid` items, CTA k taking entry k of every round.  Odd rounds
    // are stored back to front, so that the CTA with the longest item of one round gets the
    // shortest of the next; the last round is padded with empty entries (b = -1).
    const int padded = (total_items + grid - 1) / grid * grid;
    for (int i = total_items - total_items % grid + tid; i < padded; i += 1024) items[i].b = -1;
    if (tid == 0) *n_items = padded;
    __syncthreads();
    for (int u = tid; u < n_units; u += 1024) {
        const int b = u / Hkv, g = u - b * Hkv;
        const int64_t L = prefix_off[b + 1] - prefix_off[b];
        int np, plen;
        unit_parts(L, chunk, &np, &plen);
        for (int p = 0; p < np; ++p) {
            const int64_t t0 = (int64_t)p * plen;
            const int64_t t1 = t0 + plen < L ? t0 + plen : L;
            const int nt = (int)((t1 - t0 + kBN - 1) / kBN) + (p == np - 1);
            const int nrb = blocks_of(b);
            for (int rb = 0; rb < nrb; ++rb) {
                int pos = atomicAdd(&bucket[nt < 1023 ? nt : 1023], 1);
                const int round = pos / grid;
                if (round & 1) pos = round * grid + (grid - 1 - (pos - round * grid));
                AttnItem it;
                it.b = b; it.g = g; it.t0 = (int)t0; it.t1 = (int)t1; it.last = (p == np - 1);
                it.nparts = np; it.slot = units[u].first_slot + p; it.rb = rb;
                items[pos] = it;
            }
        }
    }
}

// Merge the parts of every split unit: out = sum_c O_c 2^(m_c - m) / sum_c l_c 2^(m_c - m).
__global__ void __launch_bounds__(128)
k_attn_combine(TcArgs a, const UnitParts *__restrict__ units) {
    const int layer = blockIdx.y;
    int u = blockIdx.x;
    UnitParts up;
    if (units) {
        up = units[u];
    } else {                                             // tail split: block i merges tail unit i
        up.first_slot = u * a.tail_k; up.nparts = a.tail_k;
        u += a.tail_first;
    }
    if (up.nparts <= 1) return;
    const int b = u / a.Hkv, g = u - b * a.Hkv;
    a.partial += (int64_t)layer * a.slots_per_layer * a.max_rows * 130;
    a.out += (int64_t)layer * a.q_layer_stride;
    const int n_lo = a.beam_node_off[b];
    const int M = (a.beam_node_off[b + 1] - n_lo) * a.group;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int row = warp; row < M; row += 4) {
        float m = -INFINITY;
        for (int c = 0; c < up.nparts; ++c)
            m = fmaxf(m, a.partial[((int64_t)(up.first_slot + c) * a.max_rows + row) * 130]);
        float l = 0.f;
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int c = 0; c < up.nparts; ++c) {
            const float *src = a.partial + ((int64_t)(up.first_slot + c) * a.max_rows + row) * 130;
            const float w = src[0] == -INFINITY ? 0.f : exp2f(src[0] - m);
            l += src[1] * w;
            const float2 x = *reinterpret_cast<const float2 *>(src + 2 + lane * 4);
            const float2 y = *reinterpret_cast<const float2 *>(src + 4 + lane * 4);
            o.x += x.x * w; o.y += x.y * w; o.z += y.x * w; o.w += y.y * w;
        }
        const float inv = 1.f / l;
        const int node = row / a.group, hq = g * a.group + (row - node * a.group);
        __nv_bfloat16 *dst = a.out + ((int64_t)(n_lo + node) * a.Hq + hq) * kD + lane * 4;
        uint2 w2;
        w2.x = pack_bf16(o.x * inv, o.y * inv);
        w2.y = pack_bf16(o.z * inv, o.w * inv);
        *reinterpret_cast<uint2 *>(dst) = w2;
    }
}

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
    static EncodeFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeFn>(p);
    }
    return fn;
}

// [rows, cols] bf16 row-major with `pitch` bytes between rows; boxes of 64 cols x 64 rows.
bool make_map(CUtensorMap *m, const void *base, uint64_t cols, uint64_t rows, uint64_t pitch) {
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {pitch};
    const cuuint32_t box[2] = {64, (cuuint32_t)kBN};
    const cuuint32_t el[2] = {1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, el,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// q as [nodes, Hq, 128] bf16: boxes of 64 columns x `group` heads x `nodes` nodes, i.e. the query rows
// of one KV head for a run of nodes, in (node, head) order.
bool make_map_q(CUtensorMap *m, const void *base, uint64_t Hq, uint64_t nodes_total, uint32_t group, uint32_t nodes) {
    EncodeFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)kD, Hq, nodes_total};
    const cuuint64_t strides[2] = {(cuuint64_t)kD * 2, Hq * kD * 2};
    const cuuint32_t box[3] = {64, group, nodes};
    const cuuint32_t el[3] = {1, 1, 1};
    return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, el,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Launch shape shared by the workspace query and the launch.
struct TcPlan {
    int grid, chunk;          // chunk == 0: one item per unit in unit order, no plan kernel
    bool split;               // units are cut into parts (partials + combine kernel)
    int tail_first, tail_k;   // chunk == 0 only: the units from tail_first on are cut into tail_k parts
    bool rank;                // chunk == 0 only: the CTAs order the (ragged) units themselves
    int64_t items_max;
    size_t off_items, off_units, off_partial, total;
};

// Query rows per row block.  Trees of up to 64 rows take the 64-row tile (two CTAs per SM).  So do
// forests whose AVERAGE tree has at most 64 rows even when the largest is bigger (a sampled
// forest puts most drafts under a few roots and leaves the other trees tiny): the big trees then
// run as several 64-row blocks, the many small ones at the faster shape.
int tile_rows_for(const dsbd_forest_t *f, const dsbd_attn_desc_t *d) {
    const int group = d->Hq / d->Hkv;
    if (f->max_tree_nodes * group <= 64) return 64;
    return ((int64_t)f->N * group <= (int64_t)64 * f->B && group <= 64) ? 64 : kRows;
}
// Rows of a row block: whole nodes (the copy engine fetches a block's query rows as a box of nodes x
// heads), as many as the tile holds.
int block_rows_for(const dsbd_forest_t *f, const dsbd_attn_desc_t *d) {
    const int group = d->Hq / d->Hkv;
    return tile_rows_for(f, d) / group * group;
}

TcPlan make_plan(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, int n_layers = 1) {
    TcPlan p = {};
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int group = d->Hq / d->Hkv;
    const int block_rows = block_rows_for(f, d);
    const bool small_q = tile_rows_for(f, d) == 64;
    p.grid = small_q ? 2 * sms : sms;
    const int row_blocks = (f->max_tree_nodes * group + block_rows - 1) / block_rows;
    const int64_t n_units = (int64_t)f->B * d->Hkv * row_blocks;     // counted with their row blocks
    // Splitting a unit costs a pipeline drain, a Q reload and a partial result per part, so it
    // pays only when there are fewer units than CTAs: then the prefix is cut so that about two
    // items per CTA exist, in parts of at least 512 tokens.  Ragged batches with enough units
    // are only re-ordered (longest first, rounds alternating in direction).
    int64_t c = (int64_t)d->total_prefix * d->Hkv / (2ll * p.grid);
    if (c < 512) c = 512;
    c = (c + kBN - 1) / kBN * kBN;
    p.split = n_units < p.grid && c < d->max_prefix;
    const bool ragged = (int64_t)d->max_prefix * f->B * 100 > (int64_t)d->total_prefix * 115;
    // trees with several row blocks always go through the plan, which lists only the blocks that
    // exist (in unit order most (unit, block) pairs of a ragged forest would be empty, and the
    // CTAs whose stride hits the first blocks would do all the work)
    if (!p.split && !(ragged && n_units > p.grid) && row_blocks == 1) {
        p.chunk = 0;
        p.items_max = n_units;
        if (p.grid > n_units) p.grid = (int)n_units;
        p.total = 256;
        // Equal-length units that do not fill the last round of CTAs: cut the units of that round
        // into parts so that (nearly) every CTA has a part of it.  1024 units on 296 CTAs are 3.46
        // rounds: whole units would take the time of 4, with the last 136 units in 2 parts 3.5.
        const int rem = (int)(n_units % p.grid);
        const bool uniform = (int64_t)d->max_prefix * f->B == d->total_prefix;
        if (uniform && n_units > p.grid && rem > 0) {
            const int tiles = (int)((d->max_prefix + kBN - 1) / kBN);
            int k = p.grid / rem;
            if (k > 8) k = 8;
            if (k > tiles / 8) k = tiles / 8;               // parts of at least 8 tiles
            if (k >= 2) {
                p.tail_first = (int)n_units - rem;
                p.tail_k = k;
                p.items_max = (int64_t)p.tail_first + (int64_t)rem * k;
                p.off_partial = 256;
                p.total = align_up(256 + sizeof(float) * 130 * (size_t)n_layers * (size_t)rem * k *
                                             (size_t)(f->max_tree_nodes * group), 256);
            }
        }
        return p;
    }
    // a ragged batch of whole units, few enough per CTA: no plan kernel, every CTA ranks the units
    // itself at its start (a few microseconds in parallel instead of a serial kernel ahead of it)
    if (!p.split && row_blocks == 1 && n_units <= 2048 && n_units <= (int64_t)kMaxRanked * p.grid) {
        p.chunk = 0;
        p.rank = true;
        p.items_max = n_units;
        p.total = 256;
        return p;
    }
    if (!p.split) c = (int64_t)1 << 30;                  // one part per unit
    p.chunk = (int)c;
    p.items_max = (p.split ? (int64_t)d->Hkv * row_blocks * (d->total_prefix / c + f->B) : n_units) + p.grid;
    if (p.grid > p.items_max - p.grid) p.grid = (int)(p.items_max - p.grid);
    if (p.grid < 1) p.grid = 1;
    size_t off = 256;
    p.off_items = off;   off = align_up(off + sizeof(AttnItem) * (size_t)p.items_max, 256);
    p.off_units = off;   off = align_up(off + sizeof(UnitParts) * (size_t)f->B * d->Hkv, 256);
    p.off_partial = off;
    if (p.split)
        off = align_up(off + sizeof(float) * 130 * (size_t)n_layers * (size_t)p.items_max *
                                 (size_t)(f->max_tree_nodes * group), 256);
    p.total = off;
    return p;
}

}  // namespace

namespace dsbd {

// Layer count and strides of a paged call, checked: the layers of one call share one tensor map
// per operand, so a layer stride must be a whole number of map rows.
struct LayerDims { int n_layers, pool_rows, new_rows; int64_t q_stride; bool ok; };

LayerDims layer_dims(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, const dsbd_kv_pages_t *pages) {
    LayerDims L = {1, 0, 0, 0, true};
    if (!pages || pages->n_layers <= 1) return L;
    L.n_layers = pages->n_layers;
    const int64_t page_elems = (int64_t)d->Hkv * kBN * kD, new_row = (int64_t)d->Hkv * kD;
    const int64_t ps = pages->pool_layer_stride, ns = pages->new_layer_stride, qs = pages->q_layer_stride;
    L.ok = ps >= pages->n_pages * page_elems && ps % ((int64_t)kBN * kD) == 0 &&
           ns >= (int64_t)f->N * new_row && ns % new_row == 0 &&
           qs >= (int64_t)f->N * d->Hq * kD && qs % ((int64_t)d->Hq * kD) == 0;
    if (!L.ok) return L;
    const int64_t pool_rows = ps / kD, new_rows = ns / new_row;
    // row coordinates of the maps are 32-bit
    if (pool_rows * L.n_layers >= ((int64_t)1 << 31) || new_rows * L.n_layers >= ((int64_t)1 << 31)) L.ok = false;
    L.pool_rows = (int)pool_rows; L.new_rows = (int)new_rows; L.q_stride = qs;
    return L;
}

bool attention_tc_supported(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, int64_t n_pages) {
    if (d->dtype != DSBD_DTYPE_BF16 || d->d != kD) return false;
    if (d->Hq / d->Hkv > kRows) return false;                                // a node's rows fit one tile
    if (!(d->scale > 0.f)) return false;                                     // the row maximum is taken before scaling
    if (f->max_tree_nodes * (d->Hq / d->Hkv) > kRows * 8) return false;      // up to 8 row blocks
    if (f->max_tree_nodes > 2 * kBN) return false;                           // two tree tiles
    if (d->total_prefix <= 0) return false;
    // row coordinates of the K/V maps are 32-bit
    const int64_t rows = n_pages > 0 ? n_pages * d->Hkv * kBN : (int64_t)d->total_prefix * d->Hkv;
    if (rows >= (int64_t)1 << 31) return false;
    return encode_fn() != nullptr;
}

bool attention_tc_layers_ok(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, const dsbd_kv_pages_t *pages) {
    return layer_dims(f, d, pages).ok;
}

size_t attention_tc_workspace(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, int n_layers) {
    return make_plan(f, d, n_layers < 1 ? 1 : n_layers).total;
}

int attention_tc_launches(const dsbd_forest_t *f, const dsbd_attn_desc_t *d) {
    const TcPlan p = make_plan(f, d);
    return 1 + (p.chunk > 0 ? 1 : 0) + (p.split || p.tail_k ? 1 : 0);
}

int launch_attention_tc(const dsbd_forest_t *f, const dsbd_attn_desc_t *d, const void *q, const void *k_new,
                        const void *v_new, const void *k_prefix, const void *v_prefix, const int64_t *prefix_off,
                        void *out, void *workspace, size_t workspace_bytes, int32_t *status, cudaStream_t stream,
                        const dsbd_kv_pages_t *pages) {
    CUtensorMap kp, vp, kn, vn, qm;
    const LayerDims LD = layer_dims(f, d, pages);
    if (!LD.ok) return DSBD_ERR_INVALID_ARG;
    const int nl = LD.n_layers;
    // one map per operand over all layers: layer l starts l * (layer stride in rows) further down
    const uint64_t prows = pages ? (uint64_t)pages->n_pages * d->Hkv * kBN + (uint64_t)(nl - 1) * LD.pool_rows
                                 : (uint64_t)d->total_prefix * d->Hkv;
    const uint64_t nrows = (uint64_t)f->N + (uint64_t)(nl - 1) * LD.new_rows;
    if (!make_map(&kp, k_prefix, kD, prows, kD * 2) || !make_map(&vp, v_prefix, kD, prows, kD * 2) ||
        !make_map(&kn, k_new, (uint64_t)d->Hkv * kD, nrows, (uint64_t)d->Hkv * kD * 2) ||
        !make_map(&vn, v_new, (uint64_t)d->Hkv * kD, nrows, (uint64_t)d->Hkv * kD * 2))
        return DSBD_ERR_CUDA;
    const int group = d->Hq / d->Hkv, block_rows = block_rows_for(f, d);
    const int64_t q_layer_nodes = nl > 1 ? LD.q_stride / ((int64_t)d->Hq * kD) : 0;
    if ((uint64_t)f->N + (uint64_t)(nl - 1) * q_layer_nodes >= ((uint64_t)1 << 31)) return DSBD_ERR_UNSUPPORTED;
    if (!make_map_q(&qm, q, (uint64_t)d->Hq, (uint64_t)f->N + (uint64_t)(nl - 1) * q_layer_nodes, (uint32_t)group,
                    (uint32_t)(block_rows / group)))
        return DSBD_ERR_CUDA;
    const TcPlan plan = make_plan(f, d, nl);
    if (workspace_bytes < plan.total) return DSBD_ERR_WORKSPACE_TOO_SMALL;
    char *ws = static_cast<char *>(workspace);
    TcArgs a = {};
    a.B = f->B; a.N = f->N; a.Hq = d->Hq; a.Hkv = d->Hkv; a.group = d->Hq / d->Hkv;
    a.n_units = f->B * d->Hkv;
    a.max_rows = f->max_tree_nodes * a.group;
    a.block_rows = block_rows;
    a.nodes_per_block = block_rows / group;
    a.row_blocks = (a.max_rows + a.block_rows - 1) / a.block_rows;
    a.scale_log2 = d->scale * 1.4426950408889634f;
    a.beam_node_off = f->beam_node_off; a.parent = f->parent; a.prefix_off = prefix_off;
    if (pages) { a.page_table = pages->page_table; a.page_off = pages->page_off; }
    a.q = static_cast<const __nv_bfloat16 *>(q);
    a.out = static_cast<__nv_bfloat16 *>(out);
    a.status = status;
    a.n_layers = nl; a.pool_layer_rows = LD.pool_rows; a.new_layer_rows = LD.new_rows;
    a.q_layer_stride = LD.q_stride;
    a.q_layer_nodes = (int)q_layer_nodes;
    a.slots_per_layer = plan.tail_k ? (a.n_units - plan.tail_first) * plan.tail_k : (int)plan.items_max;
    a.tail_first = plan.tail_first; a.tail_k = plan.tail_k;
    a.rank_units = plan.rank ? a.n_units : 0;
    if (plan.tail_k) {
        if (reinterpret_cast<uintptr_t>(workspace) & 255) return DSBD_ERR_INVALID_ARG;
        a.partial = reinterpret_cast<float *>(ws + plan.off_partial);
    }
    UnitParts *units = nullptr;
    if (plan.chunk > 0) {
        if (reinterpret_cast<uintptr_t>(workspace) & 255) return DSBD_ERR_INVALID_ARG;
        AttnItem *items = reinterpret_cast<AttnItem *>(ws + plan.off_items);
        units = reinterpret_cast<UnitParts *>(ws + plan.off_units);
        int *n_items = reinterpret_cast<int *>(ws);
        k_attn_plan<<<1, 1024, 0, stream>>>(f->B, d->Hkv, prefix_off, f->beam_node_off, a.group, a.block_rows,
                                            plan.chunk, plan.grid, items, n_items, units);
        a.items = items;
        a.n_items = n_items;
        a.partial = reinterpret_cast<float *>(ws + plan.off_partial);
    }
    // more layers mean more items for the same plan: the grid may grow back to the SM-filling size
    int grid = plan.grid;
    if (nl > 1) {
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int full = tile_rows_for(f, d) == 64 ? 2 * sms : sms;
        if (plan.chunk == 0) grid = (int)std::min<int64_t>((int64_t)plan.items_max * nl, full);
    }
    // up to 64 query rows: 16 KB of Q, three stages, two CTAs per SM; more rows: one CTA per SM
    const bool small_q = tile_rows_for(f, d) == 64;
#define DSBD_LAUNCH_TC(QR, ST)                                                                              \
    do {                                                                                                   \
        constexpr uint32_t bytes = smem_bytes(QR, ST);                                                     \
        if (cudaFuncSetAttribute(k_forest_attn_tc<QR, ST>, cudaFuncAttributeMaxDynamicSharedMemorySize,    \
                                 (int)bytes) != cudaSuccess)                                               \
            return DSBD_ERR_CUDA;                                                                          \
        k_forest_attn_tc<QR, ST><<<grid, kThreadsTc, bytes, stream>>>(kp, vp, kn, vn, qm, a);                  \
    } while (0)
    if (small_q) DSBD_LAUNCH_TC(64, 3);
    else DSBD_LAUNCH_TC(128, 3);
#undef DSBD_LAUNCH_TC
    if (plan.split) k_attn_combine<<<dim3(a.n_units, nl), 128, 0, stream>>>(a, units);
    else if (plan.tail_k) k_attn_combine<<<dim3(a.n_units - plan.tail_first, nl), 128, 0, stream>>>(a, nullptr);
    return cudaGetLastError() == cudaSuccess ? DSBD_OK : DSBD_ERR_CUDA;
}

}  // namespace dsbd
