"""Oracle of the paged form of the per-beam KV caches.

TEST INFRASTRUCTURE, NOT PRODUCT CODE (plain numpy; shares nothing with the CUDA library).

The paper keeps "a separate key-value cache for each input beam" and, after an iteration, the
caches "according to the output beams" (Section "Forest-based Parallel Decoding"); it does not
say how a cache is stored.  Here a cache is a list of pages of PAGE = 64 tokens in a pool
[n_pages, Hkv, PAGE, d]; beams that descend from the same input beam share its full pages, and
only the last, partly filled page is private.  What a paged cache *means* is its gathered
content, and that is what pins this file: gathering must give the packed oracle's result.

Conventions of the commit (nothing in the paper fixes them, so the page ids are "parity
unpinned": only the gathered content is pinned; the CUDA path has to match them):
  * kept output beams are selected and numbered exactly as in oracle.kv_commit;
  * new beam j keeps the first L_old // PAGE pages of its input beam, then gets
    ceil((L_old % PAGE + path length) / PAGE) fresh pages that hold the input beam's partial
    page followed by the path's keys/values;
  * fresh pages come off the top of the free stack, beam after beam: the k-th fresh page of
    the call is free_stack[free_count - 1 - k];
  * afterwards the free stack is rebuilt: every page no new beam references, ascending id.
"""
import numpy as np

from . import kv_commit as _packed

PAGE = 64


def pack_into_pages(k_prefix, v_prefix, prefix_off, Hkv, d, n_pages, rng=None):
    """Spread packed caches over a pool (page ids shuffled when rng is given).  Returns
    k_pool, v_pool [n_pages, Hkv, PAGE, d], page_table, page_off [B+1], free_stack, free_count."""
    B = len(prefix_off) - 1
    need = [int(-(-(prefix_off[b + 1] - prefix_off[b]) // PAGE)) for b in range(B)]
    total = sum(need)
    assert total <= n_pages
    ids = np.arange(n_pages)
    if rng is not None:
        ids = rng.permutation(n_pages)
    k_pool = np.zeros((n_pages, Hkv, PAGE, d), np.asarray(k_prefix).dtype)
    v_pool = np.zeros_like(k_pool)
    page_table = ids[:total].astype(np.int32)
    page_off = np.concatenate([[0], np.cumsum(need)]).astype(np.int64)
    kp, vp = np.asarray(k_prefix).reshape(-1), np.asarray(v_prefix).reshape(-1)
    for b in range(B):
        L = int(prefix_off[b + 1] - prefix_off[b])
        base = int(prefix_off[b]) * Hkv * d
        kb = kp[base:base + Hkv * L * d].reshape(Hkv, L, d)
        vb = vp[base:base + Hkv * L * d].reshape(Hkv, L, d)
        for i in range(need[b]):
            n = min(PAGE, L - i * PAGE)
            pg = page_table[page_off[b] + i]
            k_pool[pg, :, :n] = kb[:, i * PAGE:i * PAGE + n]
            v_pool[pg, :, :n] = vb[:, i * PAGE:i * PAGE + n]
    free = np.sort(ids[total:]).astype(np.int32)
    free_stack = np.zeros(n_pages, np.int32)
    free_stack[:len(free)] = free
    return k_pool, v_pool, page_table, page_off, free_stack, len(free)


def gather(k_pool, v_pool, page_table, page_off, prefix_off):
    """The packed caches a paged description stands for (beam b as [Hkv, L_b, d])."""
    B = len(prefix_off) - 1
    ks, vs = [], []
    for b in range(B):
        L = int(prefix_off[b + 1] - prefix_off[b])
        pages = page_table[int(page_off[b]):int(page_off[b + 1])]
        assert len(pages) == -(-L // PAGE)
        if L == 0:
            continue
        kb = np.concatenate([k_pool[p] for p in pages], axis=1)[:, :L]      # [Hkv, L, d]
        vb = np.concatenate([v_pool[p] for p in pages], axis=1)[:, :L]
        ks.append(kb.reshape(-1))
        vs.append(vb.reshape(-1))
    empty = np.zeros(0, k_pool.dtype)
    return (np.concatenate(ks) if ks else empty), (np.concatenate(vs) if vs else empty)


def kv_commit_paged(forest, out_off, out_width, out_parent, out_root_beam, out_logp, k_new, v_new,
                    k_pool, v_pool, page_table, page_off, prefix_off, free_stack, free_count,
                    keep_best=False):
    """Returns dict(error, new_req_beam_off, new_prefix_off, new_page_off, new_page_table,
    new_beam_slot, k_pool, v_pool, free_stack, free_count); pools are copies."""
    n_pages, Hkv, _, d = k_pool.shape
    parent = np.asarray(forest["parent"])
    k_new = np.asarray(k_new).reshape(-1, Hkv, d)
    v_new = np.asarray(v_new).reshape(-1, Hkv, d)
    kept = _packed.select_beams(forest, out_off, out_width, out_parent, out_root_beam, out_logp, prefix_off,
                                keep_best)
    R = int(forest["R"])
    plan, fresh_total = [], 0
    for _, s in kept:
        b = int(out_root_beam[s])
        L = int(prefix_off[b + 1] - prefix_off[b])
        path = _packed.path_to_root(parent, int(out_parent[s]))
        n_fresh = -(-(L % PAGE + len(path)) // PAGE)
        plan.append((s, b, L, path, fresh_total, n_fresh))
        fresh_total += n_fresh
    if fresh_total > free_count:
        return dict(error=3)
    k_pool, v_pool = k_pool.copy(), v_pool.copy()
    new_req_beam_off = np.zeros(R + 1, np.int32)
    for r, _ in kept:
        new_req_beam_off[r + 1] += 1
    new_req_beam_off = np.cumsum(new_req_beam_off).astype(np.int32)
    table, new_page_off, new_prefix_off = [], [0], [0]
    for s, b, L, path, first, n_fresh in plan:
        old = page_table[int(page_off[b]):int(page_off[b + 1])]
        full, rem = L // PAGE, L % PAGE
        fresh = [int(free_stack[free_count - 1 - (first + i)]) for i in range(n_fresh)]
        rows_k = np.concatenate([k_pool[old[full]][:, :rem] if rem else np.zeros((Hkv, 0, d), k_pool.dtype),
                                 np.transpose(k_new[path], (1, 0, 2))], axis=1)
        rows_v = np.concatenate([v_pool[old[full]][:, :rem] if rem else np.zeros((Hkv, 0, d), v_pool.dtype),
                                 np.transpose(v_new[path], (1, 0, 2))], axis=1)
        for i, pg in enumerate(fresh):
            n = min(PAGE, rows_k.shape[1] - i * PAGE)
            k_pool[pg, :, :n] = rows_k[:, i * PAGE:i * PAGE + n]
            v_pool[pg, :, :n] = rows_v[:, i * PAGE:i * PAGE + n]
        table += list(old[:full]) + fresh
        new_page_off.append(len(table))
        new_prefix_off.append(new_prefix_off[-1] + L + len(path))
    table = np.asarray(table, np.int32)
    used = np.zeros(n_pages, bool)
    used[table] = True
    free = np.nonzero(~used)[0].astype(np.int32)
    new_free = np.zeros(n_pages, np.int32)
    new_free[:len(free)] = free
    return dict(error=0, new_req_beam_off=new_req_beam_off, new_prefix_off=np.asarray(new_prefix_off, np.int64),
                new_page_off=np.asarray(new_page_off, np.int64), new_page_table=table,
                new_beam_slot=np.asarray([s for s, *_ in plan], np.int32), k_pool=k_pool, v_pool=v_pool,
                free_stack=new_free, free_count=len(free))
