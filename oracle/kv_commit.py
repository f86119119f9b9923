"""Oracle of the KV-cache update that ends a decode step.

TEST INFRASTRUCTURE, NOT PRODUCT CODE (plain numpy, loops over beams; shares nothing with the
CUDA library).

Section "Forest-based Parallel Decoding": every input beam owns a key-value cache; after the
iteration the caches are updated according to the output beams -- an output beam keeps the
cache of the input beam it descends from, extended by the keys/values of the forest nodes on
its path.  Section "Reducing Memory Cost": optionally only the output beam of lowest
perplexity is kept per request, so that a single cache survives.

Conventions (the paper fixes none of them, so the numbering of the kept beams and the tie rule
are "parity unpinned"; the content of each cache is pinned through the attention; they mirror
the attention's layout):
  * the cache of a beam holds every token of the beam except its last one (the last token is
    the root of the beam's next draft tree and brings its own key/value);
  * an output beam (parent node n, new token x) therefore keeps: cache of its input beam, then
    the keys/values of the nodes on the path root .. n, root first; x becomes the next root;
  * new beams are numbered request by request, inside a request in output-slot order;
  * perplexity of an output beam = exp(-out_logp / length), length = tokens of the new beam
    = new cache length + 1; ties go to the lower slot.
"""
import numpy as np


def path_to_root(parent, n):
    """Nodes root .. n (root first)."""
    path = []
    while n >= 0:
        path.append(int(n))
        n = parent[n]
    return path[::-1]


def select_beams(forest, out_off, out_width, out_parent, out_root_beam, out_logp, prefix_off, keep_best):
    """The output slots that survive, request by request: list of (request, slot)."""
    parent = np.asarray(forest["parent"])
    kept = []
    for r in range(int(forest["R"])):
        slots = list(range(int(out_off[r]), int(out_off[r]) + int(out_width[r])))
        if keep_best and slots:
            best, best_ppl = None, None
            for s in slots:
                b = int(out_root_beam[s])
                length = int(prefix_off[b + 1] - prefix_off[b]) + len(path_to_root(parent, int(out_parent[s]))) + 1
                ppl = np.exp(-np.float64(out_logp[s]) / length)
                if best is None or ppl < best_ppl:
                    best, best_ppl = s, ppl
            slots = [best]
        kept += [(r, s) for s in slots]
    return kept


def kv_commit(forest, Hkv, d, out_off, out_width, out_parent, out_root_beam, out_logp,
              k_new, v_new, k_prefix, v_prefix, prefix_off, keep_best=False):
    """Returns dict(new_req_beam_off[R+1], new_prefix_off[B'+1], new_beam_slot[B'],
    k_cache, v_cache): the caches of the kept output beams packed like the inputs, beam j as
    [Hkv, L'_j, d] starting at element new_prefix_off[j]*Hkv*d.  k_new/v_new: [N, Hkv, d];
    k_prefix/v_prefix: flat arrays in the attention's packed layout."""
    parent = np.asarray(forest["parent"])
    k_new = np.asarray(k_new).reshape(-1, Hkv, d)
    v_new = np.asarray(v_new).reshape(-1, Hkv, d)
    k_prefix, v_prefix = np.asarray(k_prefix).reshape(-1), np.asarray(v_prefix).reshape(-1)
    kept = select_beams(forest, out_off, out_width, out_parent, out_root_beam, out_logp, prefix_off, keep_best)
    R = int(forest["R"])
    new_req_beam_off = np.zeros(R + 1, np.int32)
    for r, _ in kept:
        new_req_beam_off[r + 1] += 1
    new_req_beam_off = np.cumsum(new_req_beam_off).astype(np.int32)
    new_prefix_off = [0]
    k_parts, v_parts = [], []
    for _, s in kept:
        b = int(out_root_beam[s])
        L = int(prefix_off[b + 1] - prefix_off[b])
        base = int(prefix_off[b]) * Hkv * d
        old_k = k_prefix[base:base + Hkv * L * d].reshape(Hkv, L, d)
        old_v = v_prefix[base:base + Hkv * L * d].reshape(Hkv, L, d)
        path = path_to_root(parent, int(out_parent[s]))
        add_k = np.transpose(k_new[path], (1, 0, 2))        # [Hkv, len(path), d]
        add_v = np.transpose(v_new[path], (1, 0, 2))
        k_parts.append(np.concatenate([old_k, add_k], axis=1).reshape(-1))
        v_parts.append(np.concatenate([old_v, add_v], axis=1).reshape(-1))
        new_prefix_off.append(new_prefix_off[-1] + L + len(path))
    empty = np.zeros(0, k_prefix.dtype)
    return dict(new_req_beam_off=new_req_beam_off,
                new_prefix_off=np.asarray(new_prefix_off, np.int64),
                new_beam_slot=np.asarray([s for _, s in kept], np.int32),
                k_cache=np.concatenate(k_parts) if k_parts else empty,
                v_cache=np.concatenate(v_parts) if v_parts else empty)
