"""Stack-distance capacity model (Section 3.2, Eq. 4; Appendix C "Prefix coverage from
a reference stream").

The reuse distance D of a reference is the number of different chunks, *other* than this one, touched
strictly between it and the previous reference to the same chunk (infinite on a first
reference).  Under a fully associative LRU tier that admits every miss, a reference
hits exactly when D < K (Mattson's inclusion property).  Host coverage of a request is
its leading run of hits; useful restoration is R_j = max{0, H_j - G_j}; summing the
uncovered prompt length predicts computed prefill.
"""
import math

INF = math.inf


def reuse_distances_definition(stream):
    """Literal definition: scan back to the previous reference, count distinct others."""
    out = []
    for i, k in enumerate(stream):
        s = None
        for j in range(i - 1, -1, -1):
            if stream[j] == k:
                s = j
                break
        if s is None:
            out.append(INF)
        else:
            out.append(len(set(stream[s + 1:i])))   # k itself cannot occur in between
    return out


def reuse_distances(stream):
    """Same distances in O(T log T): keep a mark at the latest position of every chunk;
    the distinct chunks seen since position s are the marks to the right of s."""
    T = len(stream)
    tree = [0] * (T + 1)

    def add(pos, v):
        pos += 1
        while pos <= T:
            tree[pos] += v
            pos += pos & -pos

    def prefix(pos):          # marks at positions [0, pos)
        s = 0
        while pos > 0:
            s += tree[pos]
            pos -= pos & -pos
        return s

    last = {}
    out = []
    for i, k in enumerate(stream):
        s = last.get(k)
        if s is None:
            out.append(INF)
        else:
            out.append(prefix(i) - prefix(s + 1))
            add(s, -1)
        add(i, 1)
        last[k] = i
    return out


def predicted_hits(distances, capacity):
    """Eq. 4: the reference survives (hits) iff D < K."""
    return [d < capacity for d in distances]


def request_coverage(hit_flags):
    """Leading run of hits of one request's references."""
    n = 0
    for h in hit_flags:
        if not h:
            break
        n += 1
    return n


def predict_trace(request_keys, request_tokens, gpu_prefix_blocks, capacity, block_size):
    """Per-capacity prediction for a whole trace under write-all.

    request_keys[j]      keys of request j (in request order)
    request_tokens[j]    prompt tokens of request j
    gpu_prefix_blocks[j] G_j
    Returns dict(host_cover=[H_j], restored_blocks=sum R_j, computed_tokens=sum uncovered,
                 hit_flags=[...per reference...]).
    """
    stream = [k for keys in request_keys for k in keys]
    hits = predicted_hits(reuse_distances(stream), capacity)
    pos = 0
    cover, restored, computed = [], 0, 0
    for keys, n, G in zip(request_keys, request_tokens, gpu_prefix_blocks):
        H = request_coverage(hits[pos:pos + len(keys)])
        pos += len(keys)
        cover.append(H)
        restored += max(0, H - G)
        computed += n - max(G, H) * block_size
    return dict(host_cover=cover, restored_blocks=restored, computed_tokens=computed,
                hit_flags=hits)


def working_set_full(distances):
    """Smallest capacity (in chunks) at which every re-reference hits: max finite D + 1."""
    finite = [d for d in distances if d != INF]
    return (max(finite) + 1) if finite else 0


def working_set_within(request_keys, request_tokens, gpu_prefix_blocks, block_size, percent=1):
    """Smallest capacity K (in chunks) whose predicted computed tokens are within ``percent`` % of
    the prediction for an unbounded tier: computed(K) * 100 <= computed(inf) * (100 + percent).
    Plain scan over K = 0, 1, 2, ... (computed(K) never grows with K, by inclusion)."""
    stream = [k for keys in request_keys for k in keys]
    top = working_set_full(reuse_distances(stream))
    floor_tokens = predict_trace(request_keys, request_tokens, gpu_prefix_blocks, top, block_size)["computed_tokens"]
    for K in range(0, top + 1):
        c = predict_trace(request_keys, request_tokens, gpu_prefix_blocks, K, block_size)["computed_tokens"]
        if c * 100 <= floor_tokens * (100 + percent):
            return K
    return top
