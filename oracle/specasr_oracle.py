"""CPU fp64 oracle for the target decoder's tree-verification step.  TEST INFRASTRUCTURE ONLY.

This is a plain, slow restatement of what one verification round computes
(Section II-B: the target model checks every draft token at once, stops at the
first token that fails, and the output is identical to non-speculative greedy
decoding; Section II-B / Fig. 13 and Section IV-C: a draft token *tree* is
verified in one pass with a 2-D attention mask so that every branch gets its own
outcome).  It exists so that the CUDA path can be compared against it; only the
tests, the smoke check and the benchmark's CPU-baseline leg may import it.  It
shares no code with the CUDA path and never calls it.

The paper has no equations for this step, so the definition used is the plain
one the method must reproduce exactly:

    logits[i] = Decoder(prefix ++ tokens on the root->i path)[-1]   (ordinary causal attention)
    argmax[i] = lowest-id maximiser of logits[i]
    node i != root matches   iff tokens[i] == argmax[parent[i]]
    node i is accepted       iff every non-root node on its root path matches
    result                   = deepest accepted node (lowest index among equals), its path,
                               accept_len = its depth, bonus = its argmax

`causal_forward` is that definition written out with no cache and no tree mask;
`verify_tree` is the cached, tree-masked form and is trusted only because the
tests show it equals the former node by node.

Readings taken where the paper is silent (all from the workload description,
none from the paper): pre-norm Llama block, RMSNorm eps 1e-6 with a learned
gain, rotate-half RoPE (pairs (k, k + dh/2), theta_k = base^(-2k/dh)), SwiGLU,
GQA with q-head h reading kv-head h // (Hq/Hkv), score scale 1/sqrt(dh), no
biases, untied LM head; audio-embedding vectors enter layer 0 directly at
positions 0..Ta-1 and are followed by text tokens; node 0 of a tree is the last
committed token (never verified); tree node i sits at position L + depth[i];
argmax ties go to the lowest token id.

Parity pins (tests/test_oracle_*.py): an independent library decoder
(transformers' Llama in fp64 with the same tensors) for the block wiring, RoPE
pairing and GQA grouping; torch's scaled_dot_product_attention for the masked
attention; closed forms for RMSNorm / softmax / SiLU / RoPE; brute force over
root paths for the tree forward and for the accept rule; a plain prefill of the
accepted path for the commit; scipy's softmax, a hand-computed row and a brute-force sort for
top2_probs; a full sort, hand rows and a tie for top2_gap; hand-built trees with supplied logits for
the `decisive` flag of `decide`.  The paper prints no worked numbers for this step,
so parity with numbers *in the paper* is unpinned; only its lossless property
binds, and the tests check it.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------- storage widening

def widen(a: np.ndarray) -> np.ndarray:
    """uint16 arrays are bf16 bit patterns; everything is widened to fp64."""
    a = np.asarray(a)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(F64)
    return a.astype(F64)


class Weights:
    """Adapter over any store with .layer(l) / .globals() -> dict of arrays.  Widens on access, one
    layer at a time, so that a 7B-shape model never sits in memory in fp64."""

    def __init__(self, store, cache_layers: bool = False):
        self.store = store
        self._cache = {} if cache_layers else None
        self._globals = None

    def layer(self, l: int) -> dict:
        if self._cache is not None and l in self._cache:
            return self._cache[l]
        w = {k: widen(v) for k, v in self.store.layer(l).items()}
        if self._cache is not None:
            self._cache[l] = w
        return w

    def globals(self) -> dict:
        if self._globals is None:
            self._globals = {k: widen(v) for k, v in self.store.globals().items()}
        return self._globals


# --------------------------------------------------------------------------- elementwise pieces

def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """x / sqrt(mean(x^2) + eps) * g over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * g


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def rope(x: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotate-half rotary embedding.  x: [T, H, dh]; pos: [T] integer positions."""
    dh = x.shape[-1]
    half = dh // 2
    theta = base ** (-2.0 * np.arange(half, dtype=F64) / dh)
    ang = np.asarray(pos, dtype=F64)[:, None] * theta[None, :]          # [T, half]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def masked_softmax(scores: np.ndarray, mask: np.ndarray) -> np.ndarray:
    """Row softmax over the entries where mask is True (each row has at least one)."""
    s = np.where(mask, scores, -np.inf)
    s = s - np.max(s, axis=-1, keepdims=True)
    e = np.exp(s)
    return e / np.sum(e, axis=-1, keepdims=True)


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, mask: np.ndarray) -> np.ndarray:
    """q: [T, Hq, dh]; k, v: [S, Hkv, dh]; mask: [T, S] bool (True = visible).  Returns [T, Hq, dh]."""
    T, Hq, dh = q.shape
    Hkv = k.shape[1]
    group = Hq // Hkv
    out = np.empty_like(q)
    for h in range(Hq):
        kv = h // group
        scores = (q[:, h, :] @ k[:, kv, :].T) / np.sqrt(F64(dh))
        out[:, h, :] = masked_softmax(scores, mask) @ v[:, kv, :]
    return out


# --------------------------------------------------------------------------- KV cache

class KVCache:
    """Per layer K and V of every committed position: lists of [L, Hkv, dh] fp64 arrays."""

    def __init__(self, cfg):
        self.cfg = cfg
        self.K = [np.zeros((0, cfg.n_kv_heads, cfg.head_dim), F64) for _ in range(cfg.n_layers)]
        self.V = [np.zeros((0, cfg.n_kv_heads, cfg.head_dim), F64) for _ in range(cfg.n_layers)]

    @property
    def length(self) -> int:
        return self.K[0].shape[0]

    def copy(self) -> "KVCache":
        c = KVCache(self.cfg)
        c.K = [a.copy() for a in self.K]
        c.V = [a.copy() for a in self.V]
        return c

    def append(self, new_k, new_v):
        for l in range(self.cfg.n_layers):
            self.K[l] = np.concatenate([self.K[l], new_k[l]], axis=0)
            self.V[l] = np.concatenate([self.V[l], new_v[l]], axis=0)


# --------------------------------------------------------------------------- the decoder

def embed(weights: Weights, tokens) -> np.ndarray:
    return weights.globals()["embed"][np.asarray(tokens, dtype=np.int64)]


def decoder_stack(cfg, weights: Weights, x: np.ndarray, pos: np.ndarray, mask_new: np.ndarray,
                  cache: KVCache | None):
    """Run all layers over T new rows.

    x: [T, d] layer-0 inputs; pos: [T] positions; mask_new: [T, T] visibility among the new rows;
    every cached position is visible to every new row.  Returns (final hidden [T, d] before the
    final norm, list of new K per layer, list of new V per layer).
    """
    T = x.shape[0]
    L = cache.length if cache is not None else 0
    full_mask = np.concatenate([np.ones((T, L), dtype=bool), mask_new.astype(bool)], axis=1)
    new_k, new_v = [], []
    x = x.astype(F64)
    for l in range(cfg.n_layers):
        w = weights.layer(l)
        h = rmsnorm(x, w["g_attn"], cfg.eps)
        q = (h @ w["wq"].T).reshape(T, cfg.n_heads, cfg.head_dim)
        k = (h @ w["wk"].T).reshape(T, cfg.n_kv_heads, cfg.head_dim)
        v = (h @ w["wv"].T).reshape(T, cfg.n_kv_heads, cfg.head_dim)
        q = rope(q, pos, cfg.rope_base)
        k = rope(k, pos, cfg.rope_base)
        new_k.append(k)
        new_v.append(v)
        if cache is not None:
            k_all = np.concatenate([cache.K[l], k], axis=0)
            v_all = np.concatenate([cache.V[l], v], axis=0)
        else:
            k_all, v_all = k, v
        a = attention(q, k_all, v_all, full_mask).reshape(T, cfg.q_dim)
        x = x + a @ w["wo"].T
        h = rmsnorm(x, w["g_ffn"], cfg.eps)
        x = x + (silu(h @ w["wg"].T) * (h @ w["wu"].T)) @ w["wd"].T
    return x, new_k, new_v


def lm_logits(cfg, weights: Weights, hidden: np.ndarray) -> np.ndarray:
    g = weights.globals()
    return rmsnorm(hidden, g["g_final"], cfg.eps) @ g["lm_head"].T


def causal_forward(cfg, weights: Weights, inputs: np.ndarray) -> np.ndarray:
    """The plain definition: ordinary causal decoder over a whole sequence of layer-0 input
    vectors, no cache.  Returns logits [T, V]."""
    T = inputs.shape[0]
    mask = np.tril(np.ones((T, T), dtype=bool))
    hidden, _, _ = decoder_stack(cfg, weights, inputs, np.arange(T), mask, None)
    return lm_logits(cfg, weights, hidden)


def prefill(cfg, weights: Weights, cache: KVCache, inputs: np.ndarray, want_logits: bool = False):
    """Append T positions (audio vectors or embedded tokens) to the cache under causal attention."""
    T = inputs.shape[0]
    mask = np.tril(np.ones((T, T), dtype=bool))
    pos = cache.length + np.arange(T)
    hidden, nk, nv = decoder_stack(cfg, weights, inputs, pos, mask, cache)
    cache.append(nk, nv)
    if want_logits:
        return lm_logits(cfg, weights, hidden)
    return None


# --------------------------------------------------------------------------- tree side

class TreeError(ValueError):
    pass


def tree_prep(parent) -> tuple[np.ndarray, np.ndarray]:
    """depth[n] (root = 0) and anc[n, n] with anc[i, j] = True iff j is i or an ancestor of i.
    This matrix is the 2-D attention mask of a draft token tree (Fig. 13)."""
    parent = np.asarray(parent, dtype=np.int64)
    n = len(parent)
    if n < 1 or parent[0] != -1:
        raise TreeError("node 0 must be the root with parent -1")
    depth = np.zeros(n, dtype=np.int64)
    anc = np.zeros((n, n), dtype=bool)
    anc[0, 0] = True
    for i in range(1, n):
        p = parent[i]
        if p < 0 or p >= i:
            raise TreeError(f"parent[{i}] = {p} must satisfy 0 <= parent < index")
        depth[i] = depth[p] + 1
        anc[i] = anc[p]
        anc[i, i] = True
    return depth, anc


def top2_gap(logits: np.ndarray) -> np.ndarray:
    """Largest entry minus second largest entry along the last axis (0 where the maximum is attained twice;
    +inf for a single column, where nothing can overtake the only candidate)."""
    logits = np.asarray(logits, dtype=F64)
    if logits.shape[-1] < 2:
        return np.full(logits.shape[:-1], np.inf)
    part = np.partition(logits, -2, axis=-1)
    return part[..., -1] - part[..., -2]


def top2_probs(logits: np.ndarray) -> tuple[np.ndarray, np.ndarray]:
    """The two most probable tokens of every row and their probabilities under the softmax over the whole
    vocabulary ("normalized logits", Section IV-A: drafting stops where the top-1 value falls below a threshold;
    Section IV-C: the second-ranked token seeds a side branch).  Ties go to the lower token id.
    Returns (ids [n, 2] int32, probs [n, 2] fp64)."""
    logits = np.asarray(logits, dtype=F64)
    n, v = logits.shape
    ids = np.zeros((n, 2), dtype=np.int32)
    probs = np.zeros((n, 2), dtype=F64)
    for i in range(n):
        row = logits[i]
        e = np.exp(row - row.max())
        sm = e / e.sum()
        first = int(np.argmax(row))                       # lowest id among equal maxima
        rest = row.copy()
        rest[first] = -np.inf
        second = int(np.argmax(rest)) if v > 1 else first
        ids[i] = (first, second)
        probs[i] = (sm[first], sm[second])
    return ids, probs


def accept(tokens, parent, argmax) -> dict:
    """Greedy acceptance: follow draft tokens while they equal the target's own next token and stop
    at the first that does not (Section II-B), independently on every branch."""
    tokens = np.asarray(tokens)
    parent = np.asarray(parent, dtype=np.int64)
    depth, _ = tree_prep(parent)
    n = len(parent)
    ok = np.zeros(n, dtype=bool)
    ok[0] = True
    for i in range(1, n):
        ok[i] = ok[parent[i]] and (tokens[i] == argmax[parent[i]])
    best = 0
    for i in range(1, n):
        if ok[i] and depth[i] > depth[best]:
            best = i
    path = []
    j = best
    while j >= 0:
        path.append(j)
        j = parent[j]
    path = path[::-1]
    return {
        "accept_len": int(depth[best]),
        "best": int(best),
        "path": np.asarray(path, dtype=np.int32),
        "bonus": int(argmax[best]),
        "accepted_mask": ok,
    }


def verify_tree(cfg, weights: Weights, cache: KVCache, tokens, parent, decisive_gap: float = 1e-2) -> dict:
    """One verification round over a draft token tree on top of `cache` (which is not modified)."""
    tokens = np.asarray(tokens, dtype=np.int64)
    depth, anc = tree_prep(parent)
    if np.any(tokens < 0) or np.any(tokens >= cfg.vocab):
        raise TreeError("token id out of range")
    pos = cache.length + depth
    hidden, tk, tv = decoder_stack(cfg, weights, embed(weights, tokens), pos, anc, cache)
    logits = lm_logits(cfg, weights, hidden)
    res = decide(tokens, parent, logits, decisive_gap)
    res.update({"depth": depth, "pos": pos, "tree_K": tk, "tree_V": tv})
    return res


def verify_tree_uncached(cfg, weights: Weights, prefix_inputs: np.ndarray, tokens, parent,
                         decisive_gap: float = 1e-2) -> dict:
    """The same round without a cache object: the context rows and the tree rows go through the layer
    stack together, the context under causal attention, every tree node seeing the whole context and
    its own root path (Section II-B: the tree is verified in one pass on top of the decoded text).
    One pass over the weights instead of two, which is what makes the 7B shape affordable when the
    layers are regenerated one at a time.  Equal to prefill + verify_tree (tested)."""
    tokens = np.asarray(tokens, dtype=np.int64)
    depth, anc = tree_prep(parent)
    if np.any(tokens < 0) or np.any(tokens >= cfg.vocab):
        raise TreeError("token id out of range")
    L, n = prefix_inputs.shape[0], len(tokens)
    x = np.concatenate([np.asarray(prefix_inputs, dtype=F64), embed(weights, tokens)], axis=0)
    pos = np.concatenate([np.arange(L), L + depth])
    mask = np.zeros((L + n, L + n), dtype=bool)
    mask[:L, :L] = np.tril(np.ones((L, L), dtype=bool))
    mask[L:, :L] = True
    mask[L:, L:] = anc
    hidden, nk, nv = decoder_stack(cfg, weights, x, pos, mask, None)
    res = decide(tokens, parent, lm_logits(cfg, weights, hidden[L:]), decisive_gap)
    res.update({"depth": depth, "pos": pos[L:], "tree_K": [k[L:] for k in nk], "tree_V": [v[L:] for v in nv],
                "prefix_K": [k[:L] for k in nk], "prefix_V": [v[:L] for v in nv]})
    return res


def decide(tokens, parent, logits: np.ndarray, decisive_gap: float = 1e-2) -> dict:
    """From the logits of every node to the round's outcome: greedy tokens, their margins, the accept
    result, and whether that result is unambiguous.  The accept rule reads the arg-max of every node
    that has a child (to test the child's token) and of the winning node (the bonus token); the result
    is `decisive` when each of those was decided by more than `decisive_gap`.  A narrow margin at a
    childless node that does not win changes nothing that is reported."""
    logits = np.asarray(logits, dtype=F64)
    n = len(tokens)
    argmax = np.argmax(logits, axis=-1).astype(np.int32)
    gap = top2_gap(logits)
    res = accept(tokens, parent, argmax)
    consulted = np.zeros(n, dtype=bool)
    consulted[np.asarray(parent, dtype=np.int64)[1:]] = True
    consulted[res["best"]] = True
    res.update({
        "logits": logits, "argmax": argmax, "gap": gap, "consulted": consulted,
        "decisive": bool(np.all(gap[consulted] > decisive_gap)),
    })
    return res


def commit(cache: KVCache, result: dict) -> list[tuple[int, int]]:
    """Keep the accepted path: cache slot L + j receives tree node path[j].  Returns the
    (source slot, destination slot) pairs, slots counted from the start of the cache."""
    L = cache.length
    path = result["path"]
    moves = [(L + int(p), L + j) for j, p in enumerate(path)]
    cache.append([k[path] for k in result["tree_K"]], [v[path] for v in result["tree_V"]])
    return moves


def greedy_continuation(cfg, weights: Weights, cache: KVCache, root_token: int, k: int) -> list[int]:
    """Ordinary autoregressive greedy decoding: feed root_token, then each emitted token, k times.
    `cache` is left untouched."""
    c = cache.copy()
    out = []
    tok = int(root_token)
    for _ in range(k):
        logits = prefill(cfg, weights, c, embed(weights, [tok]), want_logits=True)
        tok = int(np.argmax(logits[-1]))
        out.append(tok)
    return out


# --------------------------------------------------------------------------- draft side (Section IV)
#
# The three drafting strategies of Section IV, restated as plain control flow over a "draft step"
# callable.  They decide which tokens are proposed; they never touch what the target accepts, so the
# lossless property of Section II-B is untouched by them.  Readings taken where the paper is silent:
#   * "normalized logits" (Section IV-A) = softmax probability over the whole vocabulary (top2_probs);
#   * "corresponding or adjacent positions" (Section IV-B) = position offsets 0, -1, +1, tried in that order;
#   * a side branch of the sparse tree (Section IV-C) starts with the second-ranked token at an uncertain
#     trunk position, is extended greedily, keeps the token on which it meets the trunk or an earlier branch
#     and ends there; a branch also ends after `max_branch` tokens or when the node budget is used up.

RECYCLE_OFFSETS = (0, -1, 1)


def match_position(seq_tokens, seq_first_pos: int, token: int, pos: int, offsets=RECYCLE_OFFSETS,
                   lowest_pos: int | None = None):
    """Section IV-B, merging: does `token`, generated for position `pos`, equal the token that the
    sequence `seq_tokens` (whose first token sits at position `seq_first_pos`) carries at the same or an
    adjacent position?  Returns the index into seq_tokens of the first such position in the order of
    `offsets`, or None.  Positions below `lowest_pos` are not considered."""
    for off in offsets:
        q = pos + off
        if lowest_pos is not None and q < lowest_pos:
            continue
        i = q - seq_first_pos
        if 0 <= i < len(seq_tokens) and int(seq_tokens[i]) == int(token):
            return i
    return None


def adaptive_sequence(step_fn, root: int, max_len: int, threshold: float) -> list[int]:
    """Section IV-A: greedy single-sequence drafting that stops after the first token whose probability
    falls below `threshold` (that token is still proposed), or after `max_len` tokens.
    step_fn(path) -> next-token logits [V] of the draft model after the context and `path` (path[0] = root)."""
    path, out = [int(root)], []
    for _ in range(max_len):
        ids, probs = top2_probs(np.asarray(step_fn(path), dtype=F64)[None, :])
        out.append(int(ids[0, 0]))
        path.append(int(ids[0, 0]))
        if probs[0, 0] < threshold:
            break
    return out


def two_pass_tree(step_fn, root: int, max_len: int, threshold: float, n_nodes: int, max_branch: int) -> dict:
    """Section IV-C, two-pass sparse-tree prediction.

    Pass 1: greedy single-sequence decoding of `max_len` trunk tokens; a position whose top-1 probability
    is below `threshold` is marked together with the second-ranked token, and decoding goes on.
    Pass 2: at every mark, in trunk order, a branch starts with the second-ranked token as a sibling of the
    trunk token and is extended greedily; it ends with the token that equals the trunk's (or an earlier
    branch's) token at the corresponding or an adjacent depth, after `max_branch` tokens, or when the tree
    has `n_nodes` nodes.  Returns tokens / parent (root = node 0, trunk = nodes 1..m in order, then the
    branches in the order they were grown), the marks [(depth, second token)] and the depth of every node."""
    tokens, parent, depth = [int(root)], [-1], [0]
    path, marks = [int(root)], []
    for j in range(1, max_len + 1):
        if len(tokens) >= n_nodes:
            break
        ids, probs = top2_probs(np.asarray(step_fn(path), dtype=F64)[None, :])
        tokens.append(int(ids[0, 0]))
        parent.append(len(tokens) - 2)
        depth.append(j)
        path.append(int(ids[0, 0]))
        if probs[0, 0] < threshold and int(ids[0, 1]) != int(ids[0, 0]):
            marks.append((j, int(ids[0, 1])))
    m = len(tokens) - 1                                   # trunk nodes are 1..m, trunk token at depth d is tokens[d]
    grown = []                                            # (first depth, tokens) of the branches so far

    def rejoins(tok, d):
        if match_position(tokens[1:m + 1], 1, tok, d) is not None:
            return True
        return any(match_position(bt, d0, tok, d) is not None for d0, bt in grown)

    for j, second in marks:
        if len(tokens) >= n_nodes:
            break
        bpath = [int(root)] + tokens[1:j] + [second]
        tokens.append(second)
        parent.append(j - 1)                              # sibling of trunk node j
        depth.append(j)
        btoks = [second]
        while not rejoins(btoks[-1], j + len(btoks) - 1) and len(btoks) < max_branch and len(tokens) < n_nodes:
            nxt = int(np.argmax(np.asarray(step_fn(bpath), dtype=F64)))
            tokens.append(nxt)
            parent.append(len(tokens) - 2)
            depth.append(j + len(btoks))
            btoks.append(nxt)
            bpath.append(nxt)
        grown.append((j, btoks))
    return {"tokens": np.asarray(tokens, np.int32), "parent": np.asarray(parent, np.int32),
            "depth": np.asarray(depth, np.int64), "marks": marks, "trunk_len": m}


def recycled_draft(tree_step_fn, last_accepted: int, seq1, accept_len: int, bonus: int, max_len: int,
                   max_regen: int) -> dict:
    """Section IV-B, draft sequence recycling after a verification round.

    `seq1` is the draft sequence that was verified (trunk tokens at depths 1..m under the old root);
    `accept_len` of them were accepted and the target emitted `bonus` for depth accept_len + 1.  The draft
    model now decodes two sequences side by side in one masked token tree under the last accepted token:
    sequence 1, the unaccepted tail seq1[accept_len:], which it keeps extending, and sequence 2, which starts
    at `bonus` and regenerates what failed.  After every step the token just regenerated for depth q is
    compared with sequence 1 at depths q, q - 1, q + 1; on a match the two sequences are merged: the next
    draft is the regenerated tokens followed by what sequence 1 holds after the matching depth.

    tree_step_fn(tokens, parent) -> logits [n, V] of the draft model over a token tree whose node 0 is
    `last_accepted`, the last accepted token (the old root if nothing was accepted); its context is
    everything before that token.  Returns the next draft (the tokens proposed
    after `bonus`, at most max_len), how many regeneration steps were made and where the merge happened."""
    seq1 = [int(t) for t in seq1]
    a = int(accept_len)
    tail = seq1[a:]                                       # depths a+1 .. m; tail[0] is the rejected token
    if not tail:                                          # everything was accepted: nothing to recycle
        return {"draft": [], "steps": 0, "merged_at": None, "regenerated": [], "extended": []}
    regen, ext = [], []
    merged = None
    for step in range(max_regen):
        # node 0 = last accepted token; chain 1 = sequence 1, chain 2 = sequence 2
        c1 = tail + ext
        c2 = [int(bonus)] + regen
        tokens = [int(last_accepted)] + c1 + c2
        parent = [-1] + [0] + list(range(1, len(c1))) + [0] + list(range(len(c1) + 1, len(c1) + len(c2)))
        logits = np.asarray(tree_step_fn(np.asarray(tokens), np.asarray(parent)), dtype=F64)
        ext.append(int(np.argmax(logits[len(c1)])))       # after the tip of sequence 1
        r = int(np.argmax(logits[len(c1) + len(c2)]))     # after the tip of sequence 2
        regen.append(r)
        q = a + 1 + len(regen)                            # depth of the token just regenerated
        hit = match_position(tail + ext, a + 1, r, q, lowest_pos=a + 1)
        if hit is not None:
            merged = a + 1 + hit
            break
        if len(regen) >= max_len:
            break
    if merged is not None:
        reuse = (tail + ext)[merged - a:]                 # what sequence 1 holds after the matching depth
        draft = regen + reuse
    else:
        draft = list(regen)
    return {"draft": draft[:max_len], "steps": len(regen), "merged_at": merged, "regenerated": regen, "extended": ext}
