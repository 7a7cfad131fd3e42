"""Pins of the oracle's tree side: the cached, tree-masked forward must equal the plain causal
definition node by node, and accept / commit must satisfy what lossless draft-then-verify
(Section II-B) implies."""
import itertools

import numpy as np
import pytest

import gen
from oracle import specasr_oracle as O
from helpers import oracle_weights, filled_cache


def _root_path(parent, i):
    path = []
    while i >= 0:
        path.append(i)
        i = parent[i]
    return path[::-1]


def _scenario(name="micro", n_audio=9, n_prompt=5, seed=0):
    cfg = gen.get_config(name)
    W = oracle_weights(cfg, seed)
    cache, x, audio, prompt = filled_cache(cfg, W, n_audio, n_prompt, seed)
    return cfg, W, cache, x, prompt


def test_tree_prep_values_and_errors():
    depth, anc = O.tree_prep([-1, 0, 0, 1, 3, 2])
    assert list(depth) == [0, 1, 1, 2, 3, 2]
    assert [list(np.nonzero(r)[0]) for r in anc] == [[0], [0, 1], [0, 2], [0, 1, 3], [0, 1, 3, 4], [0, 2, 5]]
    for bad in ([0, 0], [-1, 1], [-1, -1], [-1, 0, 5], []):
        with pytest.raises(O.TreeError):
            O.tree_prep(bad)


@pytest.mark.parametrize("name,tree", [("micro", "binary"), ("micro", "sparse"), ("tiny", "binary")])
def test_tree_forward_equals_bruteforce_causal(name, tree):
    """Every node's logits equal an uncached causal forward over prefix + that node's root path."""
    cfg, W, cache, x, prompt = _scenario(name)
    parent = gen.complete_binary_tree(15) if tree == "binary" else gen.sparse_tree(20, seed=3)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=1, root_token=int(prompt[-1]))
    res = O.verify_tree(cfg, W, cache, tokens, parent)
    for i in range(len(parent)):
        path = _root_path(parent, i)
        seq = np.concatenate([x, O.embed(W, tokens[path])], axis=0)
        ref = O.causal_forward(cfg, W, seq)[-1]
        assert np.abs(res["logits"][i] - ref).max() <= 1e-10 * max(1.0, np.abs(ref).max())
        assert res["argmax"][i] == int(np.argmax(ref))


def test_chain_tree_is_sequential_greedy_decoding():
    cfg, W, cache, x, prompt = _scenario("micro")
    root = int(prompt[-1])
    k = 6
    greedy = O.greedy_continuation(cfg, W, cache, root, k + 1)
    parent = gen.chain_tree(k)
    tokens = np.array([root] + greedy[:k], dtype=np.int32)
    res = O.verify_tree(cfg, W, cache, tokens, parent)
    # one causal forward over the same sequence gives the same per-step argmax
    full = O.causal_forward(cfg, W, np.concatenate([x, O.embed(W, tokens)], axis=0))
    assert list(res["argmax"]) == list(full[len(x):].argmax(-1)) == greedy
    # a draft equal to the target's greedy continuation is accepted whole, bonus = next greedy token
    assert res["accept_len"] == k and list(res["path"]) == list(range(k + 1)) and res["bonus"] == greedy[k]
    # corrupt position j (1-based draft index): exactly j-1 drafts survive
    for j in (1, 3, 6):
        bad = tokens.copy()
        bad[j] = (bad[j] + 1) % cfg.vocab
        r = O.verify_tree(cfg, W, cache, bad, parent)
        assert r["accept_len"] == j - 1 and r["bonus"] == greedy[j - 1]
        assert list(r["argmax"][:j]) == greedy[:j]


def test_accept_matches_path_enumeration():
    """Brute force: among all root paths whose every draft token equals the argmax at its parent,
    take the longest (lowest end index among equals)."""
    rng = np.random.default_rng(0)
    for trial in range(300):
        n = int(rng.integers(1, 16))
        parent = np.array([-1] + [int(rng.integers(0, i)) for i in range(1, n)], dtype=np.int32)
        tokens = rng.integers(0, 3, size=n)
        argmax = rng.integers(0, 3, size=n)
        best, best_len = 0, 0
        for i in range(n):
            path = _root_path(parent, i)
            if all(tokens[c] == argmax[p] for p, c in zip(path[:-1], path[1:])):
                if len(path) - 1 > best_len:
                    best, best_len = i, len(path) - 1
        r = O.accept(tokens, parent, argmax)
        assert (r["best"], r["accept_len"]) == (best, best_len)
        assert list(r["path"]) == _root_path(parent, best) and r["bonus"] == argmax[best]
        depth, _ = O.tree_prep(parent)
        assert r["accept_len"] <= depth.max()


def test_branches_are_independent_and_order_does_not_matter():
    cfg, W, cache, x, prompt = _scenario("micro")
    parent = gen.sparse_tree(24, seed=4)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=2, root_token=int(prompt[-1]))
    res = O.verify_tree(cfg, W, cache, tokens, parent)
    _, anc = O.tree_prep(parent)
    # changing tokens off node i's root path leaves its logits untouched
    i = 17
    other = tokens.copy()
    off = ~anc[i]
    other[off] = (other[off] + 7) % cfg.vocab
    res2 = O.verify_tree(cfg, W, cache, other, parent)
    assert np.array_equal(res["logits"][i], res2["logits"][i])
    # any renumbering with parent < child gives the same per-node logits and the same accepted path
    p2, t2, old = gen.relabel_tree(parent, tokens, seed=9)
    res3 = O.verify_tree(cfg, W, cache, t2, p2)
    assert np.abs(res3["logits"] - res["logits"][old]).max() < 1e-12
    assert res3["accept_len"] == res["accept_len"]
    assert list(tokens[res["path"]]) == list(t2[res3["path"]])


def test_positions_shift_invariance_of_whole_stack():
    """Rotary attention only sees position differences: the same tokens verified on the same cache
    contents placed 100 positions later give the same logits."""
    cfg = gen.get_config("micro")
    W = oracle_weights(cfg, 0)
    toks = gen.prompt_tokens(8, cfg.vocab, 3)
    emb = O.embed(W, toks)
    T = len(toks)
    mask = np.tril(np.ones((T, T), bool))
    h0, _, _ = O.decoder_stack(cfg, W, emb, np.arange(T), mask, None)
    h1, _, _ = O.decoder_stack(cfg, W, emb, 100 + np.arange(T), mask, None)
    assert np.abs(h0 - h1).max() < 1e-9


def test_commit_equals_plain_prefill_of_accepted_path():
    cfg, W, cache, x, prompt = _scenario("micro")
    root = int(prompt[-1])
    greedy = O.greedy_continuation(cfg, W, cache, root, 4)
    parent = gen.complete_binary_tree(15)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=5, root_token=root, main_tokens=greedy[:3])
    res = O.verify_tree(cfg, W, cache, tokens, parent)
    assert res["accept_len"] == 3 and list(res["path"]) == [0, 1, 3, 7] and res["bonus"] == greedy[3]
    L = cache.length
    before = cache.copy()
    moves = O.commit(cache, res)
    assert moves == [(L + 0, L + 0), (L + 1, L + 1), (L + 3, L + 2), (L + 7, L + 3)]
    assert cache.length == L + 4
    ref = before.copy()
    O.prefill(cfg, W, ref, O.embed(W, tokens[res["path"]]))
    for l in range(cfg.n_layers):
        assert np.abs(cache.K[l] - ref.K[l]).max() < 1e-12 and np.abs(cache.V[l] - ref.V[l]).max() < 1e-12
        assert np.array_equal(cache.K[l][:L], before.K[l])


def test_speculative_loop_is_lossless():
    """Draft-then-verify rounds with imperfect drafts emit exactly the autoregressive greedy
    transcript (Section II-B: lossless)."""
    cfg, W, cache, x, prompt = _scenario("micro", seed=2)
    root = int(prompt[-1])
    want = O.greedy_continuation(cfg, W, cache, root, 14)
    rng = np.random.default_rng(7)
    out = []
    rounds = 0
    while len(out) < 14:
        k = min(4, 14 - len(out))
        # drafts: the true continuation with each position corrupted with p = 0.3
        truth = want[len(out):len(out) + k]
        draft = [t if rng.random() > 0.3 else (t + 1) % cfg.vocab for t in truth]
        parent = gen.chain_tree(len(draft))
        tokens = np.array([root] + draft, dtype=np.int32)
        res = O.verify_tree(cfg, W, cache, tokens, parent)
        O.commit(cache, res)
        out += [int(t) for t in tokens[res["path"]][1:]] + [res["bonus"]]
        root = res["bonus"]
        rounds += 1
    assert out[:14] == want and rounds < 14


def test_config1_scenario_accepts_three():
    """Tiny decoder, 64 audio vectors + 8 prompt tokens, 15-node binary tree whose leftmost path
    carries the greedy continuation for 3 tokens."""
    cfg, W, cache, x, prompt = _scenario("tiny", n_audio=64, n_prompt=8, seed=0)
    assert cache.length == 71
    root = int(prompt[-1])
    greedy = O.greedy_continuation(cfg, W, cache, root, 4)
    parent = gen.complete_binary_tree(15)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=0, root_token=root, main_tokens=greedy[:3])
    res = O.verify_tree(cfg, W, cache, tokens, parent)
    assert res["accept_len"] == 3 and list(res["path"]) == [0, 1, 3, 7] and res["bonus"] == greedy[3]
    assert list(res["pos"]) == [71 + d for d in [0, 1, 1, 2, 2, 2, 2, 3, 3, 3, 3, 3, 3, 3, 3]]


def test_planted_mistakes_are_caught():
    """Each pin above must be able to fail: break one convention at a time in a copy of the oracle's
    pieces and check that the brute-force / library comparison notices."""
    cfg = gen.get_config("micro")
    W = oracle_weights(cfg, 0)
    toks = gen.prompt_tokens(6, cfg.vocab, 0)
    x = O.embed(W, toks)
    good = O.causal_forward(cfg, W, x)
    saved = (O.rope, O.silu, O.rmsnorm)
    try:
        def rope_interleaved(t, pos, base):      # pairs (2k, 2k+1) instead of (k, k + dh/2)
            dh = t.shape[-1]
            theta = base ** (-2.0 * np.arange(dh // 2) / dh)
            ang = np.asarray(pos, float)[:, None] * theta[None]
            c, s = np.cos(ang)[:, None], np.sin(ang)[:, None]
            out = np.empty_like(t)
            out[..., 0::2] = t[..., 0::2] * c - t[..., 1::2] * s
            out[..., 1::2] = t[..., 1::2] * c + t[..., 0::2] * s
            return out
        O.rope = rope_interleaved
        assert np.abs(O.causal_forward(cfg, W, x) - good).max() > 1e-4
        O.rope = saved[0]
        O.rmsnorm = lambda t, g, eps: t / np.sqrt(np.mean(t * t, -1, keepdims=True) + eps)   # gain dropped
        assert np.abs(O.causal_forward(cfg, W, x) - good).max() > 1e-4
        O.rmsnorm = saved[2]
        O.silu = lambda t: 1.0 / (1.0 + np.exp(-t))                                          # sigmoid only
        assert np.abs(O.causal_forward(cfg, W, x) - good).max() > 1e-4
    finally:
        O.rope, O.silu, O.rmsnorm = saved
    # a tree mask that lets siblings see each other breaks the brute-force equality
    cache = O.KVCache(cfg)
    O.prefill(cfg, W, cache, x[:-1])
    parent = np.array([-1, 0, 0], np.int32)
    tokens = np.array([toks[-1], 5, 9], np.int32)
    res = O.verify_tree(cfg, W, cache, tokens, parent)
    ref = O.causal_forward(cfg, W, np.concatenate([x, O.embed(W, [9])]))[-1]
    assert np.abs(res["logits"][2] - ref).max() < 1e-10
    leaky = O.causal_forward(cfg, W, np.concatenate([x, O.embed(W, [5, 9])]))[-1]
    assert np.abs(leaky - ref).max() > 1e-6


def test_oracle_reproduces_the_stored_config1_values():
    """tests/golden/config1_tiny_verify.json was written by tests/golden/make_golden.py from the oracle alone; a
    change to the oracle's arithmetic (or to the seeded generators) shows up here."""
    import importlib.util
    import json
    import os
    here = os.path.dirname(os.path.abspath(__file__))
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(here, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    now = mod.compute()
    stored = json.load(open(os.path.join(here, "golden", "config1_tiny_verify.json")))
    assert stored["accept_len"] == 3 and stored["path"] == [0, 1, 3, 7]      # the workload's stated outcome
    for key in ("tokens", "parent", "greedy_continuation", "argmax", "accept_len", "path", "bonus", "top2_ids_row0"):
        assert now[key] == stored[key], key
    for key in ("logits_row0_first8", "top2_probs_row0"):
        assert np.allclose(now[key], stored[key], rtol=1e-9, atol=1e-12), key
    assert abs(now["logits_abs_sum"] - stored["logits_abs_sum"]) <= 1e-7 * stored["logits_abs_sum"]
    assert abs(now["min_top2_gap"] - stored["min_top2_gap"]) < 1e-9


def test_uncached_round_equals_prefill_then_verify():
    """verify_tree_uncached (context and tree in one pass) against prefill + verify_tree, and through that against
    the per-node brute force that pins verify_tree."""
    cfg = gen.get_config("micro")
    W = oracle_weights(cfg, 3)
    cache, x, audio, prompt = filled_cache(cfg, W, 11, 4, seed=3)
    parent = gen.sparse_tree(17, seed=3)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=3, root_token=int(prompt[-1]))
    a = O.verify_tree(cfg, W, cache, tokens, parent)
    b = O.verify_tree_uncached(cfg, W, x, tokens, parent)
    assert np.abs(a["logits"] - b["logits"]).max() < 1e-10
    assert a["accept_len"] == b["accept_len"] and list(a["path"]) == list(b["path"]) and a["bonus"] == b["bonus"]
    for l in range(cfg.n_layers):
        assert np.abs(a["tree_K"][l] - b["tree_K"][l]).max() < 1e-12
        assert np.abs(a["tree_V"][l] - b["tree_V"][l]).max() < 1e-12
        assert np.abs(cache.K[l] - b["prefix_K"][l]).max() < 1e-12
    # one node against the plain definition: causal forward over context + its root path
    i = int(np.argmax(a["depth"]))
    path = []
    j = i
    while j >= 0:
        path.append(j)
        j = int(parent[j])
    seq = np.concatenate([x, O.embed(W, tokens[path[::-1]])], 0)
    assert np.abs(O.causal_forward(cfg, W, seq)[-1] - b["logits"][i]).max() < 1e-10
