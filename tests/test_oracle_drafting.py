"""Pins of the oracle's drafting strategies (Section IV): the position-matching rule against a brute-force
restatement, and the three strategies on scripted draft models whose outcome can be worked out by hand."""
import numpy as np
import pytest

import gen
from oracle import specasr_oracle as O
from helpers import oracle_weights, filled_cache

V = 12


def _onehot(tok, second=None, p1=0.9):
    """Logits over V tokens whose softmax gives `tok` probability p1 (the largest), `second` the next largest
    (0.8 p1, or half of what is left if that is less), and spreads the rest evenly over the other tokens."""
    p = np.zeros(V)
    p[tok] = p1
    rest = 1.0 - p1
    if second is not None and second != tok:
        p[second] = min(0.8 * p1, 0.5 * rest)
        rest -= p[second]
    others = [i for i in range(V) if p[i] == 0.0]
    for i in others:
        p[i] = rest / len(others)
    assert np.argmax(p) == tok and abs(p.sum() - 1.0) < 1e-12
    return np.log(p)


def test_match_position_against_bruteforce_and_hand_cases():
    seq, first = [5, 6, 7, 6], 3                       # token 5 at position 3, 6 at 4, 7 at 5, 6 at 6
    assert O.match_position(seq, first, 6, 4) == 1     # same position
    assert O.match_position(seq, first, 5, 4) == 0     # one position earlier
    assert O.match_position(seq, first, 7, 4) == 2     # one position later
    assert O.match_position(seq, first, 7, 3) is None  # two positions away
    assert O.match_position(seq, first, 6, 5) == 1     # both neighbours carry 6: the earlier offset in the order 0, -1, +1 wins
    assert O.match_position(seq, first, 5, 2) == 0 and O.match_position(seq, first, 5, 2, lowest_pos=4) is None
    assert O.match_position(seq, first, 6, 7) == 3 and O.match_position(seq, first, 6, 8) is None
    assert O.match_position([], 0, 1, 0) is None
    rng = np.random.default_rng(0)
    for _ in range(300):
        n = int(rng.integers(1, 8))
        s = rng.integers(0, 4, size=n)
        f, tok, pos = int(rng.integers(0, 5)), int(rng.integers(0, 4)), int(rng.integers(-2, 14))
        want = None
        for off in (0, -1, 1):                          # the definition, written out
            q = pos + off
            if f <= q < f + n and s[q - f] == tok:
                want = q - f
                break
        assert O.match_position(s, f, tok, pos) == want


def test_adaptive_sequence_stops_after_the_first_uncertain_token():
    script = {1: (3, 0.9), 2: (4, 0.8), 3: (5, 0.3), 4: (6, 0.9)}        # path length -> (token, top-1 probability)
    step = lambda path: _onehot(script[len(path)][0], second=0, p1=script[len(path)][1])
    assert O.adaptive_sequence(step, 9, max_len=24, threshold=0.4) == [3, 4, 5]      # the uncertain token is still proposed
    assert O.adaptive_sequence(step, 9, max_len=2, threshold=0.4) == [3, 4]          # the length cap
    assert O.adaptive_sequence(step, 9, max_len=4, threshold=0.0) == [3, 4, 5, 6]    # threshold 0 never truncates
    assert O.adaptive_sequence(step, 9, max_len=4, threshold=0.95) == [3]


def test_two_pass_tree_on_a_scripted_draft_model():
    """Trunk 1 2 3 4 5 6 under root 0; positions 2 and 4 are uncertain with second-ranked tokens 7 and 8.
    After (.., 1, 7) the model says 9 then 4: 4 is the trunk's token at the same depth, so the branch is
    7 9 4 and ends.  After (.., 3, 8) it says 6: the trunk's token one depth later, so the branch is 8 6."""
    trunk = [1, 2, 3, 4, 5, 6]

    def step(path):
        path = list(path)
        if path == [0] + trunk[:len(path) - 1]:                    # on the trunk
            j = len(path)
            unsure = {2: 7, 4: 8}
            return _onehot(trunk[j - 1], second=unsure.get(j, 11), p1=0.3 if j in unsure else 0.9)
        table = {(0, 1, 7): 9, (0, 1, 7, 9): 4, (0, 1, 7, 9, 4): 10, (0, 1, 2, 3, 8): 6, (0, 1, 2, 3, 8, 6): 10}
        return _onehot(table[tuple(path)], second=0)

    t = O.two_pass_tree(step, 0, max_len=6, threshold=0.4, n_nodes=32, max_branch=5)
    assert t["marks"] == [(2, 7), (4, 8)] and t["trunk_len"] == 6
    assert list(t["tokens"]) == [0, 1, 2, 3, 4, 5, 6, 7, 9, 4, 8, 6]
    assert list(t["parent"]) == [-1, 0, 1, 2, 3, 4, 5, 1, 7, 8, 3, 10]
    assert list(t["depth"]) == [0, 1, 2, 3, 4, 5, 6, 2, 3, 4, 4, 5]
    O.tree_prep(t["parent"])                                       # a valid tree: parent[i] < i
    # no uncertain position -> a plain chain; a node budget cuts the second pass, then the trunk
    assert list(O.two_pass_tree(step, 0, 6, 0.0, 32, 5)["parent"]) == [-1, 0, 1, 2, 3, 4, 5]
    assert len(O.two_pass_tree(step, 0, 6, 0.4, 9, 5)["tokens"]) == 9
    assert list(O.two_pass_tree(step, 0, 6, 0.4, 4, 5)["tokens"]) == [0, 1, 2, 3]
    # a branch that never meets the trunk stops at max_branch tokens
    t2 = O.two_pass_tree(step, 0, max_len=6, threshold=0.4, n_nodes=32, max_branch=2)
    assert list(t2["tokens"]) == [0, 1, 2, 3, 4, 5, 6, 7, 9, 8, 6]
    # a later branch also stops where it meets an earlier one: second pass at depth 2 (7 9 4), then at depth 3 the
    # alternative 9 is what the first branch holds at that very depth
    def step2(path):
        path = list(path)
        if path == [0] + trunk[:len(path) - 1]:
            j = len(path)
            unsure = {2: 7, 3: 9}
            return _onehot(trunk[j - 1], second=unsure.get(j, 11), p1=0.3 if j in unsure else 0.9)
        return _onehot({(0, 1, 7): 9, (0, 1, 7, 9): 4}[tuple(path)], second=0)
    t3 = O.two_pass_tree(step2, 0, max_len=6, threshold=0.4, n_nodes=32, max_branch=5)
    assert list(t3["tokens"]) == [0, 1, 2, 3, 4, 5, 6, 7, 9, 4, 9] and list(t3["parent"])[-1] == 2


def test_recycled_draft_on_scripted_sequences():
    """Old draft 1 2 3 4 5 6 under the old root; the target accepted 1 2 and emitted 9 instead of 3."""
    seq1 = [1, 2, 3, 4, 5, 6]

    def make_step(after_bonus, ext):
        """Sequence 2 continues `after_bonus` (a list) after the bonus token; sequence 1 is extended by `ext`."""
        def step(tokens, parent):
            tokens, parent = list(tokens), list(parent)
            n = len(tokens)
            assert tokens[0] == 2 and parent[0] == -1 and all(0 <= parent[i] < i for i in range(1, n))
            start2 = [i for i in range(1, n) if parent[i] == 0][1]           # second child of node 0 = the bonus token
            assert tokens[start2] == 9 and tokens[1:4 + 1] == [3, 4, 5, 6]
            len1, len2 = start2 - 1, n - start2
            lg = np.full((n, V), -30.0)
            lg[start2 - 1, ext[len1 - 4]] = 0.0                               # tip of sequence 1
            lg[n - 1, after_bonus[len2 - 1]] = 0.0                            # tip of sequence 2
            return lg
        return step

    # substitution: after 9 the draft says 4 (what sequence 1 holds at the same depth 4): reuse 5 6 and the extension
    r = O.recycled_draft(make_step([4, 0, 0], [7, 8, 0]), 2, seq1, 2, 9, max_len=24, max_regen=6)
    assert r["regenerated"] == [4] and r["merged_at"] == 4 and r["draft"] == [4, 5, 6, 7] and r["steps"] == 1
    # insertion: the target inserted 9 before 3, so the first regenerated token is 3 itself (one depth earlier)
    r = O.recycled_draft(make_step([3, 0, 0], [7, 8, 0]), 2, seq1, 2, 9, max_len=24, max_regen=6)
    assert r["merged_at"] == 3 and r["draft"] == [3, 4, 5, 6, 7]
    # deletion: 9 replaced both 3 and 4, the regenerated token 5 sits one depth later in sequence 1
    r = O.recycled_draft(make_step([5, 0, 0], [7, 8, 0]), 2, seq1, 2, 9, max_len=24, max_regen=6)
    assert r["merged_at"] == 5 and r["draft"] == [5, 6, 7]
    # a match only at the second step: two regenerated tokens, then the reused tail
    r = O.recycled_draft(make_step([10, 5, 0], [7, 8, 0]), 2, seq1, 2, 9, max_len=24, max_regen=6)
    assert r["regenerated"] == [10, 5] and r["merged_at"] == 5 and r["draft"] == [10, 5, 6, 7, 8] and r["steps"] == 2
    # no match within the budget: the regenerated tokens alone; the draft length cap applies
    r = O.recycled_draft(make_step([10, 11, 10, 11], [7, 8, 0, 0]), 2, seq1, 2, 9, max_len=24, max_regen=3)
    assert r["merged_at"] is None and r["draft"] == [10, 11, 10] and r["steps"] == 3
    r = O.recycled_draft(make_step([4, 0, 0], [7, 8, 0]), 2, seq1, 2, 9, max_len=2, max_regen=6)
    assert r["draft"] == [4, 5]
    # everything accepted: nothing to recycle
    assert O.recycled_draft(None, 6, seq1, 6, 9, 24, 6)["draft"] == []


def test_strategies_on_a_real_decoder_are_self_consistent():
    """With the fp64 decoder as the draft model: the trunk of the two-pass tree is its greedy continuation, the
    branches start with its second-ranked tokens, and a recycled draft after a planted substitution returns to the
    greedy continuation (the draft model regenerates its own next tokens, which the old draft already holds)."""
    cfg = gen.get_config("micro")
    W = oracle_weights(cfg, 4)
    cache, x, audio, prompt = filled_cache(cfg, W, 9, 4, seed=4)
    root = int(prompt[-1])
    greedy = O.greedy_continuation(cfg, W, cache, root, 10)

    def step(path):
        c = cache.copy()
        return O.prefill(cfg, W, c, O.embed(W, list(path)), want_logits=True)[-1]

    t = O.two_pass_tree(step, root, max_len=8, threshold=2.0, n_nodes=20, max_branch=3)   # every position is "uncertain"
    assert list(t["tokens"][1:9]) == greedy[:8] and len(t["tokens"]) == 20
    for j, second in t["marks"][:3]:
        ids, _ = O.top2_probs(step([root] + greedy[:j - 1])[None, :])
        assert ids[0, 1] == second and ids[0, 0] == greedy[j - 1]
    depth, _ = O.tree_prep(t["parent"])
    assert np.array_equal(depth, t["depth"])
    assert O.adaptive_sequence(step, root, 8, 0.0) == greedy[:8]

    # recycling: the old draft is the greedy continuation with position 3 corrupted; the "target" (same model)
    # accepts two tokens and emits the true third one
    seq1 = list(greedy[:8])
    seq1[2] = (seq1[2] + 1) % cfg.vocab
    c2 = cache.copy()
    O.prefill(cfg, W, c2, O.embed(W, [root, greedy[0]]))             # context up to (not including) the last accepted token

    def tree_step(tokens, parent):
        return O.verify_tree(cfg, W, c2, tokens, parent)["logits"]

    r = O.recycled_draft(tree_step, greedy[1], seq1, 2, greedy[2], max_len=24, max_regen=6)
    assert r["regenerated"][0] == greedy[3]                          # sequence 2 regenerates the true continuation
    assert r["merged_at"] == 4 and r["steps"] == 1                   # ... which the old draft holds at the same depth
    assert r["draft"][:5] == greedy[3:8]
