"""The drafting strategies of Section IV run on the draft model through the library (tree-verification calls with the
top-2 epilogue), against the oracle's restatement of the same strategies on the fp64 decoder.

The strategies take discrete decisions from the draft model's probabilities, so the comparison is exact wherever the
oracle's decisions are clear: every arg-max it consulted decided by more than 1e-2 in the logits, and no top-1
probability within 1e-3 of the threshold.  The seeded cases below are chosen to be clear (asserted on the oracle side).
"""
import numpy as np
import pytest
import torch

import gen
from oracle import specasr_oracle as O

pytestmark = pytest.mark.gpu

GAP = 1e-2


class _Recorder:
    """Wraps the oracle's draft step so that the test knows how narrow the narrowest decision was."""

    def __init__(self, cfg, W, cache, threshold):
        self.cfg, self.W, self.cache, self.threshold = cfg, W, cache, threshold
        self.min_gap, self.min_thr = np.inf, np.inf

    def _note(self, logits):
        logits = np.atleast_2d(logits)
        self.min_gap = min(self.min_gap, float(O.top2_gap(logits).min()))
        _, probs = O.top2_probs(logits)
        self.min_thr = min(self.min_thr, float(np.abs(probs[:, 0] - self.threshold).min()))

    def chain(self, path):
        c = self.cache.copy()
        lg = O.prefill(self.cfg, self.W, c, O.embed(self.W, list(path)), want_logits=True)[-1]
        self._note(lg)
        return lg

    def tree(self, tokens, parent):
        lg = O.verify_tree(self.cfg, self.W, self.cache, tokens, parent)["logits"]
        self._note(lg[[-1, int(np.flatnonzero(np.asarray(parent) == 0)[1]) - 1]])      # the two tips that are read
        return lg


def _setup(cfg_name, seed, n_audio, n_prompt, extra_tokens=()):
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    cfg = gen.get_config(cfg_name)
    store = gen.WeightStore(cfg, seed)
    W = O.Weights(store, cache_layers=True)
    model = DeviceModel(cfg, store)
    kv = DeviceKV(model, max_tokens=256, max_nodes=64)
    audio = gen.audio_prefix(n_audio, cfg.d_model, seed)
    prompt = gen.prompt_tokens(n_prompt, cfg.vocab, seed)
    ctx = [int(t) for t in prompt[:-1]] + [int(t) for t in extra_tokens]
    cache = O.KVCache(cfg)
    O.prefill(cfg, W, cache, np.concatenate([audio.astype(np.float64), O.embed(W, ctx)], 0))
    kv.prefill_embeds(torch.from_numpy(audio).cuda())
    kv.prefill_tokens(torch.tensor(ctx, dtype=torch.int32, device="cuda"))
    return cfg, W, cache, model, kv, int(prompt[-1])


def test_top2_epilogue_matches_the_oracle_on_a_tree():
    """specasr_verify_tree_top2 against top2_probs of the oracle's logits, node by node, and against the
    stand-alone specasr_top2_probs kernel fed the library's own logits."""
    from paper_2507_18181_b200 import binding as B
    cfg, W, cache, model, kv, root = _setup("small", 3, 60, 5)
    parent = gen.sparse_tree(40, seed=3)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=3, root_token=root)
    want = O.verify_tree(cfg, W, cache, tokens, parent)
    ids_w, probs_w = O.top2_probs(want["logits"])
    d_t, d_p = torch.from_numpy(tokens).cuda(), torch.from_numpy(parent).cuda()
    kv.verify_top2(d_t, d_p)
    torch.cuda.synchronize()
    assert kv.status() == 0
    ids = kv.out_top2_ids[:40].cpu().numpy()
    probs = kv.out_top2_probs[:40].cpu().numpy()
    srt = np.sort(want["logits"], -1)
    clear = (srt[:, -1] - srt[:, -2] > GAP) & (srt[:, -2] - srt[:, -3] > GAP)     # both ranks decided clearly
    assert clear.sum() >= 20
    assert np.array_equal(ids[clear], ids_w[clear])
    assert np.array_equal(ids[:, 0], kv.out_argmax[:40].cpu().numpy())             # rank 1 is the call's arg-max
    assert np.allclose(probs[clear], probs_w[clear], rtol=2e-2, atol=1e-7)         # logits agree to 2e-2 -> probabilities to ~2 %
    assert int(kv.out_accept.item()) == O.accept(tokens, parent, ids[:, 0])["accept_len"]
    # the same numbers from a materialised logits matrix
    logits = torch.empty(40, cfg.vocab, dtype=torch.float32, device="cuda")
    kv.verify(d_t, d_p, logits)
    ids2 = torch.empty(40, 2, dtype=torch.int32, device="cuda")
    probs2 = torch.empty(40, 2, dtype=torch.float32, device="cuda")
    B.specasr_top2_probs(logits.data_ptr(), 40, cfg.vocab, ids2.data_ptr(), probs2.data_ptr())
    torch.cuda.synchronize()
    assert np.array_equal(ids2.cpu().numpy(), ids)
    assert np.allclose(probs2.cpu().numpy(), probs, rtol=1e-4, atol=1e-9)
    # a refused tree reports -1 / 0
    bad = torch.tensor([-1, 0, 5, 1], dtype=torch.int32, device="cuda")
    kv.verify_top2(d_t[:4].clone(), bad)
    torch.cuda.synchronize()
    assert kv.status() != 0 and bool((kv.out_top2_ids[:4] == -1).all())


@pytest.mark.parametrize("cfg_name,seed", [("tiny", 27), ("small", 5)])
def test_adaptive_and_two_pass_drafts_match_the_oracle(cfg_name, seed):
    from paper_2507_18181_b200.loop import DraftStrategies
    cfg, W, cache, model, kv, root = _setup(cfg_name, seed, 40, 4)
    ds = DraftStrategies(kv)
    # random weights give near-uniform next-token distributions (top-1 probability ~ 1 / vocab): thresholds are
    # placed inside that range so that some trunk positions count as certain and some as uncertain
    rec = _Recorder(cfg, W, cache, 0.0)
    probs = []
    path = [root]
    for _ in range(6):
        ids, pr = O.top2_probs(rec.chain(path)[None, :])
        probs.append(float(pr[0, 0]))
        path.append(int(ids[0, 0]))
    thr = float(np.sort(probs)[3] + np.sort(probs)[4]) / 2          # two of the six positions lie above it
    for max_len, n_nodes, max_branch in ((6, 14, 3), (5, 8, 2)):
        rec = _Recorder(cfg, W, cache, thr)
        want = O.two_pass_tree(rec.chain, root, max_len, thr, n_nodes, max_branch)
        assert rec.min_gap > GAP and rec.min_thr > 1e-5, (rec.min_gap, rec.min_thr)   # the seeded case is a clear one
        got = ds.two_pass_tree(root, max_len, thr, n_nodes, max_branch)
        assert list(got["tokens"]) == list(want["tokens"]) and list(got["parent"]) == list(want["parent"])
        assert got["marks"] == want["marks"] and len(want["marks"]) >= 1
    rec = _Recorder(cfg, W, cache, thr)
    want = O.adaptive_sequence(rec.chain, root, 6, thr)
    assert rec.min_gap > GAP
    assert ds.adaptive_sequence(root, 6, thr) == want and 1 <= len(want) < 6         # truncated inside the trunk
    assert kv.length() == cache.length                                                # drafting never moved the cache


def test_recycled_draft_matches_the_oracle():
    """The draft model is the decoder itself; the old draft is its greedy continuation with one substitution, one
    insertion or one deletion planted, so that the regeneration meets it again at offset 0, -1 or +1."""
    from paper_2507_18181_b200.loop import DraftStrategies
    cfg, W, cache0, model, kv0, root = _setup("small", 4, 40, 4)
    greedy = O.greedy_continuation(cfg, W, cache0, root, 12)
    # context up to, not including, the last accepted token greedy[1]
    cfg, W, cache, model, kv, _ = _setup("small", 4, 40, 4, extra_tokens=[root, greedy[0]])
    ds = DraftStrategies(kv)
    other = (greedy[2] + 7) % cfg.vocab
    cases = {
        "substitution": greedy[:2] + [other] + greedy[3:9],                 # position 3 is wrong, the rest still lines up
        "insertion": greedy[:2] + [other] + greedy[2:8],                    # an extra token: everything after it is one late
        "deletion": greedy[:2] + greedy[3:9],                               # a token is missing: everything is one early
    }
    for name, seq1 in cases.items():
        a = 2
        bonus = greedy[2]                                                   # what the target emits after two accepted tokens
        if name == "deletion":
            assert seq1[2] != bonus
        rec = _Recorder(cfg, W, cache, 0.0)
        want = O.recycled_draft(rec.tree, greedy[1], seq1, a, bonus, max_len=24, max_regen=6)
        assert rec.min_gap > GAP, (name, rec.min_gap)
        got = ds.recycled_draft(greedy[1], seq1, a, bonus, max_len=24, max_regen=6)
        assert got["draft"] == want["draft"] and got["merged_at"] == want["merged_at"] and got["steps"] == want["steps"], name
        assert want["merged_at"] is not None, name                          # the planted edit is found again
        assert want["draft"][:4] == greedy[3:7], name                       # and the recycled draft is the true continuation
    assert kv.length() == cache.length


@pytest.mark.parametrize("strategy,same_model", [("two_pass", True), ("two_pass", False), ("recycle", True), ("recycle", False)])
def test_whole_method_is_lossless(strategy, same_model):
    """Draft with the strategies of Section IV, verify with the target, commit: the transcript is the target's own
    greedy transcript (Section II-B), whatever the draft model proposes.  With the target's own weights as the draft
    model whole trunks are accepted; with another model hardly anything is, and recycling has rejected tails to work on."""
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    from paper_2507_18181_b200.loop import SpeculativeBatchLoop
    cfg = gen.get_config("tiny")
    store = gen.WeightStore(cfg, 0)
    W = O.Weights(store, cache_layers=True)
    target = DeviceModel(cfg, store)
    draft = target if same_model else DeviceModel(cfg, gen.WeightStore(cfg, 5))
    n_tokens, max_len = 16, 6
    kvs, dkvs, roots, truth = [], [], [], []
    for b, n_audio in enumerate((33, 58)):
        prompt = gen.prompt_tokens(4, cfg.vocab, 0, utterance=b)
        audio = gen.audio_prefix(n_audio, cfg.d_model, 0, utterance=b)
        cache = O.KVCache(cfg)
        O.prefill(cfg, W, cache, np.concatenate([audio.astype(np.float64), O.embed(W, prompt[:-1])], 0))
        for model, lst in ((target, kvs), (draft, dkvs)):
            kv = DeviceKV(model, max_tokens=256, max_nodes=64)
            kv.prefill_embeds(torch.from_numpy(audio).cuda())
            kv.prefill_tokens(torch.from_numpy(prompt[:-1].copy()).cuda())
            lst.append(kv)
        roots.append(int(prompt[-1]))
        truth.append(O.greedy_continuation(cfg, W, cache, roots[-1], n_tokens + max_len + 2))
    loop = SpeculativeBatchLoop(kvs, dkvs)
    out = loop.decode_with_strategies(roots, n_tokens, strategy=strategy, threshold=2.0 if strategy == "two_pass" else 0.0,
                                      max_len=max_len, n_nodes=20, max_branch=3, max_regen=3)
    for b in range(2):
        assert out[b] == truth[b][:n_tokens]
        assert kvs[b].status() == 0 and dkvs[b].status() == 0 and kvs[b].length() == loop.target_len[b]
    assert loop.draft_forwards > 0
    if same_model:
        assert loop.rounds <= -(-n_tokens // (max_len + 1)) + 1          # whole trunks accepted
    else:
        assert loop.rounds >= n_tokens // 2
