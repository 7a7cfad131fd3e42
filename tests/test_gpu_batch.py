"""Batched verification through the C ABI: several utterances with caches of different lengths and trees of
different shapes go through one specasr_verify_tree_batch call and must come out as the oracle computes each
of them on its own.  Bars as in test_gpu_parity.py (integer results exact where the oracle's top-2 gap is
clear, otherwise self-consistent and within tolerance of the maximum)."""
import numpy as np
import pytest
import torch

import gen
from oracle import specasr_oracle as O

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2
GAP = 1e-2


def _tree(kind, seed):
    if kind == "binary15":
        return gen.complete_binary_tree(15)
    if kind.startswith("sparse"):
        return gen.sparse_tree(int(kind[6:]), seed=seed)
    return gen.chain_tree(int(kind[5:]))


class _Utterance:
    """One utterance on both sides: oracle cache and device cache filled with the same prefix."""

    def __init__(self, cfg, W, model, index, n_audio, n_prompt, max_nodes):
        from paper_2507_18181_b200.runtime import DeviceKV
        self.cfg, self.W = cfg, W
        audio = gen.audio_prefix(n_audio, cfg.d_model, 0, utterance=index)
        prompt = gen.prompt_tokens(n_prompt, cfg.vocab, 0, utterance=index)
        self.cache = O.KVCache(cfg)
        O.prefill(cfg, W, self.cache, np.concatenate([audio.astype(np.float64), O.embed(W, prompt[:-1])], 0))
        self.kv = DeviceKV(model, max_tokens=512, max_nodes=max_nodes, shuffle_pages_seed=17 + index)
        self.kv.prefill_embeds(torch.from_numpy(audio).cuda())
        if n_prompt > 1:
            self.kv.prefill_tokens(torch.from_numpy(prompt[:-1].copy()).cuda())
        self.root = int(prompt[-1])

    def draft(self, kind, seed):
        parent = _tree(kind, seed)
        greedy = O.greedy_continuation(self.cfg, self.W, self.cache, self.root, len(gen.main_path(parent)) - 1)
        tokens = gen.fill_tree_tokens(parent, self.cfg.vocab, seed=seed, root_token=self.root, main_tokens=greedy,
                                      corrupt_p=0.2)
        return np.asarray(tokens, np.int32), np.asarray(parent, np.int32)


def _run_batch(bv, trees, vocab=None):
    offsets = np.concatenate([[0], np.cumsum([len(t) for t, _ in trees])]).astype(int)
    tokens = torch.from_numpy(np.concatenate([t for t, _ in trees])).cuda()
    parent = torch.from_numpy(np.concatenate([p for _, p in trees])).cuda()
    logits = torch.empty(int(offsets[-1]), vocab, dtype=torch.float32, device="cuda") if vocab else None
    bv.verify(tokens, parent, offsets, logits)
    torch.cuda.synchronize()
    out = []
    for b in range(len(trees)):
        lo, hi = offsets[b], offsets[b + 1]
        out.append({"argmax": bv.out_argmax[lo:hi].cpu().numpy(), "path": bv.out_path[lo:hi].cpu().numpy(),
                    "accept_len": int(bv.out_accept[b].item()), "bonus": int(bv.out_bonus[b].item())})
        if vocab:
            out[-1]["logits"] = logits[lo:hi].cpu().numpy().astype(np.float64)
    return out


def _check_utterance(got, want, tokens, parent):
    n = len(tokens)
    if "logits" in got:
        assert np.abs(got["logits"] - want["logits"]).max() < LOGIT_TOL
    clear = want["gap"] > GAP
    assert np.array_equal(got["argmax"][clear], want["argmax"][clear])
    top = want["logits"].max(-1)
    assert np.all(top - want["logits"][np.arange(n), got["argmax"]] <= LOGIT_TOL)
    mine = O.accept(tokens, parent, got["argmax"])
    a = got["accept_len"]
    assert a == mine["accept_len"] and got["bonus"] == mine["bonus"]
    assert list(got["path"][:a + 1]) == list(mine["path"]) and np.all(got["path"][a + 1:] == -1)
    if want["decisive"]:
        assert a == want["accept_len"] and list(got["path"][:a + 1]) == list(want["path"])
        assert got["bonus"] == want["bonus"]


@pytest.mark.parametrize("cfg_name,shapes", [
    ("tiny", [(64, 8, "binary15"), (150, 3, "sparse24"), (21, 5, "chain8")]),
    ("small", [(150, 9, "sparse40"), (37, 3, "chain8"), (300, 4, "sparse64"), (90, 2, "chain4")]),
])
def test_batch_matches_oracle_per_utterance_over_two_rounds(cfg_name, shapes):
    from paper_2507_18181_b200.runtime import DeviceModel, BatchVerifier
    cfg = gen.get_config(cfg_name)
    store = gen.WeightStore(cfg, 0)
    model = DeviceModel(cfg, store, gemm_path=0)
    W = O.Weights(store, cache_layers=True)
    utts = [_Utterance(cfg, W, model, i, na, npmt, 256 if i == 0 else 64) for i, (na, npmt, _) in enumerate(shapes)]
    bv = BatchVerifier([u.kv for u in utts])
    for rnd in range(2):
        trees = [u.draft(kind, seed=rnd) for u, (_, _, kind) in zip(utts, shapes)]
        wants = [O.verify_tree(cfg, W, u.cache, t, p) for u, (t, p) in zip(utts, trees)]
        gots = _run_batch(bv, trees, cfg.vocab if rnd == 0 else None)
        for u, got, want, (t, p) in zip(utts, gots, wants, trees):
            assert u.kv.status() == 0
            _check_utterance(got, want, t, p)
        lens = [u.cache.length for u in utts]
        bv.commit()
        for u, got, want, L in zip(utts, gots, wants, lens):
            a = got["accept_len"]
            assert u.kv.length() == L + a + 1
            # the oracle's cache follows the path the device took (identical to its own when decisive)
            O.commit(u.cache, dict(want, path=np.asarray(got["path"][:a + 1]), accept_len=a))
            k, v = u.kv.read_kv(cfg.n_layers - 1, L + a + 1)
            assert np.abs(k - u.cache.K[-1]).max() < 2e-3 and np.abs(v - u.cache.V[-1]).max() < 2e-3
            u.root = got["bonus"]


def test_batch_of_one_equals_plain_call_and_bad_tree_fails_alone():
    from paper_2507_18181_b200.runtime import DeviceModel, BatchVerifier
    from paper_2507_18181_b200 import binding as B
    cfg = gen.get_config("tiny")
    store = gen.WeightStore(cfg, 0)
    model = DeviceModel(cfg, store, gemm_path=0)
    W = O.Weights(store, cache_layers=True)
    utts = [_Utterance(cfg, W, model, i, na, 4, 128 if i == 0 else 64) for i, na in enumerate((40, 70, 55))]
    trees = [u.draft("sparse24", seed=3) for u in utts]

    # a batch of one is the plain call
    solo = _run_batch(BatchVerifier([utts[0].kv]), trees[:1])[0]
    t, p = trees[0]
    utts[0].kv.verify(torch.from_numpy(t).cuda(), torch.from_numpy(p).cuda())
    torch.cuda.synchronize()
    assert np.array_equal(solo["argmax"], utts[0].kv.out_argmax[:len(t)].cpu().numpy())
    assert solo["accept_len"] == int(utts[0].kv.out_accept.item())
    assert np.array_equal(solo["path"], utts[0].kv.out_path[:len(t)].cpu().numpy())

    # a malformed tree (a parent that does not precede its child) fails its own utterance only
    bad_t, bad_p = trees[1][0].copy(), trees[1][1].copy()
    bad_p[5] = 9
    bv = BatchVerifier([u.kv for u in utts])
    gots = _run_batch(bv, [trees[0], (bad_t, bad_p), trees[2]])
    assert gots[1]["accept_len"] == -1 and np.all(gots[1]["path"] == -1)
    assert utts[1].kv.status() == B.SPECASR_ERR_INVALID_TREE
    for i in (0, 2):
        assert utts[i].kv.status() == 0
        _check_utterance(gots[i], O.verify_tree(cfg, W, utts[i].cache, *trees[i]), *trees[i])
    # committing the failed utterance is a no-op on the device; the others advance
    lens = [u.kv.length() for u in utts]
    bv.commit()
    assert utts[1].kv.length() == lens[1]
    assert utts[0].kv.length() == lens[0] + gots[0]["accept_len"] + 1
    # the failed utterance recovers with a well-formed tree
    gots = _run_batch(bv, trees)
    assert utts[1].kv.status() == 0
    _check_utterance(gots[1], O.verify_tree(cfg, W, utts[1].cache, *trees[1]), *trees[1])


def test_batch_host_side_errors_enqueue_nothing():
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    from paper_2507_18181_b200 import binding as B
    cfg = gen.get_config("tiny")
    model = DeviceModel(cfg, gen.WeightStore(cfg, 0), gemm_path=0)
    kvs = [DeviceKV(model, max_tokens=128, max_nodes=16) for _ in range(2)]
    buf = torch.zeros(64, dtype=torch.int32, device="cuda")
    before = [kv.launches() for kv in kvs]

    def call(handles, offsets):
        B.specasr_verify_tree_batch(model.handle, handles, buf.data_ptr(), buf.data_ptr(), offsets, buf.data_ptr(),
                                    buf.data_ptr(), buf.data_ptr(), 0, 0, 0)

    for handles, offsets in [
        ([kvs[0].handle, kvs[0].handle], [0, 4, 8]),      # the same handle twice
        ([kvs[0].handle, kvs[1].handle], [0, 9, 18]),     # more rows than the first workspace holds
        ([kvs[0].handle, kvs[1].handle], [0, 4, 4]),      # an utterance without nodes
        ([kvs[0].handle, kvs[1].handle], [1, 4, 8]),      # offsets must start at 0
    ]:
        with pytest.raises(B.SpecasrError) as e:
            call(handles, offsets)
        assert e.value.status == B.SPECASR_ERR_INVALID_ARG
    assert [kv.launches() for kv in kvs] == before
    # a cache that cannot take the tree
    kvs[1].prefill_tokens(torch.zeros(120, dtype=torch.int32, device="cuda"))
    with pytest.raises(B.SpecasrError) as e:
        call([kvs[0].handle, kvs[1].handle], [0, 4, 16])
    assert e.value.status == B.SPECASR_ERR_KV_CAPACITY


def test_largest_batch_of_single_node_trees_equals_plain_calls():
    """32 utterances (the most one call takes) of one node each: every row is an ordinary decoding step."""
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV, BatchVerifier
    from paper_2507_18181_b200 import binding as B
    cfg = gen.get_config("tiny")
    model = DeviceModel(cfg, gen.WeightStore(cfg, 0), gemm_path=0)
    nb = B.SPECASR_MAX_BATCH
    kvs, toks = [], []
    for b in range(nb):
        kv = DeviceKV(model, max_tokens=64, max_nodes=32)
        kv.prefill_tokens(torch.from_numpy(gen.prompt_tokens(3 + b % 7, cfg.vocab, 0, utterance=b)).cuda())
        kvs.append(kv)
        toks.append(int(gen.prompt_tokens(1, cfg.vocab, 9, utterance=b)[0]))
    bv = BatchVerifier(kvs)
    d_toks = torch.tensor(toks, dtype=torch.int32, device="cuda")
    minus = torch.full((nb,), -1, dtype=torch.int32, device="cuda")
    bv.verify(d_toks, minus, list(range(nb + 1)))
    torch.cuda.synchronize()
    got = bv.out_argmax[:nb].cpu().numpy()
    assert np.all(bv.out_accept.cpu().numpy() == 0) and np.all(bv.out_path[:nb].cpu().numpy() == 0)
    assert np.array_equal(bv.out_bonus.cpu().numpy(), got)
    for b in range(nb):
        kvs[b].verify(d_toks[b:b + 1], minus[:1])
        torch.cuda.synchronize()
        assert int(kvs[b].out_argmax[0].item()) == int(got[b])
    with pytest.raises(B.SpecasrError) as e:          # one utterance more than a call takes
        B.specasr_verify_tree_batch(model.handle, [kv.handle for kv in kvs] + [kvs[0].handle], d_toks.data_ptr(),
                                    minus.data_ptr(), list(range(nb + 2)), bv.out_argmax.data_ptr(),
                                    bv.out_accept.data_ptr(), bv.out_path.data_ptr(), 0, 0, 0)
    assert e.value.status == B.SPECASR_ERR_INVALID_ARG
