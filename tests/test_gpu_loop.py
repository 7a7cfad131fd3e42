"""The batched draft-then-verify loop on the GPU: transcripts must equal the oracle's autoregressive greedy
transcripts token for token (losslessness, Section II-B), with a draft model of the 0.5B shape stepped through
the same kernels.  Also parity of that draft shape (14 query heads on 2 KV heads) against the oracle."""
import numpy as np
import pytest
import torch

import gen
from oracle import specasr_oracle as O

pytestmark = pytest.mark.gpu


def _fill(cfg, model, kv_cls, index, n_audio, prompt, W=None):
    audio = gen.audio_prefix(n_audio, cfg.d_model, 0, utterance=index)
    kv = kv_cls(model, max_tokens=256, max_nodes=64)
    kv.prefill_embeds(torch.from_numpy(audio).cuda())
    kv.prefill_tokens(torch.from_numpy(prompt[:-1].copy()).cuda())
    cache = None
    if W is not None:
        cache = O.KVCache(cfg)
        O.prefill(cfg, W, cache, np.concatenate([audio.astype(np.float64), O.embed(W, prompt[:-1])], 0))
    return kv, cache


@pytest.mark.parametrize("with_draft", [False, True])
def test_batched_loop_reproduces_greedy_transcripts(with_draft):
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    from paper_2507_18181_b200.loop import SpeculativeBatchLoop
    cfg = gen.get_config("tiny")
    store = gen.WeightStore(cfg, 0)
    W = O.Weights(store, cache_layers=True)
    target = DeviceModel(cfg, store, gemm_path=0)
    dcfg = gen.get_config("0.5b", n_layers=2)
    draft = DeviceModel(dcfg, gen.WeightStore(dcfg, 1), gemm_path=0) if with_draft else None
    n_tokens, k_max = 20, 6
    prefixes = (40, 70, 25)
    kvs, dkvs, roots, truth = [], [], [], []
    for b, n_audio in enumerate(prefixes):
        prompt = gen.prompt_tokens(4, cfg.vocab, 0, utterance=b)
        kv, cache = _fill(cfg, target, DeviceKV, b, n_audio, prompt, W)
        kvs.append(kv)
        roots.append(int(prompt[-1]))
        truth.append(O.greedy_continuation(cfg, W, cache, roots[-1], n_tokens + k_max + 2))
        if with_draft:
            dkvs.append(_fill(dcfg, draft, DeviceKV, b, n_audio, prompt)[0])
    proposer = gen.CorruptedGreedyProposer(truth, roots, cfg.vocab, seed=3, n_nodes=12, k_min=2, k_max=k_max,
                                           corrupt_p=0.25)
    loop = SpeculativeBatchLoop(kvs, dkvs if with_draft else None)
    out = loop.decode(roots, n_tokens, proposer)
    for b in range(len(prefixes)):
        assert out[b] == truth[b][:n_tokens]
        assert kvs[b].status() == 0 and kvs[b].length() == loop.target_len[b]
        assert loop.target_len[b] >= prefixes[b] + 3 + n_tokens
    assert loop.rounds < n_tokens            # speculation accepted something
    if with_draft:
        assert loop.draft_steps > 0
        for b in range(len(prefixes)):
            assert dkvs[b].status() == 0


def test_draft_shape_matches_oracle():
    """0.5B shape cut to two layers: 14 query heads share 2 KV heads (7 per group, so an attention row tile holds
    18 nodes), d_model 896, FFN 4864."""
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    cfg = gen.get_config("0.5b", n_layers=2)
    store = gen.WeightStore(cfg, 2)
    W = O.Weights(store, cache_layers=True)
    model = DeviceModel(cfg, store, gemm_path=0)
    prompt = gen.prompt_tokens(5, cfg.vocab, 2)
    kv, cache = _fill(cfg, model, DeviceKV, 0, 150, prompt, W)
    root = int(prompt[-1])
    for parent in (gen.chain_tree(0), gen.sparse_tree(40, seed=2)):
        greedy = O.greedy_continuation(cfg, W, cache, root, len(gen.main_path(parent)))
        tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=2, root_token=root, main_tokens=greedy, corrupt_p=0.2)
        want = O.verify_tree(cfg, W, cache, tokens, parent)
        n = len(tokens)
        logits = torch.empty(n, cfg.vocab, dtype=torch.float32, device="cuda")
        kv.verify(torch.from_numpy(tokens).cuda(), torch.from_numpy(parent).cuda(), logits)
        torch.cuda.synchronize()
        assert kv.status() == 0
        err = np.abs(logits.cpu().numpy().astype(np.float64) - want["logits"]).max()
        assert err < 2e-2, err
        clear = want["gap"] > 1e-2
        assert np.array_equal(kv.out_argmax[:n].cpu().numpy()[clear], want["argmax"][clear])
        if want["decisive"]:
            assert int(kv.out_accept.item()) == want["accept_len"]


def test_top2_probs_matches_oracle():
    from paper_2507_18181_b200 import binding as B
    rng = np.random.default_rng(11)
    for n, vocab, scale in ((1, 1, 1.0), (3, 2, 1.0), (5, 257, 3.0), (64, 32000, 1.5), (2, 4099, 30.0)):
        logits = (rng.standard_normal((n, vocab)) * scale).astype(np.float32)
        if vocab > 300:
            logits[0, 17] = logits[0, 230] = logits[0].max() + 1.0      # a tie at the top: lower id first
        d = torch.from_numpy(logits).cuda()
        ids = torch.empty(n, 2, dtype=torch.int32, device="cuda")
        probs = torch.empty(n, 2, dtype=torch.float32, device="cuda")
        B.specasr_top2_probs(d.data_ptr(), n, vocab, ids.data_ptr(), probs.data_ptr())
        torch.cuda.synchronize()
        want_ids, want_probs = O.top2_probs(logits)
        assert np.array_equal(ids.cpu().numpy(), want_ids)                       # decided on the same fp32 values
        assert np.allclose(probs.cpu().numpy(), want_probs, rtol=2e-5, atol=1e-9)
    with pytest.raises(B.SpecasrError):
        B.specasr_top2_probs(0, 1, 8, ids.data_ptr(), probs.data_ptr())


@pytest.mark.parametrize("same_model,threshold,max_len", [(True, 0.0, 6), (True, 2.0, 6), (False, 0.0, 4)])
def test_loop_with_the_draft_models_own_proposals(same_model, threshold, max_len):
    """Drafts come from the draft model (top-1 extends the trunk, a low-probability top-1 ends it and adds the
    second-ranked token as a sibling).  With the target's own weights as the draft every trunk token is the
    target's greedy token, so rounds accept whole trunks; with another model nearly nothing is accepted.  Either
    way the transcript is the oracle's greedy one."""
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    from paper_2507_18181_b200.loop import SpeculativeBatchLoop
    cfg = gen.get_config("tiny")
    store = gen.WeightStore(cfg, 0)
    W = O.Weights(store, cache_layers=True)
    target = DeviceModel(cfg, store, gemm_path=0)
    draft = target if same_model else DeviceModel(cfg, gen.WeightStore(cfg, 5), gemm_path=0)
    n_tokens = 18
    prefixes = (33, 58)
    kvs, dkvs, roots, truth = [], [], [], []
    for b, n_audio in enumerate(prefixes):
        prompt = gen.prompt_tokens(4, cfg.vocab, 0, utterance=b)
        kv, cache = _fill(cfg, target, DeviceKV, b, n_audio, prompt, W)
        kvs.append(kv)
        dkvs.append(_fill(cfg, draft, DeviceKV, b, n_audio, prompt)[0])
        roots.append(int(prompt[-1]))
        truth.append(O.greedy_continuation(cfg, W, cache, roots[-1], n_tokens + max_len + 2))
    loop = SpeculativeBatchLoop(kvs, dkvs)
    out = loop.decode_with_draft_model(roots, n_tokens, threshold=threshold, max_len=max_len)
    for b in range(len(prefixes)):
        assert out[b] == truth[b][:n_tokens]
        assert kvs[b].status() == 0 and dkvs[b].status() == 0
        assert kvs[b].length() == loop.target_len[b]
    if same_model and threshold == 0.0:
        assert loop.rounds <= -(-n_tokens // (max_len + 1)) + 1       # whole trunks accepted
    if same_model and threshold == 2.0:
        assert loop.rounds <= n_tokens // 2 + 1                       # one draft token + the bonus per round
    if not same_model:
        assert loop.rounds >= n_tokens - 3
