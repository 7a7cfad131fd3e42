"""Parity against the oracle at the shapes the workloads state, not only at cut-down ones:

  * the 7B-shape, 64-node, KV-1700 verification at all 32 layers (the graded point), where the error has the
    whole depth to grow;
  * the corners of the verify-cost sweep at the 7B head geometry (2-layer cut): a 256-node tree on short and
    long caches, and a chain of 33 drafts on a cache of 4096 positions;
  * the speculative loop (target + draft model, batched) checked by teacher forcing: one causal oracle pass over
    context + emitted transcript must reproduce every emitted token (Section II-B: the output equals
    non-speculative greedy decoding);
  * the same parity with every caller-owned buffer pre-filled with 0xFF bytes, so that a kernel reading memory
    that no kernel wrote cannot pass by finding zeros there.

Bars as in test_gpu_parity.py: logits within 2e-2, integer results exact where the oracle's margin is clear.
"""
import numpy as np
import pytest
import torch

import gen
from oracle import specasr_oracle as O
from test_gpu_parity import LOGIT_TOL, GAP, _check_against_oracle, _verify_gpu

pytestmark = pytest.mark.gpu


def _device_greedy(kv, root, k, L):
    """The target's greedy continuation by single-node rounds of the library itself (input construction only)."""
    out, tok = [], int(root)
    minus = torch.tensor([-1], dtype=torch.int32, device="cuda")
    for _ in range(k):
        kv.verify(torch.tensor([tok], dtype=torch.int32, device="cuda"), minus)
        kv.commit()
        tok = int(kv.out_bonus.item())
        out.append(tok)
    kv.truncate(L)
    return out


def _case(cfg, n_audio, n_text, parent, seed, max_nodes, poison=False, page_size=16, check_rows=True):
    """Fill the context on both sides, verify one tree, compare.  The oracle runs context and tree in one pass
    over the weights (verify_tree_uncached), streaming the layers."""
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    store = gen.WeightStore(cfg, seed)
    model = DeviceModel(cfg, store, page_size=page_size)
    L, n = n_audio + n_text - 1, len(parent)
    kv = DeviceKV(model, max_tokens=L + n + 64, max_nodes=max_nodes, poison=poison, shuffle_pages_seed=seed + 1)
    audio = gen.audio_prefix(n_audio, cfg.d_model, seed)
    text = gen.prompt_tokens(n_text, cfg.vocab, seed)
    kv.prefill_embeds(torch.from_numpy(audio).cuda())
    kv.prefill_tokens(torch.from_numpy(text[:-1].copy()).cuda())
    assert kv.length() == L
    root = int(text[-1])
    k = min(len(gen.main_path(parent)) - 1, 12)
    greedy = _device_greedy(kv, root, k, L)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=seed, root_token=root, main_tokens=greedy, corrupt_p=0.2)
    got = _verify_gpu(cfg, kv, tokens, parent)
    W = O.Weights(store, cache_layers=False)
    x = np.concatenate([audio.astype(np.float64), O.embed(W, text[:-1])], 0)
    want = O.verify_tree_uncached(cfg, W, x, tokens, parent)
    err = _check_against_oracle(got, want, tokens, parent)
    if check_rows:
        for layer in (0, cfg.n_layers - 1):
            kk, vv = kv.read_kv(layer, L + n)
            assert np.abs(kk[:L] - want["prefix_K"][layer]).max() < 2e-3 and np.abs(vv[:L] - want["prefix_V"][layer]).max() < 2e-3
            assert np.abs(kk[L:] - want["tree_K"][layer]).max() < 2e-3 and np.abs(vv[L:] - want["tree_V"][layer]).max() < 2e-3
    a = got["accept_len"]
    kv.commit()
    assert kv.length() == L + a + 1
    k_after, _ = kv.read_kv(cfg.n_layers - 1, L + a + 1)
    assert np.abs(k_after[L:] - want["tree_K"][-1][got["path"][:a + 1]]).max() < 2e-3
    kv.close()
    model.close()
    return err, got, want


def test_7b_shape_all_32_layers_against_the_oracle():
    """The graded workload at its stated depth: 32 layers, 1500 audio frames + 200 text tokens, 64-node tree of
    12 levels, 16-slot pages, prefill in 64-row chunks -- the launch configuration bench.py times."""
    cfg = gen.get_config("7b")
    parent = gen.sparse_tree(64, seed=1, levels=12)
    err, got, want = _case(cfg, 1500, 201, parent, seed=1, max_nodes=64)
    print(f"7b x 32 layers: max-abs logit error {err:.3e}, accept_len {got['accept_len']}, "
          f"clear nodes {int((want['gap'] > GAP).sum())}/64, decisive {want['decisive']}")
    assert err < LOGIT_TOL
    assert np.isfinite(got["logits"]).all()
    assert int((want["gap"] > GAP).sum()) >= 48          # most of the arg-max comparisons were bit-exact ones


@pytest.mark.parametrize("n_nodes,chain,kv_len", [(256, False, 4096), (256, False, 512), (34, True, 4096)])
def test_7b_head_geometry_at_the_corners_of_the_sweep(n_nodes, chain, kv_len):
    """256-node trees (the folded projection path, two accumulator sets) on a short and a long cache, and a chain of
    33 drafts (padded to 64 rows) on 4096 positions, where the key blocks of the attention no longer fit one wave."""
    cfg = gen.get_config("7b", n_layers=2)
    parent = gen.chain_tree(n_nodes - 1) if chain else gen.sparse_tree(n_nodes, seed=3)
    n_text = 33
    err, got, want = _case(cfg, kv_len + 1 - n_text, n_text, parent, seed=3, max_nodes=n_nodes)
    assert err < LOGIT_TOL


@pytest.mark.parametrize("cfg_name,n_audio,tree,max_nodes,page_size", [
    ("small", 100, "sparse40", 64, 16),
    ("small", 333, "sparse256", 256, 32),
    ("tiny", 50, "chain8", 16, 16),
])
def test_parity_holds_with_poisoned_buffers(cfg_name, n_audio, tree, max_nodes, page_size):
    """Both KV pools and the whole workspace start as 0xFF bytes instead of zeros."""
    cfg = gen.get_config(cfg_name)
    n = int(tree[6:]) if tree.startswith("sparse") else int(tree[5:]) + 1
    parent = gen.sparse_tree(n, seed=5) if tree.startswith("sparse") else gen.chain_tree(n - 1)
    err, got, want = _case(cfg, n_audio, 5, parent, seed=5, max_nodes=max_nodes, poison=True, page_size=page_size)
    assert np.isfinite(got["logits"]).all() and err < LOGIT_TOL


def test_poisoned_batched_call():
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV, BatchVerifier
    cfg = gen.get_config("small")
    store = gen.WeightStore(cfg, 6)
    model = DeviceModel(cfg, store)
    W = O.Weights(store, cache_layers=True)
    kvs, caches, trees = [], [], []
    for b, n_audio in enumerate((70, 133, 41)):
        kv = DeviceKV(model, max_tokens=256, max_nodes=128 if b == 0 else 32, poison=True, shuffle_pages_seed=b)
        audio = gen.audio_prefix(n_audio, cfg.d_model, 6, utterance=b)
        kv.prefill_embeds(torch.from_numpy(audio).cuda())
        cache = O.KVCache(cfg)
        O.prefill(cfg, W, cache, audio.astype(np.float64))
        parent = gen.sparse_tree(20 + 7 * b, seed=b)
        tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=b, root_token=3 + b)
        kvs.append(kv); caches.append(cache); trees.append((tokens, parent))
    bv = BatchVerifier(kvs)
    offs = np.concatenate([[0], np.cumsum([len(t) for t, _ in trees])])
    total = int(offs[-1])
    logits = torch.empty(total, cfg.vocab, dtype=torch.float32, device="cuda")
    bv.verify(torch.from_numpy(np.concatenate([t for t, _ in trees])).cuda(),
              torch.from_numpy(np.concatenate([p for _, p in trees])).cuda(), offs, logits)
    torch.cuda.synchronize()
    lg = logits.cpu().numpy().astype(np.float64)
    for b, (tokens, parent) in enumerate(trees):
        assert kvs[b].status() == 0
        lo, hi = int(offs[b]), int(offs[b + 1])
        got = {"logits": lg[lo:hi], "argmax": bv.out_argmax[lo:hi].cpu().numpy(), "accept_len": int(bv.out_accept[b].item()),
               "path": bv.out_path[lo:hi].cpu().numpy(), "bonus": int(bv.out_bonus[b].item())}
        _check_against_oracle(got, O.verify_tree(cfg, W, caches[b], tokens, parent), tokens, parent)


def test_speculative_loop_transcripts_by_teacher_forcing():
    """Reduced serving workload: 8-layer cuts of the 7B-shape target and the 0.5B-shape draft, three utterances,
    40 tokens each, 32-node trees verified in one batched call per round.  One causal oracle pass per utterance over
    context + root + emitted tokens yields the target's next-token logits at every emitted position; each
    emitted token must be the oracle's arg-max there wherever that is decided by more than 1e-2, and otherwise lie
    within 2e-2 of the maximum.  By induction over the positions this is token-for-token equality with the
    oracle's own greedy transcript wherever no near-tie is met."""
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    from paper_2507_18181_b200.loop import SpeculativeBatchLoop
    seed, n_tokens, n_nodes, k_max, n_prompt = 2, 40, 32, 12, 6
    cfg = gen.get_config("7b", n_layers=8)
    dcfg = gen.get_config("0.5b", n_layers=8)
    store = gen.WeightStore(cfg, seed)
    target = DeviceModel(cfg, store)
    draft = DeviceModel(dcfg, gen.WeightStore(dcfg, seed + 1))
    frames = (90, 150, 61)
    B = len(frames)
    need = n_tokens + 2 * k_max + 2
    kvs, dkvs, roots, L0, truth, prefixes = [], [], [], [], [], []
    for b, fr in enumerate(frames):
        prompt = gen.prompt_tokens(n_prompt, cfg.vocab, seed, utterance=b)
        audio = gen.audio_prefix(fr, cfg.d_model, seed, utterance=b)
        kv = DeviceKV(target, max_tokens=fr + n_prompt + need + n_nodes + 64, max_nodes=B * n_nodes)
        kv.prefill_embeds(torch.from_numpy(audio).cuda())
        kv.prefill_tokens(torch.from_numpy(prompt[:-1].copy()).cuda())
        L = fr + n_prompt - 1
        truth.append(_device_greedy(kv, int(prompt[-1]), need, L))         # proposals are built from these
        dkv = DeviceKV(draft, max_tokens=fr + n_prompt + need + n_nodes + 64, max_nodes=B * n_nodes)
        dkv.prefill_embeds(torch.from_numpy(gen.audio_prefix(fr, dcfg.d_model, seed, utterance=b)).cuda())
        dkv.prefill_tokens(torch.from_numpy(prompt[:-1].copy()).cuda())
        kvs.append(kv); dkvs.append(dkv); roots.append(int(prompt[-1])); L0.append(L)
        prefixes.append((audio, prompt))
    proposer = gen.CorruptedGreedyProposer(truth, roots, cfg.vocab, seed=seed, n_nodes=n_nodes, k_min=4, k_max=k_max,
                                           corrupt_p=0.2)
    loop = SpeculativeBatchLoop(kvs, dkvs)
    out = loop.decode(roots, n_tokens, proposer)
    torch.cuda.synchronize()
    assert loop.rounds < n_tokens and loop.draft_steps > 0
    W = O.Weights(store, cache_layers=True)
    clear_total = 0
    for b in range(B):
        assert kvs[b].status() == 0 and len(out[b]) >= n_tokens
        audio, prompt = prefixes[b]
        emitted = [int(t) for t in out[b][:n_tokens]]
        seq = np.concatenate([audio.astype(np.float64), O.embed(W, list(prompt) + emitted[:-1])], 0)
        logits = O.causal_forward(cfg, W, seq)[-n_tokens:]                  # row j predicts emitted[j]
        gap = O.top2_gap(logits)
        top = logits.max(-1)
        am = logits.argmax(-1)
        for j, t in enumerate(emitted):
            assert top[j] - logits[j, t] <= LOGIT_TOL, (b, j)
            if gap[j] > GAP:
                assert am[j] == t, (b, j)
                clear_total += 1
        # the speculative transcript is the autoregressive one wherever every position was clear
        if np.all(gap > GAP):
            assert emitted == truth[b][:n_tokens]
    assert clear_total >= B * n_tokens * 3 // 4
