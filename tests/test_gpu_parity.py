"""Parity of the CUDA path against the CPU oracle, through the C ABI, on seeded inputs.

Bars: integer work (tree prep results visible through positions, accept length, path, committed
length, compaction moves) bit-exact; logits within 2e-2 max-abs of the fp64 oracle on the same bf16
weights; argmax / accept / path exact wherever the oracle's top-2 gap exceeds 1e-2 at every node the
result reads, otherwise the GPU result must be self-consistent and its argmax within 2e-2 of the top.
"""
import numpy as np
import pytest
import torch

import gen
from oracle import specasr_oracle as O
from helpers import oracle_weights

pytestmark = pytest.mark.gpu

LOGIT_TOL = 2e-2
GAP = 1e-2


def _gpu_stack(cfg_name, seed, gemm_path, max_tokens=512, max_nodes=64, shuffle=None, page_size=16):
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    cfg = gen.get_config(cfg_name)
    store = gen.WeightStore(cfg, seed)
    model = DeviceModel(cfg, store, gemm_path=gemm_path, page_size=page_size)
    kv = DeviceKV(model, max_tokens=max_tokens, max_nodes=max_nodes, shuffle_pages_seed=shuffle)
    return cfg, store, model, kv


def _fill_both(cfg, store, kv, n_audio, n_prompt, seed):
    W = O.Weights(store, cache_layers=True)
    audio = gen.audio_prefix(n_audio, cfg.d_model, seed)
    prompt = gen.prompt_tokens(n_prompt, cfg.vocab, seed)
    cache = O.KVCache(cfg)
    O.prefill(cfg, W, cache, np.concatenate([audio.astype(np.float64), O.embed(W, prompt[:-1])], 0))
    kv.prefill_embeds(torch.from_numpy(audio).cuda())
    if n_prompt > 1:
        kv.prefill_tokens(torch.from_numpy(prompt[:-1].copy()).cuda())
    return W, cache, prompt


def _verify_gpu(cfg, kv, tokens, parent):
    n = len(tokens)
    logits = torch.empty(n, cfg.vocab, dtype=torch.float32, device="cuda")
    kv.verify(torch.from_numpy(np.asarray(tokens, np.int32)).cuda(), torch.from_numpy(np.asarray(parent, np.int32)).cuda(),
              logits)
    torch.cuda.synchronize()
    assert kv.status() == 0
    return {
        "logits": logits.cpu().numpy().astype(np.float64),
        "argmax": kv.out_argmax[:n].cpu().numpy(),
        "accept_len": int(kv.out_accept.item()),
        "path": kv.out_path[:n].cpu().numpy(),
        "bonus": int(kv.out_bonus.item()),
    }


def _check_against_oracle(got, want, tokens, parent):
    n = len(tokens)
    err = np.abs(got["logits"] - want["logits"]).max()
    assert err < LOGIT_TOL, f"max-abs logit error {err}"
    clear = want["gap"] > GAP
    assert np.array_equal(got["argmax"][clear], want["argmax"][clear])
    # wherever the gap is small the GPU's pick must still be (numerically) a maximiser
    top = want["logits"].max(-1)
    picked = want["logits"][np.arange(n), got["argmax"]]
    assert np.all(top - picked <= LOGIT_TOL)
    # self-consistency: accept rule applied to the GPU's own argmax
    mine = O.accept(tokens, parent, got["argmax"])
    assert got["accept_len"] == mine["accept_len"] and got["bonus"] == mine["bonus"]
    a = got["accept_len"]
    assert list(got["path"][:a + 1]) == list(mine["path"]) and np.all(got["path"][a + 1:] == -1)
    if want["decisive"]:
        assert a == want["accept_len"] and list(got["path"][:a + 1]) == list(want["path"])
        assert got["bonus"] == want["bonus"]
    return err


CASES = [
    # cfg, gemm_path, n_audio, n_prompt, tree
    ("tiny", 1, 64, 8, "binary15"),
    ("tiny", 0, 64, 8, "binary15"),
    ("micro", 1, 21, 6, "sparse24"),
    ("micro", 0, 21, 6, "sparse24"),
    ("small", 1, 150, 9, "sparse64"),
    ("small", 0, 150, 9, "sparse64"),
    ("small", 0, 37, 3, "chain8"),
    ("small", 0, 100, 5, "sparse40"),     # n not a power of two: several activation boxes per stage
]


def _tree(kind, seed):
    if kind == "binary15":
        return gen.complete_binary_tree(15)
    if kind.startswith("sparse"):
        n = int(kind[6:])
        return gen.sparse_tree(n, seed=seed, levels=12 if n == 64 else None)
    return gen.chain_tree(int(kind[5:]))


@pytest.mark.parametrize("cfg_name,gemm_path,n_audio,n_prompt,tree", CASES)
def test_verify_matches_oracle(cfg_name, gemm_path, n_audio, n_prompt, tree):
    cfg, store, model, kv = _gpu_stack(cfg_name, 0, gemm_path, shuffle=11)
    W, cache, prompt = _fill_both(cfg, store, kv, n_audio, n_prompt, 0)
    assert kv.length() == cache.length == n_audio + n_prompt - 1
    # the filled cache itself
    for layer in (0, cfg.n_layers - 1):
        k, v = kv.read_kv(layer, cache.length)
        assert np.abs(k - cache.K[layer]).max() < 2e-3 and np.abs(v - cache.V[layer]).max() < 2e-3
    root = int(prompt[-1])
    parent = _tree(tree, 0)
    depth_main = len(gen.main_path(parent)) - 1
    greedy = O.greedy_continuation(cfg, W, cache, root, depth_main)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=0, root_token=root, main_tokens=greedy,
                                  corrupt_p=0.0 if tree == "binary15" else 0.2)
    if tree == "binary15":
        tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=0, root_token=root, main_tokens=greedy[:3])
    want = O.verify_tree(cfg, W, cache, tokens, parent)
    got = _verify_gpu(cfg, kv, tokens, parent)
    _check_against_oracle(got, want, tokens, parent)
    # verify does not move the committed length, and is repeatable
    assert kv.length() == cache.length
    again = _verify_gpu(cfg, kv, tokens, parent)
    assert np.array_equal(again["logits"], got["logits"]) and again["accept_len"] == got["accept_len"]

    # commit: compaction moves, new length, cache contents
    L = cache.length
    a = got["accept_len"]
    before_k, before_v = kv.read_kv(cfg.n_layers - 1, L + len(tokens))
    kv.commit()
    assert kv.length() == L + a + 1
    after_k, after_v = kv.read_kv(cfg.n_layers - 1, L + a + 1)
    src = L + got["path"][:a + 1]
    assert np.array_equal(after_k[L:], before_k[src]) and np.array_equal(after_v[L:], before_v[src])   # bitwise
    assert np.array_equal(after_k[:L], before_k[:L])
    if want["decisive"]:
        moves = O.commit(cache, want)
        assert moves == [(int(s), L + j) for j, s in enumerate(src)]
        assert np.abs(after_k - cache.K[-1]).max() < 2e-3 and np.abs(after_v - cache.V[-1]).max() < 2e-3


@pytest.mark.parametrize("page_size", [8, 24, 32, 64, 208])
def test_page_sizes_and_an_exactly_full_cache(page_size):
    """Pages of 32 / 64 / 208 slots run the tensor-core attention (one TMA box per page), 8 and 24 the plain one;
    the cache is sized so that the tree's last node lands in its last slot."""
    n_audio, n_prompt, n = 150, 6, 40
    L = n_audio + n_prompt - 1
    cap = -(-(L + n) // page_size) * page_size
    extra = cap - (L + n)                       # audio frames added so that L + n == capacity
    cfg, store, model, kv = _gpu_stack("small", 4, 0, max_tokens=cap, max_nodes=64, shuffle=5, page_size=page_size)
    W, cache, prompt = _fill_both(cfg, store, kv, n_audio + extra, n_prompt, 4)
    assert kv.length() + n == kv.max_pages * page_size
    parent = gen.sparse_tree(n, seed=4)
    root = int(prompt[-1])
    greedy = O.greedy_continuation(cfg, W, cache, root, len(gen.main_path(parent)) - 1)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=4, root_token=root, main_tokens=greedy, corrupt_p=0.2)
    got = _verify_gpu(cfg, kv, tokens, parent)
    _check_against_oracle(got, O.verify_tree(cfg, W, cache, tokens, parent), tokens, parent)
    before = kv.length()
    kv.commit()
    assert kv.length() == before + got["accept_len"] + 1
    # one node more than fits is refused on the host
    from paper_2507_18181_b200 import binding as B
    kv.truncate(before)
    bigger = gen.chain_tree(n)                  # n + 1 nodes
    t = torch.zeros(n + 1, dtype=torch.int32, device="cuda")
    with pytest.raises(B.SpecasrError) as e:
        kv.verify(t, torch.from_numpy(bigger).cuda())
    assert e.value.status == B.SPECASR_ERR_KV_CAPACITY


def test_product_library_has_one_engine():
    """The plain-FMA projections and attention live in the cross-check build variant only: the product library
    refuses the shapes and the switch that would need them."""
    from paper_2507_18181_b200 import binding as B
    from paper_2507_18181_b200.runtime import DeviceModel
    cfg = gen.get_config("tiny")
    store = gen.WeightStore(cfg, 0)
    for kwargs in (dict(gemm_path=1), dict(page_size=8), dict(page_size=24)):
        with pytest.raises(B.SpecasrError) as e:
            DeviceModel(cfg, store, crosscheck=False, **kwargs)
        assert e.value.status == B.SPECASR_ERR_UNSUPPORTED
    with pytest.raises(B.SpecasrError) as e:
        DeviceModel(gen.get_config("micro"), gen.WeightStore(gen.get_config("micro"), 0), crosscheck=False)   # head_dim 32
    assert e.value.status == B.SPECASR_ERR_UNSUPPORTED
    assert DeviceModel(cfg, store).variant == "product" and DeviceModel(cfg, store, gemm_path=1).variant == "crosscheck"


def test_tensor_core_and_fma_projections_agree():
    """Same operands, two engines (the second one from the cross-check build variant of the library): the only
    difference allowed is fp32 summation order."""
    outs = []
    for path in (1, 0):
        cfg, store, model, kv = _gpu_stack("small", 3, path)
        W, cache, prompt = _fill_both(cfg, store, kv, 90, 4, 3)
        parent = gen.sparse_tree(48, seed=3)
        tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=3, root_token=int(prompt[-1]))
        outs.append(_verify_gpu(cfg, kv, tokens, parent))
    assert np.abs(outs[0]["logits"] - outs[1]["logits"]).max() < 2e-3


def _follow_device(cache, ref, got):
    """Advance the oracle's cache along the path the device committed.  On a clear round that is the oracle's
    own path (asserted by _check_against_oracle); on a near-tie the device may legitimately have picked the
    other maximiser, and the two sides must keep describing the same cache."""
    a = got["accept_len"]
    return O.commit(cache, dict(ref, path=np.asarray(got["path"][:a + 1]), accept_len=a))


def test_speculative_rounds_are_lossless_on_gpu():
    """verify -> commit rounds with corrupted chain drafts and sparse trees reproduce the oracle's
    autoregressive greedy transcript; every round is also checked against the oracle.  Where a round hangs on
    a near-tie the oracle's cache follows the device's path and the expected transcript is re-derived from there;
    no round is skipped."""
    cfg, store, model, kv = _gpu_stack("small", 2, 0, shuffle=3)
    W, cache, prompt = _fill_both(cfg, store, kv, 30, 5, 2)
    root = int(prompt[-1])
    total = 24
    want = O.greedy_continuation(cfg, W, cache, root, total + 12)      # what is still expected from here on
    out = []
    rounds = clear_rounds = 0
    while len(out) < total:
        parent = gen.chain_tree(6) if rounds % 2 == 0 else gen.sparse_tree(20, seed=rounds)
        k = len(gen.main_path(parent)) - 1
        if len(want) < k + 1:                       # `want` always continues from the current cache and root
            want = O.greedy_continuation(cfg, W, cache, root, k + 13)
        truth = want[:k]
        tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=100 + rounds, root_token=root, main_tokens=truth,
                                      corrupt_p=0.25)
        ref = O.verify_tree(cfg, W, cache, tokens, parent)
        got = _verify_gpu(cfg, kv, tokens, parent)
        _check_against_oracle(got, ref, tokens, parent)
        kv.commit()
        _follow_device(cache, ref, got)
        assert kv.length() == cache.length
        a = got["accept_len"]
        emitted = [int(t) for t in tokens[got["path"][1:a + 1]]] + [got["bonus"]]
        out += emitted
        root = got["bonus"]
        same = got["bonus"] == ref["bonus"] and list(got["path"][:a + 1]) == list(ref["path"])
        assert same or not ref["decisive"]
        if same:
            assert emitted == want[:len(emitted)]                     # lossless: the oracle's own greedy tokens
            want = want[len(emitted):]
        else:                                                         # a near-tie went the other way on the device
            want = O.greedy_continuation(cfg, W, cache, root, total + 12)
        clear_rounds += int(ref["decisive"])
        rounds += 1
    # the seeded run has nine rounds, six of them clear (the oracle side alone fixes both numbers)
    assert len(out) >= total and rounds >= 4 and clear_rounds >= 4


def test_node_order_does_not_matter_on_gpu():
    cfg, store, model, kv = _gpu_stack("micro", 2, 0)
    W, cache, prompt = _fill_both(cfg, store, kv, 17, 4, 2)
    parent = gen.sparse_tree(30, seed=2)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=2, root_token=int(prompt[-1]))
    a = _verify_gpu(cfg, kv, tokens, parent)
    p2, t2, old = gen.relabel_tree(parent, tokens, seed=4)
    b = _verify_gpu(cfg, kv, t2, p2)
    assert np.abs(b["logits"] - a["logits"][old]).max() < 1e-3
    assert b["accept_len"] == a["accept_len"]


def test_error_paths_leave_state_untouched():
    from paper_2507_18181_b200 import binding as B
    cfg, store, model, kv = _gpu_stack("tiny", 0, 0, max_tokens=64, max_nodes=32)
    W, cache, prompt = _fill_both(cfg, store, kv, 20, 3, 0)
    L = kv.length()
    dev = "cuda"
    tok = torch.zeros(8, dtype=torch.int32, device=dev)
    par = torch.tensor([-1, 0, 1, 2, 3, 4, 5, 6], dtype=torch.int32, device=dev)
    # host-visible errors
    with pytest.raises(B.SpecasrError) as e:
        B.specasr_verify_tree(model.handle, kv.handle, tok.data_ptr(), par.data_ptr(), 0, kv.out_argmax.data_ptr(),
                              kv.out_accept.data_ptr(), kv.out_path.data_ptr())
    assert e.value.status == B.SPECASR_ERR_INVALID_ARG
    with pytest.raises(B.SpecasrError) as e:
        B.specasr_verify_tree(model.handle, kv.handle, tok.data_ptr(), par.data_ptr(), 33, kv.out_argmax.data_ptr(),
                              kv.out_accept.data_ptr(), kv.out_path.data_ptr())
    assert e.value.status == B.SPECASR_ERR_INVALID_ARG
    with pytest.raises(B.SpecasrError) as e:
        B.specasr_verify_tree(model.handle, kv.handle, 0, par.data_ptr(), 8, kv.out_argmax.data_ptr(),
                              kv.out_accept.data_ptr(), kv.out_path.data_ptr())
    assert e.value.status == B.SPECASR_ERR_INVALID_ARG
    with pytest.raises(B.SpecasrError) as e:
        kv.commit()                                     # nothing pending
    assert e.value.status == B.SPECASR_ERR_STATE
    # device-visible errors: cycle / forward parent, token out of range
    for bad_par, bad_tok in (([-1, 0, 3, 2, 1, 1, 1, 1], None), ([0, 0, 1, 2, 3, 4, 5, 6], None),
                             ([-1, 0, 1, 2, 3, 4, 5, 6], cfg.vocab)):
        p = torch.tensor(bad_par, dtype=torch.int32, device=dev)
        t = tok.clone()
        if bad_tok is not None:
            t[3] = bad_tok
        kv.verify(t, p)
        torch.cuda.synchronize()
        assert kv.status() == B.SPECASR_ERR_INVALID_TREE
        assert int(kv.out_accept.item()) == -1 and bool((kv.out_path[:8] == -1).all())
        kv.commit()                                     # committing a failed verify is a no-op
        assert kv.length() == L
    # capacity: 22 committed + 32 tree slots fit in 64, a prefill that does not fit is refused
    with pytest.raises(B.SpecasrError) as e:
        kv.prefill_tokens(torch.zeros(60, dtype=torch.int32, device=dev))
    assert e.value.status == B.SPECASR_ERR_KV_CAPACITY
    assert kv.length() == L
    # a good verify still works afterwards and gives the oracle's answer
    parent = gen.chain_tree(7)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=1, root_token=int(prompt[-1]))
    got = _verify_gpu(cfg, kv, tokens, parent)
    _check_against_oracle(got, O.verify_tree(cfg, W, cache, tokens, parent), tokens, parent)
    # abandoning a round: verify twice, commit once
    kv.truncate(L)
    assert kv.length() == L


def test_context_fill_refuses_a_token_id_outside_the_vocabulary():
    """A prompt id >= vocab (or negative) is never turned into an address: the chunk's status word is set, the rest
    of the call does nothing, the length does not advance, and the handle works again afterwards."""
    from paper_2507_18181_b200 import binding as B
    cfg, store, model, kv = _gpu_stack("tiny", 0, 0, max_tokens=128, max_nodes=32)
    W, cache, prompt = _fill_both(cfg, store, kv, 20, 3, 0)
    L = kv.length()
    for bad in (cfg.vocab, -1, 2 ** 30):
        toks = torch.tensor([5, 6, bad, 7], dtype=torch.int32, device="cuda")
        kv.prefill_tokens(toks)
        torch.cuda.synchronize()
        assert kv.status() == B.SPECASR_ERR_INVALID_TREE
        assert kv.length() == L                          # nothing of the call was appended, not even the good ids before the bad one's chunk ended
        kv.truncate(L)                                   # clears the status
    parent = gen.chain_tree(5)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=2, root_token=int(prompt[-1]))
    got = _verify_gpu(cfg, kv, tokens, parent)
    _check_against_oracle(got, O.verify_tree(cfg, W, cache, tokens, parent), tokens, parent)


def test_single_node_tree_and_max_nodes():
    cfg, store, model, kv = _gpu_stack("micro", 1, 0, max_tokens=600, max_nodes=256)
    W, cache, prompt = _fill_both(cfg, store, kv, 10, 2, 1)
    root = int(prompt[-1])
    # n = 1: plain autoregressive step
    got = _verify_gpu(cfg, kv, np.array([root], np.int32), np.array([-1], np.int32))
    want = O.verify_tree(cfg, W, cache, [root], [-1])
    _check_against_oracle(got, want, np.array([root]), np.array([-1]))
    assert got["accept_len"] == 0 and got["path"][0] == 0
    # n = 256: the largest tree the ancestor bitmask holds
    parent = gen.sparse_tree(256, seed=1)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=1, root_token=root)
    got = _verify_gpu(cfg, kv, tokens, parent)
    _check_against_oracle(got, O.verify_tree(cfg, W, cache, tokens, parent), tokens, parent)


def test_13b_shape_two_layers():
    """13B-class head geometry: 40 query heads = 40 KV heads (a row tile holds 128 nodes of one head), d_model 5120,
    120 weight tiles in the QKV projection (no k-split)."""
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    cfg = gen.get_config("13b", n_layers=2)
    store = gen.WeightStore(cfg, 6)
    model = DeviceModel(cfg, store, gemm_path=0)
    kv = DeviceKV(model, max_tokens=512, max_nodes=64, shuffle_pages_seed=2)
    W2, cache, prompt = _fill_both(cfg, store, kv, 230, 5, 6)
    root = int(prompt[-1])
    parent = gen.sparse_tree(64, seed=6, levels=12)
    greedy = O.greedy_continuation(cfg, W2, cache, root, len(gen.main_path(parent)) - 1)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=6, root_token=root, main_tokens=greedy, corrupt_p=0.2)
    got = _verify_gpu(cfg, kv, tokens, parent)
    _check_against_oracle(got, O.verify_tree(cfg, W2, cache, tokens, parent), tokens, parent)


def _bench_shape_case(cfg, n_audio, n_text, parent, seed, max_nodes):
    """Same launch configuration as bench.py for that shape: prefill in chunks of max_nodes, page size 16,
    tensor-core path; the oracle runs the same seeded inputs in fp64."""
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    store = gen.WeightStore(cfg, seed)
    model = DeviceModel(cfg, store)
    L = n_audio + n_text - 1
    n = len(parent)
    kv = DeviceKV(model, max_tokens=L + n + 64, max_nodes=max_nodes)
    W = O.Weights(store, cache_layers=True)
    audio = gen.audio_prefix(n_audio, cfg.d_model, seed)
    text = gen.prompt_tokens(n_text, cfg.vocab, seed)
    cache = O.KVCache(cfg)
    O.prefill(cfg, W, cache, np.concatenate([audio.astype(np.float64), O.embed(W, text[:-1])], 0))
    kv.prefill_embeds(torch.from_numpy(audio).cuda())
    kv.prefill_tokens(torch.from_numpy(text[:-1].copy()).cuda())
    assert kv.length() == cache.length == L
    root = int(text[-1])
    k = len(gen.main_path(parent)) - 1
    greedy = O.greedy_continuation(cfg, W, cache, root, k)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=seed, root_token=root, main_tokens=greedy, corrupt_p=0.2)
    want = O.verify_tree(cfg, W, cache, tokens, parent)
    got = _verify_gpu(cfg, kv, tokens, parent)
    err = _check_against_oracle(got, want, tokens, parent)
    # cache rows of the tree itself (last layer), then the commit
    kk, vv = kv.read_kv(cfg.n_layers - 1, L + n)
    assert np.abs(kk[L:] - want["tree_K"][-1]).max() < 2e-3 and np.abs(vv[L:] - want["tree_V"][-1]).max() < 2e-3
    kv.commit()
    assert kv.length() == L + got["accept_len"] + 1
    return err, got, want


def test_7b_shape_two_layers_in_the_benchmarked_launch_configuration():
    """Config 3 with the layer count cut to two (the per-layer kernels, tile counts, split counts and the
    1700 + 64 position attention are exactly those of the 32-layer benchmark run)."""
    cfg = gen.get_config("7b", n_layers=2)
    parent = gen.sparse_tree(64, seed=1, levels=12)
    err, got, want = _bench_shape_case(cfg, 1500, 201, parent, seed=1, max_nodes=64)
    assert err < LOGIT_TOL


def test_1b_shape_chain_draft_full_size():
    """Config 2 at full size: 16 layers, d 2048, 32 / 8 heads of 64, KV prefix 750 + 32, chain of 8 drafts."""
    cfg = gen.get_config("1b")
    parent = gen.chain_tree(8)
    err, got, want = _bench_shape_case(cfg, 750, 33, parent, seed=2, max_nodes=16)
    assert err < LOGIT_TOL
    assert got["accept_len"] <= 8


def test_7b_full_size_properties():
    """Config 3 at full size (32 layers, 14 GB of weights), where the fp64 oracle would need minutes: properties
    that hold at any size.  Determinism, the accept rule applied to the GPU's own arg-max, invariance under
    renumbering of the tree, agreement of a node with the same node verified as a chain (its root path), and
    the cache after commit."""
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    cfg = gen.get_config("7b")
    store = gen.WeightStore(cfg, 1)
    model = DeviceModel(cfg, store)
    L, n = 1700, 64
    kv = DeviceKV(model, max_tokens=L + n + 64, max_nodes=64)
    kv.prefill_embeds(torch.from_numpy(gen.audio_prefix(1500, cfg.d_model, 1)).cuda())
    text = gen.prompt_tokens(201, cfg.vocab, 1)
    kv.prefill_tokens(torch.from_numpy(text[:-1].copy()).cuda())
    assert kv.length() == L
    root = int(text[-1])
    parent = gen.sparse_tree(n, seed=1, levels=12)
    # the target's own greedy continuation, by single-node rounds of the library itself
    greedy, tok = [], root
    for _ in range(11):
        kv.verify(torch.tensor([tok], dtype=torch.int32, device="cuda"), torch.tensor([-1], dtype=torch.int32, device="cuda"))
        kv.commit()
        tok = int(kv.out_bonus.item())
        greedy.append(tok)
    kv.truncate(L)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=1, root_token=root, main_tokens=greedy, corrupt_p=0.2)
    a = _verify_gpu(cfg, kv, tokens, parent)
    b = _verify_gpu(cfg, kv, tokens, parent)
    assert np.array_equal(a["logits"], b["logits"]) and np.array_equal(a["path"], b["path"])
    assert np.isfinite(a["logits"]).all()
    mine = O.accept(tokens, parent, a["argmax"])
    assert a["accept_len"] == mine["accept_len"] and a["bonus"] == mine["bonus"]
    assert list(a["path"][:a["accept_len"] + 1]) == list(mine["path"])
    assert np.array_equal(a["argmax"], a["logits"].argmax(-1))
    # greedy drafts up to the first corrupted position are accepted (lossless acceptance of the target's own tokens)
    mp = gen.main_path(parent)
    k_ok = 0
    while k_ok < 11 and tokens[mp[k_ok + 1]] == greedy[k_ok]:
        k_ok += 1
    assert a["accept_len"] >= k_ok
    # renumbering
    p2, t2, old = gen.relabel_tree(parent, tokens, seed=3)
    c = _verify_gpu(cfg, kv, t2, p2)
    assert np.abs(c["logits"] - a["logits"][old]).max() < 2e-3
    assert c["accept_len"] == a["accept_len"]
    # the deepest node of the main path, verified as a plain chain (= causal decoding of its root path)
    chain_tokens = tokens[mp].astype(np.int32)
    d = _verify_gpu(cfg, kv, chain_tokens, gen.chain_tree(len(mp) - 1))
    assert np.abs(d["logits"] - a["logits"][mp]).max() < 2e-3
    # commit of the tree result
    res = _verify_gpu(cfg, kv, tokens, parent)
    k_before, v_before = kv.read_kv(31, L + n)
    kv.commit()
    al = res["accept_len"]
    assert kv.length() == L + al + 1
    k_after, _ = kv.read_kv(31, L + al + 1)
    assert np.array_equal(k_after[L:], k_before[L + res["path"][:al + 1]])


@pytest.mark.parametrize("cfg_name", ["tiny", "micro", "small"])
def test_random_tree_shapes(cfg_name):
    """Seeded random topologies (any parent[i] < i: bushy, stringy, stars) and sizes from 1 to 70 nodes, several
    rounds on one cache with commits in between, so that ragged tile tails, odd page offsets and every padding
    width (16 / 32 / 64 / 128) are hit."""
    cfg, store, model, kv = _gpu_stack(cfg_name, 8, 0, max_tokens=640, max_nodes=128, shuffle=9)
    W, cache, prompt = _fill_both(cfg, store, kv, 45, 4, 8)
    rng = np.random.default_rng(1234)
    root = int(prompt[-1])
    sizes = [1, 2, 3, 7, 15, 17, 31, 33, 48, 63, 65, 70]
    sizes_run = []
    for rnd, n in enumerate(sizes):
        shape = rnd % 3
        if shape == 0:
            parent = np.array([-1] + [int(rng.integers(0, i)) for i in range(1, n)], np.int32)              # bushy
        elif shape == 1:
            parent = np.array([-1] + [max(0, i - 1 - int(rng.integers(0, 2))) for i in range(1, n)], np.int32)  # stringy
        else:
            parent = np.array([-1] + [0 if rng.random() < 0.5 else int(rng.integers(0, i)) for i in range(1, n)], np.int32)
        depth_main = len(gen.main_path(parent)) - 1
        greedy = O.greedy_continuation(cfg, W, cache, root, depth_main) if depth_main else []
        tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=50 + rnd, root_token=root, main_tokens=greedy,
                                      corrupt_p=0.15)
        want = O.verify_tree(cfg, W, cache, tokens, parent)
        got = _verify_gpu(cfg, kv, tokens, parent)
        _check_against_oracle(got, want, tokens, parent)
        kv.commit()
        _follow_device(cache, want, got)                # a near-tie does not end the run: the oracle follows
        assert kv.length() == cache.length
        root = got["bonus"]
        sizes_run.append(n)
    assert sizes_run == sizes                           # every listed size reached the comparison


_TRACE_SCRIPT = r"""
import numpy as np, torch, gen
from paper_2507_18181_b200 import binding as B, build
from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
assert B.TRACE_LIB
build.build(trace=True)
cfg = gen.get_config("tiny")
model = DeviceModel(cfg, gen.WeightStore(cfg, 0))
kv = DeviceKV(model, max_tokens=256, max_nodes=64)
kv.prefill_embeds(torch.from_numpy(gen.audio_prefix(40, cfg.d_model, 0)).cuda())
parent = gen.complete_binary_tree(15)
tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=0, root_token=7)
d_t, d_p = torch.from_numpy(tokens).cuda(), torch.from_numpy(parent).cuda()
kv.verify(d_t, d_p)
torch.cuda.synchronize()
plain = kv.out_argmax[:15].clone()
rec = kv.trace(lambda: kv.verify(d_t, d_p))
kinds = [B.KIND_NAMES[int(k) & 0xFF] for k in rec[:, 0]]    # bits 8.. carry layer + 1 for the steps of the fused stack
# one launch each of prep, embedding and accept; per layer 2 norms, 4 projections, rotary, attention, merge, then the LM head
assert kinds.count("accept") == 1 and "gemm_lm" in kinds
for name in ("norm", "gemm_qkv", "rope", "attn", "attn_merge", "gemm_o", "gemm_gu", "gemm_down"):
    assert name in kinds, name
assert np.all(rec[:, 2] >= rec[:, 1])                              # every block ended after it started
assert np.all((rec[:, 3] == 0) | ((rec[:, 3] >= rec[:, 1]) & (rec[:, 3] <= rec[:, 2])))
assert kinds[0] == "prep" and int(np.argmax(rec[:, 2])) == kinds.index("accept")
assert torch.equal(kv.out_argmax[:15], plain)                      # tracing does not change results
# a buffer that is too small keeps counting but writes only what fits
small = torch.zeros(2 + 4 * 8 + 4, dtype=torch.int64, device="cuda")
B.specasr_trace_set(kv.handle, small.data_ptr(), 8)
kv.verify(d_t, d_p)
torch.cuda.synchronize()
B.specasr_trace_set(kv.handle, 0, 0)
assert int(small[0].item()) == len(rec) and int(small[2 + 4 * 8:].abs().sum().item()) == 0
small.zero_()                                                      # off again: nothing is written
kv.verify(d_t, d_p)
torch.cuda.synchronize()
assert int(small.abs().sum().item()) == 0
print("trace ok", len(rec))
"""


def test_device_trace_variant_records_every_block_and_product_library_refuses():
    """The device-side trace is a build variant (libspecasr_trace.so, selected by SPECASR_TRACE_LIB=1), exercised
    in a child process; the product library accepts only 'off'."""
    import os
    import subprocess
    import sys
    from paper_2507_18181_b200 import binding as B
    cfg, store, model, kv = _gpu_stack("tiny", 0, 0)
    buf = torch.zeros(64, dtype=torch.int64, device="cuda")
    B.specasr_trace_set(kv.handle, 0, 0)
    with pytest.raises(B.SpecasrError) as e:
        B.specasr_trace_set(kv.handle, buf.data_ptr(), 8)
    assert e.value.status == B.SPECASR_ERR_UNSUPPORTED
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, SPECASR_TRACE_LIB="1", PYTHONPATH=root + os.pathsep + os.environ.get("PYTHONPATH", ""))
    res = subprocess.run([sys.executable, "-c", _TRACE_SCRIPT], env=env, cwd=root, capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0 and "trace ok" in res.stdout, res.stdout + res.stderr


def test_config1_matches_the_stored_oracle_values():
    """Config 1 against tests/golden/config1_tiny_verify.json (written from the oracle alone by make_golden.py)."""
    import json
    import os
    stored = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden",
                                         "config1_tiny_verify.json")))
    cfg, store, model, kv = _gpu_stack("tiny", 0, 0)
    kv.prefill_embeds(torch.from_numpy(gen.audio_prefix(64, cfg.d_model, 0)).cuda())
    prompt = gen.prompt_tokens(8, cfg.vocab, 0)
    kv.prefill_tokens(torch.from_numpy(prompt[:-1].copy()).cuda())
    tokens, parent = np.asarray(stored["tokens"], np.int32), np.asarray(stored["parent"], np.int32)
    got = _verify_gpu(cfg, kv, tokens, parent)
    assert stored["min_top2_gap"] > GAP                     # every arg-max of this workload is decided clearly
    assert list(got["argmax"]) == stored["argmax"]
    assert got["accept_len"] == stored["accept_len"] == 3
    assert list(got["path"][:4]) == stored["path"] and got["bonus"] == stored["bonus"]
    assert np.allclose(got["logits"][0, :8], stored["logits_row0_first8"], rtol=0, atol=LOGIT_TOL)
    assert abs(np.abs(got["logits"]).sum() - stored["logits_abs_sum"]) < 1e-4 * stored["logits_abs_sum"]
