"""Pins of the oracle's building blocks against things other than itself: closed forms,
library routines, and an independent library decoder."""
import math

import numpy as np
import pytest
import torch

import gen
from oracle import specasr_oracle as O
from helpers import oracle_weights


def test_widen_reads_bf16_bits():
    x = np.array([1.0, -2.5, 0.0, 0.00390625], np.float32)
    assert np.array_equal(O.widen(gen.f32_to_bf16_bits(x)), x.astype(np.float64))
    # 0x3F80 is 1.0, 0xC000 is -2.0 in bf16
    assert list(O.widen(np.array([0x3F80, 0xC000], np.uint16))) == [1.0, -2.0]


def test_rmsnorm_closed_forms():
    # constant row c: mean square c^2, so output = c / sqrt(c^2 + eps) * g
    g = np.array([1.0, 2.0, -1.0, 0.5])
    y = O.rmsnorm(np.full((1, 4), 3.0), g, 1e-6)
    assert np.allclose(y[0], 3.0 / math.sqrt(9.0 + 1e-6) * g, rtol=0, atol=1e-15)
    # (3,4,0,0): mean square 6.25 -> rms 2.5
    y = O.rmsnorm(np.array([[3.0, 4.0, 0.0, 0.0]]), np.ones(4), 0.0)
    assert np.allclose(y[0], [1.2, 1.6, 0.0, 0.0])
    # eps matters for a zero row (no division by zero) and scale invariance holds without it
    assert np.all(O.rmsnorm(np.zeros((1, 4)), np.ones(4), 1e-6) == 0.0)
    x = np.random.default_rng(0).standard_normal((3, 16))
    assert np.allclose(O.rmsnorm(x, g=np.ones(16), eps=0.0), O.rmsnorm(7.0 * x, np.ones(16), 0.0))
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (16,), eps=1e-6).numpy()
    assert np.allclose(O.rmsnorm(x, np.ones(16), 1e-6), ref, atol=1e-14)


def test_silu_and_softmax_closed_forms():
    assert O.silu(np.array([0.0]))[0] == 0.0
    assert np.allclose(O.silu(np.array([1.0, -1.0])), [1 / (1 + math.exp(-1)), -1 / (1 + math.e)])
    x = np.linspace(-5, 5, 11)
    assert np.allclose(O.silu(x), torch.nn.functional.silu(torch.from_numpy(x)).numpy(), atol=1e-15)
    s = np.array([[0.0, math.log(2.0), math.log(5.0), 100.0]])
    m = np.array([[True, True, True, False]])
    p = O.masked_softmax(s, m)
    assert np.allclose(p, [[1 / 8, 2 / 8, 5 / 8, 0.0]])
    assert np.allclose(O.masked_softmax(s + 1234.5, m), p)          # shift invariance
    assert np.allclose(O.masked_softmax(np.random.default_rng(0).standard_normal((5, 9)),
                                        np.ones((5, 9), bool)).sum(-1), 1.0)


def test_rope_closed_forms():
    rng = np.random.default_rng(0)
    dh, base = 8, 1e4
    x = rng.standard_normal((1, 1, dh))
    assert np.array_equal(O.rope(x, np.array([0]), base), x)                      # position 0 = identity
    # pair (k, k + dh/2) is rotated by angle pos * base^(-2k/dh): check one pair by hand
    pos, k = 3, 1
    ang = pos * base ** (-2.0 * k / dh)
    y = O.rope(x, np.array([pos]), base)[0, 0]
    assert np.isclose(y[k], x[0, 0, k] * math.cos(ang) - x[0, 0, k + dh // 2] * math.sin(ang))
    assert np.isclose(y[k + dh // 2], x[0, 0, k + dh // 2] * math.cos(ang) + x[0, 0, k] * math.sin(ang))
    # pair 0 turns by exactly `pos` radians
    y0 = O.rope(np.array([[[1.0, 0, 0, 0, 0.0, 0, 0, 0]]]), np.array([2]), base)[0, 0]
    assert np.isclose(y0[0], math.cos(2.0)) and np.isclose(y0[4], math.sin(2.0))
    # norms preserved; inner products depend on the position difference only
    q = rng.standard_normal((1, 2, dh))
    kk = rng.standard_normal((1, 2, dh))
    assert np.isclose(np.linalg.norm(O.rope(q, np.array([17]), base)), np.linalg.norm(q))
    d1 = np.sum(O.rope(q, np.array([9]), base) * O.rope(kk, np.array([4]), base))
    d2 = np.sum(O.rope(q, np.array([1005]), base) * O.rope(kk, np.array([1000]), base))
    assert np.isclose(d1, d2, atol=1e-11)


@pytest.mark.parametrize("hq,hkv", [(4, 4), (4, 2), (8, 2)])
def test_attention_matches_library_sdpa(hq, hkv):
    rng = np.random.default_rng(hq * 10 + hkv)
    T, S, dh = 5, 11, 16
    q = rng.standard_normal((T, hq, dh))
    k = rng.standard_normal((S, hkv, dh))
    v = rng.standard_normal((S, hkv, dh))
    mask = rng.random((T, S)) < 0.6
    mask[:, 0] = True
    out = O.attention(q, k, v, mask)
    rep = hq // hkv
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(rep, dim=0)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(rep, dim=0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=torch.from_numpy(mask)[None, None])
    assert np.allclose(out, ref[0].permute(1, 0, 2).numpy(), atol=1e-13)


def _hf_model(cfg, W):
    from transformers import LlamaConfig, LlamaForCausalLM
    hc = LlamaConfig(vocab_size=cfg.vocab, hidden_size=cfg.d_model, intermediate_size=cfg.ffn,
                     num_hidden_layers=cfg.n_layers, num_attention_heads=cfg.n_heads,
                     num_key_value_heads=cfg.n_kv_heads, head_dim=cfg.head_dim, rms_norm_eps=cfg.eps,
                     rope_theta=cfg.rope_base, attention_bias=False, mlp_bias=False,
                     tie_word_embeddings=False, max_position_embeddings=4096)
    model = LlamaForCausalLM(hc).double().eval()
    g = W.globals()
    sd = {"model.embed_tokens.weight": g["embed"], "lm_head.weight": g["lm_head"], "model.norm.weight": g["g_final"]}
    names = {"wq": "self_attn.q_proj", "wk": "self_attn.k_proj", "wv": "self_attn.v_proj", "wo": "self_attn.o_proj",
             "wg": "mlp.gate_proj", "wu": "mlp.up_proj", "wd": "mlp.down_proj",
             "g_attn": "input_layernorm", "g_ffn": "post_attention_layernorm"}
    for l in range(cfg.n_layers):
        w = W.layer(l)
        for k, v in names.items():
            sd[f"model.layers.{l}.{v}.weight"] = w[k]
    model.load_state_dict({k: torch.from_numpy(np.ascontiguousarray(v)) for k, v in sd.items()}, strict=True)
    return model


@pytest.mark.parametrize("name", ["micro", "tiny"])
def test_causal_forward_matches_library_llama(name):
    """Block wiring, RoPE pairing, GQA grouping, SwiGLU, norms, audio vectors as inputs_embeds:
    an independent implementation fed the same tensors must give the same logits.  (The library
    builds its rotary table in fp32, hence 1e-6 rather than 1e-12.)"""
    pytest.importorskip("transformers")
    cfg = gen.get_config(name)
    W = oracle_weights(cfg, seed=1)
    model = _hf_model(cfg, W)
    audio = gen.audio_prefix(12, cfg.d_model, 1).astype(np.float64)
    toks = gen.prompt_tokens(9, cfg.vocab, 1)
    x = np.concatenate([audio, O.embed(W, toks)], axis=0)
    ours = O.causal_forward(cfg, W, x)
    with torch.no_grad():
        ref = model(inputs_embeds=torch.from_numpy(x)[None]).logits[0].numpy()
    assert np.abs(ours - ref).max() < 1e-6
    assert np.array_equal(ours.argmax(-1), ref.argmax(-1))
    # pure-token input goes through the embedding table on both sides
    ours_t = O.causal_forward(cfg, W, O.embed(W, toks))
    with torch.no_grad():
        ref_t = model(input_ids=torch.from_numpy(toks.astype(np.int64))[None]).logits[0].numpy()
    assert np.abs(ours_t - ref_t).max() < 1e-6


def test_top2_probs_against_library_softmax_hand_values_and_sorting():
    from scipy.special import softmax
    # a row worked by hand: logits (0, ln 2, ln 5) -> probabilities (1/8, 2/8, 5/8)
    ids, probs = O.top2_probs(np.array([[0.0, np.log(2.0), np.log(5.0)]]))
    assert ids.tolist() == [[2, 1]]
    assert np.allclose(probs, [[5 / 8, 2 / 8]], rtol=0, atol=1e-15)
    # ties: the lower id first, then the other holder of the maximum
    ids, probs = O.top2_probs(np.array([[1.0, 3.0, 3.0, -1.0], [2.0, 2.0, 2.0, 2.0]]))
    assert ids.tolist() == [[1, 2], [0, 1]]
    assert np.allclose(probs[1], [0.25, 0.25])
    # random rows: library softmax and a full stable sort
    rng = np.random.default_rng(7)
    logits = rng.standard_normal((9, 501)) * 4.0
    ids, probs = O.top2_probs(logits)
    sm = softmax(logits, axis=-1)
    order = np.argsort(-logits, axis=-1, kind="stable")
    assert np.array_equal(ids, order[:, :2].astype(np.int32))
    assert np.allclose(probs, np.take_along_axis(sm, order[:, :2], axis=-1), rtol=1e-13, atol=0)
    assert np.all(probs[:, 0] >= probs[:, 1]) and np.all(probs.sum(-1) <= 1.0 + 1e-15)
    # shifting a row by a constant changes nothing; a huge offset must not overflow
    ids2, probs2 = O.top2_probs(logits + 1000.0)
    assert np.array_equal(ids2, ids) and np.allclose(probs2, probs, rtol=1e-10)


def test_top2_gap_against_a_full_sort_hand_rows_and_a_tie():
    """The margin that decides which arg-max entries are compared bit-exactly: pinned to a full sort, to rows
    worked by hand, to a tie (margin 0) and to the one-column case."""
    rng = np.random.default_rng(3)
    x = rng.standard_normal((7, 50))
    s = np.sort(x, axis=-1)
    assert np.array_equal(O.top2_gap(x), s[:, -1] - s[:, -2])
    assert np.all(O.top2_gap(x) > 0)
    # hand rows: 1-D input, 2-D input, negative values, the maximum in first / last place
    assert O.top2_gap(np.array([0.25, -1.0, 0.75])) == 0.5
    assert list(O.top2_gap(np.array([[3.0, 1.0, 2.0], [-5.0, -7.0, -4.0], [0.0, 0.0, 9.0]]))) == [1.0, 1.0, 9.0]
    # a tie for the maximum has margin exactly 0, wherever the two entries sit
    assert O.top2_gap(np.array([1.0, 5.0, 3.0, 5.0])) == 0.0
    assert O.top2_gap(np.array([[2.0, 2.0]]))[0] == 0.0
    # 3-D input keeps the leading axes
    y = rng.standard_normal((2, 3, 9))
    sy = np.sort(y, axis=-1)
    assert np.array_equal(O.top2_gap(y), sy[..., -1] - sy[..., -2])
    # a single column: nothing can overtake
    assert np.all(np.isinf(O.top2_gap(np.array([[1.5], [2.5]]))))
    # the margin is what separates a perturbed arg-max from the original: shifting the runner-up by more than
    # the margin changes the arg-max, by less does not
    row = x[0].copy()
    first, second = np.argsort(row)[-1], np.argsort(row)[-2]
    g = O.top2_gap(row)
    bumped = row.copy(); bumped[second] += 0.99 * g
    assert np.argmax(bumped) == first
    bumped[second] = row[second] + 1.01 * g
    assert np.argmax(bumped) == second


def _hand_logits(n, vocab, winners, margins):
    """Rows whose largest entry is winners[i] and whose runner-up sits margins[i] below it."""
    lg = np.full((n, vocab), -3.0)
    for i, (w, m) in enumerate(zip(winners, margins)):
        lg[i, w] = 1.0
        lg[i, (w + 1) % vocab] = 1.0 - m
    return lg


def test_decisive_flag_on_hand_built_trees():
    """Tree 0 -> 1 -> 2 with a side leaf 3 below the root.  Node 1 carries the target's token after the root,
    node 2 the target's token after node 1, so the path 0, 1, 2 is accepted and node 2 wins; node 3 carries
    another token and is rejected.  The result reads the arg-max of nodes 0 and 1 (they have children) and of
    node 2 (the bonus token); node 3's arg-max is read by nothing."""
    parent = np.array([-1, 0, 1, 0])
    vocab = 8
    winners = [4, 6, 2, 5]                  # the target's greedy token after each node
    tokens = np.array([7, 4, 6, 1])         # node 1 = winners[0], node 2 = winners[1], node 3 != winners[0]
    wide = [1.0, 1.0, 1.0, 1.0]
    r = O.decide(tokens, parent, _hand_logits(4, vocab, winners, wide))
    assert r["accept_len"] == 2 and list(r["path"]) == [0, 1, 2] and r["bonus"] == 2 and r["decisive"]
    assert list(r["consulted"]) == [True, True, True, False]
    assert np.allclose(r["gap"], wide)
    # a narrow margin at the rejected leaf changes nothing that is reported
    r = O.decide(tokens, parent, _hand_logits(4, vocab, winners, [1.0, 1.0, 1.0, 1e-3]))
    assert r["decisive"] and abs(r["gap"][3] - 1e-3) < 1e-12
    # the same narrow margin at a node with a child, or at the winner, makes the round ambiguous
    for node in (0, 1, 2):
        m = list(wide)
        m[node] = 1e-3
        r = O.decide(tokens, parent, _hand_logits(4, vocab, winners, m))
        assert not r["decisive"], node
        assert r["accept_len"] == 2                      # the oracle's own outcome is unchanged
    # the threshold is exclusive and adjustable: a margin equal to it is not clear
    r = O.decide(tokens, parent, _hand_logits(4, vocab, winners, [0.5, 1.0, 1.0, 1.0]), decisive_gap=0.5)
    assert not r["decisive"]
    assert O.decide(tokens, parent, _hand_logits(4, vocab, winners, [0.5, 1.0, 1.0, 1.0]), decisive_gap=0.49)["decisive"]
    # when the draft fails at the first step the winner is the root: only node 0 and the parents are read
    tokens2 = np.array([7, 3, 6, 1])
    r = O.decide(tokens2, parent, _hand_logits(4, vocab, winners, [1.0, 1.0, 1e-3, 1e-3]))
    assert r["accept_len"] == 0 and r["best"] == 0 and r["decisive"]
    assert list(r["consulted"]) == [True, True, False, False]
    # a gap of zero everywhere (what a broken margin would report) must make every round ambiguous
    flat = np.zeros((4, vocab))
    assert not O.decide(tokens, parent, flat)["decisive"]
