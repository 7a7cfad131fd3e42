"""Writes tests/golden/config1_tiny_verify.json: what the CPU oracle computes for the smallest workload (2-layer
decoder of width 256, 64 audio vectors + 8 prompt tokens, complete binary tree of 15 nodes whose leftmost path
carries the greedy continuation for 3 tokens).  Calls only gen/ and oracle/; the paper prints no numbers for the
verification step, so these are the oracle's own values, kept so that a later change to the oracle's arithmetic
shows up as a diff.

    python tests/golden/make_golden.py
"""
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import gen  # noqa: E402
from oracle import specasr_oracle as O  # noqa: E402


def compute():
    cfg = gen.get_config("tiny")
    store = gen.WeightStore(cfg, 0)
    W = O.Weights(store, cache_layers=True)
    audio = gen.audio_prefix(64, cfg.d_model, 0)
    prompt = gen.prompt_tokens(8, cfg.vocab, 0)
    cache = O.KVCache(cfg)
    O.prefill(cfg, W, cache, np.concatenate([audio.astype(np.float64), O.embed(W, prompt[:-1])], 0))
    root = int(prompt[-1])
    greedy = O.greedy_continuation(cfg, W, cache, root, 4)
    parent = gen.complete_binary_tree(15)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=0, root_token=root, main_tokens=greedy[:3])
    res = O.verify_tree(cfg, W, cache, tokens, parent)
    ids, probs = O.top2_probs(res["logits"])
    return {
        "workload": "tiny decoder, seed 0, 64 audio vectors + 8 prompt tokens, complete binary tree of 15 nodes",
        "tokens": [int(t) for t in tokens],
        "parent": [int(p) for p in parent],
        "greedy_continuation": [int(t) for t in greedy],
        "argmax": [int(t) for t in res["argmax"]],
        "accept_len": int(res["accept_len"]),
        "path": [int(p) for p in res["path"]],
        "bonus": int(res["bonus"]),
        "min_top2_gap": float(res["gap"].min()),
        "logits_row0_first8": [float(x) for x in res["logits"][0, :8]],
        "logits_abs_sum": float(np.abs(res["logits"]).sum()),
        "top2_ids_row0": [int(x) for x in ids[0]],
        "top2_probs_row0": [float(x) for x in probs[0]],
    }


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "config1_tiny_verify.json")
    with open(out, "w") as f:
        json.dump(compute(), f, indent=1)
        f.write("\n")
    print("wrote", out)
