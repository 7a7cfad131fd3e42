"""Scenario builders shared by the CPU and GPU tests (inputs only; expected values come from the oracle)."""
import numpy as np

import gen
from oracle import specasr_oracle as O


def oracle_weights(cfg, seed=0, round_bf16=True):
    return O.Weights(gen.WeightStore(cfg, seed, round_bf16=round_bf16), cache_layers=True)


def prefix_inputs(cfg, W, n_audio, n_prompt, seed=0):
    """Layer-0 inputs of the context: audio vectors then all prompt tokens but the last (which
    becomes the root of the first tree).  Returns (inputs [T, d] fp64, audio fp32, prompt ids)."""
    audio = gen.audio_prefix(n_audio, cfg.d_model, seed)
    prompt = gen.prompt_tokens(n_prompt, cfg.vocab, seed)
    x = np.concatenate([audio.astype(np.float64), O.embed(W, prompt[:-1])], axis=0)
    return x, audio, prompt


def filled_cache(cfg, W, n_audio, n_prompt, seed=0):
    x, audio, prompt = prefix_inputs(cfg, W, n_audio, n_prompt, seed)
    cache = O.KVCache(cfg)
    O.prefill(cfg, W, cache, x)
    return cache, x, audio, prompt
