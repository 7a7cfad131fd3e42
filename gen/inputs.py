"""Seeded context inputs: audio-embedding vectors and token ids.

The audio encoder of an LLM-based ASR model hands the decoder a sequence of
vectors already projected to the decoder width (Section II-A); here they are
N(0,1) draws of that shape.  Text is uniform over the vocabulary.
"""
import numpy as np

_STREAM_AUDIO = 0xA0D1
_STREAM_PROMPT = 0x9207
_STREAM_TOKENS = 0x70CE


def _rng(seed: int, stream: int, *extra: int) -> np.random.Generator:
    ss = np.random.SeedSequence(entropy=[int(seed), stream, *[int(e) for e in extra]])
    return np.random.Generator(np.random.PCG64(ss))


def audio_prefix(n_frames: int, d_model: int, seed: int = 0, utterance: int = 0) -> np.ndarray:
    """[n_frames, d_model] fp32 ~ N(0,1)."""
    return _rng(seed, _STREAM_AUDIO, utterance).standard_normal((n_frames, d_model), dtype=np.float32)


def prompt_tokens(n: int, vocab: int, seed: int = 0, utterance: int = 0) -> np.ndarray:
    return _rng(seed, _STREAM_PROMPT, utterance).integers(0, vocab, size=n, dtype=np.int32)


def uniform_tokens(n: int, vocab: int, seed: int = 0, stream: int = 0) -> np.ndarray:
    return _rng(seed, _STREAM_TOKENS, stream).integers(0, vocab, size=n, dtype=np.int32)
