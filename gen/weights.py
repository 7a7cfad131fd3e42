"""Random-init decoder weights, regenerable one tensor at a time.

Every tensor has its own PCG64 stream keyed by (seed, layer, tensor name), so a
7B-shape model never has to be held whole in host memory: the oracle streams one
layer at a time and the GPU loader uploads tensor by tensor.

Matrices are stored [out_features, in_features] (row-major), drawn as
0.02 * N(0,1) in fp32 and rounded once to bf16; the bit patterns are what both
the oracle and the CUDA path consume.  Norm gains are 1 + 0.02 * N(0,1) and
stay fp32 (a gain of exactly zero-mean noise would erase the residual stream,
and a gain of exactly one would hide a missing multiply).
"""
from concurrent.futures import ThreadPoolExecutor
import os
import threading

import numpy as np

from .bf16 import f32_to_bf16_bits
from .configs import ModelConfig

_STREAM_WEIGHTS = 0x5EC0
_scratch = threading.local()


def _scratch_f32(n: int) -> np.ndarray:
    """Per-thread reusable fp32 buffer: large draws do not pay for fresh pages every time."""
    buf = getattr(_scratch, "buf", None)
    if buf is None or buf.size < n:
        buf = np.empty(n, dtype=np.float32)
        _scratch.buf = buf
    return buf[:n]

# name -> (code, shape function)
LAYER_TENSORS = {
    "wq": (1, lambda c: (c.q_dim, c.d_model)),
    "wk": (2, lambda c: (c.kv_dim, c.d_model)),
    "wv": (3, lambda c: (c.kv_dim, c.d_model)),
    "wo": (4, lambda c: (c.d_model, c.q_dim)),
    "wg": (5, lambda c: (c.ffn, c.d_model)),
    "wu": (6, lambda c: (c.ffn, c.d_model)),
    "wd": (7, lambda c: (c.d_model, c.ffn)),
    "g_attn": (8, lambda c: (c.d_model,)),
    "g_ffn": (9, lambda c: (c.d_model,)),
}
GLOBAL_TENSORS = {
    "embed": (20, lambda c: (c.vocab, c.d_model)),
    "lm_head": (21, lambda c: (c.vocab, c.d_model)),
    "g_final": (22, lambda c: (c.d_model,)),
}


class WeightStore:
    """Seeded weights of one decoder.  `round_bf16=False` keeps the fp32 draws (oracle-only use)."""

    def __init__(self, cfg: ModelConfig, seed: int = 0, round_bf16: bool = True):
        self.cfg = cfg
        self.seed = int(seed)
        self.round_bf16 = round_bf16

    def _rng(self, layer: int, code: int) -> np.random.Generator:
        ss = np.random.SeedSequence(entropy=[self.seed, _STREAM_WEIGHTS, layer + 1, code])
        return np.random.Generator(np.random.PCG64(ss))

    def _draw(self, layer: int, name: str) -> np.ndarray:
        table = GLOBAL_TENSORS if layer < 0 else LAYER_TENSORS
        code, shape_fn = table[name]
        shape = shape_fn(self.cfg)
        if len(shape) == 1:
            z = self._rng(layer, code).standard_normal(shape, dtype=np.float32)
            z *= np.float32(0.02)
            z += np.float32(1.0)
            return z
        z = _scratch_f32(int(np.prod(shape))).reshape(shape)
        self._rng(layer, code).standard_normal(dtype=np.float32, out=z)
        z *= np.float32(0.02)
        return z          # view of the thread's scratch buffer: consume before the next draw

    def tensor(self, layer: int, name: str) -> np.ndarray:
        """Matrix: uint16 bf16 bit patterns (or fp32 if round_bf16=False).  Gain vector: fp32.
        `layer` = -1 addresses the global tensors (embed, lm_head, g_final)."""
        z = self._draw(layer, name)
        if z.ndim == 2:
            return f32_to_bf16_bits(z) if self.round_bf16 else z.copy()
        return z

    def layer(self, layer: int) -> dict:
        return {name: self.tensor(layer, name) for name in LAYER_TENSORS}

    def globals(self) -> dict:
        return {name: self.tensor(-1, name) for name in GLOBAL_TENSORS}

    def map_tensors(self, fn, keys, threads: int | None = None):
        """Call fn(layer, name, array) for every (layer, name) in keys, drawing in a thread pool
        (numpy generators release the GIL) while fn itself runs on the calling thread."""
        threads = threads or max(1, min(16, len(os.sched_getaffinity(0))))
        with ThreadPoolExecutor(threads) as pool:
            pending = []
            keys = list(keys)
            it = iter(keys)
            # keep at most `threads + 2` tensors in flight to bound host memory
            for _ in range(threads + 2):
                k = next(it, None)
                if k is None:
                    break
                pending.append((k, pool.submit(self.tensor, *k)))
            while pending:
                k, fut = pending.pop(0)
                arr = fut.result()
                nxt = next(it, None)
                if nxt is not None:
                    pending.append((nxt, pool.submit(self.tensor, *nxt)))
                fn(k[0], k[1], arr)

    def all_keys(self):
        keys = [(-1, n) for n in GLOBAL_TENSORS]
        for l in range(self.cfg.n_layers):
            keys += [(l, n) for n in LAYER_TENSORS]
        return keys
