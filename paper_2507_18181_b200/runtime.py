"""Device-memory plumbing around the C ABI: torch allocates and owns every buffer, the library
borrows them.  No arithmetic of the verification path lives here."""
import ctypes as C

import numpy as np
import torch

from . import binding as B


def pack_weight(w: "torch.Tensor") -> "torch.Tensor":
    """[M, K] row-major bf16 -> the tile-packed layout include/specasr.h asks for: 128 x 64 tiles, each contiguous,
    ordered [row tile][column tile], M and K padded with zeros to multiples of 128 (data movement only)."""
    M, K = w.shape
    Mp, Kp = -(-M // 128) * 128, -(-K // 128) * 128
    if (Mp, Kp) != (M, K):
        w = torch.nn.functional.pad(w, (0, Kp - K, 0, Mp - M))
    return w.view(Mp // 128, 128, Kp // 64, 64).permute(0, 2, 1, 3).contiguous().view(-1)


def _routed(cls):
    """Every method of the class runs with the binding routed to the library variant the object was made with
    (self.variant), so that handles never reach another build of the library."""
    import functools
    for name, fn in list(vars(cls).items()):
        if isinstance(fn, staticmethod) or not callable(fn) or name in ("__init__", "__del__"):
            continue

        def make(f):
            @functools.wraps(f)
            def wrapped(self, *a, **k):
                with B.use(getattr(self, "variant", "product")):
                    return f(self, *a, **k)
            return wrapped
        setattr(cls, name, make(fn))
    return cls


def _bf16_from_bits(bits: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


@_routed
class DeviceModel:
    """Weights of one decoder on the GPU in the layouts include/specasr.h asks for.

    `cfg` needs n_layers, d_model, n_heads, n_kv_heads, head_dim, ffn, vocab, eps, rope_base.
    `store` needs tensor(layer, name) -> numpy array (uint16 bf16 bit patterns for matrices, fp32 for
    gains; layer -1 = embed / lm_head / g_final) and optionally map_tensors(fn, keys) for threaded draws.
    """

    def __init__(self, cfg, store, page_size=16, max_positions=8192, gemm_path=0, device="cuda:0", crosscheck=None):
        """crosscheck=True loads the cross-check build variant of the library (plain-FMA projections with
        gemm_path=1, head_dim 32, page sizes that are not a multiple of 16); by default it is chosen exactly when
        the shape asks for something the product library does not have."""
        if crosscheck is None:
            crosscheck = gemm_path != 0 or cfg.head_dim not in (64, 128) or page_size % 16 != 0
        self.variant = "crosscheck" if crosscheck else "product"
        if crosscheck:
            from . import build as _build
            _build.build(crosscheck=True)
        self._setup(cfg, store, page_size, max_positions, gemm_path, device)

    def _setup(self, cfg, store, page_size, max_positions, gemm_path, device):
        self.cfg = cfg
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.page_size = page_size
        L = cfg.n_layers
        got = {}
        # rotary-paired row order of the fused QKV matrix (see include/specasr.h): within every head,
        # stored row 32 g + 16 h + j holds feature 16 g + j + h * head_dim / 2
        dh = cfg.head_dim
        rho = np.arange(dh)
        feat = (rho // 32) * 16 + rho % 16 + ((rho % 32) // 16) * (dh // 2)
        n_heads_all = cfg.n_heads + 2 * cfg.n_kv_heads
        self._qkv_rows = torch.from_numpy((np.arange(n_heads_all)[:, None] * dh + feat[None, :]).reshape(-1)).to(self.device)

        def put(layer, name, arr):
            if arr.dtype == np.uint16:
                got[(layer, name)] = _bf16_from_bits(arr, self.device)
            else:
                got[(layer, name)] = torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32)).to(self.device)
            if layer >= 0 and all((layer, k) in got for k in ("wq", "wk", "wv")):
                fused = torch.cat([got.pop((layer, k)) for k in ("wq", "wk", "wv")], dim=0)
                got[(layer, "wqkv")] = pack_weight(fused[self._qkv_rows])
            if layer >= 0 and all((layer, k) in got for k in ("wg", "wu")):
                g, u = got.pop((layer, "wg")), got.pop((layer, "wu"))
                got[(layer, "wgu")] = pack_weight(torch.stack([g, u], dim=1).reshape(2 * cfg.ffn, cfg.d_model))
            if name in ("wo", "wd", "lm_head"):
                got[(layer, name)] = pack_weight(got[(layer, name)])

        keys = [(-1, n) for n in ("embed", "lm_head", "g_final")]
        for l in range(L):
            keys += [(l, n) for n in ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "g_attn", "g_ffn")]
        if hasattr(store, "map_tensors"):
            store.map_tensors(put, keys)
        else:
            for k in keys:
                put(k[0], k[1], store.tensor(*k))
        self.t = got
        self._arrays = {}
        wp = B.WeightPtrs()
        wp.embed = got[(-1, "embed")].data_ptr()
        wp.lm_head = got[(-1, "lm_head")].data_ptr()
        wp.g_final = got[(-1, "g_final")].data_ptr()
        for field in ("wqkv", "wo", "wgu", "wd", "g_attn", "g_ffn"):
            arr = (C.c_void_p * L)(*[got[(l, field)].data_ptr() for l in range(L)])
            self._arrays[field] = arr
            setattr(wp, field, C.cast(arr, C.POINTER(C.c_void_p)))
        mc = B.ModelConfig(n_layers=L, d_model=cfg.d_model, n_heads=cfg.n_heads, n_kv_heads=cfg.n_kv_heads,
                           head_dim=cfg.head_dim, ffn=cfg.ffn, vocab=cfg.vocab, page_size=page_size,
                           max_positions=max_positions, rms_eps=cfg.eps, rope_base=cfg.rope_base,
                           gemm_path=gemm_path)
        self.handle = B.specasr_model_create(mc, wp)

    def weight_bytes(self) -> int:
        return sum(v.numel() * v.element_size() for v in self.t.values())

    def close(self):
        if self.handle:
            B.specasr_model_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


@_routed
class DeviceKV:
    """Paged KV cache + workspace for one utterance."""

    def __init__(self, model: DeviceModel, max_tokens: int, max_nodes: int = 256, shuffle_pages_seed=None,
                 poison: bool = False):
        self.variant = model.variant
        self._setup(model, max_tokens, max_nodes, shuffle_pages_seed, poison)

    def _setup(self, model, max_tokens, max_nodes, shuffle_pages_seed, poison):
        """`poison` fills both pools and the workspace with 0xFF bytes (NaN as bf16 and fp32, -1 as int32)
        instead of zeros before the handle is created: a kernel that reads something no kernel wrote then
        produces NaN or an error instead of a silently plausible result."""
        self.model = model
        cfg = model.cfg
        dev = model.device
        ps = model.page_size
        self.max_pages = (max_tokens + ps - 1) // ps
        self.n_pages = self.max_pages
        self.max_nodes = max_nodes
        pool_bytes = B.specasr_kv_pool_bytes(model.handle, self.n_pages)
        self.k_pool = torch.zeros(pool_bytes // 2, dtype=torch.bfloat16, device=dev)
        self.v_pool = torch.zeros(pool_bytes // 2, dtype=torch.bfloat16, device=dev)
        if poison:
            self.k_pool.view(torch.uint8).fill_(0xFF)
            self.v_pool.view(torch.uint8).fill_(0xFF)
        if shuffle_pages_seed is None:
            table = np.arange(self.max_pages, dtype=np.int32)
        else:
            table = np.random.default_rng(shuffle_pages_seed).permutation(self.max_pages).astype(np.int32)
        self.page_table_host = table
        self.page_table = torch.from_numpy(table).to(dev)
        ws_bytes = B.specasr_workspace_bytes(model.handle, max_nodes)
        self.workspace = torch.full((ws_bytes + 256,), 0xFF if poison else 0, dtype=torch.uint8, device=dev)
        ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
        self.handle = B.specasr_kv_create(model.handle, self.k_pool.data_ptr(), self.v_pool.data_ptr(), self.n_pages,
                                          self.page_table.data_ptr(), self.max_pages, ws_ptr, max_nodes)
        self.out_argmax = torch.empty(max_nodes, dtype=torch.int32, device=dev)
        self.out_path = torch.empty(max_nodes, dtype=torch.int32, device=dev)
        self.out_accept = torch.empty(1, dtype=torch.int32, device=dev)
        self.out_bonus = torch.empty(1, dtype=torch.int32, device=dev)

    @staticmethod
    def _stream() -> int:
        return torch.cuda.current_stream().cuda_stream

    def length(self) -> int:
        return B.specasr_kv_length(self.handle, self._stream())

    def truncate(self, n: int):
        B.specasr_kv_truncate(self.handle, n, self._stream())

    def prefill_embeds(self, embeds: torch.Tensor):
        assert embeds.dtype == torch.float32 and embeds.is_cuda and embeds.is_contiguous()
        B.specasr_prefill_embeds(self.model.handle, self.handle, embeds.data_ptr(), embeds.shape[0], self._stream())

    def prefill_tokens(self, tokens: torch.Tensor):
        assert tokens.dtype == torch.int32 and tokens.is_cuda and tokens.is_contiguous()
        B.specasr_prefill_tokens(self.model.handle, self.handle, tokens.data_ptr(), tokens.shape[0], self._stream())

    def verify(self, tokens: torch.Tensor, parent: torch.Tensor, logits: torch.Tensor | None = None):
        """Enqueues one verification round; results land in out_argmax / out_accept / out_path / out_bonus."""
        n = tokens.shape[0]
        B.specasr_verify_tree_ex(self.model.handle, self.handle, tokens.data_ptr(), parent.data_ptr(), n,
                                 self.out_argmax.data_ptr(), self.out_accept.data_ptr(), self.out_path.data_ptr(),
                                 logits.data_ptr() if logits is not None else 0, self.out_bonus.data_ptr(),
                                 self._stream())

    def verify_top2(self, tokens: torch.Tensor, parent: torch.Tensor):
        """As verify(), and the two most probable next tokens of every node with their probabilities land in
        out_top2_ids / out_top2_probs ([n, 2] each), computed in the vocabulary projection's epilogue."""
        n = tokens.shape[0]
        if not hasattr(self, "out_top2_ids"):
            self.out_top2_ids = torch.empty(self.max_nodes, 2, dtype=torch.int32, device=self.model.device)
            self.out_top2_probs = torch.empty(self.max_nodes, 2, dtype=torch.float32, device=self.model.device)
        B.specasr_verify_tree_top2(self.model.handle, self.handle, tokens.data_ptr(), parent.data_ptr(), n,
                                   self.out_argmax.data_ptr(), self.out_accept.data_ptr(), self.out_path.data_ptr(),
                                   self.out_bonus.data_ptr(), self.out_top2_ids.data_ptr(), self.out_top2_probs.data_ptr(),
                                   self._stream())

    def commit(self):
        B.specasr_commit_kv(self.model.handle, self.handle, self.out_path.data_ptr(), self.out_accept.data_ptr(),
                            self._stream())

    def status(self) -> int:
        return B.specasr_poll_status(self.handle, self._stream())

    def launches(self) -> int:
        return B.specasr_launch_count(self.handle)

    def trace(self, fn, capacity: int = 1 << 16):
        """Runs fn() with the device-side trace on and returns the records as an int64 array [records, 4]
        (kind, start ns, end ns, wait-end ns), sorted by start time."""
        buf = torch.zeros(2 + 4 * capacity, dtype=torch.int64, device=self.model.device)
        torch.cuda.synchronize()
        B.specasr_trace_set(self.handle, buf.data_ptr(), capacity)
        try:
            fn()
            torch.cuda.synchronize()
        finally:
            B.specasr_trace_set(self.handle, 0, 0)
        host = buf.cpu().numpy()
        n = min(int(host[0]), capacity)
        rec = host[2:2 + 4 * n].reshape(n, 4)
        return rec[np.argsort(rec[:, 1], kind="stable")]

    def read_kv(self, layer: int, n_slots: int):
        """Host copy of K and V of slots [0, n_slots) of one layer as fp64 [n, Hkv, dh] (hi + lo)."""
        cfg = self.model.cfg
        ps = self.model.page_size
        shape = (cfg.n_layers, self.n_pages, cfg.n_kv_heads, 2, ps, cfg.head_dim)
        out = []
        for pool in (self.k_pool, self.v_pool):
            p = pool.view(shape)[layer].float().cpu().numpy().astype(np.float64)   # [pages, Hkv, 2, ps, dh]
            logical = p[self.page_table_host]                                      # logical page order
            val = logical[:, :, 0] + logical[:, :, 1]                              # [pages, Hkv, ps, dh]
            val = val.transpose(0, 2, 1, 3).reshape(-1, cfg.n_kv_heads, cfg.head_dim)
            out.append(val[:n_slots])
        return out[0], out[1]

    def close(self):
        if self.handle:
            B.specasr_kv_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


@_routed
class BatchVerifier:
    """Output buffers for specasr_verify_tree_batch over a fixed list of utterances.  The first
    utterance's workspace carries the rows of all of them, so its max_nodes bounds the total."""

    def __init__(self, kvs):
        self.kvs = list(kvs)
        self.variant = self.kvs[0].variant
        self.model = self.kvs[0].model
        dev = self.model.device
        total = self.kvs[0].max_nodes
        self.out_argmax = torch.empty(total, dtype=torch.int32, device=dev)
        self.out_path = torch.empty(total, dtype=torch.int32, device=dev)
        self.out_accept = torch.empty(len(self.kvs), dtype=torch.int32, device=dev)
        self.out_bonus = torch.empty(len(self.kvs), dtype=torch.int32, device=dev)
        self.offsets = [0] * (len(self.kvs) + 1)

    def verify(self, tokens: torch.Tensor, parent: torch.Tensor, node_offsets, logits: torch.Tensor | None = None):
        """tokens / parent: int32 device tensors over all utterances back to back (parents local to the
        utterance); node_offsets: batch + 1 host ints; logits: optional fp32 [total nodes, vocab] output."""
        self.offsets = [int(o) for o in node_offsets]
        B.specasr_verify_tree_batch(self.model.handle, [kv.handle for kv in self.kvs], tokens.data_ptr(),
                                    parent.data_ptr(), self.offsets, self.out_argmax.data_ptr(),
                                    self.out_accept.data_ptr(), self.out_path.data_ptr(),
                                    logits.data_ptr() if logits is not None else 0, self.out_bonus.data_ptr(),
                                    DeviceKV._stream())

    def verify_top2(self, tokens: torch.Tensor, parent: torch.Tensor, node_offsets):
        """As verify(), with the top-2 tokens and probabilities of every node in out_top2_ids / out_top2_probs."""
        self.offsets = [int(o) for o in node_offsets]
        if not hasattr(self, "out_top2_ids"):
            total = self.kvs[0].max_nodes
            self.out_top2_ids = torch.empty(total, 2, dtype=torch.int32, device=self.model.device)
            self.out_top2_probs = torch.empty(total, 2, dtype=torch.float32, device=self.model.device)
        B.specasr_verify_tree_batch_top2(self.model.handle, [kv.handle for kv in self.kvs], tokens.data_ptr(),
                                         parent.data_ptr(), self.offsets, self.out_argmax.data_ptr(),
                                         self.out_accept.data_ptr(), self.out_path.data_ptr(), self.out_bonus.data_ptr(),
                                         self.out_top2_ids.data_ptr(), self.out_top2_probs.data_ptr(), DeviceKV._stream())

    def commit(self):
        item = self.out_path.element_size()
        for b, kv in enumerate(self.kvs):
            B.specasr_commit_kv(self.model.handle, kv.handle, self.out_path.data_ptr() + item * self.offsets[b],
                                self.out_accept.data_ptr() + item * b, DeviceKV._stream())

    def commit_chains(self):
        """After a verify() whose trees were chains: keeps every node of every chain (the caller's own choice of
        path, which specasr_commit_kv allows), whatever the model's arg-max said.  Used to feed known tokens."""
        sizes = [self.offsets[b + 1] - self.offsets[b] for b in range(len(self.kvs))]
        path = torch.tensor([i for n in sizes for i in range(n)], dtype=torch.int32, device=self.model.device)
        accept = torch.tensor([n - 1 for n in sizes], dtype=torch.int32, device=self.model.device)
        item = path.element_size()
        for b, kv in enumerate(self.kvs):
            B.specasr_commit_kv(self.model.handle, kv.handle, path.data_ptr() + item * self.offsets[b],
                                accept.data_ptr() + item * b, DeviceKV._stream())
        self._chain_commit = (path, accept)              # alive until the stream has run the copies
