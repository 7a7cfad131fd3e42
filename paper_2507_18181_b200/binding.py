"""ctypes binding of libspecasr.so: same names and arguments as include/specasr.h.

Argument marshalling only.  Device buffers are passed as integer addresses (e.g.
`tensor.data_ptr()`), streams as the integer value of a cudaStream_t.  Nothing here computes
anything; if the shared library is missing the import of any entry point fails loudly.
"""
import ctypes as C
import os

import contextlib

_HERE = os.path.dirname(os.path.abspath(__file__))
# SPECASR_TRACE_LIB=1 selects the variant built with -DSPECASR_TRACE (specasr_trace_set records; ~2 % slower)
TRACE_LIB = os.environ.get("SPECASR_TRACE_LIB") == "1"
LIB_PATH = os.path.join(_HERE, "libspecasr_trace.so" if TRACE_LIB else "libspecasr.so")
# The cross-check variant (-DSPECASR_CROSSCHECK) also carries the plain-FMA projections and attention.  It can be
# loaded beside the product library: handles made by one library are only ever passed back to that library, which
# `use("crosscheck")` arranges for the calls made inside it.
VARIANT_PATHS = {"product": LIB_PATH, "crosscheck": os.path.join(_HERE, "libspecasr_crosscheck.so")}
_current = ["product"]


@contextlib.contextmanager
def use(variant: str):
    """Route the binding's calls to another build variant of the library for the duration of the block."""
    _current.append(variant)
    try:
        yield
    finally:
        _current.pop()


SPECASR_MAX_NODES = 256
SPECASR_MAX_BATCH = 32
(SPECASR_OK, SPECASR_ERR_INVALID_ARG, SPECASR_ERR_INVALID_TREE, SPECASR_ERR_KV_CAPACITY, SPECASR_ERR_STATE,
 SPECASR_ERR_UNSUPPORTED, SPECASR_ERR_TIMEOUT, SPECASR_ERR_CUDA) = range(8)
STATUS_NAMES = ["OK", "INVALID_ARG", "INVALID_TREE", "KV_CAPACITY", "STATE", "UNSUPPORTED", "TIMEOUT", "CUDA"]

EXPORTS = [
    "specasr_model_create", "specasr_model_destroy", "specasr_workspace_bytes", "specasr_kv_pool_bytes",
    "specasr_kv_create", "specasr_kv_destroy", "specasr_kv_length", "specasr_kv_truncate",
    "specasr_prefill_embeds", "specasr_prefill_tokens", "specasr_verify_tree", "specasr_verify_tree_ex",
    "specasr_verify_tree_batch", "specasr_verify_tree_top2", "specasr_verify_tree_batch_top2", "specasr_commit_kv", "specasr_poll_status", "specasr_launch_count", "specasr_last_error",
    "specasr_profile_enable", "specasr_profile_read", "specasr_trace_set", "specasr_accept_logits_static", "specasr_top2_probs",
]
KIND_NAMES = ["prep", "norm", "gemm_qkv", "rope", "attn", "attn_merge", "gemm_o", "gemm_gu", "gemm_down", "gemm_lm",
              "accept", "commit", "stack"]


class ModelConfig(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32), ("page_size", C.c_int32),
                ("max_positions", C.c_int32), ("rms_eps", C.c_float), ("rope_base", C.c_float),
                ("gemm_path", C.c_int32), ("reserved", C.c_int32 * 3)]


class WeightPtrs(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("g_final", C.c_void_p),
                ("wqkv", C.POINTER(C.c_void_p)), ("wo", C.POINTER(C.c_void_p)), ("wgu", C.POINTER(C.c_void_p)),
                ("wd", C.POINTER(C.c_void_p)), ("g_attn", C.POINTER(C.c_void_p)), ("g_ffn", C.POINTER(C.c_void_p))]


_libs = {}


def lib() -> C.CDLL:
    variant = _current[-1]
    if variant not in _libs:
        path = VARIANT_PATHS[variant]
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -m paper_2507_18181_b200.build` "
                               "(there is no fallback path)")
        L = C.CDLL(path)
        vp, i32, st = C.c_void_p, C.c_int32, C.c_int
        L.specasr_model_create.argtypes = [C.POINTER(ModelConfig), C.POINTER(WeightPtrs), C.POINTER(vp)]
        L.specasr_model_create.restype = st
        L.specasr_model_destroy.argtypes = [vp]
        L.specasr_model_destroy.restype = None
        L.specasr_workspace_bytes.argtypes = [vp, i32]
        L.specasr_workspace_bytes.restype = C.c_size_t
        L.specasr_kv_pool_bytes.argtypes = [vp, i32]
        L.specasr_kv_pool_bytes.restype = C.c_size_t
        L.specasr_kv_create.argtypes = [vp, vp, vp, i32, vp, i32, vp, i32, C.POINTER(vp)]
        L.specasr_kv_create.restype = st
        L.specasr_kv_destroy.argtypes = [vp]
        L.specasr_kv_destroy.restype = None
        L.specasr_kv_length.argtypes = [vp, C.POINTER(i32), vp]
        L.specasr_kv_length.restype = st
        L.specasr_kv_truncate.argtypes = [vp, i32, vp]
        L.specasr_kv_truncate.restype = st
        L.specasr_prefill_embeds.argtypes = [vp, vp, vp, i32, vp]
        L.specasr_prefill_embeds.restype = st
        L.specasr_prefill_tokens.argtypes = [vp, vp, vp, i32, vp]
        L.specasr_prefill_tokens.restype = st
        L.specasr_verify_tree.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp]
        L.specasr_verify_tree.restype = st
        L.specasr_verify_tree_ex.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]
        L.specasr_verify_tree_ex.restype = st
        L.specasr_verify_tree_batch.argtypes = [vp, i32, C.POINTER(vp), vp, vp, C.POINTER(i32), vp, vp, vp, vp, vp, vp]
        L.specasr_verify_tree_batch.restype = st
        L.specasr_verify_tree_top2.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp, vp]
        L.specasr_verify_tree_top2.restype = st
        L.specasr_verify_tree_batch_top2.argtypes = [vp, i32, C.POINTER(vp), vp, vp, C.POINTER(i32), vp, vp, vp, vp, vp, vp, vp]
        L.specasr_verify_tree_batch_top2.restype = st
        L.specasr_commit_kv.argtypes = [vp, vp, vp, vp, vp]
        L.specasr_commit_kv.restype = st
        L.specasr_poll_status.argtypes = [vp, C.POINTER(i32), vp]
        L.specasr_poll_status.restype = st
        L.specasr_launch_count.argtypes = [vp]
        L.specasr_launch_count.restype = C.c_int64
        L.specasr_profile_enable.argtypes = [vp, i32]
        L.specasr_profile_enable.restype = st
        L.specasr_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64), vp]
        L.specasr_profile_read.restype = st
        L.specasr_trace_set.argtypes = [vp, vp, C.c_int64]
        L.specasr_trace_set.restype = st
        L.specasr_accept_logits_static.argtypes = [vp, i32, vp, vp, i32, vp, vp, vp, vp, vp]
        L.specasr_accept_logits_static.restype = st
        L.specasr_top2_probs.argtypes = [vp, i32, i32, vp, vp, vp]
        L.specasr_top2_probs.restype = st
        L.specasr_last_error.argtypes = []
        L.specasr_last_error.restype = C.c_char_p
        _libs[variant] = L
    return _libs[variant]


class SpecasrError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"SPECASR_ERR_{STATUS_NAMES[status]}: {message}")
        self.status = status


def specasr_last_error() -> str:
    return lib().specasr_last_error().decode()


def _check(status: int):
    if status != SPECASR_OK:
        raise SpecasrError(status, specasr_last_error())


def specasr_model_create(cfg: ModelConfig, weights: WeightPtrs) -> int:
    out = C.c_void_p()
    _check(lib().specasr_model_create(C.byref(cfg), C.byref(weights), C.byref(out)))
    return out.value


def specasr_model_destroy(model: int) -> None:
    lib().specasr_model_destroy(model)


def specasr_workspace_bytes(model: int, max_nodes: int) -> int:
    return lib().specasr_workspace_bytes(model, max_nodes)


def specasr_kv_pool_bytes(model: int, n_pages: int) -> int:
    return lib().specasr_kv_pool_bytes(model, n_pages)


def specasr_kv_create(model: int, k_pool: int, v_pool: int, n_pages: int, page_table: int, max_pages: int,
                      workspace: int, max_nodes: int) -> int:
    out = C.c_void_p()
    _check(lib().specasr_kv_create(model, k_pool, v_pool, n_pages, page_table, max_pages, workspace, max_nodes,
                                   C.byref(out)))
    return out.value


def specasr_kv_destroy(kv: int) -> None:
    lib().specasr_kv_destroy(kv)


def specasr_kv_length(kv: int, stream: int = 0) -> int:
    out = C.c_int32()
    _check(lib().specasr_kv_length(kv, C.byref(out), stream))
    return out.value


def specasr_kv_truncate(kv: int, length: int, stream: int = 0) -> None:
    _check(lib().specasr_kv_truncate(kv, length, stream))


def specasr_prefill_embeds(model: int, kv: int, embeds: int, n: int, stream: int = 0) -> None:
    _check(lib().specasr_prefill_embeds(model, kv, embeds, n, stream))


def specasr_prefill_tokens(model: int, kv: int, tokens: int, n: int, stream: int = 0) -> None:
    _check(lib().specasr_prefill_tokens(model, kv, tokens, n, stream))


def specasr_verify_tree(model: int, kv: int, tokens: int, parent_idx: int, n_nodes: int, out_argmax: int,
                        out_accept_len: int, out_path: int, stream: int = 0) -> None:
    _check(lib().specasr_verify_tree(model, kv, tokens, parent_idx, n_nodes, out_argmax, out_accept_len, out_path,
                                     stream))


def specasr_verify_tree_ex(model: int, kv: int, tokens: int, parent_idx: int, n_nodes: int, out_argmax: int,
                           out_accept_len: int, out_path: int, out_logits: int = 0, out_bonus: int = 0,
                           stream: int = 0) -> None:
    _check(lib().specasr_verify_tree_ex(model, kv, tokens, parent_idx, n_nodes, out_argmax, out_accept_len, out_path,
                                        out_logits or None, out_bonus or None, stream))


def specasr_verify_tree_batch(model: int, kv_handles, tokens: int, parent_idx: int, node_offsets, out_argmax: int,
                              out_accept_len: int, out_path: int, out_logits: int = 0, out_bonus: int = 0,
                              stream: int = 0) -> None:
    """kv_handles: sequence of handles; node_offsets: sequence of batch + 1 ints (both host side);
    the other arguments are device addresses covering all utterances back to back."""
    batch = len(kv_handles)
    handles = (C.c_void_p * batch)(*kv_handles)
    offsets = (C.c_int32 * len(node_offsets))(*node_offsets)
    if len(node_offsets) != batch + 1:
        raise ValueError("node_offsets needs batch + 1 entries")
    _check(lib().specasr_verify_tree_batch(model, batch, handles, tokens, parent_idx, offsets, out_argmax,
                                           out_accept_len, out_path, out_logits or None, out_bonus or None, stream))


def specasr_verify_tree_top2(model: int, kv: int, tokens: int, parent_idx: int, n_nodes: int, out_argmax: int,
                             out_accept_len: int, out_path: int, out_bonus: int, out_top2_ids: int, out_top2_probs: int,
                             stream: int = 0) -> None:
    _check(lib().specasr_verify_tree_top2(model, kv, tokens, parent_idx, n_nodes, out_argmax, out_accept_len, out_path,
                                          out_bonus or None, out_top2_ids, out_top2_probs, stream))


def specasr_verify_tree_batch_top2(model: int, kv_handles, tokens: int, parent_idx: int, node_offsets, out_argmax: int,
                                   out_accept_len: int, out_path: int, out_bonus: int, out_top2_ids: int,
                                   out_top2_probs: int, stream: int = 0) -> None:
    batch = len(kv_handles)
    handles = (C.c_void_p * batch)(*kv_handles)
    offsets = (C.c_int32 * len(node_offsets))(*node_offsets)
    if len(node_offsets) != batch + 1:
        raise ValueError("node_offsets needs batch + 1 entries")
    _check(lib().specasr_verify_tree_batch_top2(model, batch, handles, tokens, parent_idx, offsets, out_argmax,
                                                out_accept_len, out_path, out_bonus or None, out_top2_ids,
                                                out_top2_probs, stream))


def specasr_commit_kv(model: int, kv: int, path: int, accept_len: int, stream: int = 0) -> None:
    _check(lib().specasr_commit_kv(model, kv, path, accept_len, stream))


def specasr_accept_logits_static(logits: int, vocab: int, tokens: int, parent_idx: int, n_nodes: int, out_argmax: int,
                                 out_accept_len: int, out_path: int, out_bonus: int = 0, stream: int = 0) -> None:
    """Accept step from a logits matrix for callers that cannot allocate device memory (see the header):
    all arguments are device addresses of caller-owned buffers; the library's built-in array is the only scratch."""
    _check(lib().specasr_accept_logits_static(logits, vocab, tokens, parent_idx, n_nodes, out_argmax, out_accept_len,
                                              out_path, out_bonus or None, stream))


def specasr_top2_probs(logits: int, n_rows: int, vocab: int, out_ids: int, out_probs: int, stream: int = 0) -> None:
    _check(lib().specasr_top2_probs(logits, n_rows, vocab, out_ids, out_probs, stream))


def specasr_poll_status(kv: int, stream: int = 0) -> int:
    out = C.c_int32()
    _check(lib().specasr_poll_status(kv, C.byref(out), stream))
    return out.value


def specasr_launch_count(kv: int) -> int:
    return lib().specasr_launch_count(kv)


def specasr_profile_enable(kv: int, enable: int) -> None:
    _check(lib().specasr_profile_enable(kv, enable))


def specasr_trace_set(kv: int, buffer: int, capacity_records: int) -> None:
    _check(lib().specasr_trace_set(kv, buffer or None, capacity_records))


def specasr_profile_read(kv: int, stream: int = 0):
    """Returns ({kind name: ms}, {kind name: launches}) accumulated since the last read."""
    n = len(KIND_NAMES)
    ms = (C.c_double * n)()
    cnt = (C.c_int64 * n)()
    _check(lib().specasr_profile_read(kv, ms, cnt, stream))
    return dict(zip(KIND_NAMES, list(ms))), dict(zip(KIND_NAMES, list(cnt)))
