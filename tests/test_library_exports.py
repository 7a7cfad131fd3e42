"""The C-ABI library builds, loads without a GPU, and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2507_18181_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "specasr.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(specasr_[a-z0-9_]+)\s*\(", text)))


def test_header_and_binding_agree_and_symbols_exist():
    build.build()
    declared = _declared()
    assert declared == sorted(binding.EXPORTS)
    lib = ctypes.CDLL(binding.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name
    for name in binding.EXPORTS:
        assert callable(getattr(binding, name))


def test_host_side_argument_errors_need_no_gpu():
    lib = binding.lib()
    out = ctypes.c_void_p()
    assert lib.specasr_model_create(None, None, ctypes.byref(out)) == binding.SPECASR_ERR_INVALID_ARG
    assert b"null" in lib.specasr_last_error()
    cfg = binding.ModelConfig(n_layers=1, d_model=64, n_heads=2, n_kv_heads=1, head_dim=48, ffn=64, vocab=100,
                              page_size=16, max_positions=128, rms_eps=1e-6, rope_base=1e4)
    arr = (ctypes.c_void_p * 1)(1)
    wp = binding.WeightPtrs(embed=1, lm_head=1, g_final=1)
    for f in ("wqkv", "wo", "wgu", "wd", "g_attn", "g_ffn"):
        setattr(wp, f, ctypes.cast(arr, ctypes.POINTER(ctypes.c_void_p)))
    assert lib.specasr_model_create(ctypes.byref(cfg), ctypes.byref(wp), ctypes.byref(out)) == binding.SPECASR_ERR_UNSUPPORTED
    assert lib.specasr_workspace_bytes(None, 64) == 0
    assert lib.specasr_verify_tree(None, None, None, None, 4, None, None, None, None) == binding.SPECASR_ERR_INVALID_ARG
    assert lib.specasr_commit_kv(None, None, None, None, None) == binding.SPECASR_ERR_INVALID_ARG
    n = ctypes.c_int32()
    assert lib.specasr_kv_length(None, ctypes.byref(n), None) == binding.SPECASR_ERR_INVALID_ARG


def test_pack_weight_follows_the_offset_formula_of_the_header():
    """The tile-packed weight layout (include/specasr.h): element (m, k) of a [M, K] matrix sits at
    (((m / 128) * Kt + k / 64) * 128 + m % 128) * 64 + k % 64 with Kt = 2 * ceil(K / 128); padding reads as zero."""
    import torch
    from paper_2507_18181_b200.runtime import pack_weight
    for M, K in ((128, 128), (200, 72), (384, 320), (96, 64)):
        w = torch.arange(1, M * K + 1, dtype=torch.float32).reshape(M, K)
        packed = pack_weight(w)
        Kt = 2 * -(-K // 128)
        assert packed.numel() == -(-M // 128) * Kt * 128 * 64
        m = torch.arange(M)[:, None].expand(M, K)
        k = torch.arange(K)[None, :].expand(M, K)
        off = (((m // 128) * Kt + k // 64) * 128 + m % 128) * 64 + k % 64
        assert torch.equal(packed[off.reshape(-1)], w.reshape(-1))
        assert float(packed.sum()) == float(w.sum())          # everything else is padding
