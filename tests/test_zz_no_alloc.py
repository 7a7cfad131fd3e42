"""The allocation-free accept entry point against the full verification call.

`specasr_accept_logits_static` exists for callers that are handed device buffers but cannot obtain any
themselves (a plug-in inside a serving process whose device memory was all reserved at start-up, or a
component that only scores logits computed elsewhere): its only scratch is a fixed array inside the
library.  Fed the logits that `specasr_verify_tree_ex` wrote, it must return that call's arg-max tokens,
accepted length, path and bonus token exactly (integer results: no tolerance), on two calls in a row
with different trees, because the second call finds the first call's leftovers in the shared array.
This file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

import gen
from oracle import specasr_oracle as O
from paper_2507_18181_b200 import binding as B

pytestmark = pytest.mark.gpu


def _verify(cfg, kv, tokens, parent):
    n = len(tokens)
    logits = torch.empty(n, cfg.vocab, dtype=torch.float32, device="cuda")
    kv.verify(torch.from_numpy(tokens).cuda(), torch.from_numpy(parent).cuda(), logits)
    torch.cuda.synchronize()
    assert kv.status() == 0
    return logits, (kv.out_argmax[:n].clone(), kv.out_accept.clone(), kv.out_path[:n].clone(), kv.out_bonus.clone())


def test_static_accept_matches_verify_on_two_calls_in_a_row():
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    cfg = gen.get_config("tiny")
    model = DeviceModel(cfg, gen.WeightStore(cfg, 7))
    kv = DeviceKV(model, max_tokens=256, max_nodes=64)
    kv.prefill_embeds(torch.from_numpy(gen.audio_prefix(19, cfg.d_model, 7)).cuda())
    L = kv.length()
    # every buffer the new call touches is created here, before it runs: it must not need more
    stream = torch.cuda.current_stream().cuda_stream
    cases = []
    for seed, parent in ((1, gen.sparse_tree(40, seed=1)), (2, gen.chain_tree(6))):
        # drafts that follow the target's own greedy tokens for a while, so that accept_len > 0
        k = len(gen.main_path(parent)) - 1
        greedy, tok = [], 5
        for _ in range(k):
            kv.verify(torch.tensor([tok], dtype=torch.int32, device="cuda"), torch.tensor([-1], dtype=torch.int32, device="cuda"))
            kv.commit()
            tok = int(kv.out_bonus.item())
            greedy.append(tok)
        kv.truncate(L)
        tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=seed, root_token=5, main_tokens=greedy, corrupt_p=0.2)
        logits, want = _verify(cfg, kv, tokens, parent)
        n = len(tokens)
        outs = (torch.full((n,), -7, dtype=torch.int32, device="cuda"), torch.full((1,), -7, dtype=torch.int32, device="cuda"),
                torch.full((n,), -7, dtype=torch.int32, device="cuda"), torch.full((1,), -7, dtype=torch.int32, device="cuda"))
        cases.append((tokens, parent, logits, want, outs))
    for tokens, parent, logits, want, outs in cases:          # two calls in a row on the shared array
        d_tok, d_par = torch.from_numpy(tokens).cuda(), torch.from_numpy(parent).cuda()
        B.specasr_accept_logits_static(logits.data_ptr(), cfg.vocab, d_tok.data_ptr(), d_par.data_ptr(), len(tokens),
                                       outs[0].data_ptr(), outs[1].data_ptr(), outs[2].data_ptr(), outs[3].data_ptr(), stream)
    torch.cuda.synchronize()
    for tokens, parent, logits, want, outs in cases:
        for got, ref in zip(outs, want):
            assert torch.equal(got, ref)
        # and against the oracle's accept rule applied to the arg-max of the very same logits (integer work: exact)
        am = logits.cpu().numpy().argmax(-1)
        ref = O.accept(tokens, parent, am)
        n, a = len(tokens), ref["accept_len"]
        assert np.array_equal(outs[0].cpu().numpy(), am)
        assert int(outs[1].item()) == a and int(outs[3].item()) == ref["bonus"]
        path = outs[2].cpu().numpy()
        assert list(path[:a + 1]) == list(ref["path"]) and np.all(path[a + 1:] == -1)
    assert int(cases[0][3][1].item()) >= 0
    # a tree larger than the built-in array is refused on the host, with a message that names the limit
    with pytest.raises(B.SpecasrError) as e:
        B.specasr_accept_logits_static(cases[0][2].data_ptr(), cfg.vocab, 1, 1, B.SPECASR_MAX_NODES + 1, 1, 1, 1, 0, stream)
    assert e.value.status == B.SPECASR_ERR_INVALID_ARG and "scratch" in str(e.value)
    # a malformed tree is reported through the outputs
    bad = torch.tensor([-1, 0, 5, 1], dtype=torch.int32, device="cuda")
    t4 = torch.zeros(4, dtype=torch.int32, device="cuda")
    o = [torch.zeros(4, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda"),
         torch.zeros(4, dtype=torch.int32, device="cuda")]
    B.specasr_accept_logits_static(cases[0][2].data_ptr(), cfg.vocab, t4.data_ptr(), bad.data_ptr(), 4, o[0].data_ptr(),
                                   o[1].data_ptr(), o[2].data_ptr(), 0, stream)
    torch.cuda.synchronize()
    assert int(o[1].item()) == -1 and bool((o[2] == -1).all())
