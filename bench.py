#!/usr/bin/env python
"""Benchmark of the tree-verification step (verify + commit) on the 7B-shape, 64-node workload.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload config3]

One step = one pass of the whole hot path: tree prep, embedding, 32 decoder layers over the tree
(projections, rotary + KV append, tree attention, SwiGLU), vocabulary projection + argmax, accept,
KV compaction.  Prints ONE JSON line on rank 0.  With --gpus N > 1 (under torchrun) every rank runs
an independent replica (the path does not shard) and the value is the sum over ranks divided by the
slowest rank's time.  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import gen  # noqa: E402

WORKLOADS = {
    # name: (model, n_audio, n_text (decoded tokens incl. the root), n_nodes, tree kind, page size)
    "config3": dict(model="7b", n_audio=1500, n_text=201, n_nodes=64, levels=12, chain=False),
    "config2": dict(model="1b", n_audio=750, n_text=33, n_nodes=9, levels=None, chain=True),
    "config1": dict(model="tiny", n_audio=64, n_text=8, n_nodes=15, levels=None, chain=False),
    # config3 cut to two layers: same kernels and launch shapes, small enough for a profiler capture
    "config3_2layers": dict(model="7b", n_layers=2, n_audio=1500, n_text=201, n_nodes=64, levels=12, chain=False),
    "config4_kv2048": dict(model="7b", n_audio=1848, n_text=201, n_nodes=64, levels=12, chain=False),
    "config4_n16": dict(model="7b", n_audio=1500, n_text=201, n_nodes=16, levels=None, chain=False),
    "config3_4layers": dict(model="7b", n_layers=4, n_audio=1500, n_text=201, n_nodes=64, levels=12, chain=False),
    # the 13B-class shape as a second target (same tree and context as config 3)
    "config3_13b": dict(model="13b", n_audio=1500, n_text=201, n_nodes=64, levels=12, chain=False),
    # a 256-node point of the config 4 sweep cut to two layers, for a profiler capture of the large-tree regime
    "config4_n256_2layers": dict(model="7b", n_layers=2, n_audio=1500, n_text=201, n_nodes=256, levels=None, chain=False),
}
METRIC = "tree_tokens_per_s"
UNIT = "tree tokens/s"


def workload_keys(wl):
    """The workload's parameters for the JSON line (the decoder shape is named `decoder_shape`)."""
    return {("decoder_shape" if k == "model" else k): v for k, v in wl.items()}


def model_config(wl):
    over = {"n_layers": wl["n_layers"]} if "n_layers" in wl else {}
    return gen.get_config(wl["model"], **over)


def algorithmic_bytes(cfg, L, n):
    w = 2 * (cfg.n_layers * (cfg.d_model * (cfg.q_dim + 2 * cfg.kv_dim) + cfg.q_dim * cfg.d_model
                             + 3 * cfg.d_model * cfg.ffn) + cfg.d_model * cfg.vocab)
    kv_row = cfg.n_layers * 2 * cfg.n_kv_heads * cfg.head_dim * 4          # K and V, hi + lo bf16 planes
    return {"weights": w, "kv_read": (L + n) * kv_row, "kv_write": n * kv_row,
            "total": w + (L + 2 * n) * kv_row}


def gemm_weight_bytes(cfg):
    d, F = cfg.d_model, cfg.ffn
    return {"gemm_qkv": 2 * d * (cfg.q_dim + 2 * cfg.kv_dim), "gemm_o": 2 * cfg.q_dim * d, "gemm_gu": 4 * d * F,
            "gemm_down": 2 * d * F, "gemm_lm": 2 * d * cfg.vocab}


def algorithmic_flops(cfg, L, n):
    params = cfg.n_layers * (cfg.d_model * (cfg.q_dim + 2 * cfg.kv_dim) + cfg.q_dim * cfg.d_model
                             + 3 * cfg.d_model * cfg.ffn) + cfg.d_model * cfg.vocab
    return 2 * n * params + 4 * n * cfg.q_dim * (L + n) * cfg.n_layers


# DRAM traffic (read + write) of one launch of the fused layer-stack kernel from the ncu captures summarised in
# profiles/k_stack_config3.md: the 2-layer and the 4-layer cut of config 3 (7B shape, 64 tokens, KV 1700).  Traffic
# grows by a fixed amount per layer, so a full launch is the 2-layer figure plus (layers - 2) times the per-layer
# difference.  Valid only for the kernel source it was taken on.
STACK_TRAFFIC_MB = {"cut2": 1252.6, "cut4": 2228.0}
STACK_TRAFFIC_SOURCE_SHA256 = {
    "fused_stack.cu": "077073dfca1a59de599181e079301eaf000d98cb0b6fb51e392c4d8b4cd71ab5",
    "sm100_ptx.cuh": "f811f56641d5fa39c0c575ce57fecebd5da4265ce577e5678d955814594e3f4d",
    "device_utils.cuh": "a35abef135a039a872df2c3961d941f9636495b6918adef1293a236f9905c175",
}


def stack_traffic_per_launch(wl, cfg):
    """DRAM bytes of one fused-stack launch from the committed captures, or None when they do not describe this run
    (another shape, or the kernel source changed since)."""
    import hashlib
    if wl.get("model") != "7b" or wl.get("n_nodes") != 64 or STACK_TRAFFIC_MB["cut2"] is None:
        return None
    for name, want in STACK_TRAFFIC_SOURCE_SHA256.items():
        path = os.path.join(ROOT, "paper_2507_18181_b200", "csrc", name)
        if not os.path.exists(path) or hashlib.sha256(open(path, "rb").read()).hexdigest() != want:
            return None
    per_layer = (STACK_TRAFFIC_MB["cut4"] - STACK_TRAFFIC_MB["cut2"]) / 2.0
    return (STACK_TRAFFIC_MB["cut2"] + (cfg.n_layers - 2) * per_layer) * 1e6


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        rows = [r.strip().split(", ") for r in open(self.file.name) if r.strip()]
        os.unlink(self.file.name)
        rows = [r for r in rows if len(r) == 6 and r[0].replace(".", "").isdigit()]
        if rows:
            out["sm_mhz"] = float(np.median([float(r[0]) for r in rows]))
            out["sm_max_mhz"] = float(rows[0][1])
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            out["reasons"] = [nm for j, nm in enumerate(names) if any(r[2 + j].strip() == "Active" for r in rows)]
            out["samples"] = len(rows)
        return out


# ------------------------------------------------------------------------------------------------ CPU oracle leg

class _DictStore:
    def __init__(self, layers, glob):
        self._layers, self._glob = layers, glob

    def layer(self, l):
        return self._layers[l]

    def globals(self):
        return self._glob


def oracle_sample(wl, seed=1):
    """Bounded sample of the workload for the CPU oracle: the oracle's own steps of the same verify
    call (same tree, same KV length, same shapes) run over ONE of the model's layers plus the embedding
    and vocabulary projection, each part timed; the full call is extrapolated as
    t_globals + n_layers * t_layer + t_head.  Returns a closure that runs the sample once and returns
    (extrapolated seconds per full call, seconds actually timed)."""
    from oracle import specasr_oracle as O
    cfg_full = model_config(wl)
    cfg = gen.get_config(wl["model"], n_layers=1)
    store = gen.WeightStore(cfg_full, seed)
    layers = [store.layer(0)]
    glob = store.globals()
    L = wl["n_audio"] + wl["n_text"] - 1
    n = wl["n_nodes"]
    parent = gen.chain_tree(n - 1) if wl["chain"] else gen.sparse_tree(n, seed=seed, levels=wl["levels"])
    tokens = gen.fill_tree_tokens(parent, cfg_full.vocab, seed=seed, root_token=1)
    rng = np.random.default_rng(seed)
    cache = O.KVCache(cfg)
    cache.K = [rng.standard_normal((L, cfg.n_kv_heads, cfg.head_dim))]
    cache.V = [rng.standard_normal((L, cfg.n_kv_heads, cfg.head_dim))]

    def run_once():
        W = O.Weights(_DictStore(layers, glob))          # fresh: nothing widened ahead of the timed call
        t0 = time.perf_counter()
        depth, anc = O.tree_prep(parent)
        x = O.embed(W, tokens)                           # widens embedding, vocabulary matrix, final gain
        t1 = time.perf_counter()
        hidden, _, _ = O.decoder_stack(cfg, W, x, cache.length + depth, anc, cache)
        t2 = time.perf_counter()
        logits = O.lm_logits(cfg, W, hidden)
        O.accept(tokens, parent, np.argmax(logits, axis=-1))
        t3 = time.perf_counter()
        return (t1 - t0) + cfg_full.n_layers * (t2 - t1) + (t3 - t2), t3 - t0

    desc = (f"oracle steps of verify_tree on the {wl['model']} shape, {n}-node tree, KV length {L} (seeded N(0,1) "
            f"K/V): embedding + 1 of {cfg_full.n_layers} layers + vocabulary projection + accept, full call = "
            f"t_embed + {cfg_full.n_layers} * t_layer + t_head")
    return run_once, desc


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    run_once, desc = oracle_sample(wl)
    for _ in range(args.warmup):
        run_once()
    runs = [run_once() for _ in range(args.steps)]
    per_call = float(np.mean([r[0] for r in runs]))
    timed = float(np.mean([r[1] for r in runs]))
    n = wl["n_nodes"]
    cores = len(os.sched_getaffinity(0))
    value = n / per_call
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_call * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, **workload_keys(wl)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                         "extrapolated": True, "timed_seconds_per_step": timed},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ CUDA leg

def in_flow_times(kv, step, kind_names):
    """Where the time of one step goes, from the library's device-side trace.  Worker thread 0 of every CTA of the
    fused layer-stack kernel writes one record per step of the stack {kind | (layer + 1) << 8, start, end, wait end};
    the other kernels (tree prep, embedding, accept) write one record per block.  A step of the stack is charged the
    time from the moment the last CTA finished the step before it to the moment the last CTA finished this one.
    Returns {name: {"launches": occurrences, "us_per_step": total}} or None if nothing was recorded."""
    import torch
    n_sm = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count
    rec = kv.trace(step, capacity=1 << 18)
    if len(rec) == 0:
        return None
    kind = rec[:, 0] & 0xFF
    layer = (rec[:, 0] >> 8).astype(np.int64) - 1
    groups = []                                  # [name, first start, last end]
    plain = rec[layer < 0]
    for k in sorted(set(int(x) for x in plain[:, 0] & 0xFF)):
        r = plain[(plain[:, 0] & 0xFF) == k]
        groups.append([kind_names[k], int(r[:, 1].min()), int(r[:, 2].max())])
    stack = rec[layer >= 0]
    for l in sorted(set(int(x) for x in layer[layer >= 0])):
        for k in sorted(set(int(x) for x in (stack[:, 0] & 0xFF)[((stack[:, 0] >> 8) - 1) == l])):
            r = stack[((stack[:, 0] & 0xFF) == k) & (((stack[:, 0] >> 8) - 1) == l)]
            r = r[np.argsort(r[:, 1], kind="stable")]
            name = kind_names[k]
            if name == "norm" and len(r) > n_sm:     # two norms per layer: the earlier half is the attention norm
                h = len(r) // 2
                groups.append(["norm", int(r[:h, 1].min()), int(r[:h, 2].max())])
                r = r[h:]
            groups.append([name, int(r[:, 1].min()), int(r[:, 2].max())])
    groups.sort(key=lambda g: g[2])
    out = {}
    latest = min(g[1] for g in groups)
    for name, _, end in groups:
        d = out.setdefault(name, {"launches": 0, "us_per_step": 0.0})
        d["launches"] += 1
        d["us_per_step"] += max(0, end - latest) / 1e3
        latest = max(latest, end)
    return out


def run_in_flow(args, wl):
    """Child mode (--in-flow, with SPECASR_TRACE_LIB=1): one traced step of the workload, result as a JSON line."""
    import torch
    from paper_2507_18181_b200 import binding as B
    device = "cuda:0"
    torch.cuda.set_device(0)
    cfg, model, kv, L, tokens, parent = build_workload(wl, device)
    d_tokens, d_parent = torch.from_numpy(tokens).to(device), torch.from_numpy(parent).to(device)

    def step():
        kv.verify(d_tokens, d_parent)
        kv.commit()
        kv.truncate(L)

    for _ in range(5):
        step()
    print(json.dumps({"in_flow": in_flow_times(kv, step, B.KIND_NAMES)}))


def in_flow_from_child(args):
    """The device-side trace lives in a build variant of the library (it costs ~2 % even when off), so the traced
    step runs in a child process that loads that variant."""
    env = dict(os.environ, SPECASR_TRACE_LIB="1")
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        env.pop(k, None)
    try:
        res = subprocess.run([sys.executable, os.path.abspath(__file__), "--workload", args.workload, "--in-flow"],
                             env=env, capture_output=True, text=True, timeout=600)
        lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
        return json.loads(lines[-1])["in_flow"] if res.returncode == 0 and lines else None
    except Exception:
        return None


def slowest_rank(elapsed, world, device):
    """Replicas do not exchange data: the job's time is the slowest rank's (max over ranks)."""
    if world <= 1:
        return float(elapsed)
    import torch
    import torch.distributed as dist
    t = torch.tensor([elapsed], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_step, steps, world, elapsed_s):
    """Aggregate throughput of `world` independent replicas that each did `steps` steps in `elapsed_s`."""
    return world * units_per_rank_step * steps / elapsed_s


def build_workload(wl, device, seed=1):
    import torch
    from paper_2507_18181_b200 import build as _build
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    from paper_2507_18181_b200 import binding as _binding
    _build.build(trace=_binding.TRACE_LIB)
    cfg = model_config(wl)
    store = gen.WeightStore(cfg, seed)
    model = DeviceModel(cfg, store, device=device)
    L = wl["n_audio"] + wl["n_text"] - 1
    n = wl["n_nodes"]
    kv = DeviceKV(model, max_tokens=L + n + 64, max_nodes=max(n, 16))
    audio = gen.audio_prefix(wl["n_audio"], cfg.d_model, seed)
    text = gen.prompt_tokens(wl["n_text"], cfg.vocab, seed)
    kv.prefill_embeds(torch.from_numpy(audio).to(device))
    kv.prefill_tokens(torch.from_numpy(text[:-1].copy()).to(device))
    assert kv.length() == L
    root = int(text[-1])
    parent = gen.chain_tree(n - 1) if wl["chain"] else gen.sparse_tree(n, seed=seed, levels=wl["levels"])
    # the target's own greedy continuation (input construction: autoregressive single-node rounds)
    k = len(gen.main_path(parent)) - 1
    greedy = []
    tok = root
    one_p = torch.tensor([-1], dtype=torch.int32, device=device)
    for _ in range(k):
        kv.verify(torch.tensor([tok], dtype=torch.int32, device=device), one_p)
        kv.commit()
        tok = int(kv.out_bonus.item())
        greedy.append(tok)
    kv.truncate(L)
    tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=seed, root_token=root, main_tokens=greedy, corrupt_p=0.2)
    return cfg, model, kv, L, tokens, parent


def run_ours(args, wl):
    import torch
    from paper_2507_18181_b200 import binding as B
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: there is no CPU fallback for the verification path")
    device = f"cuda:{local}"
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(device))
    cfg, model, kv, L, tokens, parent = build_workload(wl, device)
    n = len(tokens)
    d_tokens = torch.from_numpy(tokens).to(device)
    d_parent = torch.from_numpy(parent).to(device)
    stream = torch.cuda.current_stream()

    def step():
        kv.verify(d_tokens, d_parent)
        kv.commit()
        kv.truncate(L)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    launches0 = kv.launches()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_events = []
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        step()
        b.record(stream)
        step_events.append((a, b))
    e1.record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else {}
    elapsed_ms = e0.elapsed_time(e1)
    launches = kv.launches() - launches0
    per_step = sorted(a.elapsed_time(b) for a, b in step_events)
    accept_len = int(kv.out_accept.item())
    elapsed_ms = slowest_rank(elapsed_ms, world, device)

    # end to end through the C ABI with host buffers: H2D of the tree, D2H of the results, every step
    h_tokens = torch.from_numpy(tokens).pin_memory()
    h_parent = torch.from_numpy(parent).pin_memory()
    h_out = torch.empty(2 * n + 2, dtype=torch.int32).pin_memory()
    dd_tokens, dd_parent = torch.empty_like(d_tokens), torch.empty_like(d_parent)

    def e2e_step():
        dd_tokens.copy_(h_tokens, non_blocking=True)
        dd_parent.copy_(h_parent, non_blocking=True)
        kv.verify(dd_tokens, dd_parent)
        kv.commit()
        h_out[:n].copy_(kv.out_argmax[:n], non_blocking=True)
        h_out[n:2 * n].copy_(kv.out_path[:n], non_blocking=True)
        h_out[2 * n:2 * n + 1].copy_(kv.out_accept, non_blocking=True)
        h_out[2 * n + 1:].copy_(kv.out_bonus, non_blocking=True)
        torch.cuda.synchronize()          # the caller needs accept_len and the bonus token to go on
        kv.truncate(L)

    for _ in range(3):
        e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        e2e_step()
    barrier()
    e2e_s = time.perf_counter() - t0
    e2e_s = slowest_rank(e2e_s, world, device)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # per-kernel times with events around every launch (separate pass, same steps)
    B.specasr_profile_enable(kv.handle, 1)
    prof_steps = min(args.steps, 10)
    for _ in range(prof_steps):
        step()
    ms, cnt = B.specasr_profile_read(kv.handle, stream.cuda_stream)
    B.specasr_profile_enable(kv.handle, 0)
    kernels = {k: {"launches_per_step": cnt[k] / prof_steps, "ms_per_step": ms[k] / prof_steps} for k in ms if cnt[k]}
    in_flow = in_flow_from_child(args) if world == 1 and not args.no_in_flow else None
    gb = gemm_weight_bytes(cfg)
    gemm_bytes_step = cfg.n_layers * (gb["gemm_qkv"] + gb["gemm_o"] + gb["gemm_gu"] + gb["gemm_down"]) + gb["gemm_lm"]
    peaks = measured_peaks()
    ab = algorithmic_bytes(cfg, L, n)
    if cnt.get("stack"):
        # the whole layer stack is one persistent kernel: its algorithmic bytes are the weights it streams plus the
        # cache rows it reads and writes, i.e. those of the step
        dom = {"kernel": "k_stack (fused layer stack: norms, projections, rotary, attention, arg-max)",
               "bytes": ab["total"], "ms": ms["stack"] / cnt["stack"], "traffic": stack_traffic_per_launch(wl, cfg)}
    else:
        gemm_ms = sum(ms[k] for k in gb)
        gemm_n = sum(cnt[k] for k in gb)
        dom = {"kernel": "k_proj (all projections)", "bytes": gemm_bytes_step * prof_steps / gemm_n,
               "ms": gemm_ms / gemm_n, "traffic": None}
        for k in gb:
            per = gb[k] * (cfg.n_layers if k != "gemm_lm" else 1)
            kernels[k]["achieved_gbs"] = per / (ms[k] / prof_steps * 1e-3) / 1e9
    achieved = dom["bytes"] / (dom["ms"] * 1e-3) / 1e9

    ms_per_step = elapsed_ms / args.steps
    value = whole_job_rate(n, args.steps, world, elapsed_ms * 1e-3)
    fl = algorithmic_flops(cfg, L, n)
    t_roof_ms = max(ab["total"] / (peaks["hbm_gbs"] * 1e9), fl / (peaks["bf16_tflops"] * 1e12)) * 1e3
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, **workload_keys(wl), "kv_len": L, "page_size": model.page_size,
                   "kv_storage": "bf16 hi+lo planes (4 bytes/element)", "l2": "inputs larger than L2 (weights "
                   f"{ab['weights'] / 1e9:.2f} GB per step)", "parallelism": "replicas" if world > 1 else "single"},
        "latency_ms": {"mean": ms_per_step, "median": per_step[len(per_step) // 2], "min": per_step[0]},
        "accept_len": accept_len, "accepted_tokens_per_s": world * (accept_len + 1) * args.steps / (elapsed_ms * 1e-3),
        "step_roofline": {"algorithmic_bytes": ab["total"], "algorithmic_flops": fl, "roof_ms": t_roof_ms,
                          "frac_of_" + peaks["source"]: t_roof_ms / ms_per_step,
                          "frac_of_nominal_8TBs": (ab["total"] / 8e12 * 1e3) / ms_per_step},
        "roofline": {"kernel": dom["kernel"], "bound": "hbm", "achieved": achieved,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                     "peak_source": peaks["source"], "traffic": dom["traffic"],
                     "algorithmic_bytes_per_launch": dom["bytes"], "avg_launch_ms": dom["ms"]},
        "kernels": kernels,
        "in_flow": None,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "e2e": {"value": world * n * args.steps / e2e_s, "unit": UNIT, "ms_per_step": e2e_s / args.steps * 1e3,
                "h2d_bytes_per_step": int(2 * n * 4), "d2h_bytes_per_step": int((2 * n + 2) * 4)},
    }
    if in_flow:
        gemm_us = sum(in_flow[k]["us_per_step"] for k in gb if k in in_flow)
        line["in_flow"] = {
            "how": "one extra step with the device-side trace on: every step of the fused layer stack (and every other "
                   "kernel) is charged the time from the end of the step before it on its last CTA to its own end "
                   "on its last CTA (%globaltimer)",
            "us_per_launch": {k: round(v["us_per_step"] / v["launches"], 2) for k, v in in_flow.items()},
            "projections": {"us_per_step": gemm_us, "achieved_gbs": gemm_bytes_step / (gemm_us * 1e-6) / 1e9,
                            "frac_of_" + peaks["source"]: gemm_bytes_step / (gemm_us * 1e-6) / 1e9 / peaks["hbm_gbs"]},
        }
    if world == 1 and not args.no_cpu_baseline:
        run_once, desc = oracle_sample(wl)
        run_once()
        reps, t_start, runs = 0, time.perf_counter(), []
        while reps < 3 and time.perf_counter() - t_start < 25:
            runs.append(run_once())
            reps += 1
        per_call = float(np.mean([r[0] for r in runs]))
        line["cpu_baseline"] = {"value": n / per_call, "unit": UNIT, "cores": len(os.sched_getaffinity(0)),
                                "kind": "oracle", "sample": desc, "ms_per_step": per_call * 1e3, "extrapolated": True,
                                "timed_seconds_per_step": float(np.mean([r[1] for r in runs]))}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Verify-cost sweep (draft / target latency balance): the 7B shape, chain drafts of 4 / 8 / 16 / 32 tokens and
    sparse trees of 16 / 64 / 256 nodes at KV lengths 512 .. 4096.  One JSON line per point, the model is built
    once.  Latency is the CUDA-event time of verify + commit (+ length reset) averaged over --steps rounds."""
    import torch
    from paper_2507_18181_b200 import build as _build
    from paper_2507_18181_b200.runtime import DeviceModel, DeviceKV
    _build.build()
    device = "cuda:0"
    torch.cuda.set_device(0)
    seed = 1
    cfg = gen.get_config("7b")
    model = DeviceModel(cfg, gen.WeightStore(cfg, seed), device=device)
    peaks = measured_peaks()
    stream = torch.cuda.current_stream()
    shapes = [("chain", k + 1) for k in (4, 8, 16, 32)] + [("tree", n) for n in (16, 64, 256)]
    for L in (512, 1024, 2048, 4096):
        kv = DeviceKV(model, max_tokens=L + 256 + 64, max_nodes=256)
        n_text = 200
        kv.prefill_embeds(torch.from_numpy(gen.audio_prefix(L - n_text + 1, cfg.d_model, seed)).to(device))
        text = gen.prompt_tokens(n_text, cfg.vocab, seed)
        kv.prefill_tokens(torch.from_numpy(text[:-1].copy()).to(device))
        assert kv.length() == L
        root = int(text[-1])
        one_p = torch.tensor([-1], dtype=torch.int32, device=device)
        greedy, tok = [], root
        for _ in range(32):
            kv.verify(torch.tensor([tok], dtype=torch.int32, device=device), one_p)
            kv.commit()
            tok = int(kv.out_bonus.item())
            greedy.append(tok)
        kv.truncate(L)
        for kind, n in shapes:
            parent = gen.chain_tree(n - 1) if kind == "chain" else gen.sparse_tree(n, seed=seed)
            tokens = gen.fill_tree_tokens(parent, cfg.vocab, seed=seed, root_token=root, main_tokens=greedy, corrupt_p=0.2)
            d_tokens, d_parent = torch.from_numpy(tokens).to(device), torch.from_numpy(parent).to(device)

            def step():
                kv.verify(d_tokens, d_parent)
                kv.commit()
                kv.truncate(L)

            for _ in range(max(args.warmup, 3)):
                step()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.steps):
                step()
            e1.record(stream)
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1) / args.steps
            ab, fl = algorithmic_bytes(cfg, L, n), algorithmic_flops(cfg, L, n)
            t_hbm = ab["total"] / (peaks["hbm_gbs"] * 1e9) * 1e3
            t_tc = fl / (peaks["bf16_tflops"] * 1e12) * 1e3
            print(json.dumps({
                "workload": f"config4 {kind} n_nodes={n} kv_len={L}", "ms_per_step": ms, "tree_tokens_per_s": n / (ms * 1e-3),
                "accept_len": int(kv.out_accept.item()), "algorithmic_bytes": ab["total"], "algorithmic_flops": fl,
                "roof_ms": max(t_hbm, t_tc), "bound": "hbm" if t_hbm >= t_tc else "tensor",
                "frac_of_" + peaks["source"]: max(t_hbm, t_tc) / ms,
                "frac_of_nominal_8TBs": (ab["total"] / 8e12 * 1e3) / ms}), flush=True)
        kv.close()
        del kv
        torch.cuda.empty_cache()


def run_loop(args):
    """Config 5: the batched draft-then-verify loop end to end.  8 utterances with audio prefixes of 300..1500
    frames decode 200 tokens each: per round the 0.5B-shape draft model is stepped autoregressively (all
    utterances per step in one batched call), the 7B-shape target verifies one 32-node sparse tree per utterance
    in one batched call, accepted paths are committed, and accept lengths / bonus tokens go back to the host.
    Proposals are the target's greedy transcript (computed beforehand, untimed, by the library itself running
    autoregressively) corrupted per position with p = 0.2, with the tail past a rejection recycled.  A step is
    one full decode of the batch; the transcript of every step is checked token for token against the
    autoregressive one.  One JSON line: emitted tokens per second, host control and copies included."""
    import torch
    from paper_2507_18181_b200 import build as _build
    from paper_2507_18181_b200.loop import SpeculativeBatchLoop
    from paper_2507_18181_b200.runtime import BatchVerifier, DeviceModel, DeviceKV
    _build.build()
    device = "cuda:0"
    torch.cuda.set_device(0)
    seed, B, n_tokens, n_nodes, k_max, n_prompt = 1, 8, 200, 32, 16, 8
    small = args.workload == "config5_small"       # same loop on 2-layer cuts, for a quick functional run
    cfg = gen.get_config("7b", **({"n_layers": 2} if small else {}))
    dcfg = gen.get_config("0.5b", **({"n_layers": 2} if small else {}))
    target = DeviceModel(cfg, gen.WeightStore(cfg, seed), device=device)
    draft = DeviceModel(dcfg, gen.WeightStore(dcfg, seed + 1), device=device)
    frames = np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, 0x5E55]))).integers(300, 1501, size=B)
    margin = n_tokens + 2 * k_max + n_nodes + 64
    need = n_tokens + 2 * k_max + 2
    min_gap = 3e-4
    kvs, dkvs, roots, L0, truth, redrawn = [], [], [], [], [], 0
    one_p = torch.tensor([-1], dtype=torch.int32, device=device)
    logits = torch.empty(1, cfg.vocab, dtype=torch.float32, device=device)
    utt = 0
    while len(kvs) < B:
        # the target's autoregressive greedy transcript of this utterance (input construction and the reference
        # of the check).  Token-for-token equality is only defined away from ties (two computation orders of
        # the same fp32 sums differ by ~1e-5 in a logit), so an utterance whose transcript has a top-2 logit
        # gap below min_gap anywhere is redrawn.
        b = len(kvs)
        prompt = gen.prompt_tokens(n_prompt, cfg.vocab, seed, utterance=utt)
        kv = DeviceKV(target, max_tokens=int(frames[b]) + n_prompt + margin, max_nodes=B * n_nodes)
        kv.prefill_embeds(torch.from_numpy(gen.audio_prefix(int(frames[b]), cfg.d_model, seed, utterance=utt)).to(device))
        kv.prefill_tokens(torch.from_numpy(prompt[:-1].copy()).to(device))
        L = int(frames[b]) + n_prompt - 1
        tok, seq, gap = int(prompt[-1]), [], float("inf")
        for _ in range(need):
            kv.verify(torch.tensor([tok], dtype=torch.int32, device=device), one_p, logits)
            kv.commit()
            top = torch.topk(logits[0], 2).values
            gap = min(gap, float(top[0] - top[1]))
            tok = int(kv.out_bonus.item())
            seq.append(tok)
            if gap < min_gap:
                break
        if gap < min_gap:
            redrawn += 1
            utt += 1
            kv.close()
            continue
        kv.truncate(L)
        dkv = DeviceKV(draft, max_tokens=int(frames[b]) + n_prompt + margin, max_nodes=B * n_nodes)
        dkv.prefill_embeds(torch.from_numpy(gen.audio_prefix(int(frames[b]), dcfg.d_model, seed, utterance=utt)).to(device))
        dkv.prefill_tokens(torch.from_numpy(prompt[:-1].copy()).to(device))
        kvs.append(kv)
        dkvs.append(dkv)
        roots.append(int(prompt[-1]))
        L0.append(L)
        truth.append(seq)
        utt += 1
    # batched one-token-per-step decoding with the same library, as the autoregressive baseline of the loop
    bv = BatchVerifier(kvs)
    toks = torch.tensor(roots, dtype=torch.int32, device=device)
    minus = torch.full((B,), -1, dtype=torch.int32, device=device)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for _ in range(n_tokens):
        bv.verify(toks, minus, list(range(B + 1)))
        bv.commit()
        toks = bv.out_bonus.clone()
        toks.cpu()
    autoregressive_s = time.perf_counter() - t0

    def reset():
        for b in range(B):
            kvs[b].truncate(L0[b])
            dkvs[b].truncate(L0[b])

    def one_decode():
        reset()
        proposer = gen.CorruptedGreedyProposer(truth, roots, cfg.vocab, seed=seed, n_nodes=n_nodes, k_min=4,
                                               k_max=k_max, corrupt_p=0.2)
        loop = SpeculativeBatchLoop(kvs, dkvs)
        out = loop.decode(roots, n_tokens, proposer)
        torch.cuda.synchronize()
        return loop, out

    warm = max(1, min(args.warmup, 2))
    steps = max(1, min(args.steps, 5))
    for _ in range(warm):
        one_decode()
    launches0 = sum(kv.launches() for kv in kvs + dkvs)
    sampler = ClockSampler(0)
    sampler.start()
    t0 = time.perf_counter()
    for _ in range(steps):
        loop, out = one_decode()
    elapsed = time.perf_counter() - t0
    clocks = sampler.stop()
    launches = sum(kv.launches() for kv in kvs + dkvs) - launches0
    lossless = all(out[b] == truth[b][:n_tokens] for b in range(B))
    per = elapsed / steps
    line = {
        "metric": "end_to_end_tokens_per_s", "value": B * n_tokens / per, "unit": "emitted tokens/s", "n_gpus": 1,
        "steps": steps, "warmup": warm, "ms_per_step": per * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "target": cfg.name, "target_layers": cfg.n_layers, "draft": dcfg.name,
                   "draft_layers": dcfg.n_layers, "utterances": B, "audio_frames": [int(f) for f in frames],
                   "tokens_per_utterance": n_tokens, "tree_nodes": n_nodes, "draft_len": [4, k_max], "corrupt_p": 0.2,
                   "utterances_redrawn_for_near_ties": redrawn, "min_top2_gap": min_gap,
                   "timing": "host wall clock around the whole decode (host control, H2D of trees, D2H of results)"},
        "lossless": lossless, "rounds_per_decode": loop.rounds, "draft_steps_per_decode": loop.draft_steps,
        "tokens_per_tree": sum(len(o) for o in out) / max(1, loop.utterance_rounds),
        "autoregressive_batched_tokens_per_s": B * n_tokens / autoregressive_s,
        "speedup_over_autoregressive": autoregressive_s / per,
        "gpu_launches": int(launches // steps), "clocks": clocks,
    }
    print(json.dumps(line))
    if not lossless:
        for b in range(B):
            d = [i for i in range(n_tokens) if out[b][i] != truth[b][i]]
            if d:
                print(f"utterance {b}: first difference at token {d[0]}: {out[b][d[0]]} vs {truth[b][d[0]]}", file=sys.stderr)
        raise SystemExit("speculative transcript differs from the autoregressive one")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="config3", choices=sorted(WORKLOADS) + ["config5", "config5_small"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="config 4: one JSON line per (draft shape, KV length) point")
    ap.add_argument("--in-flow", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--no-in-flow", action="store_true", help="skip the traced step (it runs in a child process)")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.workload.startswith("config5"):
        if args.impl == "reference" or args.gpus != 1:
            raise SystemExit("config5 runs the CUDA loop on one GPU only")
        run_loop(args)
        return
    wl = WORKLOADS[args.workload]
    if args.in_flow:
        run_in_flow(args, wl)
        return
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
