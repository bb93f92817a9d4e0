#!/usr/bin/env python
"""Benchmark of the streamed layer backward on one B200 (or N independent replicas).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--chunk C] [--impl reference]

A step is one streambp_layer_backward call (K/V prologue, every chunk's re-forward and
backward, all weight gradients) over one synthetic sequence.  Prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "streamed_layer_backward_tokens_per_s"
UNIT = "tokens/s"


def layer_flops(s, T):
    """Algorithmic FLOPs of one streamed layer backward: 6 forward products (no down projection),
    14 backward products, attention (2 forward + 5 backward products) over the causal half."""
    d, dq, dkv, I = s.d_model, s.dq, s.dkv, s.d_ff
    P = d * dq + 2 * d * dkv + dq * d + 3 * d * I
    fwd = 2 * T * (P - d * I)
    bwd = 4 * T * P
    pairs = T * (T + 1) / 2
    att = 7 * 2 * s.head_dim * s.n_q_heads * pairs
    return fwd + bwd + att


def attn_bwd_bytes(s, kv_len, n):
    """Algorithmic DRAM bytes of one attention-backward launch (n queries against kv_len keys): K, V read (storage
    dtype), fp32 dK, dV read and written, Q, dO read, fp32 dQ written, lse / delta read."""
    e = 2
    return kv_len * s.dkv * (2 * e + 2 * 2 * 4) + n * s.dq * (2 * e + 4) + 2 * 4 * n * s.n_q_heads


def attn_fwd_bytes(s, kv_len, n):
    """K, V read, Q read, O written, lse written."""
    e = 2
    return kv_len * s.dkv * 2 * e + n * s.dq * 2 * e + 4 * n * s.n_q_heads


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of ONE captured launch per kernel class, from the ncu
# captures summarised under profiles/ -- (config, chunk, class) -> (bytes, what was captured, algorithmic bytes of
# that launch).  The step's average launch is this figure scaled by the ratio of algorithmic bytes (product launches
# depend on the chunk only; attention launches grow with the key prefix, and their traffic in proportion).
NCU_TRAFFIC = {
    ("qwen7b_layer", 1024, "gemm"): (2142.5e6, "MLP-backward group of a chunk, profiles/gemm_pair_kernel_chunk_products.md", None),
    ("llama8b_layer", 2048, "gemm"): (2421.9e6, "MLP-backward group of a chunk, profiles/gemm_pair_kernel_chunk_products.md", None),
    ("llama8b_layer", 2048, "attention_bwd"): (488.6e6, "2048 queries against a 16384-key prefix, "
                                               "profiles/attention_tc_kernels_llama8b_chunk2048.md", (16384, 2048)),
    ("llama8b_layer", 2048, "attention_fwd"): (88.4e6, "2048 queries against a 16384-key prefix, "
                                               "profiles/attention_tc_kernels_llama8b_chunk2048.md", (16384, 2048)),
}


def class_traffic(cfg, chunk, cls):
    """(bytes per average launch or None, note).  Never silently None: the note says why a figure is absent."""
    rec = NCU_TRAFFIC.get((cfg.name, chunk, cls))
    if rec is None:
        return None, f"no ncu capture of the {cls} class at ({cfg.name}, chunk {chunk}) under profiles/"
    nbytes, what, at = rec
    if at is None:
        return nbytes, f"dram bytes under ncu of: {what}"
    s, T = cfg.layer, cfg.T
    fn = attn_bwd_bytes if cls == "attention_bwd" else attn_fwd_bytes
    ends = [min(T, r0 + chunk) for r0 in range(0, T, chunk)]
    avg = sum(fn(s, e, min(chunk, e)) for e in ends) / len(ends)
    return nbytes * avg / fn(s, at[0], at[1]), (f"dram bytes under ncu of: {what}; scaled to the step's average launch "
                                                 f"by algorithmic bytes ({avg / fn(s, at[0], at[1]):.3f}x)")


CLASS_NAMES = {"gemm": "linear products (gemm_pair_kernel, all GEMM launches of the step)",
               "attention_fwd": "partitioned attention forward (attn_fwd_2q_kernel / attn_fwd_tc16_kernel)",
               "attention_bwd": "partitioned attention backward (attn_bwd_tc_kernel)"}


def roofline_object(prof, steps, peaks, cfg, chunk, profiled_ms, flops_scale=1.0):
    """The roofline entry is the kernel class that takes the largest share of the step that was actually run; the
    other classes ride along with their own achieved rate and fraction.  All three are tensor-core bound (dense
    contractions); the denominator is the measured sustained bf16 peak (kernels timed inside a long step)."""
    peak = peaks["sustained"]
    classes = {}
    for k, (ms, calls, fl) in prof.items():
        fl *= flops_scale
        tf = fl / (ms * 1e-3) / 1e12 if ms > 0 else 0.0
        classes[k] = {"ms_per_step": ms / steps, "launches_per_step": calls / steps, "tflops": tf, "frac": tf / peak,
                      "frac_of_burst": tf / peaks["burst"], "frac_of_nominal_2250": tf / 2250.0}
    dom = max(classes, key=lambda k: classes[k]["ms_per_step"])
    traffic, note = class_traffic(cfg, chunk, dom) if cfg.layer is not None and not cfg.n_layers else \
        (None, "no ncu capture of this workload's launches under profiles/ (captures are made on the layer workloads)")
    return dom, classes, {
        "bound": "tensor", "kernel": CLASS_NAMES[dom], "class": dom, "achieved": classes[dom]["tflops"], "peak": peak,
        "unit": "TFLOP/s", "frac": classes[dom]["frac"], "peak_source": peaks["source"] + " sustained bf16",
        "traffic": traffic, "traffic_note": note,
        "launches": int(prof[dom][1]), "ms_per_step": classes[dom]["ms_per_step"],
        "algorithmic_flops_per_launch": prof[dom][2] * flops_scale / max(1, prof[dom][1]),
        "timed": "a second run of the same K steps with CUDA events around every launch of the class",
        "step_ms_with_events": profiled_ms / steps,
        "classes": {k: {"achieved": v["tflops"], "frac": v["frac"], "ms_per_step": v["ms_per_step"]} for k, v in classes.items()},
    }


def check_outputs(tensors) -> str:
    """After the warm-up steps, outside any timed region: every output tensor is finite and not identically zero, so a
    step that skipped its work cannot produce a number.  (Values are checked against the oracle by the tests.)"""
    import torch
    for name, t in tensors.items():
        f = t.float()
        assert bool(torch.isfinite(f).all()), f"bench: output {name} is not finite"
        assert float(f.abs().max()) > 0.0, f"bench: output {name} is identically zero"
    return "finite and non-zero: " + ", ".join(tensors)


def max_over_ranks(ms: float, world: int, device) -> float:
    """Timing rule for N > 1: every rank reports the slowest rank's device time."""
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_seed(base_seed: int, rank: int) -> int:
    """Replicas see different sequences; the weights are the same on every rank."""
    return base_seed + 1000 * rank


def aggregate_tokens_per_s(T: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: tokens all replicas processed in a step / the slowest replica's step time."""
    return world * T / (ms_per_step * 1e-3)


def read_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm=j["hbm_gbs"], burst=j["bf16_tflops"], sustained=j["bf16_tflops_sustained"], source="measured")
    return dict(hbm=6650.0, burst=1590.0, sustained=1400.0, source="fallback")


class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


_ORACLE_INPUTS = {}


def oracle_sample(cfg, T_sample):
    """Times the CPU oracle (as it stands) on the first T_sample tokens of the workload.
    Input generation is outside the timed region."""
    from oracle import streambp_oracle as O
    from paper_2506_03077_b200 import synth
    s = cfg.layer
    key = (cfg.name, T_sample)
    if key not in _ORACLE_INPUTS:
        W = synth.make_layer_weights(s, cfg.seed, cfg.bf16)
        X, dY = synth.make_layer_io(s, cfg.seed, T_sample, cfg.bf16)
        _ORACLE_INPUTS[key] = (W, X, dY)
    W, X, dY = _ORACLE_INPUTS[key]
    oc = O.LayerCfg(s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ff, s.qkv_bias, s.rope_theta, s.rms_eps)
    t0 = time.perf_counter()
    O.layer_backward(oc, W, X, dY)
    return time.perf_counter() - t0


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    T_sample = args.ref_tokens
    for _ in range(args.warmup):
        oracle_sample(cfg, T_sample)
    times = [oracle_sample(cfg, T_sample) for _ in range(args.steps)]
    total = sum(times)
    value = T_sample * args.steps / total
    cores = os.cpu_count()
    sample = (f"first {T_sample} tokens of {cfg.name} (full widths), fp64 numpy oracle, full-sequence backward; a "
              f"{T_sample}-token prefix under-counts the attention term, which is quadratic in T")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "T": cfg.T, "chunk": cfg.chunk, "sample_tokens": T_sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def head_flops(h, T):
    """Three products of 2 T d V each (logits, dH, dW_vocab)."""
    return 3 * 2 * T * h.d_model * h.vocab


def run_head_or_model(args, cfg):
    """Secondary workloads (one JSON line, same keys where they apply): the streamed LM head alone
    (qwen7b_head) and the whole model on layer-input checkpoints (qwen7b_model).  Weights of the model
    workload are drawn on the device (7.6 G parameters), everything else as in the layer workloads."""
    import torch
    from paper_2506_03077_b200 import binding as B
    from paper_2506_03077_b200 import synth
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        raise SystemExit("head / model workloads run on one GPU")
    torch.cuda.set_device(0)
    B.lib()
    dt = torch.bfloat16
    h, T = cfg.head, cfg.T
    hc = B.HeadConfig(h.d_model, h.vocab, h.rms_eps, h.ignore_index, dt)
    gen = torch.Generator(device="cuda").manual_seed(cfg.seed)
    rn = lambda *shape, mean=0.0, std=1.0: (torch.randn(*shape, generator=gen, device="cuda") * std + mean).to(dt)
    loss = torch.zeros(1, device="cuda")
    peaks = read_peaks()
    if cfg.n_layers == 0:
        g, Wv, H, labels = synth.make_head_inputs(h, cfg.seed, T, True, cfg.masked_prefix)
        gd, Wd, Hd = (torch.from_numpy(a).to("cuda", dt) for a in (g, Wv, H))
        ld = torch.from_numpy(labels).cuda()
        nv = torch.zeros(1, dtype=torch.int64, device="cuda")
        dH, dW, dg = torch.empty_like(Hd), torch.empty(h.vocab, h.d_model, device="cuda"), torch.empty(h.d_model, device="cuda")
        ws_bytes = B.lmhead_workspace_bytes(hc, T, cfg.chunk, args.wgrad_group)
        ws_full = B.lmhead_workspace_bytes(hc, T, T)
        ws = B.alloc_workspace(ws_bytes)
        step = lambda: B.lmhead_ce_backward(hc, gd, Wd, Hd, ld, cfg.chunk, loss, nv, dH, dW, dg, ws,
                                            wgrad_group=args.wgrad_group)
        flops, name = head_flops(h, T), "streamed_lmhead_ce_backward_tokens_per_s"
        if args.objective != "sft":
            # synthetic per-token inputs of the RL objectives: behaviour / reference log-probabilities around the
            # ln V of a random-init policy, unit-variance advantages, uniform weights (GRPO) or +-1 signs (DPO)
            n_part = int((labels != h.ignore_index).sum())
            lp0 = -float(__import__("math").log(h.vocab))
            old = torch.from_numpy(synth.normal(cfg.seed, "logp_old", (T,), lp0, 0.3)).cuda()
            ref = torch.from_numpy(synth.normal(cfg.seed, "logp_ref", (T,), lp0, 0.3)).cuda()
            adv = torch.from_numpy(synth.normal(cfg.seed, "advantage", (T,))).cuda()
            if args.objective == "grpo":
                wt = torch.full((T,), 1.0 / n_part, device="cuda")
                obj, beta, eps = B.OBJ_GRPO, 0.04, 0.2
            else:
                half = (T + cfg.masked_prefix) // 2
                wt = torch.where(torch.arange(T, device="cuda") < half, 1.0, -1.0).float()
                obj, beta, eps = B.OBJ_DPO, 0.1, 0.0
            step = lambda: B.lmhead_rl_backward(hc, obj, beta, eps, gd, Wd, Hd, ld, old, ref, adv, wt, cfg.chunk, loss,
                                                dH, dW, dg, ws, wgrad_group=args.wgrad_group)
            name = f"streamed_lmhead_{args.objective}_backward_tokens_per_s"
        H_host, l_host = torch.from_numpy(H).to(dt).pin_memory(), torch.from_numpy(labels).pin_memory()
        dH_host, loss_host = torch.empty_like(H_host).pin_memory(), torch.zeros(1).pin_memory()
        e2e_io = lambda: ([(Hd, H_host), (ld, l_host)], [(dH_host, dH), (loss_host, loss)])
        # chunks (with --wgrad-group, groups of chunks) whose labels are all ignored are skipped on the device (their
        # gradient is exactly zero)
        gate_rows = cfg.chunk * max(1, args.wgrad_group)
        live = sum(min(gate_rows, T - r0) for r0 in range(0, T, gate_rows)
                   if (labels[r0:r0 + gate_rows] != h.ignore_index).any())
        executed_flops = head_flops(h, live)
    else:
        s, L = cfg.layer, cfg.n_layers
        lc = B.LayerConfig(s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ff, s.qkv_bias, s.rope_theta, s.rms_eps, dt)
        shapes = B.layer_grad_shapes(lc)
        layers = [{k: rn(*shp, mean=1.0 if k in ("g1", "g2") else 0.0, std=0.02) for k, shp in shapes.items()}
                  for _ in range(L)]
        grads = [B.alloc_layer_grads(lc) for _ in range(L)]
        E, Wv, gf = rn(h.vocab, h.d_model, std=0.02), rn(h.vocab, h.d_model, std=0.02), rn(h.d_model, mean=1.0, std=0.02)
        ids, labels = synth.make_model_tokens(h.vocab, cfg.seed, T, cfg.prompt_frac)
        idd, ld = torch.from_numpy(ids).cuda(), torch.from_numpy(labels).cuda()
        dE, dWv, dg = torch.empty(h.vocab, h.d_model, device="cuda"), torch.empty(h.vocab, h.d_model, device="cuda"), torch.empty(h.d_model, device="cuda")
        ch = cfg.chunk_head or cfg.chunk
        ws_bytes = B.model_workspace_bytes(L, lc, hc, T, cfg.chunk, ch)
        ws_full = B.model_workspace_bytes(L, lc, hc, T, T, T)
        ws = B.alloc_workspace(ws_bytes)
        step = lambda: B.model_backward(lc, hc, layers, gf, Wv, ld, cfg.chunk, ch, loss, grads, dg, dWv, ws,
                                        embed=E, ids=idd, d_embed=dE)
        id_host, l_host = torch.from_numpy(ids).pin_memory(), torch.from_numpy(labels).pin_memory()
        loss_host = torch.zeros(1).pin_memory()
        e2e_io = lambda: ([(idd, id_host), (ld, l_host)], [(loss_host, loss)])
        P = s.d_model * s.dq + 2 * s.d_model * s.dkv + s.dq * s.d_model + 3 * s.d_model * s.d_ff
        fwd_extra = 2 * T * P + 4 * s.head_dim * s.n_q_heads * T * (T + 1) / 2      # checkpointing forward
        flops = L * (layer_flops(s, T) + fwd_extra) + head_flops(h, T)
        executed_flops = flops
        name = "streamed_model_backward_tokens_per_s"
    for _ in range(args.warmup):
        step()
    assert B.last_device_status(ws) == B.OK
    launches = B.last_launch_count()
    torch.cuda.synchronize()
    checked = check_outputs({"loss": loss, "d_w_vocab": dW if cfg.layer is None else dWv, "d_g_final": dg})
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(0)
    sampler.start()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    # class timing: the same steps again with CUDA events around every product launch
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    B.profile_enable(True)
    p0.record()
    for _ in range(args.steps):
        step()
    p1.record()
    torch.cuda.synchronize()
    prof = {k: B.profile_read(k) for k in B.KERNEL_CLASSES}
    B.profile_enable(False)
    profiled_ms = p0.elapsed_time(p1)
    ms = e0.elapsed_time(e1) / args.steps
    # launches of chunks that are skipped on the device return at once but are still bracketed: count only the
    # executed share of their FLOPs (the head workload has product launches only)
    _, classes, roofline = roofline_object(prof, args.steps, peaks, cfg, cfg.chunk, profiled_ms,
                                           flops_scale=executed_flops / flops if cfg.n_layers == 0 else 1.0)
    out = {
        "metric": name, "value": T / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic", "loss": loss.item(),
        "config": {"workload": cfg.name, "T": T, "chunk": cfg.chunk,
                   "wgrad_group": args.wgrad_group if cfg.n_layers == 0 else 1, "n_layers": cfg.n_layers, "vocab": h.vocab,
                   "l2": "inputs larger than L2", "product_kernel": B.product_kernel()},
        "algorithmic_tflop_per_step": flops / 1e12, "tflops": flops / (ms * 1e-3) / 1e12,
        "frac_of_measured_sustained_bf16": flops / (ms * 1e-3) / 1e12 / peaks["sustained"],
        "executed_tflop_per_step": executed_flops / 1e12,
        "tflops_executed": executed_flops / (ms * 1e-3) / 1e12,
        "frac_of_measured_sustained_bf16_executed": executed_flops / (ms * 1e-3) / 1e12 / peaks["sustained"],
        "peak_activation_gb": ws_bytes / 1e9, "peak_activation_gb_unchunked": ws_full / 1e9,
        "gpu_launches": int(launches * args.steps), "outputs_checked": checked,
        "roofline": roofline, "kernel_classes": classes, "clocks": clocks,
    }
    if not args.no_e2e:
        # the same call fed from pinned host memory: every step copies its inputs in and its result out on the
        # launching stream (serial: nothing overlaps), inside the timed region
        h2d, d2h = e2e_io()
        nb = lambda ts: sum(t.numel() * t.element_size() for _, t in ts)
        def e2e_step():
            for dev, host in h2d:
                dev.copy_(host, non_blocking=True)
            step()
            for host, dev in d2h:
                host.copy_(dev, non_blocking=True)
        e2e_step()
        torch.cuda.synchronize()
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        q0.record()
        for _ in range(args.steps):
            e2e_step()
        q1.record()
        torch.cuda.synchronize()
        out["e2e"] = {"value": T / (q0.elapsed_time(q1) / args.steps * 1e-3), "unit": UNIT,
                      "h2d_bytes_per_step": nb(h2d), "d2h_bytes_per_step": nb(d2h),
                      "mode": "serial: copies and kernels of a step on one stream, nothing overlapped"}
    if not args.no_cpu_baseline:
        out["cpu_baseline"] = head_model_cpu_baseline(cfg, args)
    print(json.dumps(out))


def head_model_cpu_baseline(cfg, args):
    """The oracle, as it stands, on a bounded sample: rows of the head workload at the full widths; for the model
    workload the per-token cost of one full-width layer (a token prefix) and of the head (rows), combined as
    n_layers * layer + head.  A reported baseline, not the target."""
    from oracle import streambp_oracle as O
    from paper_2506_03077_b200 import synth
    h = cfg.head
    rows = min(cfg.T, args.cpu_baseline_head_rows)
    g, Wv, H, labels = synth.make_head_inputs(h, cfg.seed, rows, True, rows // 4)
    t0 = time.perf_counter()
    O.lmhead_ce_backward(O.HeadCfg(h.d_model, h.vocab, h.rms_eps, h.ignore_index), g, Wv, H, labels)
    head_s = (time.perf_counter() - t0) / rows
    if cfg.n_layers == 0:
        return {"value": 1.0 / head_s, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                "sample": f"{rows} rows of {cfg.name} (d {h.d_model}, vocab {h.vocab}), fp64 numpy oracle, "
                          f"{head_s * rows:.1f} s"}
    Ts = min(args.cpu_baseline_tokens, cfg.T)
    layer_s = oracle_sample(cfg, Ts) / Ts
    per_token = cfg.n_layers * layer_s + head_s
    return {"value": 1.0 / per_token, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"per-token cost of one full-width layer backward on the first {Ts} tokens "
                      f"({layer_s * Ts:.1f} s) x {cfg.n_layers} layers + of the head on {rows} rows ({head_s * rows:.1f} s); "
                      f"the layers' forward pass is not counted and a {Ts}-token prefix under-counts the quadratic "
                      f"attention term, both in the oracle's favour"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="llama8b_layer",
                    choices=["qwen7b_layer", "llama8b_layer", "qwen7b_head", "qwen7b_model"])
    ap.add_argument("--layers", type=int, default=0, help="override the layer count of the model configuration")
    ap.add_argument("--objective", default="sft", choices=["sft", "grpo", "dpo"],
                    help="objective of the qwen7b_head workload (Sec. 3.2.1)")
    ap.add_argument("--chunk", type=int, default=0)
    ap.add_argument("--wgrad-group", type=int, default=1,
                    help="layer and head workloads: chunks per weight-gradient pass (the second partition size, Sec. 4.3)")
    ap.add_argument("--T", type=int, default=0, help="override the sequence length (profiling on small cases)")
    ap.add_argument("--ref-tokens", type=int, default=512)
    ap.add_argument("--cpu-baseline-tokens", type=int, default=1024)
    ap.add_argument("--cpu-baseline-head-rows", type=int, default=256)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--dp", action="store_true",
                    help="data parallel instead of independent replicas: every step ends with one reduce-scatter of "
                         "the layer's fp32 gradient bucket over all ranks (Sec. 3.3 / App. A.3 of the paper)")
    args = ap.parse_args()

    from paper_2506_03077_b200 import synth
    import copy
    cfg = copy.copy(synth.CONFIGS[args.config])
    if args.chunk:
        cfg.chunk = args.chunk
    if args.T:
        cfg.T = args.T
    if args.layers:
        cfg.n_layers = args.layers
    if args.impl == "reference":
        if cfg.layer is None or cfg.n_layers:
            raise SystemExit("--impl reference times the oracle on the layer workloads only")
        return run_reference(args, cfg)
    if cfg.layer is None or cfg.n_layers:
        return run_head_or_model(args, cfg)

    import torch
    import torch.distributed as dist
    from paper_2506_03077_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the streamed backward has no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.lib()   # fail loudly if the CUDA library is absent

    s = cfg.layer
    dt = torch.bfloat16 if cfg.bf16 else torch.float32
    T, chunk = cfg.T, cfg.chunk
    bcfg = B.LayerConfig(s.d_model, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ff, s.qkv_bias, s.rope_theta,
                         s.rms_eps, dt)
    seed = replica_seed(cfg.seed, rank)
    Wn = synth.make_layer_weights(s, cfg.seed, cfg.bf16)
    Xn, dYn = synth.make_layer_io(s, seed, T, cfg.bf16)
    W = {k: torch.from_numpy(v).to("cuda", dt) for k, v in Wn.items()}
    X_host = torch.from_numpy(Xn).to(dt).pin_memory()
    dY_host = torch.from_numpy(dYn).to(dt).pin_memory()
    dX_host = torch.empty_like(X_host).pin_memory()
    X, dY = X_host.cuda(), dY_host.cuda()
    dX = torch.empty_like(X)
    grads = B.alloc_layer_grads(bcfg)
    ws_bytes = B.layer_workspace_bytes(bcfg, T, chunk, args.wgrad_group)
    ws_full = B.layer_workspace_bytes(bcfg, T, T)
    ws = B.alloc_workspace(ws_bytes)
    stream = torch.cuda.current_stream()

    dpr = None
    if args.dp:
        from paper_2506_03077_b200 import dp as DP
        dpr = DP.DataParallelLayerBackward(bcfg, W, T, chunk)
        grads, ws = dpr.bucket.views, dpr.ws

    def step():
        if dpr is not None:
            dpr.step(X, dY, dX)     # backward, then the gradient exchange on the communication stream
            dpr.wait()
        else:
            B.layer_backward(bcfg, W, X, dY, chunk, grads, dX, ws, wgrad_group=args.wgrad_group)

    fed = B.HostFedLayerBackward(bcfg, W, grads, T, chunk, ws, wgrad_group=args.wgrad_group)

    def run_e2e(steps):
        """Every step's X, dY come from pinned host memory and its dX goes back, inside the timed region; the
        copies of neighbouring steps overlap the kernels (see HostFedLayerBackward)."""
        fed.prefetch(X_host, dY_host)
        for k in range(steps):
            if k + 1 < steps:
                fed.prefetch(X_host, dY_host)      # the next step's inputs travel while this step computes
            fed.step(dX_host)
        fed.drain(stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(run, steps):
        """run(steps) enqueues `steps` steps; device time between barriers, max over ranks."""
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        run(steps)
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, "cuda")

    def run_steps(steps):
        for _ in range(steps):
            step()

    for _ in range(args.warmup):
        step()
    assert B.last_device_status(ws) == B.OK
    launches_per_step = B.last_launch_count()
    checked = check_outputs({"dX": dX, **{"d_" + k: v for k, v in grads.items()}})

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    # the headline number: K calls exactly as a user makes them
    total_ms = timed(run_steps, args.steps)
    # the same K calls again with every product / attention launch bracketed by CUDA events on the launching
    # stream (two event records per bracket: ~3 % of the step, which is why they are not in the region above)
    B.profile_enable(True)
    profiled_ms = timed(run_steps, args.steps)
    prof = {k: B.profile_read(k) for k in B.KERNEL_CLASSES}
    B.profile_enable(False)
    clocks = sampler.stop() if rank == 0 else None

    e2e_ms = None
    if not args.no_e2e:
        run_e2e(2)
        e2e_ms = timed(run_e2e, args.steps)

    ms_per_step = total_ms / args.steps
    value = aggregate_tokens_per_s(T, world, ms_per_step)
    peaks = read_peaks()
    flops = layer_flops(s, T)
    _, classes, roofline = roofline_object(prof, args.steps, peaks, cfg, chunk, profiled_ms)
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg.bf16 else "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "T": T, "chunk": chunk, "wgrad_group": args.wgrad_group, "d_model": s.d_model, "n_q_heads": s.n_q_heads,
                   "n_kv_heads": s.n_kv_heads, "head_dim": s.head_dim, "d_ff": s.d_ff, "qkv_bias": s.qkv_bias,
                   "l2": "inputs larger than L2 (weights + gradients > 1 GB per step)",
                   "product_kernel": B.product_kernel(),
                   "multi_gpu": ("data parallel: one NCCL reduce-scatter of the layer's fp32 gradient bucket per step"
                                 if args.dp else "replicas only")},
        "algorithmic_tflop_per_step": flops / 1e12,
        "tflops": flops / (ms_per_step * 1e-3) / 1e12,
        "frac_of_measured_sustained_bf16": flops / (ms_per_step * 1e-3) / 1e12 / peaks["sustained"],
        "frac_of_measured_burst_bf16": flops / (ms_per_step * 1e-3) / 1e12 / peaks["burst"],
        "frac_of_nominal_bf16": flops / (ms_per_step * 1e-3) / 1e12 / 2250.0,
        "peak_activation_gb": ws_bytes / 1e9, "peak_activation_gb_unchunked": ws_full / 1e9,
        "gpu_launches": int(launches_per_step * args.steps), "outputs_checked": checked,
        "roofline": roofline,
        "kernel_classes": classes,
        "clocks": clocks,
    }
    if e2e_ms is not None:
        nbytes = X_host.numel() * X_host.element_size()
        out["e2e"] = {"value": aggregate_tokens_per_s(T, world, e2e_ms / args.steps), "unit": UNIT,
                      "h2d_bytes_per_step": 2 * nbytes, "d2h_bytes_per_step": nbytes,
                      "mode": "pipelined: two buffer sets, a step's copies overlap the neighbouring steps' kernels "
                              "(throughput, not the latency of one isolated step)"}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        Ts = min(args.cpu_baseline_tokens, T)
        sec = oracle_sample(cfg, Ts)
        out["cpu_baseline"] = {"value": Ts / sec, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
                               "sample": f"first {Ts} tokens of {cfg.name} (full widths), fp64 numpy oracle, "
                                         f"full-sequence backward, {sec:.1f} s; a {Ts}-token prefix under-counts the "
                                         f"attention term, which is quadratic in T: at T = {T} the oracle's "
                                         f"tokens/s would be lower"}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
