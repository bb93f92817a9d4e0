"""Host-side logic of bench.py on CPU: FLOP accounting, replica bookkeeping and the
max-over-ranks timing rule with two gloo ranks."""
import json
import os
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402
from paper_2506_03077_b200 import synth  # noqa: E402


def test_layer_flops_match_the_published_totals():
    # algorithmic totals of the two layer workloads: qwen7b layer T 8192 -> 12.03 TFLOP, llama8b layer T 32768 -> 69.82 TFLOP
    assert abs(bench.layer_flops(synth.QWEN7B_LAYER, 8192) / 1e12 - 12.03) < 0.01
    assert abs(bench.layer_flops(synth.LLAMA8B_LAYER, 32768) / 1e12 - 69.82) < 0.01


def test_replica_bookkeeping():
    assert bench.replica_seed(1, 0) == 1 and bench.replica_seed(1, 3) == 3001
    assert bench.aggregate_tokens_per_s(8192, 4, 20.0) == pytest.approx(4 * 8192 / 0.02)
    p = bench.read_peaks()
    assert p["sustained"] > 0 and p["source"] in ("measured", "fallback")


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 10.0 + 5.0 * rank                     # rank 1 is the slow replica
    agreed = bench.max_over_ranks(mine, world, "cpu")
    dist.barrier()
    out.put((rank, agreed))
    dist.destroy_process_group()


def test_max_over_ranks_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == {0: 15.0, 1: 15.0}


def test_reference_arm_prints_one_json_line():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1",
                        "--warmup", "0", "--ref-tokens", "32", "--config", "qwen7b_layer"],
                       capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["cpu_baseline"]["kind"] == "oracle"
    assert j["e2e"]["h2d_bytes_per_step"] == 0 and j["value"] > 0


def test_output_check_rejects_skipped_work():
    import torch
    ok = {"a": torch.ones(4), "b": torch.tensor([0.0, -2.0])}
    assert "a, b" in bench.check_outputs(ok)
    with pytest.raises(AssertionError):
        bench.check_outputs({"a": torch.zeros(4)})                       # a step that never wrote its output
    with pytest.raises(AssertionError):
        bench.check_outputs({"a": torch.tensor([1.0, float("nan")])})


def test_roofline_object_names_the_dominant_class_and_carries_the_others():
    """The roofline entry is the kernel class with the largest share of the step that was run; every class keeps its own
    achieved rate; traffic is looked up per (config, chunk, class) and never silently absent."""
    import copy
    peaks = dict(hbm=6484.6, burst=1648.7, sustained=1392.7, source="measured")
    steps = 4
    # (milliseconds over all steps, launches, algorithmic FLOPs): attention backward is the largest here
    prof = {"gemm": (4 * 30.0, 4 * 128, 4 * 39.0e12), "attention_fwd": (4 * 10.0, 4 * 16, 4 * 8.8e12),
            "attention_bwd": (4 * 32.0, 4 * 16, 4 * 22.0e12)}
    cfg = copy.copy(synth.CONFIGS["llama8b_layer"])
    dom, classes, roof = bench.roofline_object(prof, steps, peaks, cfg, cfg.chunk, 4 * 78.0)
    assert dom == "attention_bwd" and roof["class"] == "attention_bwd" and roof["bound"] == "tensor"
    assert roof["achieved"] == pytest.approx(22.0e12 / 32.0e-3 / 1e12) and roof["frac"] == pytest.approx(roof["achieved"] / 1392.7)
    assert set(roof["classes"]) == {"gemm", "attention_fwd", "attention_bwd"}
    assert classes["gemm"]["tflops"] == pytest.approx(1300.0) and classes["gemm"]["launches_per_step"] == 128
    assert roof["launches"] == 64 and roof["ms_per_step"] == pytest.approx(32.0)
    # traffic: the captured 16384-key launch scaled to the step's average launch by algorithmic bytes
    s = cfg.layer
    ends = [min(cfg.T, r0 + cfg.chunk) for r0 in range(0, cfg.T, cfg.chunk)]
    avg = sum(bench.attn_bwd_bytes(s, e, cfg.chunk) for e in ends) / len(ends)
    assert roof["traffic"] == pytest.approx(488.6e6 * avg / bench.attn_bwd_bytes(s, 16384, 2048))
    assert "profiles/" in roof["traffic_note"]
    # products dominate on the short-sequence layer: the entry switches class; an uncaptured chunk says why it has no figure
    prof2 = dict(prof, gemm=(4 * 40.0, 4 * 64, 4 * 40e12))
    q = copy.copy(synth.CONFIGS["qwen7b_layer"])
    dom2, _, roof2 = bench.roofline_object(prof2, steps, peaks, q, 512, 4 * 90.0)
    assert dom2 == "gemm" and roof2["traffic"] is None and "no ncu capture" in roof2["traffic_note"]
    _, _, roof3 = bench.roofline_object(prof2, steps, peaks, q, 1024, 4 * 90.0)
    assert roof3["traffic"] == pytest.approx(2142.5e6)


def test_attention_byte_model():
    s = synth.LLAMA8B_LAYER
    # K, V read (bf16), dK, dV read + written (fp32), Q, dO read (bf16), dQ written (fp32), lse and delta read
    assert bench.attn_bwd_bytes(s, 16384, 2048) == 16384 * 1024 * (4 + 16) + 2048 * 4096 * (4 + 4) + 8 * 2048 * 32
    assert bench.attn_fwd_bytes(s, 16384, 2048) == 16384 * 1024 * 4 + 2048 * 4096 * 4 + 4 * 2048 * 32
