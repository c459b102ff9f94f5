#!/usr/bin/env python
"""Benchmark of the Mirror-SD target-side verify step on B200.

One "step" is one whole pass of the hot path over one batch of synthetic input: branch-tree attention
for all layers -> LM head with fused reductions -> acceptance / branch selection, through the C-ABI
call mirror_verify_step.  The headline workload is the largest configuration that fits one GPU, the
66B-class one (80 layers, 16 requests with prefixes of 1024..8192 tokens in 16-token pages, kappa 8 x
gamma 8, vocab 128256, speculative-sampling acceptance; about 31 GB on the device).  The other
configurations are timed in the same run and reported under "workloads" (shorter loops).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Prints ONE JSON line.  With --impl reference the CPU oracle is timed instead (a deliberately plain
program: the ratio to it says nothing about kernel quality; parity and the roofline fraction do).
N > 1 runs independent replicas (the path does not shard): bench.py starts the N ranks itself (it re-runs
itself under torch.distributed.run on 127.0.0.1) unless it is already running under a launcher.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "verify_steps_per_sec"
UNIT = "steps/s"
HEADLINE = "opt66b_b16"                       # the largest single-GPU configuration
OTHERS = ["qwen14b", "qwen14b_b8", "qwen32b_long", "paper_native"]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="mirror", choices=["mirror", "reference"])
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--others", default=",".join(OTHERS),
                    help="comma-separated workloads also timed (short loops) and reported under 'workloads'; '' for none")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="the K-step block is repeated until this much device time has been timed; the median block is reported")
    ap.add_argument("--rendezvous-only", action="store_true",
                    help="start the ranks, run the barrier and the max-over-ranks reduction on a dummy timing and print a "
                         "skeleton line (gloo when there is no CUDA device): checks the launch path without a GPU")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-low-precision", action="store_true",
                    help="leave out stages.lmhead_fp8 and stages.attn_fp8 (the opt-in e4m3 modes timed beside the bf16 path, "
                         "outside the timed region; on by default when the head dimension is 128)")
    ap.add_argument("--accept-mode", default=None, choices=["greedy", "spec_sampling", "spec_tree"],
                    help="override the workload's acceptance rule")
    ap.add_argument("--skip-e2e", action="store_true",
                    help="profiling aid: leave the end-to-end loop out (e2e.value is null), so that a launch list holds the "
                         "device-resident steps only")
    ap.add_argument("--attn-per-layer", action="store_true",
                    help="also time attention launched layer by layer (plain launches and a CUDA-graph replay); reported under "
                         "stages.attn_per_layer_ms, outside the timed region")
    ap.add_argument("--overlap-draft", action="store_true",
                    help="also run the verify step next to a synthetic draft on a second stream (latency law of Sec. 3.2: the "
                         "step should cost max{target, draft}, not their sum); reported under stages.overlap_draft")
    ap.add_argument("--target-layers", type=int, default=0,
                    help="also time mirror_target_forward (projections, rotary embedding, attention, MLP) over this many "
                         "decoder layers of the workload's shape with seeded random weights (0.66 GB per layer for the default "
                         "workload); reported under stages.target_forward, outside the timed region")
    ap.add_argument("--intermediate", type=int, default=17408, help="MLP width for --target-layers")
    ap.add_argument("--lmhead-fp8", action="store_true",
                    help="also time the low-precision LM head (e4m3 weights and hidden rows, one scale per row) next to the bf16 "
                         "head on the workload's rows; reported under stages.lmhead_fp8, outside the timed region")
    ap.add_argument("--attn-fp8", action="store_true",
                    help="also time the attention over an e4m3 KV cache next to the bf16 one on the workload (head dimension 128); "
                         "reported under stages.attn_fp8, outside the timed region")
    ap.add_argument("--layers", type=int, default=None,
                    help="profiling aid: run the workload with this many attention layers (config.layers reports it); "
                         "the default, the workload's own layer count, is the only valid bench configuration")
    return ap.parse_args()


# ---------------------------------------------------------------------------------------------------
# algorithmic work of one step (what the method must move / compute), used for the roofline
# ---------------------------------------------------------------------------------------------------
def algorithmic_work(cfg, prefix_lens):
    d, Hq, Hkv, n, L, B = cfg.head_dim, cfg.n_q_heads, cfg.n_kv_heads, cfg.n_nodes, cfg.layers, cfg.batch
    kv_tokens = sum(int(l) for l in prefix_lens)
    attn_bytes = L * (2 * kv_tokens * Hkv * d * 2          # prefix K and V, read once
                      + 2 * B * n * Hkv * d * 2            # the tree's K and V
                      + 2 * B * n * Hq * d * 2)            # Q read, O written
    attn_flops = L * sum(4 * d * Hq * n * (int(l) + n) for l in prefix_lens)
    lm_bytes = cfg.vocab * cfg.hidden * 2 + cfg.rows * cfg.hidden * 2
    lm_flops = 2 * cfg.rows * cfg.vocab * cfg.hidden
    return dict(attn_bytes=attn_bytes, attn_flops=attn_flops, lm_bytes=lm_bytes, lm_flops=lm_flops)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1400.0, source="fallback")


def profiled_traffic(kernel_md: str, scale: float = 1.0):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary (None if absent).  A summary that was
    captured on a cut-down case says so with a line `dram_bytes_per_layer:`; it is scaled by `scale` (the layers of a
    full launch: traffic grows in proportion to the layers, each layer has its own cache)."""
    path = os.path.join(ROOT, "profiles", kernel_md)
    if not os.path.exists(path):
        return None
    text = open(path).read()
    m = re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", text)
    if m:
        return float(m.group(1))
    m = re.search(r"dram_bytes_per_layer:\s*([0-9.eE+]+)", text)
    return float(m.group(1)) * scale if m else None


# ---------------------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML)
# ---------------------------------------------------------------------------------------------------
class ClockSampler:
    def __init__(self, index: int):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.005)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        s = sorted(self.samples)
        return dict(sm_mhz=(s[len(s) // 2] if s else None), sm_max_mhz=self.max_mhz, reasons=sorted(self.reasons),
                    samples=len(s))


# ---------------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------------
def oracle_sample_seconds(x, cfg, target_seconds: float = 15.0):
    """Times the oracle, as it stands, on a bounded sample of one step.  A short calibration (one attention
    layer, 1/16 of the vocabulary) sizes the sample to about `target_seconds` of CPU work: `n_layers` of the
    attention layers (all requests and rows; layers cost the same, so one layer's tensors are reused) and the
    LM head + reductions + acceptance on all rows over the first `vocab_frac` of the vocabulary.  Returns
    (sample seconds, extrapolated seconds for a whole step, description)."""
    import numpy as np
    from oracle import oracle as O
    from paper_2510_13161_b200 import inputs as I
    anc, _ = O.tree(x.parent)
    scale = 1.0 / np.sqrt(cfg.head_dim)
    pt, pl = x.page_table.cpu().numpy(), x.prefix_len.cpu().numpy()
    args = (I.bf16_bits(x.q[0]), I.bf16_bits(x.k_pool[0]), I.bf16_bits(x.v_pool[0]), pt, pl,
            I.bf16_bits(x.k_new[0]), I.bf16_bits(x.v_new[0]), anc, scale)
    tok = x.tokens.cpu().numpy()

    def attn_layers(n):
        t = time.perf_counter()
        out = None
        for _ in range(n):
            out, _, _ = O.attention_layer(*args)
        return time.perf_counter() - t, out

    def lm_slice(out, rows_v):
        t = time.perf_counter()
        hid = I.bf16_bits(x.hidden) if x.hidden is not None else out.reshape(cfg.rows, -1)
        logits = O.lmhead_logits(hid, I.bf16_bits(x.W[:rows_v]))
        red = O.row_reduce(logits)
        O.accept_greedy(tok, red["argmax"].reshape(tok.shape), x.parent, cfg.gamma)
        return time.perf_counter() - t

    # calibration (not part of the timed sample)
    t_layer, out = attn_layers(1)
    v_cal = max(1024, cfg.vocab // 16)
    t_lm_cal = lm_slice(out, v_cal)
    n_layers = int(max(1, min(cfg.layers, round(0.5 * target_seconds / max(t_layer, 1e-6)))))
    rows_v = int(max(v_cal, min(cfg.vocab, round(v_cal * 0.5 * target_seconds / max(t_lm_cal, 1e-6)))))
    # timed sample
    t_attn, out = attn_layers(n_layers)
    t_lm = lm_slice(out, rows_v)
    sample = t_attn + t_lm
    full = t_attn * cfg.layers / n_layers + t_lm * cfg.vocab / rows_v
    desc = (f"{n_layers} of {cfg.layers} attention layers (all rows) + LM head / reductions / acceptance over the first "
            f"{rows_v} of {cfg.vocab} vocabulary rows; whole-step time extrapolated linearly")
    return sample, full, desc


def run_reference(args):
    """--impl reference: the CPU oracle on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import torch
    from oracle import oracle as O
    from paper_2510_13161_b200 import inputs as I
    cfg = I.CONFIGS[args.workload]
    if args.accept_mode:
        cfg = I.shrink(cfg, mode=args.accept_mode)
    if args.layers is not None:
        cfg = I.shrink(cfg, layers=args.layers)
    x = I.gen_verify_inputs(cfg, args.seed, "cpu", layers=1, force_hidden=cfg.explicit_hidden)
    steps, warm = max(1, min(args.steps, 4)), max(0, min(args.warmup, 1))
    for _ in range(warm):
        oracle_sample_seconds(x, cfg, 5.0)
    fulls, samples, desc = [], [], ""
    for _ in range(steps):
        s, f, desc = oracle_sample_seconds(x, cfg)
        samples.append(s); fulls.append(f)
    full = sum(fulls) / len(fulls)
    value = 1.0 / full
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warm, "ms_per_step": full * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "draft_tokens_per_sec": value * cfg.draft_tokens,
            "config": config_dict(cfg, int(os.environ.get("WORLD_SIZE", "1"))),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": desc,
                             "sample_seconds": sum(samples) / len(samples)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def max_over_ranks(value: float, device=None) -> float:
    """Max of a per-rank scalar over the process group (the slowest rank sets the job's time); identity
    without a process group.  Works on any backend: the multi-process CPU test drives it under gloo."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(steps_per_rank: int, world: int, ms_max: float) -> float:
    """Whole-job steps/s of `world` independent replicas that each ran `steps_per_rank` steps in `ms_max` ms."""
    return world * steps_per_rank * 1e3 / ms_max


# ---------------------------------------------------------------------------------------------------
# the CUDA arm
# ---------------------------------------------------------------------------------------------------
def attn_per_layer(m, x, tree, cfg, reps: int = 10):
    """Attention launched layer by layer (one mirror_attn_verify call per layer): ms for all layers, as plain launches and
    as a CUDA-graph replay.  The fused step passes all layers in one launch because its Q tensors are inputs."""
    import torch
    L = x.q.shape[0]
    kvs = [m.kv(x.k_pool[l:l + 1], x.v_pool[l:l + 1], x.page_table, x.prefix_len) for l in range(L)]
    out = torch.empty_like(x.q)
    s = torch.cuda.Stream()

    def run():
        for l in range(L):
            m.mirror_attn_verify(kvs[l], tree, x.q[l:l + 1], x.k_new[l:l + 1], x.v_new[l:l + 1], out=out[l:l + 1], stream=s)

    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    res = {}
    with torch.cuda.stream(s):
        for _ in range(3):
            run()
        s.synchronize()
        e0.record(s)
        for _ in range(reps):
            run()
        e1.record(s)
        s.synchronize()
        res["launches"] = e0.elapsed_time(e1) / reps
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            run()
        for _ in range(3):
            g.replay()
        s.synchronize()
        e0.record(s)
        for _ in range(reps):
            g.replay()
        e1.record(s)
        s.synchronize()
        res["graph"] = e0.elapsed_time(e1) / reps
    code, detail = m.device_status()
    if code != 0:
        raise SystemExit(f"device status {code} (detail {detail}) in the per-layer attention variant")
    res["kernel_launches"] = 2 * L
    return res


def overlap_draft_stage(step, stream, reps: int = 20):
    """The verify step next to a synthetic draft on a second stream of the same GPU.  Two stand-ins for the draft's
    generation phase, sized to take about as long as the verify step alone: a weight stream (a small model's
    matrix-vector products: memory-bound like the verify step) and a chain of square tensor-core GEMMs (compute-bound).
    For each: time alone, time of both launched together, and how much of the shorter one was hidden
    (1 = the step costs max{target, draft}, 0 = it costs their sum)."""
    import torch
    s2 = torch.cuda.Stream()
    dev = torch.cuda.current_device()
    w_stream = torch.empty((24, 8192, 4096), dtype=torch.bfloat16, device=dev).normal_(0, 0.02)      # 1.6 GB of weights
    v = torch.empty((4096, 8), dtype=torch.bfloat16, device=dev).normal_()
    a = torch.empty((2048, 2048), dtype=torch.bfloat16, device=dev).normal_(0, 0.02)
    b = torch.empty((2048, 2048), dtype=torch.bfloat16, device=dev).normal_(0, 0.02)

    def draft_stream():
        for i in range(w_stream.shape[0]):
            torch.matmul(w_stream[i], v)

    def draft_gemm():
        x = a
        for _ in range(24):
            x = torch.matmul(x, b)

    def timed(fn_main, fn_side):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        done = torch.cuda.Event()
        for it in range(3 + reps):
            if it == 3:
                torch.cuda.synchronize()
                e0.record(stream)
            if fn_side is not None:
                s2.wait_stream(stream)
                with torch.cuda.stream(s2):
                    fn_side()
                    done.record(s2)
            if fn_main is not None:
                fn_main()
            if fn_side is not None:
                stream.wait_event(done)
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    t_verify = timed(step, None)
    out = {"verify_ms": t_verify}
    for name, fn in (("weight_stream", draft_stream), ("tensor_gemms", draft_gemm)):
        t_draft = timed(None, fn)
        t_both = timed(step, fn)
        out[name] = {"draft_ms": t_draft, "both_ms": t_both, "max_ms": max(t_verify, t_draft), "sum_ms": t_verify + t_draft,
                     "hidden_frac": (t_verify + t_draft - t_both) / min(t_verify, t_draft)}
    return out


def lmhead_fp8_stage(m, x, cfg, hbm_gbs: float, reps: int = 20):
    """bf16 LM head against the e4m3 one on the same rows (random rows of the workload's shape): ms and weight GB/s each.
    The weights are quantised once, outside the timing; the per-step quantisation of the hidden rows is timed with it."""
    import torch
    dev = x.W.device
    hid = torch.empty((cfg.rows, cfg.hidden), dtype=torch.bfloat16, device=dev).normal_(0, 1.0)
    W8, ws = m.mirror_quantize_rows_fp8(x.W)

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    def fp8():
        h8, hs = m.mirror_quantize_rows_fp8(hid)
        m.mirror_lmhead_reduce_fp8(h8, hs, W8, ws)

    t16 = timed(lambda: m.mirror_lmhead_reduce(hid, x.W))
    t8 = timed(fp8)
    code, detail = m.device_status()
    if code != 0:
        raise SystemExit(f"device status {code} (detail {detail}) in the fp8 LM head")
    wb = cfg.vocab * cfg.hidden
    return {"rows": cfg.rows, "bf16_ms": t16, "fp8_ms": t8, "bf16_weight_gbs": 2 * wb / t16 / 1e6, "fp8_weight_gbs": wb / t8 / 1e6,
            "fp8_frac_hbm": wb / t8 / 1e6 / hbm_gbs, "speedup": t16 / t8,
            "note": "both include the merge kernel; fp8 also includes quantising the hidden rows"}


def attn_fp8_stage(m, x, tree, kv, cfg, peaks: dict, algo: dict, reps: int = 5):
    """bf16 attention against the e4m3-cache one over the workload's layers: ms, flop/s and cache bytes per second each.
    The cache is quantised once, outside the timing (as a serving engine would when it writes the cache)."""
    import torch
    P, d = x.k_pool.shape[3], x.k_pool.shape[4]
    ks, vs = m.mirror_kv_scales_fp8(x.k_pool, P * d), m.mirror_kv_scales_fp8(x.v_pool, P * d)
    k8, v8 = m.mirror_kv_quantize_fp8(x.k_pool, P * d, ks), m.mirror_kv_quantize_fp8(x.v_pool, P * d, vs)
    kn8, vn8 = m.mirror_kv_quantize_fp8(x.k_new, d, ks), m.mirror_kv_quantize_fp8(x.v_new, d, vs)
    kv8 = m.kv_fp8(k8, v8, x.page_table, x.prefix_len)
    q_scale = float(x.q[0].float().abs().max()) / 448.0
    out = torch.empty_like(x.q)

    def timed(fn):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / reps

    t16 = timed(lambda: m.mirror_attn_verify(kv, tree, x.q, x.k_new, x.v_new, out=out))
    t8 = timed(lambda: m.mirror_attn_verify_fp8(kv8, tree, x.q, kn8, vn8, ks, vs, q_scale, out=out))
    code, detail = m.device_status()
    if code != 0:
        raise SystemExit(f"device status {code} (detail {detail}) in the fp8 attention")
    kv_bytes = algo["attn_bytes"]          # (cache, tree rows, Q and O: the cache is nearly all of it)
    return {"bf16_ms": t16, "fp8_ms": t8, "speedup": t16 / t8,
            "bf16_tflops": algo["attn_flops"] / t16 / 1e9, "fp8_tflops": algo["attn_flops"] / t8 / 1e9,
            "bf16_gbs": kv_bytes / t16 / 1e6, "fp8_gbs": kv_bytes / 2 / t8 / 1e6,
            "fp8_frac_hbm": kv_bytes / 2 / t8 / 1e6 / peaks["hbm_gbs"],
            "note": "all layers, inputs larger than L2; merge kernel included in both"}


def target_forward_stage(m, x, tree, kv, cfg, n_layers: int, intermediate: int, hbm_gbs: float, reps: int = 5):
    """mirror_target_forward over n_layers decoder layers of the workload's shape (random weights): ms, weight bytes per
    second against the HBM peak.  The layers are weight streams at these row counts."""
    import torch
    from paper_2510_13161_b200 import inputs as I
    dev = x.q.device
    layers, norm_final, emb = I.gen_layer_weights(cfg, intermediate, n_layers, 0, dev)
    tgt = m.target(layers, norm_final, intermediate, 1.0e6, 1e-6)
    scratch = m.target_scratch(tree, tgt)
    out = m.mirror_target_forward(tgt, kv, tree, emb, scratch=scratch)
    for _ in range(2):
        m.mirror_target_forward(tgt, kv, tree, emb, scratch=scratch, out=out)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    l0 = m.launch_count()
    e0.record()
    for _ in range(reps):
        m.mirror_target_forward(tgt, kv, tree, emb, scratch=scratch, out=out)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    code, detail = m.device_status()
    if code != 0:
        raise SystemExit(f"device status {code} (detail {detail}) in mirror_target_forward")
    H, Hq, Hkv, d = cfg.hidden, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    w_bytes = 2 * ((Hq + 2 * Hkv) * d * H + H * Hq * d + 2 * intermediate * H + H * intermediate)
    kv_bytes = 2 * 2 * sum(int(l) for l in x.prefix_len.cpu().tolist()) * Hkv * d
    gbs = (w_bytes + kv_bytes) * n_layers / (ms * 1e-3) / 1e9
    return {"layers": n_layers, "intermediate": intermediate, "ms": ms, "us_per_layer": ms / n_layers * 1e3,
            "bytes_per_layer": w_bytes + kv_bytes, "gbs": gbs, "frac_hbm": gbs / hbm_gbs,
            "kernel_launches": (m.launch_count() - l0) // reps}


def config_dict(cfg, world: int):
    """The `config` object of the JSON line: the same keys and values in both arms."""
    return {"workload": cfg.name, "kappa": cfg.kappa, "gamma": cfg.gamma, "batch": cfg.batch, "layers": cfg.layers,
            "prefix": [cfg.prefix_lo, cfg.prefix_hi], "vocab": cfg.vocab, "hidden": cfg.hidden, "accept": cfg.mode,
            "l2": "inputs (KV cache + LM-head weights, gigabytes) are far larger than L2; no flush",
            "parallelism": "replicas only" if world > 1 else "single GPU"}


def stage_rooflines(work, peaks):
    """Binding roofline of each stage (the slower of its HBM and tensor time) and of the step, in ms."""
    attn = max(work["attn_bytes"] / peaks["hbm_gbs"] / 1e6, work["attn_flops"] / peaks["bf16_tflops"] / 1e9)
    lm = max(work["lm_bytes"] / peaks["hbm_gbs"] / 1e6, work["lm_flops"] / peaks["bf16_tflops"] / 1e9)
    return {"attn_ms": attn, "lmhead_ms": lm, "step_ms": attn + lm,
            "attn_bound": "hbm" if work["attn_bytes"] / peaks["hbm_gbs"] / 1e6 >= attn else "tensor",
            "lmhead_bound": "hbm" if work["lm_bytes"] / peaks["hbm_gbs"] / 1e6 >= lm else "tensor"}


class Workload:
    """One configuration resident on the device with everything a step needs."""

    def __init__(self, name, args, rank, local, dev):
        import torch
        from paper_2510_13161_b200 import binding, inputs as I
        cfg = I.CONFIGS[name]
        if args.accept_mode:
            cfg = I.shrink(cfg, mode=args.accept_mode)
        if args.layers is not None:
            cfg = I.shrink(cfg, layers=args.layers)
        self.cfg = cfg
        self.x = x = I.gen_verify_inputs(cfg, args.seed + rank, dev)          # replicas: each rank draws its own problem
        self.m = m = binding.Mirror(cfg.hidden, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.vocab,
                                    temperature=cfg.temperature, device=local)
        self.kv = m.kv(x.k_pool, x.v_pool, x.page_table, x.prefix_len)
        self.tree = m.tree(x.tokens, cfg.kappa, cfg.gamma)
        mode = {"spec_sampling": binding.ACCEPT_SPEC_SAMPLING, "spec_tree": binding.ACCEPT_SPEC_TREE}.get(cfg.mode, binding.ACCEPT_GREEDY)
        self.acc = m.accept_in(mode, True, q_probs=x.q_probs, u_accept=x.u_accept, u_resample=x.u_resample)
        self.attn_out = torch.empty_like(x.q)
        self.res = binding.AcceptResult(cfg.batch, cfg.gamma, dev)
        self.stream = torch.cuda.current_stream()
        self.work = algorithmic_work(cfg, x.prefix_len.cpu().tolist())
        self.resident_gb = sum(t.numel() * t.element_size() for t in (x.k_pool, x.v_pool, x.W)) / 1e9

    def step(self):
        x = self.x
        self.m.mirror_verify_step(self.kv, self.tree, x.q, x.k_new, x.v_new, x.hidden, x.W, self.acc, self.attn_out,
                                  out=self.res, stream=self.stream)

    def check(self, where):
        code, detail = self.m.device_status()
        if code != 0:
            raise SystemExit(f"device status {code} (detail {detail}) {where} ({self.cfg.name})")


def time_blocks(w: Workload, K: int, warmup: int, min_seconds: float, barrier, world, dev, max_blocks: int = 50):
    """Warm-up, then blocks of exactly K steps, each bracketed by CUDA events on the launching stream (resident inputs),
    repeated until `min_seconds` of device time has been timed.  Per-stage events ride on every step of a long step (an
    event record between two kernels keeps the second from being scheduled early, which matters for sub-millisecond
    steps only: there they ride on every fourth step).  Returns the median block and the stage means."""
    import torch
    for _ in range(max(warmup, 3)):
        w.step()
    barrier()
    w.check("during warm-up")
    # one probe block sizes the stage-event stride and the number of blocks
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(w.stream)
    for _ in range(3):
        w.step()
    e1.record(w.stream)
    torch.cuda.synchronize()
    est_ms = e0.elapsed_time(e1) / 3
    every = 1 if est_ms >= 1.0 else 4
    n_blocks = int(min(max_blocks, max(1, -(-min_seconds * 1e3 // (est_ms * K)), -(-20 * every // K))))
    stage_ev, blocks = [], []
    launches0 = w.m.launch_count()
    barrier()
    for b in range(n_blocks):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(w.stream)
        for k in range(K):
            if (b * K + k) % every == 0:
                stage_ev.append([torch.cuda.Event(enable_timing=True) for _ in range(4)])
                w.m.set_stage_events(stage_ev[-1])
            else:
                w.m.set_stage_events(None)
            w.step()
        ev1.record(w.stream)
        blocks.append((ev0, ev1))
    w.m.set_stage_events(None)
    barrier()
    launches = w.m.launch_count() - launches0
    w.check("during the timed region")
    block_ms = sorted(max_over_ranks(a.elapsed_time(b), dev) for a, b in blocks)
    med = block_ms[len(block_ms) // 2]
    mean = lambda i: sum(e[i].elapsed_time(e[i + 1]) for e in stage_ev) / len(stage_ev)
    return {"block_ms": med, "ms_per_step": med / K, "blocks": len(block_ms), "block_ms_min": block_ms[0], "block_ms_max": block_ms[-1],
            "attn_ms": mean(0), "lmhead_ms": mean(1), "tail_ms": mean(2), "stage_samples": len(stage_ev),
            "launches_per_block": launches // len(block_ms)}


def stages_of(t, work, peaks):
    ms_step = t["ms_per_step"]
    return {"attn_ms": t["attn_ms"], "lmhead_ms": t["lmhead_ms"], "merge_accept_ms": t["tail_ms"], "stage_samples": t["stage_samples"],
            "attn_gbs": work["attn_bytes"] / (t["attn_ms"] * 1e-3) / 1e9,
            "attn_frac_hbm": work["attn_bytes"] / (t["attn_ms"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
            "attn_tflops": work["attn_flops"] / (t["attn_ms"] * 1e-3) / 1e12,
            "attn_frac_tensor": work["attn_flops"] / (t["attn_ms"] * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "lmhead_gbs": work["lm_bytes"] / (t["lmhead_ms"] * 1e-3) / 1e9,
            "lmhead_tflops": work["lm_flops"] / (t["lmhead_ms"] * 1e-3) / 1e12,
            "lmhead_frac_tensor": work["lm_flops"] / (t["lmhead_ms"] * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "step_hbm_frac": (work["attn_bytes"] + work["lm_bytes"]) / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"]}


def run_mirror(args):
    import torch
    import torch.distributed as dist
    from paper_2510_13161_b200 import inputs as I

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verify path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = measured_peaks()
    w = Workload(args.workload, args, rank, local, dev)
    cfg, x, m = w.cfg, w.x, w.m
    K = args.steps

    # ---- timed region: blocks of K steps, resident inputs, CUDA events on the launching stream, clocks sampled throughout
    sampler = ClockSampler(local)
    sampler.start()
    t = time_blocks(w, K, args.warmup, args.min_seconds, barrier, world, dev)
    clocks = sampler.stop()
    ms_step = t["ms_per_step"]
    value = job_throughput(K, world, t["block_ms"])

    # ---- end to end: per step, this step's inputs come from pinned host memory and the decision goes back
    from paper_2510_13161_b200 import binding
    h_in = {k: getattr(x, k).cpu().pin_memory() for k in ("q", "k_new", "v_new", "tokens")}
    d_in = {k: torch.empty_like(getattr(x, k)) for k in h_in}
    tree_e = m.tree(d_in["tokens"], cfg.kappa, cfg.gamma)
    h_out = {k: torch.empty_like(getattr(w.res, k), device="cpu").pin_memory() for k in ("n_accepted", "n_emitted", "emitted", "best_branch")}
    h2d = sum(v.numel() * v.element_size() for v in h_in.values())
    d2h = sum(v.numel() * v.element_size() for v in h_out.values())

    def e2e_step():
        # one C-ABI call with host buffers: it copies this step's inputs in on its own stream, piece by piece, runs the
        # step and copies the decision back
        m.mirror_verify_step_host(w.kv, tree_e, h_in, d_in, x.hidden, x.W, w.acc, w.attn_out, w.res, h_out=h_out, stream=w.stream)
        w.stream.synchronize()      # the caller needs the decision before it can build the next step

    e2e_value = None
    if not args.skip_e2e:
        for _ in range(3):
            e2e_step()
        Ke = max(5, min(K, 200))
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(w.stream)
        for _ in range(Ke):
            e2e_step()
        e1.record(w.stream)
        barrier()
        e2e_value = job_throughput(Ke, world, max_over_ranks(e0.elapsed_time(e1), dev))
        w.check("in the end-to-end loop")
    del h_in, d_in, tree_e

    work = w.work
    stages = stages_of(t, work, peaks)
    rl = stage_rooflines(work, peaks)
    stages["roofline_ms"] = rl
    stages["step_frac_of_binding_roofline"] = rl["step_ms"] / ms_step
    # the dominant kernel of the step and the roofline that binds it
    if t["attn_ms"] >= t["lmhead_ms"]:
        tensor = rl["attn_bound"] == "tensor"
        ach = stages["attn_tflops"] if tensor else stages["attn_gbs"]
        roofline = {"kernel": "attn_verify_kernel", "bound": "tensor" if tensor else "hbm", "achieved": ach,
                    "peak": peaks["bf16_tflops"] if tensor else peaks["hbm_gbs"], "unit": "TFLOP/s" if tensor else "GB/s",
                    "frac": ach / (peaks["bf16_tflops"] if tensor else peaks["hbm_gbs"]), "peak_source": peaks["source"] + (" (sustained bf16)" if tensor else " (copy)"),
                    "traffic": profiled_traffic(f"attn_verify_kernel_{cfg.name}.md", scale=cfg.layers),
                    "algorithmic_flops_per_launch": work["attn_flops"], "algorithmic_bytes_per_launch": work["attn_bytes"],
                    "ms_per_launch": t["attn_ms"], "note": "ms_per_launch covers the attention stage (the main kernel and the small merge kernel behind it)"}
    else:
        tensor = rl["lmhead_bound"] == "tensor"
        ach = stages["lmhead_tflops"] if tensor else stages["lmhead_gbs"]
        roofline = {"kernel": "lmhead_pair_kernel", "bound": "tensor" if tensor else "hbm", "achieved": ach,
                    "peak": peaks["bf16_tflops"] if tensor else peaks["hbm_gbs"], "unit": "TFLOP/s" if tensor else "GB/s",
                    "frac": ach / (peaks["bf16_tflops"] if tensor else peaks["hbm_gbs"]), "peak_source": peaks["source"] + (" (sustained bf16)" if tensor else " (copy: a read + write stream; a read-only weight stream can read slightly above it)"),
                    "traffic": profiled_traffic(f"lmhead_pair_kernel_{cfg.name}.md"),
                    "algorithmic_flops_per_launch": work["lm_flops"], "algorithmic_bytes_per_launch": work["lm_bytes"],
                    "ms_per_launch": t["lmhead_ms"]}

    # ---- optional extra stages (outside the timed region)
    if args.attn_per_layer:
        stages["attn_per_layer_ms"] = attn_per_layer(m, x, w.tree, cfg)
    if args.overlap_draft:
        stages["overlap_draft"] = overlap_draft_stage(w.step, w.stream)
    low_precision = not args.no_low_precision and cfg.head_dim == 128 and cfg.hidden % 128 == 0 and args.layers is None
    if args.lmhead_fp8 or low_precision:
        stages["lmhead_fp8"] = lmhead_fp8_stage(m, x, cfg, peaks["hbm_gbs"])
    if args.attn_fp8 or low_precision:
        stages["attn_fp8"] = attn_fp8_stage(m, x, w.tree, w.kv, cfg, peaks, work)
    if args.target_layers > 0:
        stages["target_forward"] = target_forward_stage(m, x, w.tree, w.kv, cfg, min(args.target_layers, cfg.layers), args.intermediate,
                                                        peaks["hbm_gbs"])

    headline = {"ms_per_step": ms_step, "steps_per_sec": value, "draft_tokens_per_sec": value * cfg.draft_tokens,
                "attn_ms": t["attn_ms"], "lmhead_ms": t["lmhead_ms"], "merge_accept_ms": t["tail_ms"],
                "roofline_step_ms": rl["step_ms"], "frac_of_binding_roofline": rl["step_ms"] / ms_step,
                "attn_bound": rl["attn_bound"], "lmhead_bound": rl["lmhead_bound"], "step_hbm_frac": stages["step_hbm_frac"],
                "attn_frac": rl["attn_ms"] / t["attn_ms"], "lmhead_frac": rl["lmhead_ms"] / t["lmhead_ms"]}
    resident_gb = w.resident_gb
    del w, x, m
    torch.cuda.empty_cache()

    # ---- the other configurations, one after the other (shorter loops; same step, same events)
    workloads = {cfg.name: headline}
    for name in [n for n in args.others.split(",") if n and n != cfg.name]:
        wo = Workload(name, args, rank, local, dev)
        to = time_blocks(wo, K, 3, min(args.min_seconds, 0.3), barrier, world, dev, max_blocks=20)
        ro = stage_rooflines(wo.work, peaks)
        so = stages_of(to, wo.work, peaks)
        vo = job_throughput(K, world, to["block_ms"])
        workloads[name] = {"ms_per_step": to["ms_per_step"], "steps_per_sec": vo, "draft_tokens_per_sec": vo * wo.cfg.draft_tokens,
                           "attn_ms": to["attn_ms"], "lmhead_ms": to["lmhead_ms"], "merge_accept_ms": to["tail_ms"],
                           "roofline_step_ms": ro["step_ms"], "frac_of_binding_roofline": ro["step_ms"] / to["ms_per_step"],
                           "attn_bound": ro["attn_bound"], "lmhead_bound": ro["lmhead_bound"], "step_hbm_frac": so["step_hbm_frac"],
                           "attn_frac": ro["attn_ms"] / to["attn_ms"], "lmhead_frac": ro["lmhead_ms"] / to["lmhead_ms"],
                           "blocks": to["blocks"]}
        del wo
        torch.cuda.empty_cache()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        from oracle import oracle as O
        xs = I.gen_verify_inputs(cfg, args.seed, "cpu", layers=1, force_hidden=cfg.explicit_hidden)
        sec, full, desc = oracle_sample_seconds(xs, cfg)
        cpu = {"value": 1.0 / full, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": desc,
               "sample_seconds": sec}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "draft_tokens_per_sec": value * cfg.draft_tokens,
            "timing": {"blocks": t["blocks"], "steps_per_block": K, "block_ms_median": t["block_ms"], "block_ms_min": t["block_ms_min"],
                       "block_ms_max": t["block_ms_max"], "value_from": "median block"},
            "config": config_dict(cfg, world), "resident_gb": resident_gb,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "resident": "KV cache and LM-head weights (and, for stochastic acceptance, the draft distributions) stay on the "
                                "device; Q of every layer, the tree's K/V and the tokens are inputs of the synthetic step and are "
                                "copied every step: Q dominates the copies"},
            "gpu_launches": t["launches_per_block"], "clocks": clocks, "roofline": roofline, "stages": stages, "workloads": workloads,
            "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def rendezvous_only(args):
    """The launch path without the GPU work: process group (nccl with a CUDA device, gloo without), barrier, max-over-ranks of a
    dummy per-rank time, and a skeleton line from rank 0."""
    import torch
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("nccl" if torch.cuda.is_available() else "gloo")
        dist.barrier()
    ms = max_over_ranks(10.0 + 5.0 * rank, torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0"))) if torch.cuda.is_available() else None)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "rendezvous_only": True, "n_gpus": world, "requested_gpus": args.gpus, "ms_max": ms,
                          "value": job_throughput(args.steps, world, ms), "unit": UNIT}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(args) -> int:
    """--gpus N without a launcher: run this script again under torch.distributed.run with N ranks on this node."""
    import socket
    import subprocess
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    args = parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    if args.rendezvous_only:
        rendezvous_only(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_mirror(args)


if __name__ == "__main__":
    main()
