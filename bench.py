#!/usr/bin/env python
"""Benchmark of the Mirror-SD target-side verify step on B200.

One "step" is one whole pass of the hot path over one batch of synthetic input: branch-tree attention
for all layers -> LM head with fused reductions -> acceptance / branch selection, through the C-ABI
call mirror_verify_step.  The workload is the 14B-shaped configuration (48 layers, prefix 2048 in
16-token pages, kappa 4 x gamma 4, vocab 152064, greedy), which fits one GPU.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Prints ONE JSON line.  With --impl reference the CPU oracle is timed instead (a deliberately plain
program: the ratio to it says nothing about kernel quality; parity and the roofline fraction do).
N > 1 runs independent replicas (the path does not shard): launch under torch.distributed.run.
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


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="mirror", choices=["mirror", "reference"])
    ap.add_argument("--workload", default="qwen14b")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
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


def profiled_traffic(kernel_md: str):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary (None if absent)."""
    path = os.path.join(ROOT, "profiles", kernel_md)
    if not os.path.exists(path):
        return None
    m = re.search(r"dram_bytes_per_launch:\s*([0-9.eE+]+)", open(path).read())
    return float(m.group(1)) if m else None


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
            "config": {"workload": cfg.name, "kappa": cfg.kappa, "gamma": cfg.gamma, "batch": cfg.batch,
                       "layers": cfg.layers, "prefix": [cfg.prefix_lo, cfg.prefix_hi], "vocab": cfg.vocab},
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


def run_mirror(args):
    import torch
    import torch.distributed as dist
    from paper_2510_13161_b200 import binding, inputs as I

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verify path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)

    cfg = I.CONFIGS[args.workload]
    if args.accept_mode:
        cfg = I.shrink(cfg, mode=args.accept_mode)
    if args.layers is not None:
        cfg = I.shrink(cfg, layers=args.layers)
    x = I.gen_verify_inputs(cfg, args.seed + rank, dev)          # replicas: each rank draws its own problem
    m = binding.Mirror(cfg.hidden, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.vocab, temperature=cfg.temperature,
                       device=local)
    kv = m.kv(x.k_pool, x.v_pool, x.page_table, x.prefix_len)
    tree = m.tree(x.tokens, cfg.kappa, cfg.gamma)
    mode = {"spec_sampling": binding.ACCEPT_SPEC_SAMPLING, "spec_tree": binding.ACCEPT_SPEC_TREE}.get(cfg.mode, binding.ACCEPT_GREEDY)
    acc = m.accept_in(mode, True, q_probs=x.q_probs, u_accept=x.u_accept, u_resample=x.u_resample)
    attn_out = torch.empty_like(x.q)
    res = binding.AcceptResult(cfg.batch, cfg.gamma, dev)
    stream = torch.cuda.current_stream()

    def step():
        m.mirror_verify_step(kv, tree, x.q, x.k_new, x.v_new, x.hidden, x.W, acc, attn_out, out=res, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    code, detail = m.device_status()
    if code != 0:
        raise SystemExit(f"device status {code} (detail {detail}) during warm-up")

    # ---- timed region: K steps, resident inputs, CUDA events on the launching stream; per-stage events ride along
    K = args.steps
    # (an event record between two kernels also keeps the second from being scheduled early, so the per-stage events
    # ride on every eighth step only; ev0 / ev1 bracket all K steps)
    EVERY = 8
    stage_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range((K + EVERY - 1) // EVERY)]
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    launches0 = m.launch_count()
    barrier()
    sampler.start()
    ev0.record(stream)
    for k in range(K):
        m.set_stage_events(stage_ev[k // EVERY] if k % EVERY == 0 else None)
        step()
    ev1.record(stream)
    m.set_stage_events(None)
    barrier()
    clocks = sampler.stop()
    launches = m.launch_count() - launches0
    ms_total = max_over_ranks(ev0.elapsed_time(ev1), dev)
    ms_step = ms_total / K
    value = job_throughput(K, world, ms_total)
    attn_ms = sum(e[0].elapsed_time(e[1]) for e in stage_ev) / len(stage_ev)
    lm_ms = sum(e[1].elapsed_time(e[2]) for e in stage_ev) / len(stage_ev)
    tail_ms = sum(e[2].elapsed_time(e[3]) for e in stage_ev) / len(stage_ev)
    code, detail = m.device_status()
    if code != 0:
        raise SystemExit(f"device status {code} (detail {detail}) during the timed region")

    # ---- end to end: per step, this step's inputs come from pinned host memory and the decision goes back
    h_in = {k: getattr(x, k).cpu().pin_memory() for k in ("q", "k_new", "v_new", "tokens")}
    d_in = {k: torch.empty_like(getattr(x, k)) for k in h_in}
    tree_e = m.tree(d_in["tokens"], cfg.kappa, cfg.gamma)
    h_out = {k: torch.empty_like(getattr(res, k), device="cpu").pin_memory() for k in ("n_accepted", "n_emitted", "emitted", "best_branch")}
    h2d = sum(v.numel() * v.element_size() for v in h_in.values())
    d2h = sum(v.numel() * v.element_size() for v in h_out.values())

    def e2e_step():
        # one C-ABI call with host buffers: it copies this step's inputs in on its own stream, piece by piece, runs the
        # step and copies the decision back
        m.mirror_verify_step_host(kv, tree_e, h_in, d_in, x.hidden, x.W, acc, attn_out, res, h_out=h_out, stream=stream)
        stream.synchronize()      # the caller needs the decision before it can build the next step

    e2e_value = None
    if not args.skip_e2e:
        for _ in range(3):
            e2e_step()
        Ke = max(10, min(K, 200))
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(Ke):
            e2e_step()
        e1.record(stream)
        barrier()
        e2e_value = job_throughput(Ke, world, max_over_ranks(e0.elapsed_time(e1), dev))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    work = algorithmic_work(cfg, x.prefix_len.cpu().tolist())
    peaks = measured_peaks()
    lm_gbs = work["lm_bytes"] / (lm_ms * 1e-3) / 1e9
    attn_gbs = work["attn_bytes"] / (attn_ms * 1e-3) / 1e9
    roofline = {"kernel": "lmhead_pair_kernel", "bound": "hbm", "achieved": lm_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": lm_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
                "traffic": profiled_traffic("lmhead_pair_kernel_qwen14b.md"),
                "algorithmic_bytes_per_launch": work["lm_bytes"], "ms_per_launch": lm_ms}
    stages = {"attn_ms": attn_ms, "lmhead_ms": lm_ms, "merge_accept_ms": tail_ms,
              "attn_gbs": attn_gbs, "attn_frac_hbm": attn_gbs / peaks["hbm_gbs"],
              "attn_tflops": work["attn_flops"] / (attn_ms * 1e-3) / 1e12,
              "lmhead_tflops": work["lm_flops"] / (lm_ms * 1e-3) / 1e12,
              "step_hbm_frac": (work["attn_bytes"] + work["lm_bytes"]) / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"]}

    # ---- attention with one launch pair per layer: the order a real target enforces (layer l+1's queries depend on
    # layer l's output), as plain stream-ordered launches and replayed from a CUDA graph.  Outside the timed region.
    if args.attn_per_layer:
        stages["attn_per_layer_ms"] = attn_per_layer(m, x, tree, cfg)
    if args.overlap_draft:
        stages["overlap_draft"] = overlap_draft_stage(step, stream)
    if args.target_layers > 0:
        stages["target_forward"] = target_forward_stage(m, x, tree, kv, cfg, min(args.target_layers, cfg.layers), args.intermediate,
                                                        peaks["hbm_gbs"])

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        from oracle import oracle as O
        xs = I.gen_verify_inputs(cfg, args.seed, "cpu", layers=1, force_hidden=cfg.explicit_hidden)
        s, full, desc = oracle_sample_seconds(xs, cfg)
        cpu = {"value": 1.0 / full, "unit": UNIT, "cores": O.num_threads(), "kind": "oracle", "sample": desc,
               "sample_seconds": s}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": max(args.warmup, 3),
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "draft_tokens_per_sec": value * cfg.draft_tokens,
            "config": {"workload": cfg.name, "kappa": cfg.kappa, "gamma": cfg.gamma, "batch": cfg.batch, "layers": cfg.layers,
                       "prefix": [cfg.prefix_lo, cfg.prefix_hi], "vocab": cfg.vocab, "hidden": cfg.hidden, "accept": cfg.mode,
                       "l2": "inputs (KV cache + LM-head weights, about 2 GB) are larger than L2; no flush",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "resident": "KV cache and LM-head weights stay on the device; Q, tree K/V and tokens are copied every step"},
            "gpu_launches": launches, "clocks": clocks, "roofline": roofline, "stages": stages, "cpu_baseline": cpu}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_mirror(args)


if __name__ == "__main__":
    main()
