#!/usr/bin/env python
"""Benchmark of the hot path: one Llama-7B-shaped decoder layer, FP16, on B200.

A step = one pass of the whole path over one batch of synthetic input:
prefill of `batch` prompts of 512 tokens, then 128 decode steps over the FP16
KV cache.  The headline value is decode tokens/s (batch x 128 / decode time);
prefill tokens/s and both roofline fractions are reported beside it.

  python bench.py --gpus 1 --steps K --warmup W          # this library
  python bench.py --impl reference ...                    # the CPU oracle, timed on the host cores

With N > 1 (under torchrun) every rank runs an independent replica of the same
workload on its own GPU: the path has no exchange step, so there is no
collective on the data path; times are the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2605_25655_b200 import synth  # noqa: E402

PROMPT = 512
GEN = 128
SHAPE = synth.LLAMA_7B_LAYER
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def captured_traffic(key, batch):
    """DRAM bytes per launch from the committed ncu capture (batch 16 only; None otherwise)."""
    path = os.path.join(ROOT, "paper_2605_25655_b200", "ncu_traffic.json")
    if batch != 16 or not os.path.exists(path):
        return None
    return json.load(open(path)).get(key, {}).get("traffic_bytes")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# --------------------------------------------------------------------------- #
# algorithmic bytes / flops of the workload
# --------------------------------------------------------------------------- #
def layer_weight_elems(s):
    qd, kvd = s.n_q_heads * s.head_dim, s.n_kv_heads * s.head_dim
    return s.hidden * (qd + 2 * kvd) + qd * s.hidden + 3 * s.ffn * s.hidden


def decode_step_bytes(s, batch, t_len):
    """Weights once + gains, KV read (t_len keys) and append, activations in/out."""
    kv = batch * 2 * t_len * s.n_kv_heads * s.head_dim * 2
    app = batch * 2 * s.n_kv_heads * s.head_dim * 2
    act = batch * s.hidden * 2 * 2
    return 2 * layer_weight_elems(s) + 2 * 2 * s.hidden + kv + app + act


def gateup_gemv_bytes(s, batch):
    return 2 * (2 * s.ffn * s.hidden) + 2 * s.hidden + batch * s.hidden * 2 + batch * s.ffn * 2


def prefill_flops(s, rows, seq):
    gemm = 2.0 * rows * layer_weight_elems(s)
    attn = 2.0 * rows * seq * s.head_dim * s.n_q_heads      # causal: QK^T and PV, half of 4*S^2*d
    return gemm, attn


def gateup_gemm_flops(s, rows):
    return 2.0 * rows * 2 * s.ffn * s.hidden


# --------------------------------------------------------------------------- #
# clocks
# --------------------------------------------------------------------------- #
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.rows, self.proc, self.index = [], None, index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); power.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        busy = [s for s, p in zip(sm, power) if p > 250.0] or sm
        return {"sm_mhz": float(np.median(busy)) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- #
# oracle legs (host cores)
# --------------------------------------------------------------------------- #
def _oracle_sample(batch, n_steps, seed=0):
    """Times the oracle, as it stands, on `n_steps` decode steps of the workload (KV length PROMPT)."""
    from oracle import oracle as O
    cfg = O.Config(hidden=SHAPE.hidden, n_q_heads=SHAPE.n_q_heads, n_kv_heads=SHAPE.n_kv_heads,
                   head_dim=SHAPE.head_dim, ffn=SHAPE.ffn)
    w = synth.layer_weights(SHAPE, seed)
    rng = np.random.default_rng(seed)
    kc = rng.standard_normal((batch, SHAPE.n_kv_heads, PROMPT, SHAPE.head_dim)).astype(np.float16)
    vc = rng.standard_normal((batch, SHAPE.n_kv_heads, PROMPT, SHAPE.head_dim)).astype(np.float16)
    x = synth.hidden_states(SHAPE, seed, (batch, n_steps))
    times = []
    k, v = kc, vc
    for i in range(n_steps):
        t0 = time.perf_counter()
        _, k, v = O.layer_decode(cfg, w, x[:, i], k, v, PROMPT + i)
        times.append(time.perf_counter() - t0)
    return times


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info()]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    times = _oracle_sample(args.batch, args.warmup + args.steps)
    timed = times[args.warmup:]
    total = sum(timed)
    value = args.batch * len(timed) / total
    sample = f"{len(timed)} oracle decode steps of batch {args.batch} at KV length {PROMPT} (one step = {args.batch} tokens)"
    line = {
        "impl": "reference", "metric": "decode_tokens_per_s", "value": value, "unit": "tok/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(timed),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args.batch), "batch": args.batch, "prompt": PROMPT, "generate": GEN},
        "cpu_baseline": {"value": value, "unit": "tok/s", "cores": host_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tok/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def reduce_max_over_ranks(values, dist, device):
    """Element-wise maximum over ranks of a list of floats (times are reported as the slowest rank's)."""
    import torch
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_rate(units_per_rank, world, seconds):
    """Aggregate throughput of `world` independent replicas: all units processed / slowest rank's time."""
    return world * units_per_rank / seconds


def workload_name(batch):
    return (f"Llama-7B-shaped single decoder layer (hidden 4096, 32x128 MHA, FFN 11008), FP16, batch {batch}, "
            f"prompt {PROMPT}, {GEN} decode steps")


# --------------------------------------------------------------------------- #
# this library
# --------------------------------------------------------------------------- #
def run_ours(args):
    import torch
    from paper_2605_25655_b200 import thinfer

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    B = args.batch
    peaks, peak_kind = measured_peaks()

    w_np = synth.layer_weights(SHAPE, seed=0)
    layers = thinfer.to_device_layers([w_np], device=dev)
    x_np = synth.hidden_states(SHAPE, 0, (B, PROMPT + GEN))
    x_all = torch.from_numpy(x_np)
    x_prompt = x_all[:, :PROMPT].contiguous().to(dev)
    x_dec = [x_all[:, PROMPT + i].contiguous().to(dev) for i in range(GEN)]
    ctx = thinfer.Context(SHAPE, layers, None, max_batch=B, max_seq=PROMPT + GEN, buf_slots=1, device=dev)
    out_dec = torch.empty(B, SHAPE.hidden, dtype=torch.float16, device=dev)

    def one_step(events=None):
        if events:
            events[0].record()
        ctx.prefill(x_prompt)
        if events:
            events[1].record()
        for i in range(GEN):
            ctx.decode_step(x_dec[i], out=out_dec)
        if events:
            events[2].record()
        ctx.release_slot(0)

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step()
    sync_all()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = ctx.launch_count()
    sync_all()
    wall0 = time.perf_counter()
    for s in range(args.steps):
        one_step(evs[s])
    sync_all()
    wall = time.perf_counter() - wall0
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    if ctx.status() != 0:
        raise SystemExit(f"device status {ctx.status()} after the timed region")
    pre_ms = sum(e[0].elapsed_time(e[1]) for e in evs)
    dec_ms = sum(e[1].elapsed_time(e[2]) for e in evs)
    tot_ms = sum(e[0].elapsed_time(e[2]) for e in evs)
    pre_ms, dec_ms, tot_ms = reduce_max_over_ranks([pre_ms, dec_ms, tot_ms], dist, dev)

    # ---- end to end through the host-buffer entry points (pinned memory, copies inside the timed region)
    h_prompt = x_all[:, :PROMPT].contiguous().pin_memory()
    h_prompt_out = torch.empty_like(h_prompt).pin_memory()
    h_dec = [x_all[:, PROMPT + i].contiguous().pin_memory() for i in range(GEN)]
    h_dec_out = torch.empty(B, SHAPE.hidden, dtype=torch.float16).pin_memory()

    def one_step_host():
        ctx.prefill_host(h_prompt, h_prompt_out)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(GEN):
            ctx.decode_step_host(h_dec[i], h_dec_out)
            torch.cuda.synchronize()          # the caller reads each step's result before the next one
        dt = time.perf_counter() - t0
        ctx.release_slot(0)
        return dt

    one_step_host()
    e2e_s = sum(one_step_host() for _ in range(max(1, min(args.steps, 3))))
    e2e_steps = max(1, min(args.steps, 3))
    e2e_s = reduce_max_over_ranks([e2e_s], dist, dev)[0]

    # ---- dominant kernels, timed with CUDA events around each of their launches
    def kernel_time(kid, fn):
        ctx.profile_select(kid)
        fn()
        torch.cuda.synchronize()
        n, ms = ctx.profile_read()
        ctx.profile_select(-1)
        return n, ms

    def decode_only():
        ctx.prefill(x_prompt)
        for i in range(GEN):
            ctx.decode_step(x_dec[i], out=out_dec)
        ctx.release_slot(0)

    n_gu, ms_gu = kernel_time(thinfer.K_GATEUP, decode_only)     # 1 prefill launch + GEN decode launches
    ctx.profile_select(thinfer.K_GATEUP)
    ctx.prefill(x_prompt)
    torch.cuda.synchronize()
    n_pre, ms_pre_gu = ctx.profile_read()
    ctx.profile_select(-1)
    ctx.release_slot(0)
    ms_dec_gu = (ms_gu - ms_pre_gu) / max(1, n_gu - n_pre)
    ms_pre_gu = ms_pre_gu / max(1, n_pre)

    pre_tokens = world * B * PROMPT * args.steps
    value = whole_job_rate(B * GEN * args.steps, world, dec_ms * 1e-3)
    dec_bytes = sum(decode_step_bytes(SHAPE, B, PROMPT + i + 1) for i in range(GEN))
    dec_gbs = dec_bytes * args.steps / (dec_ms * 1e-3) / 1e9
    gemm_fl, attn_fl = prefill_flops(SHAPE, B * PROMPT, PROMPT)
    pre_tflops = (gemm_fl + attn_fl) * args.steps / (pre_ms * 1e-3) / 1e12
    hbm_peak = float(peaks["hbm_gbs"])
    tc_peak = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    gu_gbs = gateup_gemv_bytes(SHAPE, B) / (ms_dec_gu * 1e-3) / 1e9
    gu_tflops = gateup_gemm_flops(SHAPE, B * PROMPT) / (ms_pre_gu * 1e-3) / 1e12

    line = {
        "metric": "decode_tokens_per_s", "value": value, "unit": "tok/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": tot_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16", "data": "synthetic",
        "config": {"workload": workload_name(B), "batch": B, "prompt": PROMPT, "generate": GEN,
                   "value_is": "batch x generate / decode-phase time; ms_per_step covers prefill + decode",
                   "l2": "no flush: the 405 MB of layer weights streamed by every decode step and the prefill "
                         "activations exceed the 126 MB L2",
                   "multi_gpu": "independent replicas, no collective"},
        "decode": {"ms_per_token_step": dec_ms / (args.steps * GEN), "achieved_GBs": dec_gbs,
                   "frac_of_hbm_peak": dec_gbs / hbm_peak, "peak_GBs": hbm_peak, "peak_kind": peak_kind},
        "prefill": {"value": pre_tokens / (pre_ms * 1e-3), "unit": "tok/s", "ms": pre_ms / args.steps,
                    "achieved_TFLOPs": pre_tflops, "frac_of_tensor_peak": pre_tflops / tc_peak,
                    "peak_TFLOPs": tc_peak, "peak_kind": peak_kind + " bf16 sustained (same tensor-pipe rate as fp16)"},
        "roofline": {"kernel": ("skinny_mma_kernel<SWIGLU>" if B <= 16 else "tc_gemm_kernel<32..64, SWIGLU> stream-K")
                     + " (decode gate/up projection)", "bound": "hbm",
                     "achieved": gu_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gu_gbs / hbm_peak,
                     "traffic": captured_traffic("decode_gateup_b16", B), "peak_kind": peak_kind, "avg_us": ms_dec_gu * 1e3,
                     "algorithmic_bytes": gateup_gemv_bytes(SHAPE, B)},
        "roofline_prefill": {"kernel": "tc_gemm_kernel<256, SWIGLU interleaved> (prefill gate/up projection)", "bound": "tensor",
                             "achieved": gu_tflops, "peak": tc_peak, "unit": "TFLOP/s", "frac": gu_tflops / tc_peak,
                             "traffic": captured_traffic("prefill_gateup_b16", B), "peak_kind": peak_kind, "avg_us": ms_pre_gu * 1e3},
        "e2e": {"value": world * B * GEN * e2e_steps / e2e_s, "unit": "tok/s",
                "h2d_bytes_per_step": B * SHAPE.hidden * 2, "d2h_bytes_per_step": B * SHAPE.hidden * 2,
                "note": "per decode step: pinned host input -> device, layer, result -> host, stream synchronised"},
        "gpu_launches": launches, "clocks": clocks, "wall_s": wall,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n = 4
        times = _oracle_sample(B, n)
        line["cpu_baseline"] = {"value": B * n / sum(times), "unit": "tok/s", "cores": host_threads(), "kind": "oracle",
                                "sample": f"{n} oracle decode steps of batch {B} at KV length {PROMPT}"}
    if rank == 0:
        print(json.dumps(line))
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()
    return 0


def run_profile_case(args):
    """A small, self-ending case for ncu: one warm-up pass, then one pass of the chosen phase."""
    import torch
    from paper_2605_25655_b200 import thinfer
    B, n_dec = args.batch, args.profile_decode_steps
    w = thinfer.to_device_layers([synth.layer_weights(SHAPE, seed=0)])
    x = torch.from_numpy(synth.hidden_states(SHAPE, 0, (B, PROMPT + n_dec)))
    xp = x[:, :PROMPT].contiguous().cuda()
    xd = [x[:, PROMPT + i].contiguous().cuda() for i in range(n_dec)]
    ctx = thinfer.Context(SHAPE, w, None, max_batch=B, max_seq=PROMPT + n_dec)
    for rep in range(2):
        ctx.prefill(xp)
        if args.profile == "decode" or rep == 0:
            for t in xd:
                ctx.decode_step(t)
        ctx.release_slot(0)
        torch.cuda.synchronize()
    assert ctx.status() == 0
    print(json.dumps({"profile_case": args.profile, "batch": B, "launches": ctx.launch_count()}))
    ctx.close()
    return 0


# Operator latencies the paper prints for MT-3000 (one cluster for Linear; cluster count not stated for
# attention), quoted for context beside the B200 numbers: Table 8 (FP16 Linear, input dim 4096, ms) and
# Table 9 ("MT Attention", batch 4, head_dim 128, ms).
PAPER_TABLE8_FP16_MS = {
    1024: [0.52, 0.64, 0.90, 1.62, 2.03, 2.93, 3.88], 2048: [0.66, 1.05, 1.45, 1.95, 3.38, 5.05, 6.53],
    4096: [1.59, 2.19, 3.28, 3.62, 6.80, 9.54, 12.52], 8192: [3.05, 4.45, 5.81, 7.67, 12.93, 18.47, 24.17]}
TABLE8_OUT = [256, 512, 768, 1024, 2048, 3072, 4096]
PAPER_TABLE9_MT_MS = {32: [9.72, 25.13, 32.45, 79.00, 107.61, 119.39, 191.98, 248.26],
                      64: [18.20, 49.29, 63.20, 156.56, 212.08, 236.59, 381.52, 496.23]}
TABLE9_SEQ = [512, 1024, 1536, 2048, 2560, 3072, 3584, 4096]


def run_tables(args):
    """Operator micro-benchmarks at the shapes of the paper's Tables 8 and 9 (context, not the headline)."""
    import torch
    from paper_2605_25655_b200 import thinfer

    def timed(fn, reps=5, inner=20):
        # `inner` back-to-back launches per measurement so that the device, not the host call path, is timed
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(inner):
                fn()
            e1.record(); torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1) / inner)
        return float(np.median(ts))

    g = torch.Generator(device="cuda").manual_seed(0)
    rows = []
    for s_len in (1024, 2048, 4096, 8192):
        x = torch.randn(s_len, 4096, device="cuda", dtype=torch.float16, generator=g)
        for j, n_out in enumerate(TABLE8_OUT):
            w = torch.randn(n_out, 4096, device="cuda", dtype=torch.float16, generator=g) * 0.02
            y = torch.empty(s_len, n_out, device="cuda", dtype=torch.float16)
            ms = timed(lambda: thinfer.op_linear(x, w, path=0, out=y))
            rows.append({"op": "linear_fp16", "rows": s_len, "in": 4096, "out": n_out, "ms": ms,
                         "tflops": 2.0 * s_len * 4096 * n_out / (ms * 1e-3) / 1e12,
                         "paper_mt3000_ms": PAPER_TABLE8_FP16_MS[s_len][j]})
    for heads in (32, 64):
        for j, s_len in enumerate(TABLE9_SEQ):
            q = torch.randn(4, heads, s_len, 128, device="cuda", dtype=torch.float16, generator=g)
            k = torch.randn(4, heads, s_len, 128, device="cuda", dtype=torch.float16, generator=g)
            v = torch.randn(4, heads, s_len, 128, device="cuda", dtype=torch.float16, generator=g)
            o = torch.empty(4, s_len, heads * 128, device="cuda", dtype=torch.float16)
            ms = timed(lambda: thinfer.op_attention_prefill(q, k, v, out=o))
            rows.append({"op": "attention_causal_fp16", "batch": 4, "heads": heads, "seq": s_len, "head_dim": 128,
                         "ms": ms, "tflops": 2.0 * 4 * heads * s_len * s_len * 128 / (ms * 1e-3) / 1e12,
                         "paper_mt3000_ms": PAPER_TABLE9_MT_MS[heads][j]})
            del q, k, v
    print(json.dumps({"tables": rows, "note": "B200 latencies at the shapes of the paper's Tables 8 and 9; the paper "
                      "column is MT-3000 hardware (context only); attention FLOPs counted causal (2*S^2*d per head)"}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--batch", type=int, default=16)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile", choices=["prefill", "decode"], default=None,
                    help="run one small pass of a phase and exit (the case ncu captures)")
    ap.add_argument("--profile-decode-steps", type=int, default=2)
    ap.add_argument("--tables", action="store_true", help="operator micro-benchmarks at the paper's Table 8 / 9 shapes")
    args = ap.parse_args()
    if args.tables:
        return run_tables(args)
    if args.profile:
        return run_profile_case(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
