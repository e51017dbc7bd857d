#!/usr/bin/env python
"""Benchmark of the hot path on B200: FP16 Llama-shaped decoder stacks, prefill then greedy decode.

A step = one pass of the whole path over one batch of synthetic input: prefill of `batch` prompts (which
emits the first token), then the remaining tokens one decode step at a time over the FP16 KV cache, the ids
fed back on the device.  The headline value is decode tokens/s; prefill tokens/s, the paper-style end-to-end
rate (batch x generated / total latency, Section 3.4.1) and the roofline fractions are reported beside it.

  python bench.py --gpus 1 --steps K --warmup W            # this library, configuration 5 (70B stack)
  python bench.py --config {c2,c3,c4,c5} ...               # 7B layer / 7B stack / 13B stack / 70B stack
  python bench.py --impl reference ...                      # the CPU oracle, timed on the host cores
  python bench.py --tables                                  # operator latencies at the paper's Table 8 / 9 shapes
  python bench.py --pipeline --config c4                    # prefill of the next batch overlapped with decode (2 KV slots)
  python bench.py --profile {prefill,decode} --config cX    # one layer of that configuration: the case ncu captures
  python bench.py --profile stack --config cX               # two layers + head: the case of the ncu launch list
  python bench.py --profile attention --config cX --seq S   # the prefill attention operator alone, batch 4

With N > 1 (under torchrun) every rank runs an independent replica of the same workload on its own GPU: the
path has no exchange step, so there is no collective on the data path; times are the maximum over ranks.
"""
from __future__ import annotations

import argparse
import dataclasses
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

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_GBS = 8000.0       # the HBM3e figure the target bars are quoted against
NOMINAL_TFLOPS = 2250.0    # dense FP16 / BF16 tensor peak


@dataclasses.dataclass(frozen=True)
class Workload:
    key: str
    shape: synth.Shape
    batch: int
    prompt: int
    gen: int            # stack: tokens generated per request (1 by the prefill, gen - 1 by decode steps);
    label: str          # layer-only: decode steps on seeded hidden states

    @property
    def stack(self):
        return self.shape.vocab > 0

    @property
    def decode_steps(self):
        return self.gen - 1 if self.stack else self.gen

    def name(self, batch=None):
        b = self.batch if batch is None else batch
        s = self.shape
        heads = f"{s.n_q_heads}x{s.head_dim} MHA" if s.n_q_heads == s.n_kv_heads else \
            f"{s.n_q_heads} query / {s.n_kv_heads} KV heads x {s.head_dim} (GQA)"
        if self.stack:
            return (f"{self.label} full stack ({s.n_layers} layers, hidden {s.hidden}, {heads}, FFN {s.ffn}, vocab "
                    f"{s.vocab}), FP16, batch {b}, prompt {self.prompt}, {self.gen} tokens generated greedily")
        return (f"{self.label} single decoder layer (hidden {s.hidden}, {heads}, FFN {s.ffn}), FP16, batch {b}, "
                f"prompt {self.prompt}, {self.gen} decode steps")


WORKLOADS = {
    "c2": Workload("c2", synth.LLAMA_7B_LAYER, 16, 512, 128, "Llama-7B-shaped"),
    "c3": Workload("c3", synth.LLAMA_7B, 8, 512, 256, "Llama-7B-shaped"),
    "c4": Workload("c4", synth.LLAMA_13B, 16, 1024, 256, "Llama-13B-shaped"),
    "c5": Workload("c5", synth.LLAMA_70B, 4, 512, 128, "Llama-2-70B-shaped"),
}
DEFAULT_WORKLOAD = "c5"    # the largest configuration that fits one GPU (138 GB of weights)


def captured(key, field="traffic_bytes"):
    """A figure of the committed ncu captures (profiles/ncu_traffic.json): DRAM bytes per launch, tensor-pipe
    activity, DRAM throughput; None when the kernel of this workload has no capture."""
    path = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if not os.path.exists(path):
        return None
    return json.load(open(path)).get(key, {}).get(field)


def captured_traffic(key):
    return captured(key, "traffic_bytes")


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
    """One decode step of the whole model.  Per layer: weights once + gains, KV read (t_len keys) and append;
    plus activations in/out and, for a stack, the vocabulary projection, the final gain and the embedding rows."""
    kv = batch * 2 * t_len * s.n_kv_heads * s.head_dim * 2
    app = batch * 2 * s.n_kv_heads * s.head_dim * 2
    per_layer = 2 * layer_weight_elems(s) + 2 * 2 * s.hidden + kv + app
    total = s.n_layers * per_layer + batch * s.hidden * 2 * 2
    if s.vocab > 0:
        total += 2 * s.vocab * s.hidden + 2 * s.hidden + batch * s.vocab * 4
    return total


def gateup_gemv_bytes(s, batch):
    return 2 * (2 * s.ffn * s.hidden) + 2 * s.hidden + batch * s.hidden * 2 + batch * s.ffn * 2


def prefill_flops(s, rows, seq, batch):
    gemm = 2.0 * rows * layer_weight_elems(s) * s.n_layers
    attn = 2.0 * rows * seq * s.head_dim * s.n_q_heads * s.n_layers   # causal: QK^T and PV, half of 4*S^2*d
    head = 2.0 * batch * s.vocab * s.hidden
    return gemm, attn, head


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
def _oracle_sample(wl, batch, n_steps, seed=0):
    """Times the oracle, as it stands, on a bounded sample of the decode workload: `n_steps` decode steps of ONE
    layer at KV length wl.prompt, and (stack configurations) as many calls of the final norm + vocabulary
    projection.  Returns (seconds per layer step, seconds per head call) lists."""
    from oracle import oracle as O
    s = wl.shape
    cfg = O.Config(hidden=s.hidden, n_q_heads=s.n_q_heads, n_kv_heads=s.n_kv_heads, head_dim=s.head_dim, ffn=s.ffn)
    w = synth.layer_weights(s, seed)
    rng = np.random.default_rng(seed)
    kc = rng.standard_normal((batch, s.n_kv_heads, wl.prompt, s.head_dim)).astype(np.float16)
    vc = rng.standard_normal((batch, s.n_kv_heads, wl.prompt, s.head_dim)).astype(np.float16)
    x = synth.hidden_states(s, seed, (batch, n_steps))
    sw = None
    if wl.stack:
        sw = {"final_norm": synth.stack_tensor(s, seed, "final_norm"), "lm_head": synth.stack_tensor(s, seed, "lm_head")}
    layer_s, head_s = [], []
    k, v = kc, vc
    for i in range(n_steps):
        t0 = time.perf_counter()
        y, k, v = O.layer_decode(cfg, w, x[:, i], k, v, wl.prompt + i)
        layer_s.append(time.perf_counter() - t0)
        if sw is not None:
            t0 = time.perf_counter()
            O.argmax_lowest(O.head_logits(cfg, sw, y))
            head_s.append(time.perf_counter() - t0)
        else:
            head_s.append(0.0)
    return layer_s, head_s


def _oracle_sample_text(wl, batch, n):
    s = wl.shape
    if wl.stack:
        return (f"{n} oracle decode steps of ONE layer (+ final norm, vocabulary projection, argmax) at batch {batch}, "
                f"KV length {wl.prompt}; a model step is taken as {s.n_layers} x the layer time + the head time "
                f"(one step = {batch} tokens)")
    return f"{n} oracle decode steps of batch {batch} at KV length {wl.prompt} (one step = {batch} tokens)"


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info()]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count()


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    B = args.batch or wl.batch
    layer_s, head_s = _oracle_sample(wl, B, args.warmup + args.steps)
    L = wl.shape.n_layers
    step_s = [L * a + b for a, b in zip(layer_s, head_s)][args.warmup:]
    total = sum(step_s)
    value = B * len(step_s) / total
    line = {
        "impl": "reference", "metric": "decode_tokens_per_s", "value": value, "unit": "tok/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(step_s),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name(B), "batch": B, "prompt": wl.prompt, "generate": wl.gen},
        "cpu_baseline": {"value": value, "unit": "tok/s", "cores": host_threads(), "kind": "oracle",
                         "sample": _oracle_sample_text(wl, B, len(step_s))},
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


# --------------------------------------------------------------------------- #
# this library
# --------------------------------------------------------------------------- #
class Runner:
    """One workload on one device: weights, context, inputs, and the step functions the legs time."""

    def __init__(self, wl, batch, dev, torch, thinfer, storage="f16"):
        self.wl, self.B, self.dev, self.torch, self.thinfer = wl, batch, dev, torch, thinfer
        s, B = wl.shape, batch
        dt = torch.bfloat16 if storage == "bf16" else torch.float16
        self.steps_dec = wl.decode_steps
        max_seq = wl.prompt + wl.decode_steps
        if wl.stack:
            sw = synth.device_stack_weights(s, seed=0, device=dev, dtype=dt)
            self.sw = sw
            self.ctx = thinfer.Context(s, sw["layers"], {n: sw[n] for n in ("embed", "final_norm", "lm_head")},
                                       max_batch=B, max_seq=max_seq, device=dev)
            ids = synth.token_ids(s, 0, (B, wl.prompt))
            self.h_prompt = torch.from_numpy(ids).pin_memory()
            self.prompt = self.h_prompt.to(dev)
            self.id_buf = [torch.zeros(B, dtype=torch.int32, device=dev) for _ in range(2)]
            self.h_ids = torch.zeros(B, dtype=torch.int32).pin_memory()
            self.h_ids_out = torch.zeros(B, dtype=torch.int32).pin_memory()
            self.h2d, self.d2h = B * 4, B * 4
        else:
            if storage == "bf16":
                self.layers = [synth.device_layer_weights(s, 0, 0, device=dev, dtype=dt)]
            else:
                self.layers = thinfer.to_device_layers([synth.layer_weights(s, seed=0)], device=dev)
            self.ctx = thinfer.Context(s, self.layers, None, max_batch=B, max_seq=max_seq, device=dev)
            x_all = torch.from_numpy(synth.hidden_states(s, 0, (B, wl.prompt + wl.gen))).to(dt)
            self.h_prompt = x_all[:, :wl.prompt].contiguous().pin_memory()
            self.prompt = self.h_prompt.to(dev)
            self.h_prompt_out = torch.empty_like(self.h_prompt).pin_memory()
            self.h_dec = [x_all[:, wl.prompt + i].contiguous().pin_memory() for i in range(wl.gen)]
            self.x_dec = [t.to(dev) for t in self.h_dec]
            self.out_dec = torch.empty(B, s.hidden, dtype=dt, device=dev)
            self.h_dec_out = torch.empty(B, s.hidden, dtype=dt).pin_memory()
            self.h2d, self.d2h = B * s.hidden * 2, B * s.hidden * 2

    def prefill(self):
        if self.wl.stack:
            return self.ctx.prefill(self.prompt)
        self.ctx.prefill(self.prompt)
        return None

    def decode(self, first_ids, n_steps=None):
        n = self.steps_dec if n_steps is None else n_steps
        if self.wl.stack:
            cur = first_ids
            for i in range(n):
                cur = self.ctx.decode_step(cur, out=self.id_buf[i & 1])     # ids stay on the device
            return cur
        for i in range(n):
            self.ctx.decode_step(self.x_dec[i], out=self.out_dec)
        return None

    def one_step(self, events=None):
        if events:
            events[0].record()
        first = self.prefill()
        if events:
            events[1].record()
        self.decode(first)
        if events:
            events[2].record()
        self.ctx.release_slot(0)

    def one_step_host(self):
        """The same step through the host-buffer entry points: every decode step copies its input from pinned
        host memory, copies its result back, and the host reads it before it issues the next step."""
        torch, ctx = self.torch, self.ctx
        if self.wl.stack:
            ctx.prefill_host(self.h_prompt, self.h_ids_out)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for _ in range(self.steps_dec):
                self.h_ids.copy_(self.h_ids_out)                  # the token just read is the next input
                ctx.decode_step_host(self.h_ids, self.h_ids_out)
                torch.cuda.synchronize()
            dt = time.perf_counter() - t0
        else:
            ctx.prefill_host(self.h_prompt, self.h_prompt_out)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            for i in range(self.steps_dec):
                ctx.decode_step_host(self.h_dec[i], self.h_dec_out)
                torch.cuda.synchronize()
            dt = time.perf_counter() - t0
        ctx.release_slot(0)
        return dt


def run_ours(args, wl):
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
    B = args.batch or wl.batch
    S, s = wl.prompt, wl.shape
    peaks, peak_kind = measured_peaks()
    R = Runner(wl, B, dev, torch, thinfer, args.storage)
    ctx = R.ctx
    n_dec = wl.decode_steps

    def sync_all():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        R.one_step()
    sync_all()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = ctx.launch_count()
    sync_all()
    wall0 = time.perf_counter()
    for i in range(args.steps):
        R.one_step(evs[i])
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
    e2e_steps = max(1, min(args.steps, 2 if wl.stack else 3))
    R.one_step_host()
    e2e_s = sum(R.one_step_host() for _ in range(e2e_steps))
    e2e_s = reduce_max_over_ranks([e2e_s], dist, dev)[0]

    # ---- dominant kernels (gate/up projection), timed with CUDA events around each of their own launches
    def kernel_time(kid, fn):
        ctx.profile_select(kid)
        fn()
        torch.cuda.synchronize()
        n, ms = ctx.profile_read()
        ctx.profile_select(-1)
        return n, ms

    first = R.prefill()                                   # untimed: fills the slot for the decode sample
    torch.cuda.synchronize()
    k_steps = min(n_dec, 8)
    n_dgu, ms_dgu = kernel_time(thinfer.K_GATEUP, lambda: R.decode(first, k_steps))
    ctx.release_slot(0)
    n_pgu, ms_pgu = kernel_time(thinfer.K_GATEUP, R.prefill)
    ctx.release_slot(0)
    ms_dec_gu = ms_dgu / max(1, n_dgu)
    ms_pre_gu = ms_pgu / max(1, n_pgu)

    pre_tokens = world * B * S * args.steps
    value = whole_job_rate(B * n_dec * args.steps, world, dec_ms * 1e-3)
    dec_bytes = sum(decode_step_bytes(s, B, S + i + 1) for i in range(n_dec))
    dec_gbs = dec_bytes * args.steps / (dec_ms * 1e-3) / 1e9
    gemm_fl, attn_fl, head_fl = prefill_flops(s, B * S, S, B)
    pre_tflops = (gemm_fl + attn_fl + head_fl) * args.steps / (pre_ms * 1e-3) / 1e12
    hbm_peak = float(peaks["hbm_gbs"])
    tc_sustained = float(peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]))
    tc_burst = float(peaks["bf16_tflops"])
    gu_gbs = gateup_gemv_bytes(s, B) / (ms_dec_gu * 1e-3) / 1e9
    gu_tflops = gateup_gemm_flops(s, B * S) / (ms_pre_gu * 1e-3) / 1e12
    weights_gb = synth.model_bytes(s) / 1e9 if wl.stack else 2 * layer_weight_elems(s) / 1e9
    tc_pre_rows = "tc_gemm_kernel<256, SWIGLU interleaved>" if B * S > 64 else "tc_gemm_kernel<SWIGLU>"
    dec_kernel = ("skinny_mma_kernel<SWIGLU>" if B <= 16 else "tc_gemm_kernel<32..64, SWIGLU> stream-K")

    line = {
        "metric": "decode_tokens_per_s", "value": value, "unit": "tok/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": tot_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": args.storage, "data": "synthetic",
        "config": {"workload": wl.name(B).replace("FP16", "BF16") if args.storage == "bf16" else wl.name(B), "key": wl.key, "batch": B, "prompt": S, "generate": wl.gen,
                   "decode_steps_per_pass": n_dec,
                   "value_is": "batch x decode steps / decode-phase time; ms_per_step covers prefill + decode",
                   "l2": f"no flush: the {weights_gb:.1f} GB of weights streamed by every decode step and the prefill "
                         "activations exceed the 126 MB L2",
                   "multi_gpu": "independent replicas, no collective"},
        "decode": {"ms_per_token_step": dec_ms / (args.steps * n_dec), "algorithmic_bytes_per_pass": dec_bytes,
                   "achieved_GBs": dec_gbs, "frac_of_hbm_peak": dec_gbs / hbm_peak, "peak_GBs": hbm_peak,
                   "peak_kind": peak_kind, "frac_of_nominal_peak": dec_gbs / NOMINAL_GBS, "nominal_GBs": NOMINAL_GBS},
        "prefill": {"value": pre_tokens / (pre_ms * 1e-3), "unit": "tok/s", "ms": pre_ms / args.steps,
                    "achieved_TFLOPs": pre_tflops, "frac_of_tensor_peak": pre_tflops / tc_sustained,
                    "peak_TFLOPs": tc_sustained,
                    "peak_kind": peak_kind + " bf16 sustained (same tensor-pipe rate as fp16)",
                    "frac_of_nominal_peak": pre_tflops / NOMINAL_TFLOPS, "nominal_TFLOPs": NOMINAL_TFLOPS},
        "end_to_end_paper_style": {"value": world * B * wl.gen * args.steps / (tot_ms * 1e-3), "unit": "tok/s",
                                   "is": "batch x generated tokens / (prefill + decode) time, Section 3.4.1"},
        "roofline": {"kernel": dec_kernel + " (decode gate/up projection)", "bound": "hbm",
                     "achieved": gu_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gu_gbs / hbm_peak,
                     "traffic": captured_traffic(f"decode_gateup_{wl.key}_b{B}"),
                     "dram_throughput_pct_captured": captured(f"decode_gateup_{wl.key}_b{B}", "dram_throughput_pct"),
                     "traffic_kind": "captured (committed profile of the same launch, profiles/ncu_traffic.json)",
                     "peak_kind": peak_kind, "avg_us": ms_dec_gu * 1e3, "launches_timed": n_dgu,
                     "algorithmic_bytes": gateup_gemv_bytes(s, B), "frac_of_nominal_peak": gu_gbs / NOMINAL_GBS},
        "roofline_prefill": {"kernel": tc_pre_rows + " (prefill gate/up projection)", "bound": "tensor",
                             "achieved": gu_tflops, "peak": tc_burst, "unit": "TFLOP/s", "frac": gu_tflops / tc_burst,
                             "traffic": captured_traffic(f"prefill_gateup_{wl.key}_b{B}"),
                             "tensor_pipe_active_pct_captured": captured(f"prefill_gateup_{wl.key}_b{B}", "tensor_pipe_active_pct"),
                             "traffic_kind": "captured (committed profile of the same launch, profiles/ncu_traffic.json)",
                             "peak_kind": peak_kind + " bf16 burst (the kernel is timed alone)",
                             "avg_us": ms_pre_gu * 1e3, "launches_timed": n_pgu,
                             "frac_of_sustained": gu_tflops / tc_sustained,
                             "frac_of_nominal_peak": gu_tflops / NOMINAL_TFLOPS},
        "e2e": {"value": world * B * n_dec * e2e_steps / e2e_s, "unit": "tok/s",
                "h2d_bytes_per_step": R.h2d, "d2h_bytes_per_step": R.d2h,
                "note": "per decode step: pinned host input -> device, all layers, result -> host, stream synchronised; "
                        "the host feeds the token it read back in"},
        "gpu_launches": launches, "clocks": clocks, "wall_s": wall,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n = 3 if wl.stack else 4
        layer_s, head_s = _oracle_sample(wl, B, n)
        step = s.n_layers * sum(layer_s) / n + sum(head_s) / n
        line["cpu_baseline"] = {"value": B / step, "unit": "tok/s", "cores": host_threads(), "kind": "oracle",
                                "sample": _oracle_sample_text(wl, B, n)}
    if rank == 0:
        print(json.dumps(line))
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()
    return 0


def run_pipeline(args, wl):
    """The Prefill -> Buffer -> Decode schedule of Section 3.4.2 on one device, measured: two KV slots, the prefill
    of the next batch on one stream while the current batch decodes on another (the library's hand-off events order
    the stages of each slot), against the same work issued on a single stream.  Reports generated tokens / s of
    both schedules; a side measurement, not the headline."""
    import torch
    from paper_2605_25655_b200 import thinfer
    if not wl.stack:
        raise SystemExit("--pipeline needs a stack configuration (c3, c4, c5)")
    B, s, n_dec = args.batch or wl.batch, wl.shape, wl.decode_steps
    dev = torch.device("cuda", 0)
    sw = synth.device_stack_weights(s, seed=0, device=dev)
    ctx = thinfer.Context(s, sw["layers"], {n: sw[n] for n in ("embed", "final_norm", "lm_head")}, max_batch=B,
                          max_seq=wl.prompt + n_dec, buf_slots=2, device=dev)
    prompts = [torch.from_numpy(synth.token_ids(s, 0, (B, wl.prompt), stream=i)).to(dev) for i in range(2)]
    bufs = [[torch.zeros(B, dtype=torch.int32, device=dev) for _ in range(2)] for _ in range(2)]
    first = [torch.zeros(B, dtype=torch.int32, device=dev) for _ in range(2)]

    def batches(n_batches, sp, sd):
        # batch r lives in slot r % 2: its prefill is issued while batch r - 1 decodes
        def prefill(r):  # every buffer is allocated up front: nothing is freed while another stream may still read it
            return ctx.prefill(prompts[r % 2], slot=r % 2, stream=sp, out=first[r % 2])
        outs = [None, None]
        outs[0] = prefill(0)
        for r in range(n_batches):
            if r + 1 < n_batches:
                outs[(r + 1) % 2] = prefill(r + 1)
            cur = outs[r % 2]
            for i in range(n_dec):
                cur = ctx.decode_step(cur, slot=r % 2, stream=sd, out=bufs[r % 2][i & 1])
            ctx.release_slot(r % 2, stream=sd)

    n_batches = max(2, args.steps)
    res = {}
    for name in ("serial", "pipelined"):
        if name == "serial":
            sp = sd = torch.cuda.current_stream()
        else:
            sp, sd = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()
        batches(2, sp, sd)                       # warm-up
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        batches(n_batches, sp, sd)
        torch.cuda.synchronize()
        res[name] = time.perf_counter() - t0
        if ctx.status() != 0:
            raise SystemExit(f"device status {ctx.status()}")
    tokens = n_batches * B * wl.gen
    print(json.dumps({"pipeline": {"workload": wl.name(B), "batches": n_batches, "kv_slots": 2,
                                   "tok_s": {k: tokens / v for k, v in res.items()},
                                   "seconds": res,
                                   "speedup_over_serial": {k: res["serial"] / v for k, v in res.items() if k != "serial"},
                                   "is": "generated tokens / wall time over all batches, prefill included "
                                         "(Section 3.4.1's throughput); pipelined = prefill of batch r + 1 on a second "
                                         "stream while batch r decodes"}}))
    ctx.close()
    return 0


def run_profile_stack(args, wl):
    """The launch list's case: a TWO-layer stack of the configuration with its vocabulary head, real batch and
    prompt - every kernel of the benchmark's step appears with the arguments it has in the full model (layer 0
    with the norm prologue, layer 1 with the folded norm, embedding, head, argmax).  One warm-up pass, then one
    pass of prefill + `--profile-decode-steps` decode steps.  The full model repeats the per-layer launches of
    layer 1 (n_layers - 1) times: the summary under profiles/ scales the shares accordingly."""
    import torch
    from paper_2605_25655_b200 import thinfer
    B, n_dec = args.batch or wl.batch, args.profile_decode_steps
    s = dataclasses.replace(wl.shape, n_layers=2)
    sw = synth.device_stack_weights(s, 0)
    ctx = thinfer.Context(s, sw["layers"], {n: sw[n] for n in ("embed", "final_norm", "lm_head")}, max_batch=B,
                          max_seq=wl.prompt + n_dec)
    ids = torch.from_numpy(synth.token_ids(s, 0, (B, wl.prompt))).cuda()
    for rep in range(2):
        cur = ctx.prefill(ids)
        for _ in range(n_dec):
            cur = ctx.decode_step(cur)
        ctx.release_slot(0)
        torch.cuda.synchronize()
    assert ctx.status() == 0
    print(json.dumps({"profile_case": "stack", "config": wl.key, "batch": B, "layers": 2, "decode_steps": n_dec,
                      "launches": ctx.launch_count()}))
    ctx.close()
    return 0


def run_profile_case(args, wl):
    """A small, self-ending case for ncu: ONE layer of the configuration (its shapes, batch and prompt, so every
    launch equals the one in the full model), one warm-up pass, then one pass of the chosen phase."""
    import torch
    from paper_2605_25655_b200 import thinfer
    B, n_dec = args.batch or wl.batch, args.profile_decode_steps
    s = dataclasses.replace(wl.shape, n_layers=1, vocab=0)
    w = [synth.device_layer_weights(s, 0, 0)]
    g = torch.Generator(device="cuda").manual_seed(1)
    x = torch.randn(B, wl.prompt + n_dec, s.hidden, device="cuda", dtype=torch.float16, generator=g)
    xp = x[:, :wl.prompt].contiguous()
    xd = [x[:, wl.prompt + i].contiguous() for i in range(n_dec)]
    ctx = thinfer.Context(s, w, None, max_batch=B, max_seq=wl.prompt + n_dec)
    for rep in range(2):
        ctx.prefill(xp)
        if args.profile == "decode" or rep == 0:
            for t in xd:
                ctx.decode_step(t)
        ctx.release_slot(0)
        torch.cuda.synchronize()
    assert ctx.status() == 0
    print(json.dumps({"profile_case": args.profile, "config": wl.key, "batch": B, "launches": ctx.launch_count()}))
    ctx.close()
    return 0


def run_profile_attention(args, wl):
    """The prefill attention operator alone at Table 9's shape (batch 4, the configuration's heads, `--seq` keys):
    three launches, for an ncu capture at a sequence length no configuration reaches."""
    import torch
    from paper_2605_25655_b200 import thinfer
    s, S = wl.shape, args.seq
    g = torch.Generator(device="cuda").manual_seed(1)
    q = torch.randn(4, s.n_q_heads, S, s.head_dim, device="cuda", dtype=torch.float16, generator=g)
    k, v = (torch.randn(4, s.n_kv_heads, S, s.head_dim, device="cuda", dtype=torch.float16, generator=g) for _ in range(2))
    out = thinfer.op_attention_prefill(q, k, v)
    for _ in range(2):
        thinfer.op_attention_prefill(q, k, v, out=out)
    torch.cuda.synchronize()
    print(json.dumps({"profile_case": "attention", "heads": [s.n_q_heads, s.n_kv_heads], "head_dim": s.head_dim, "seq": S}))
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
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS),
                    help="c2: 7B layer; c3: 7B stack; c4: 13B stack; c5: 70B stack (default)")
    ap.add_argument("--batch", type=int, default=0, help="override the configuration's batch (c2: 1, 4, 16)")
    ap.add_argument("--storage", default="f16", choices=["f16", "bf16"],
                    help="16-bit storage type of weights, activations and KV cache (the BF16 build of the library)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profile", choices=["prefill", "decode", "stack", "attention"], default=None,
                    help="run one small pass and exit (the cases ncu captures): one layer of the configuration, "
                         "prefill or decode phase; a two-layer stack with the head (the launch list); or the prefill "
                         "attention operator alone at --seq keys")
    ap.add_argument("--seq", type=int, default=4096, help="--profile attention: sequence length")
    ap.add_argument("--profile-decode-steps", type=int, default=2)
    ap.add_argument("--pipeline", action="store_true",
                    help="measure the two-slot prefill / decode overlap of Section 3.4.2 against the serial schedule")
    ap.add_argument("--tables", action="store_true", help="operator micro-benchmarks at the paper's Table 8 / 9 shapes")
    args = ap.parse_args()
    wl = WORKLOADS[args.config]
    if args.tables:
        return run_tables(args)
    if args.pipeline:
        return run_pipeline(args, wl)
    if args.profile == "stack":
        return run_profile_stack(args, wl)
    if args.profile == "attention":
        return run_profile_attention(args, wl)
    if args.profile:
        return run_profile_case(args, wl)
    if args.impl == "reference":
        return run_reference(args, wl)
    return run_ours(args, wl)


if __name__ == "__main__":
    sys.exit(main())
