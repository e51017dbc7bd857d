"""Memory / time model and configuration search of Section 3.4.3, for B200 memory budgets.

Host-side arithmetic only (no GPU, no extension needed).  The paper sizes its
Prefill / Buffer / Decode pools with three ingredients, restated here:

  memory      parameters per device + KV cache per device + overhead < budget
              (the paper's budget is 20 GB per MT-3000 cluster; a B200 has 180 GB)
  traffic     All-Reduce volume of tensor parallelism in decode,
              Comm_TP = B * 2 * D_emb * D_size * (TP - 1)
  time        one layer with TP:  T = 2 T_norm + (T_attn + T_ffn) / TP + 2 T_allreduce + 2 T_launch
              pool cost:          Clu_pool = DP_P * PP_P + TP_D * PP_D + B_P
              objective:          minimise over DP_P   Clu_pool * max(T_p / DP_P, T_d)

`plan_single_device` answers the question this library can act on: for one GPU that holds the whole
model (TP = PP = 1), how many requests fit per slot and how many KV slots (the bounded buffer, Buf_max)
fit beside the weights.  The multi-device formulas are provided for completeness; the library itself
runs independent replicas only.
"""
from __future__ import annotations

import dataclasses
from typing import Iterable, Optional

from .synth import Shape

FP16_BYTES = 2
B200_HBM_BYTES = 180 * 10**9          # usable HBM3e per GPU
B200_HBM_GBS_MEASURED = 6545.6        # copy bandwidth measured on this machine (GB/s)
B200_TENSOR_TFLOPS_SUSTAINED = 1433.0  # dense BF16/FP16 cuBLAS, sustained (TFLOP/s)


# ----------------------------------------------------------------------------- memory (Section 3.4.3)
def layer_param_count(shape: Shape) -> int:
    """Parameters of one decoder layer: Q, K, V, O projections, gate / up / down, two norm gains."""
    d, qd, kvd, f = shape.hidden, shape.n_q_heads * shape.head_dim, shape.n_kv_heads * shape.head_dim, shape.ffn
    return qd * d + 2 * kvd * d + d * qd + 3 * f * d + 2 * d


def model_param_count(shape: Shape) -> int:
    """All layers, plus embedding, final norm and LM head when the configuration has a vocabulary."""
    n = shape.n_layers * layer_param_count(shape)
    if shape.vocab > 0:
        n += 2 * shape.vocab * shape.hidden + shape.hidden
    return n


def params_bytes_per_device(shape: Shape, tp: int = 1, pp: int = 1, d_size: int = FP16_BYTES) -> float:
    """Params_per_cluster = Model_size / (TP * PP)."""
    return model_param_count(shape) * d_size / (tp * pp)


def kv_bytes_per_device(shape: Shape, batch: int, s_max: int, tp: int = 1, d_size: int = FP16_BYTES) -> float:
    """Decode stage: KV_per_cluster = B_micro * S_max * 2 * D_size * D_kv * L / TP.

    The paper writes D_emb for the width of a key / value row (its models use multi-head attention); with
    grouped-query attention the row is n_kv_heads * head_dim wide, which is D_emb when the two coincide.
    """
    kv_dim = shape.n_kv_heads * shape.head_dim
    return batch * s_max * 2 * d_size * kv_dim * shape.n_layers / tp


def fits(params_bytes: float, kv_bytes: float, overhead_bytes: float, budget_bytes: float) -> bool:
    """The constraint Params + KV + Overhead < budget."""
    return params_bytes + kv_bytes + overhead_bytes < budget_bytes


# ----------------------------------------------------------------------------- traffic
def comm_tp_bytes(batch: int, d_emb: int, tp: int, d_size: int = FP16_BYTES) -> int:
    """Comm_TP = B * 2 * D_emb * D_size * (TP - 1): All-Reduce volume of one decode step of one layer
    (two reductions per layer, after attention and after the FFN)."""
    return batch * 2 * d_emb * d_size * (tp - 1)


# ----------------------------------------------------------------------------- time
def layer_time_tp(t_norm: float, t_attn: float, t_ffn: float, tp: int = 1, t_all_reduce: float = 0.0,
                  t_launch_group: float = 0.0) -> float:
    """T_clu = T_norm + T_attn / TP + T_norm + T_ffn / TP + 2 T_allreduce + 2 T_launch_group
    (TP = 1: no reduction and no group launch, the single-device time)."""
    if tp == 1:
        return 2 * t_norm + t_attn + t_ffn
    return 2 * t_norm + (t_attn + t_ffn) / tp + 2 * t_all_reduce + 2 * t_launch_group


def pool_devices(dp_p: int, pp_p: int, tp_d: int, pp_d: int, b_p: int) -> int:
    """Clu_pool = DP_P * PP_P + TP_D * PP_D + B_P."""
    return dp_p * pp_p + tp_d * pp_d + b_p


def search_dp_p(t_p: float, t_d: float, pp_p: int, tp_d: int, pp_d: int, b_p: int,
                candidates: Iterable[int] = range(1, 65)):
    """argmin over DP_P of Clu_pool * max(T_p / DP_P, T_d); returns (DP_P, objective).
    Ties go to the smaller DP_P (fewer devices)."""
    best = None
    for dp in candidates:
        cost = pool_devices(dp, pp_p, tp_d, pp_d, b_p) * max(t_p / dp, t_d)
        if best is None or cost < best[1]:
            best = (dp, cost)
    return best


# ----------------------------------------------------------------------------- B200 roofline estimates
def decode_step_seconds(shape: Shape, batch: int, keys: int, hbm_gbs: float = B200_HBM_GBS_MEASURED,
                        efficiency: float = 0.75) -> float:
    """One decode step of the whole stack at the HBM roofline: every weight once, every cached key and
    value of every request once.  `efficiency` is the fraction of the copy bandwidth the step reaches
    (0.75 - 0.81 measured for 1 - 16 requests on the 7B layer)."""
    weights = model_param_count(shape) * FP16_BYTES
    if shape.vocab > 0:
        weights -= shape.vocab * shape.hidden * FP16_BYTES  # the embedding is gathered, not streamed
    kv = kv_bytes_per_device(shape, batch, keys)
    return (weights + kv) / (hbm_gbs * 1e9 * efficiency)


def prefill_seconds(shape: Shape, batch: int, seq: int, tflops: float = B200_TENSOR_TFLOPS_SUSTAINED,
                    efficiency: float = 0.85) -> float:
    """Prefill of batch x seq tokens at the tensor roofline: 2 FLOPs per parameter and token for the
    projections plus causal attention 2 S^2 d per head and request (0.85 of sustained measured)."""
    tokens = batch * seq
    params = shape.n_layers * (layer_param_count(shape) - 2 * shape.hidden)
    if shape.vocab > 0:
        params_head = shape.vocab * shape.hidden  # only the last position of each request
        gemm = 2.0 * tokens * params + 2.0 * batch * params_head
    else:
        gemm = 2.0 * tokens * params
    attn = 2.0 * batch * shape.n_q_heads * seq * seq * shape.head_dim * shape.n_layers
    return (gemm + attn) / (tflops * 1e12 * efficiency)


# ----------------------------------------------------------------------------- single-device plan
@dataclasses.dataclass(frozen=True)
class Plan:
    max_batch: int          # requests per KV slot
    buf_slots: int          # Buf_max: slots of the bounded buffer between prefill and decode
    params_bytes: int
    kv_bytes_per_slot: int
    scratch_bytes: int
    free_bytes: int
    decode_step_s: float    # estimate at the full sequence length
    prefill_s: float        # estimate for one slot's prompts
    decode_tokens_per_s: float


def _scratch_estimate(shape: Shape, batch: int, s_max: int) -> int:
    """Activation scratch of one context (dominant terms of what thinfer_workspace_bytes asks for): the
    prefill activations of a full slot - normalised input, q, attention output, two residual buffers,
    two ping-pong buffers, the FFN activation - plus the FP32 logits of one row per request."""
    rows = batch * s_max
    qd = shape.n_q_heads * shape.head_dim
    act = rows * (5 * shape.hidden + 2 * qd + shape.ffn) * FP16_BYTES
    return act + 2 * batch * max(shape.vocab, 1) * 4


def plan_single_device(shape: Shape, s_max: int, prompt: int, budget_bytes: int = B200_HBM_BYTES,
                       want_slots: int = 2, max_batch_cap: int = 64, overhead_bytes: int = 2 * 10**9,
                       scratch_bytes: Optional[int] = None) -> Optional[Plan]:
    """Largest batch per slot (up to the library's limit of 64 decode rows) such that the weights,
    `want_slots` KV slots and the scratch fit the budget; then as many extra slots as still fit.
    Returns None when not even one request fits beside the weights."""
    params = int(params_bytes_per_device(shape))
    best = None
    for batch in range(max_batch_cap, 0, -1):
        kv_slot = int(kv_bytes_per_device(shape, batch, s_max))
        scratch = scratch_bytes if scratch_bytes is not None else _scratch_estimate(shape, batch, s_max)
        if fits(params, want_slots * kv_slot + scratch, overhead_bytes, budget_bytes):
            free = budget_bytes - params - scratch - overhead_bytes
            slots = max(want_slots, int(free // kv_slot)) if kv_slot > 0 else want_slots
            while slots > want_slots and not fits(params, slots * kv_slot + scratch, overhead_bytes, budget_bytes):
                slots -= 1
            t_d = decode_step_seconds(shape, batch, s_max)
            best = Plan(batch, slots, params, kv_slot, scratch, free - slots * kv_slot, t_d,
                        prefill_seconds(shape, batch, prompt), batch / t_d)
            break
    return best


def main(argv=None) -> int:
    import argparse
    import json
    from . import synth
    ap = argparse.ArgumentParser(description="batch and buffer sizes for one B200 (Section 3.4.3 memory model)")
    ap.add_argument("--model", choices=["7b", "13b", "70b"], default="7b")
    ap.add_argument("--s-max", type=int, default=640, help="positions per request (prompt + generated)")
    ap.add_argument("--prompt", type=int, default=512)
    ap.add_argument("--mem-gb", type=float, default=180.0)
    ap.add_argument("--slots", type=int, default=2, help="KV slots wanted at least (Buf_max)")
    a = ap.parse_args(argv)
    shape = {"7b": synth.LLAMA_7B, "13b": synth.LLAMA_13B, "70b": synth.LLAMA_70B}[a.model]
    plan = plan_single_device(shape, a.s_max, a.prompt, int(a.mem_gb * 1e9), a.slots)
    print(json.dumps(dataclasses.asdict(plan) if plan else {"fits": False}))
    return 0


if __name__ == "__main__":
    raise SystemExit(main())
