"""Seeded synthetic inputs shared by the tests, the smoke check and the benchmark.

This module holds none of the method's arithmetic: it only draws random FP16
tensors with the shapes and value distributions of the workloads (Section 4.1:
Llama-2 shaped models, prompts padded to a uniform length).  The trained
weights and the prompt data set the paper used are replaced by:

  matrices (projections, embedding, LM head)   FP16, N(0, 0.02)
  RMSNorm gains                                FP16, 1 + N(0, 0.02)
  hidden states (layer-only configurations)    FP16, N(0, 1)
  token ids                                    uniform in [0, vocab)

Every tensor has its own stream, keyed by (seed, layer, tensor id), so any one
of them can be regenerated without the others.

Two generators with the same recipe: numpy on the host for the small cases, and
torch's counter-based CUDA generator for the full-depth configurations, whose
weights (up to 138 GB) are drawn on the device tensor by tensor and never exist
on the host as a whole; a consumer on the host copies the one layer it needs.
The two generators give different values for the same key; a case uses one of
them throughout.
"""
from __future__ import annotations

import dataclasses
import numpy as np

LAYER_TENSORS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")
_STACK_TENSORS = ("embed", "final_norm", "lm_head")
_HIDDEN_ID = 100
_IDS_ID = 101


@dataclasses.dataclass(frozen=True)
class Shape:
    """Layer shapes of one configuration (names follow the C header)."""
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    n_layers: int = 1
    vocab: int = 0
    rms_eps: float = 1e-5
    rope_base: float = 10000.0


TINY = Shape(hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64, ffn=688)
LLAMA_7B_LAYER = Shape(hidden=4096, n_q_heads=32, n_kv_heads=32, head_dim=128, ffn=11008)
LLAMA_7B = dataclasses.replace(LLAMA_7B_LAYER, n_layers=32, vocab=32000)
LLAMA_13B = Shape(hidden=5120, n_q_heads=40, n_kv_heads=40, head_dim=128, ffn=13824,
                  n_layers=40, vocab=32000)
LLAMA_70B = Shape(hidden=8192, n_q_heads=64, n_kv_heads=8, head_dim=128, ffn=28672,
                  n_layers=80, vocab=32000)


def _rng(seed, layer, tensor_id):
    return np.random.default_rng(np.random.SeedSequence([int(seed), int(layer), int(tensor_id)]))


def _normal16(rng, shape, mean, std):
    # float32 draws keep the generation of the large matrices fast; the value a
    # consumer sees is the FP16 rounding of the draw.
    a = rng.standard_normal(size=shape, dtype=np.float32)
    a *= np.float32(std)
    if mean != 0.0:
        a += np.float32(mean)
    return a.astype(np.float16)


def layer_tensor_shape(shape: Shape, name: str):
    d, qd, kvd, f = shape.hidden, shape.n_q_heads * shape.head_dim, shape.n_kv_heads * shape.head_dim, shape.ffn
    return {
        "attn_norm": (d,), "ffn_norm": (d,),
        "wq": (qd, d), "wk": (kvd, d), "wv": (kvd, d), "wo": (d, qd),
        "w_gate": (f, d), "w_up": (f, d), "w_down": (d, f),
    }[name]


def layer_tensor(shape: Shape, seed: int, layer: int, name: str) -> np.ndarray:
    tid = LAYER_TENSORS.index(name)
    rng = _rng(seed, layer, tid)
    if name.endswith("_norm"):
        return _normal16(rng, layer_tensor_shape(shape, name), 1.0, 0.02)
    return _normal16(rng, layer_tensor_shape(shape, name), 0.0, 0.02)


def layer_weights(shape: Shape, seed: int = 0, layer: int = 0) -> dict:
    """All nine tensors of one layer, FP16, [out, in] row-major matrices."""
    return {n: layer_tensor(shape, seed, layer, n) for n in LAYER_TENSORS}


def stack_tensor(shape: Shape, seed: int, name: str) -> np.ndarray:
    tid = 50 + _STACK_TENSORS.index(name)
    rng = _rng(seed, 1 << 20, tid)
    if name == "final_norm":
        return _normal16(rng, (shape.hidden,), 1.0, 0.02)
    return _normal16(rng, (shape.vocab, shape.hidden), 0.0, 0.02)


def stack_weights(shape: Shape, seed: int = 0) -> dict:
    return {
        "layers": [layer_weights(shape, seed, l) for l in range(shape.n_layers)],
        "embed": stack_tensor(shape, seed, "embed"),
        "final_norm": stack_tensor(shape, seed, "final_norm"),
        "lm_head": stack_tensor(shape, seed, "lm_head"),
    }


def hidden_states(shape: Shape, seed: int, dims, stream: int = 0) -> np.ndarray:
    """FP16 N(0,1) hidden states of shape dims + (hidden,)."""
    rng = _rng(seed, stream, _HIDDEN_ID)
    return _normal16(rng, tuple(dims) + (shape.hidden,), 0.0, 1.0)


def token_ids(shape: Shape, seed: int, dims, stream: int = 0) -> np.ndarray:
    rng = _rng(seed, stream, _IDS_ID)
    return rng.integers(0, shape.vocab, size=tuple(dims), dtype=np.int32)


# --------------------------------------------------------------------------- #
# the same recipe drawn on the device (full-depth configurations)
# --------------------------------------------------------------------------- #
def _device_normal16(shape_, mean, std, key, device, dtype=None):
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(int(key))
    t = torch.empty(shape_, dtype=dtype or torch.float16, device=device)
    t.normal_(mean, std, generator=g)
    return t


def _key(seed, layer, tensor_id):
    return (int(seed) * 1_000_003 + int(layer)) * 1_009 + int(tensor_id) + 12_345


def device_layer_weights(shape: Shape, seed: int, layer: int, device="cuda:0", dtype=None) -> dict:
    """The nine tensors of one layer as CUDA tensors drawn on the device (float16, or dtype=torch.bfloat16)."""
    out = {}
    for tid, name in enumerate(LAYER_TENSORS):
        mean = 1.0 if name.endswith("_norm") else 0.0
        out[name] = _device_normal16(layer_tensor_shape(shape, name), mean, 0.02, _key(seed, layer, tid), device, dtype)
    return out


def device_stack_weights(shape: Shape, seed: int = 0, device="cuda:0", dtype=None) -> dict:
    """Whole model on the device: {"layers": [dict per layer], "embed", "final_norm", "lm_head"}."""
    out = {"layers": [device_layer_weights(shape, seed, l, device, dtype) for l in range(shape.n_layers)]}
    for i, name in enumerate(_STACK_TENSORS):
        dims = (shape.hidden,) if name == "final_norm" else (shape.vocab, shape.hidden)
        out[name] = _device_normal16(dims, 1.0 if name == "final_norm" else 0.0, 0.02,
                                     _key(seed, 1 << 20, 50 + i), device, dtype)
    return out


def model_bytes(shape: Shape) -> int:
    """FP16 bytes of all weights of a stack configuration."""
    per_layer = sum(int(np.prod(layer_tensor_shape(shape, n))) for n in LAYER_TENSORS)
    stack = (2 * shape.vocab * shape.hidden + shape.hidden) if shape.vocab > 0 else 0
    return 2 * (per_layer * shape.n_layers + stack)
