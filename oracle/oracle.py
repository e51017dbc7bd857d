"""CPU oracle for the FP16 Llama-style decoder forward (prefill and decode).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition of what the
CUDA path must compute.  It shares no code with the CUDA path and is imported
only by the tests, by the smoke check and by the benchmark's CPU-baseline leg.
The product never routes through it.

Arithmetic: every input is taken as the exact value of its FP16 bit pattern,
converted to float64, and everything after that is float64 (the paper asks for
FP16 storage with FP32 accumulation and FP32 reductions, Section 3.2.4; float64
is the wider stand-in for "exact").  No blocking, fusion or re-ordering: each
function is the textbook definition of its operator, with numpy's matmul as the
only library step.

What each function follows:
  rmsnorm            Section 3.2.4 (RMSNorm, reductions at higher precision)
  rope               Algorithm 1 (Linear-RoPE fusion: rotate output pairs by
                     row-position times theta)
  linear             Section 3.2.1, Y = X W with W given as [out, in]
  causal_attention   Eq. 6 with the three stages of Section 3.3.2 in order
                     (scores, scale + softmax, weights times V), causal
  decode_attention   Eq. 6 for a single query row over a cache of T keys
  swiglu             the FFN of the Llama layer the paper evaluates (Section 4.1)
  layer_prefill /    the per-layer order norm -> attention -> norm -> FFN of the
  layer_decode       time model in Section 3.4.3
  stack_*            embedding, L layers, final norm, LM head, greedy argmax

Pins (tests/test_oracle_*.py): closed forms, brute-force loops on tiny inputs,
invariants (RoPE norm / relative position, decode == last prefill row, batch
independence), torch CPU float64 library routines, and for the layer loop of
stack_prefill / stack_decode a hand-chained composition of independent torch
float64 layers with torch's embedding lookup, rms_norm and linear for the head.  Hidden-state values at
the large configurations have no printed reference in the paper: they are
pinned only through these functions ("parity unpinned by the paper" for the
large-shape values themselves).
"""
from __future__ import annotations

import dataclasses
import numpy as np


@dataclasses.dataclass(frozen=True)
class Config:
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    n_layers: int = 1
    vocab: int = 0
    rms_eps: float = 1e-5
    rope_base: float = 10000.0


def f64(a):
    """Exact widening of an FP16/FP32 array to float64 (an array that already is
    float64 is passed through, not copied)."""
    return np.asarray(a).astype(np.float64, copy=False)


# --------------------------------------------------------------------------- #
# operators
# --------------------------------------------------------------------------- #
def rmsnorm(x, gamma, eps):
    """y = x * gamma / sqrt(mean(x^2) + eps) over the last axis (no mean
    subtraction, no bias; eps inside the square root)."""
    x = f64(x)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x * f64(gamma) / np.sqrt(ms + eps)


def rope_angles(pos, head_dim, base):
    """angle[..., j] = pos * base**(-2j/head_dim), j = 0 .. head_dim/2 - 1."""
    j = np.arange(head_dim // 2, dtype=np.float64)
    theta = np.power(float(base), -2.0 * j / float(head_dim))
    return f64(pos)[..., None] * theta


def rope(y, pos, base):
    """Rotate adjacent pairs (2j, 2j+1) of the last axis (one head) by
    pos * theta_j (Algorithm 1: result = y*cos + mix*sin, where mix is the
    pair-swapped copy of y with the first of each pair negated).

    y: [..., head_dim]; pos: broadcastable to y.shape[:-1].
    """
    y = f64(y)
    d = y.shape[-1]
    ang = rope_angles(np.broadcast_to(f64(pos), y.shape[:-1]), d, base)
    c, s = np.cos(ang), np.sin(ang)
    even, odd = y[..., 0::2], y[..., 1::2]
    out = np.empty_like(y)
    out[..., 0::2] = even * c - odd * s
    out[..., 1::2] = odd * c + even * s
    return out


def linear(x, w):
    """y[r, n] = sum_k x[r, k] * w[n, k]   (w stored [out, in])."""
    return f64(x) @ f64(w).T


def silu(z):
    z = f64(z)
    return z / (1.0 + np.exp(-z))


def swiglu(gate, up):
    return silu(gate) * f64(up)


def softmax_rows(s):
    """Max-subtracted softmax over the last axis; -inf entries get weight 0."""
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def causal_attention(q, k, v):
    """One request.  q [Hq, S, d], k and v [Hkv, S, d] -> [S, Hq*d].

    Query head h uses kv head h // (Hq // Hkv).  Stage 1: scores = q k^T.
    Stage 2: scale by 1/sqrt(d), mask keys t > s to -inf, softmax.
    Stage 3: weights times v."""
    q, k, v = f64(q), f64(k), f64(v)
    hq, s_len, d = q.shape
    g = hq // k.shape[0]
    out = np.empty((s_len, hq * d), dtype=np.float64)
    future = np.triu(np.ones((s_len, s_len), dtype=bool), k=1)
    for h in range(hq):
        scores = q[h] @ k[h // g].T                      # stage 1
        scores = scores / np.sqrt(float(d))              # stage 2
        scores = np.where(future, -np.inf, scores)
        p = softmax_rows(scores)
        out[:, h * d:(h + 1) * d] = p @ v[h // g]        # stage 3
    return out


def decode_attention(q, k, v):
    """One request, one new token.  q [Hq, d]; k, v [Hkv, T, d] hold every key
    and value up to and including the new token -> [Hq*d]."""
    q, k, v = f64(q), f64(k), f64(v)
    hq, d = q.shape
    g = hq // k.shape[0]
    out = np.empty(hq * d, dtype=np.float64)
    for h in range(hq):
        scores = (k[h // g] @ q[h]) / np.sqrt(float(d))
        p = softmax_rows(scores)
        out[h * d:(h + 1) * d] = p @ v[h // g]
    return out


def argmax_lowest(logits):
    """Greedy pick; exact ties go to the lowest index."""
    return np.argmax(f64(logits), axis=-1).astype(np.int64)


# --------------------------------------------------------------------------- #
# layer
# --------------------------------------------------------------------------- #
def _round16(a, on):
    """Diagnostic only: emulate an FP16 store."""
    return a.astype(np.float16).astype(np.float64) if on else a


def qkv_rope(cfg, w, x, pos, emulate_fp16=False):
    """RMSNorm -> q, k, v projections -> RoPE on q and k.

    x [..., D], pos broadcastable to x.shape[:-1].
    Returns q [..., Hq, d], k [..., Hkv, d] (rotated), v [..., Hkv, d]."""
    d = cfg.head_dim
    h = rmsnorm(x, w["attn_norm"], cfg.rms_eps)
    lead = h.shape[:-1]
    h2 = h.reshape(-1, cfg.hidden)
    q = linear(h2, w["wq"]).reshape(*lead, cfg.n_q_heads, d)
    k = linear(h2, w["wk"]).reshape(*lead, cfg.n_kv_heads, d)
    v = linear(h2, w["wv"]).reshape(*lead, cfg.n_kv_heads, d)
    p = np.broadcast_to(f64(pos), lead)[..., None]
    q = rope(q, p, cfg.rope_base)
    k = rope(k, p, cfg.rope_base)
    return _round16(q, emulate_fp16), _round16(k, emulate_fp16), _round16(v, emulate_fp16)


def ffn_block(cfg, w, x1, emulate_fp16=False):
    """x2 = x1 + down(silu(gate(h2)) * up(h2)),  h2 = RMSNorm(x1)."""
    lead = x1.shape[:-1]
    h2 = rmsnorm(x1, w["ffn_norm"], cfg.rms_eps).reshape(-1, cfg.hidden)
    a = _round16(swiglu(linear(h2, w["w_gate"]), linear(h2, w["w_up"])), emulate_fp16)
    return _round16(f64(x1) + linear(a, w["w_down"]).reshape(*lead, cfg.hidden), emulate_fp16)


def layer_prefill(cfg, w, x, emulate_fp16=False):
    """x [B, S, D] -> (x2 [B, S, D], K [B, Hkv, S, d], V [B, Hkv, S, d]).

    Positions are the index inside each sequence (0 .. S-1); K is returned
    after RoPE, which is what the cache holds."""
    x = f64(x)
    b_sz, s_len, _ = x.shape
    pos = np.arange(s_len, dtype=np.float64)[None, :]
    q, k, v = qkv_rope(cfg, w, x, pos, emulate_fp16)
    kc = np.ascontiguousarray(k.transpose(0, 2, 1, 3))   # [B, Hkv, S, d]
    vc = np.ascontiguousarray(v.transpose(0, 2, 1, 3))
    attn = np.empty((b_sz, s_len, cfg.n_q_heads * cfg.head_dim), dtype=np.float64)
    for b in range(b_sz):                                # attention is per request
        attn[b] = causal_attention(q[b].transpose(1, 0, 2), kc[b], vc[b])
    attn = _round16(attn, emulate_fp16)
    x1 = _round16(x + linear(attn.reshape(-1, attn.shape[-1]), w["wo"]).reshape(x.shape), emulate_fp16)
    x2 = ffn_block(cfg, w, x1, emulate_fp16)
    return x2, kc, vc


def layer_decode(cfg, w, x, k_cache, v_cache, pos, emulate_fp16=False):
    """One new token per request.  x [B, D]; k_cache, v_cache [B, Hkv, pos, d]
    hold positions 0 .. pos-1.  Returns (x2 [B, D], k_cache', v_cache') with the
    new token's key and value appended at index pos."""
    x = f64(x)
    b_sz = x.shape[0]
    q, k, v = qkv_rope(cfg, w, x, np.full((b_sz,), float(pos)), emulate_fp16)
    k_cache = np.concatenate([f64(k_cache), k[:, :, None, :]], axis=2)
    v_cache = np.concatenate([f64(v_cache), v[:, :, None, :]], axis=2)
    attn = np.empty((b_sz, cfg.n_q_heads * cfg.head_dim), dtype=np.float64)
    for b in range(b_sz):
        attn[b] = decode_attention(q[b], k_cache[b], v_cache[b])
    attn = _round16(attn, emulate_fp16)
    x1 = _round16(x + linear(attn, w["wo"]), emulate_fp16)
    x2 = ffn_block(cfg, w, x1, emulate_fp16)
    return x2, k_cache, v_cache


# --------------------------------------------------------------------------- #
# stack
# --------------------------------------------------------------------------- #
def head_logits(cfg, sw, x_last):
    """Final RMSNorm then LM head; x_last [B, D] -> logits [B, V]."""
    return linear(rmsnorm(x_last, sw["final_norm"], cfg.rms_eps), sw["lm_head"])


def stack_prefill(cfg, sw, ids, emulate_fp16=False):
    """ids int [B, S] -> (logits of the last position [B, V], next ids [B],
    caches: list over layers of (K, V), hidden states after every layer)."""
    x = f64(sw["embed"])[np.asarray(ids)]
    caches, hiddens = [], []
    for w in sw["layers"]:
        x, kc, vc = layer_prefill(cfg, w, x, emulate_fp16)
        caches.append((kc, vc))
        hiddens.append(x)
    logits = head_logits(cfg, sw, x[:, -1, :])
    return logits, argmax_lowest(logits), caches, hiddens


def stack_decode(cfg, sw, ids, caches, pos, emulate_fp16=False):
    """ids int [B] (one token per request at position pos) ->
    (logits [B, V], next ids [B], updated caches, hidden after every layer)."""
    x = f64(sw["embed"])[np.asarray(ids)]
    new_caches, hiddens = [], []
    for w, (kc, vc) in zip(sw["layers"], caches):
        x, kc, vc = layer_decode(cfg, w, x, kc, vc, pos, emulate_fp16)
        new_caches.append((kc, vc))
        hiddens.append(x)
    logits = head_logits(cfg, sw, x)
    return logits, argmax_lowest(logits), new_caches, hiddens


# --------------------------------------------------------------------------- #
# the paper's roofline arithmetic (Section 3.2.1), used to pin the benchmark's
# own roofline calculator
# --------------------------------------------------------------------------- #
def gemm_intensity_mac_per_byte(m, k, n, elem_bytes=4):
    """Eq. (intensity): multiply-accumulates per byte, I = MKN / (e (MK + KN + MN))."""
    return (m * k * n) / (elem_bytes * (m * k + k * n + m * n))


def intensity_threshold(peak_mac_per_s, bytes_per_s):
    """Eq. (threshold): peak / bandwidth."""
    return peak_mac_per_s / bytes_per_s


def attainable(peak, bandwidth, intensity):
    """Eq. (pmax): min(peak, bandwidth * intensity)."""
    return min(peak, bandwidth * intensity)


def linear_gmacs(rows, in_dim, out_dim, ms):
    """Section 4.4's Linear throughput: multiply-accumulates per second in
    units of 1e9 (the printed 5686.34 needs decimal giga)."""
    return rows * in_dim * out_dim / (ms * 1e-3) / 1e9
