"""Pins for the oracle's layer and stack: invariants the method fixes
(incremental decode == last row of a full prefill, batch independence),
degenerate cases with a known answer, and an independent torch float64 layer
assembled from library routines."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2605_25655_b200 import synth


def _cfg(shape):
    return O.Config(hidden=shape.hidden, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                    head_dim=shape.head_dim, ffn=shape.ffn, n_layers=shape.n_layers, vocab=shape.vocab,
                    rms_eps=shape.rms_eps, rope_base=shape.rope_base)


SMALL = synth.Shape(hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=96)
SMALL_STACK = synth.Shape(hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=96, n_layers=3, vocab=50)


def test_decode_equals_last_row_of_prefill():
    cfg = _cfg(synth.TINY)
    w = synth.layer_weights(synth.TINY, seed=0)
    x = synth.hidden_states(synth.TINY, 0, (2, 12))
    full, kc, vc = O.layer_prefill(cfg, w, x)
    # prefill 8 tokens, then decode tokens 8..11 one at a time
    out8, k, v = O.layer_prefill(cfg, w, x[:, :8])
    np.testing.assert_allclose(out8, full[:, :8], rtol=1e-9, atol=1e-12)
    for t in range(8, 12):
        xt, k, v = O.layer_decode(cfg, w, x[:, t], k, v, t)
        np.testing.assert_allclose(xt, full[:, t], rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(k, kc, rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(v, vc, rtol=1e-10, atol=1e-13)


def test_batch_independence():
    cfg = _cfg(SMALL)
    w = synth.layer_weights(SMALL, seed=3)
    x = synth.hidden_states(SMALL, 3, (3, 6)).astype(np.float64)
    base, _, _ = O.layer_prefill(cfg, w, x)
    x2 = x.copy()
    x2[1] = -7.0 * x2[1] + 1.0
    out, _, _ = O.layer_prefill(cfg, w, x2)
    np.testing.assert_array_equal(out[0], base[0])
    np.testing.assert_array_equal(out[2], base[2])
    assert not np.allclose(out[1], base[1])


def test_zero_output_projections_make_the_layer_the_identity():
    cfg = _cfg(SMALL)
    w = synth.layer_weights(SMALL, seed=1)
    w["wo"] = np.zeros_like(w["wo"])
    w["w_down"] = np.zeros_like(w["w_down"])
    x = synth.hidden_states(SMALL, 1, (1, 5))
    out, _, _ = O.layer_prefill(cfg, w, x)
    np.testing.assert_array_equal(out, x.astype(np.float64))


def test_cache_holds_rotated_keys_and_plain_values():
    cfg = _cfg(SMALL)
    w = synth.layer_weights(SMALL, seed=2)
    x = synth.hidden_states(SMALL, 2, (1, 4))
    _, kc, vc = O.layer_prefill(cfg, w, x)
    h = O.rmsnorm(x[0], w["attn_norm"], cfg.rms_eps)
    v_plain = (h @ w["wv"].astype(np.float64).T).reshape(4, SMALL.n_kv_heads, SMALL.head_dim)
    np.testing.assert_allclose(vc[0], v_plain.transpose(1, 0, 2), rtol=1e-12)
    k_plain = (h @ w["wk"].astype(np.float64).T).reshape(4, SMALL.n_kv_heads, SMALL.head_dim).transpose(1, 0, 2)
    np.testing.assert_allclose(kc[0][:, 0], k_plain[:, 0], rtol=1e-12)        # position 0: no rotation
    assert not np.allclose(kc[0][:, 3], k_plain[:, 3])                         # position 3: rotated
    np.testing.assert_allclose(np.linalg.norm(kc[0], axis=-1), np.linalg.norm(k_plain, axis=-1), rtol=1e-12)


def _torch_layer(shape, w, x):
    """An independent float64 layer built from torch library routines, with the
    rotation written as a complex multiply (not the oracle's even/odd form)."""
    t = lambda a: torch.from_numpy(np.asarray(a).astype(np.float64))
    xb = t(x)
    b_sz, s_len, dm = xb.shape
    hq, hkv, d = shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    F = torch.nn.functional
    h = F.rms_norm(xb, (dm,), t(w["attn_norm"]), eps=shape.rms_eps)
    q = F.linear(h, t(w["wq"])).view(b_sz, s_len, hq, d)
    k = F.linear(h, t(w["wk"])).view(b_sz, s_len, hkv, d)
    v = F.linear(h, t(w["wv"])).view(b_sz, s_len, hkv, d)
    freqs = torch.outer(torch.arange(s_len, dtype=torch.float64),
                        shape.rope_base ** (-torch.arange(0, d, 2, dtype=torch.float64) / d))
    rot = torch.polar(torch.ones_like(freqs), freqs)[None, :, None, :]
    rope = lambda a: torch.view_as_real(torch.view_as_complex(a.reshape(*a.shape[:-1], d // 2, 2)) * rot).flatten(-2)
    q, k = rope(q), rope(k)
    kr = k.repeat_interleave(hq // hkv, dim=2)
    vr = v.repeat_interleave(hq // hkv, dim=2)
    a = F.scaled_dot_product_attention(q.transpose(1, 2), kr.transpose(1, 2), vr.transpose(1, 2), is_causal=True)
    a = a.transpose(1, 2).reshape(b_sz, s_len, hq * d)
    x1 = xb + F.linear(a, t(w["wo"]))
    h2 = F.rms_norm(x1, (dm,), t(w["ffn_norm"]), eps=shape.rms_eps)
    x2 = x1 + F.linear(F.silu(F.linear(h2, t(w["w_gate"]))) * F.linear(h2, t(w["w_up"])), t(w["w_down"]))
    return x2.numpy(), k.permute(0, 2, 1, 3).numpy(), v.permute(0, 2, 1, 3).numpy()


@pytest.mark.parametrize("shape", [SMALL, synth.TINY])
def test_layer_matches_torch_library_layer(shape):
    cfg = _cfg(shape)
    w = synth.layer_weights(shape, seed=5)
    x = synth.hidden_states(shape, 5, (2, 10))
    out, kc, vc = O.layer_prefill(cfg, w, x)
    ref, kref, vref = _torch_layer(shape, w, x)
    np.testing.assert_allclose(out, ref, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(kc, kref, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(vc, vref, rtol=1e-10, atol=1e-12)


def test_stack_decode_continues_prefill():
    cfg = _cfg(SMALL_STACK)
    sw = synth.stack_weights(SMALL_STACK, seed=7)
    ids = synth.token_ids(SMALL_STACK, 7, (2, 9))
    logits_full, _, _, hid_full = O.stack_prefill(cfg, sw, ids)
    _, _, caches, _ = O.stack_prefill(cfg, sw, ids[:, :8])
    logits_inc, nxt, caches, hid_inc = O.stack_decode(cfg, sw, ids[:, 8], caches, 8)
    np.testing.assert_allclose(logits_inc, logits_full, rtol=1e-8, atol=1e-10)
    for a, b in zip(hid_inc, hid_full):
        np.testing.assert_allclose(a, b[:, -1], rtol=1e-8, atol=1e-10)
    np.testing.assert_array_equal(nxt, np.argmax(logits_full, axis=-1))
    assert caches[0][0].shape == (2, SMALL_STACK.n_kv_heads, 9, SMALL_STACK.head_dim)


def test_stack_loop_matches_a_composition_of_independent_torch_layers():
    # pins the layer loop of the stack: embedding lookup, L independent torch float64 layers chained by hand,
    # torch rms_norm + linear for the head.  The synthetic weights are scaled up so that every layer changes
    # the hidden state by a large fraction of its size; a loop that reused layer 0's weights, skipped a layer
    # or fed a layer the wrong hidden state fails here (and the variants below prove that this check can fail).
    cfg = _cfg(SMALL_STACK)
    sw = synth.stack_weights(SMALL_STACK, seed=21)
    for w in sw["layers"]:
        for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"):
            w[n] = (w[n].astype(np.float32) * 8).astype(np.float16)
    ids = synth.token_ids(SMALL_STACK, 21, (2, 7))
    logits, nxt, caches, hid = O.stack_prefill(cfg, sw, ids)

    F = torch.nn.functional
    x = torch.from_numpy(sw["embed"].astype(np.float64))[torch.from_numpy(ids.astype(np.int64))].numpy()
    per_layer = []
    for l, w in enumerate(sw["layers"]):
        x_prev = x
        x, k, v = _torch_layer(SMALL_STACK, w, x)
        per_layer.append(x)
        np.testing.assert_allclose(hid[l], x, rtol=1e-9, atol=1e-11, err_msg=f"hidden state after layer {l}")
        np.testing.assert_allclose(caches[l][0], k, rtol=1e-9, atol=1e-11, err_msg=f"K cache of layer {l}")
        np.testing.assert_allclose(caches[l][1], v, rtol=1e-9, atol=1e-11, err_msg=f"V cache of layer {l}")
        # the layers are far from the identity and from each other, so the comparisons above can tell them apart
        assert np.linalg.norm(x - x_prev) > 0.05 * np.linalg.norm(x_prev)
    hn = F.rms_norm(torch.from_numpy(x[:, -1]), (SMALL_STACK.hidden,),
                    torch.from_numpy(sw["final_norm"].astype(np.float64)), eps=cfg.rms_eps)
    ref_logits = F.linear(hn, torch.from_numpy(sw["lm_head"].astype(np.float64))).numpy()
    np.testing.assert_allclose(logits, ref_logits, rtol=1e-9, atol=1e-11)
    np.testing.assert_array_equal(nxt, np.argmax(ref_logits, axis=-1))

    # the mistakes this pin is there to catch do change the result: layer 0's weights used everywhere,
    # and two layers swapped
    wrong = dict(sw, layers=[sw["layers"][0]] * 3)
    _, _, _, hid_wrong = O.stack_prefill(cfg, wrong, ids)
    assert not np.allclose(hid_wrong[1], per_layer[1], rtol=1e-3, atol=1e-6)
    swapped = dict(sw, layers=[sw["layers"][1], sw["layers"][0], sw["layers"][2]])
    _, _, _, hid_swapped = O.stack_prefill(cfg, swapped, ids)
    assert not np.allclose(hid_swapped[2], per_layer[2], rtol=1e-3, atol=1e-6)

    # the decode loop: one more token through stack_decode equals the torch composition over 8 tokens
    ids8 = np.concatenate([ids, synth.token_ids(SMALL_STACK, 22, (2, 1))], axis=1)
    lg_dec, _, caches2, hid_dec = O.stack_decode(cfg, sw, ids8[:, 7], caches, 7)
    x = torch.from_numpy(sw["embed"].astype(np.float64))[torch.from_numpy(ids8.astype(np.int64))].numpy()
    for l, w in enumerate(sw["layers"]):
        x, k, v = _torch_layer(SMALL_STACK, w, x)
        np.testing.assert_allclose(hid_dec[l], x[:, -1], rtol=1e-8, atol=1e-10, err_msg=f"decode hidden, layer {l}")
        np.testing.assert_allclose(caches2[l][0], k, rtol=1e-8, atol=1e-10)
    hn = F.rms_norm(torch.from_numpy(x[:, -1]), (SMALL_STACK.hidden,),
                    torch.from_numpy(sw["final_norm"].astype(np.float64)), eps=cfg.rms_eps)
    np.testing.assert_allclose(lg_dec, F.linear(hn, torch.from_numpy(sw["lm_head"].astype(np.float64))).numpy(),
                               rtol=1e-8, atol=1e-10)


def test_oracle_accepts_float64_inputs_without_changing_results():
    # weights that were widened to float64 beforehand (the large-configuration tests do that once per layer)
    # give bit-identical results to the FP16 arrays they came from
    cfg = _cfg(SMALL)
    w = synth.layer_weights(SMALL, seed=4)
    x = synth.hidden_states(SMALL, 4, (2, 6))
    a, ka, va = O.layer_prefill(cfg, w, x)
    w64 = {k: v.astype(np.float64) for k, v in w.items()}
    b, kb, vb = O.layer_prefill(cfg, w64, x.astype(np.float64))
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(ka, kb)
    np.testing.assert_array_equal(va, vb)


def test_stack_embedding_and_head():
    # zero projections everywhere: hidden == embedding row; logits = head(RMSNorm(embedding row))
    cfg = _cfg(SMALL_STACK)
    sw = synth.stack_weights(SMALL_STACK, seed=8)
    for w in sw["layers"]:
        w["wo"] = np.zeros_like(w["wo"])
        w["w_down"] = np.zeros_like(w["w_down"])
    ids = np.array([[3, 11, 49]], dtype=np.int32)
    logits, nxt, _, hid = O.stack_prefill(cfg, sw, ids)
    e = sw["embed"].astype(np.float64)
    np.testing.assert_array_equal(hid[-1][0], e[[3, 11, 49]])
    ref = torch.nn.functional.rms_norm(torch.from_numpy(e[49]), (64,),
                                       torch.from_numpy(sw["final_norm"].astype(np.float64)), eps=cfg.rms_eps)
    np.testing.assert_allclose(logits[0], (sw["lm_head"].astype(np.float64) @ ref.numpy()), rtol=1e-11)


def test_fp16_storage_emulation_stays_close_but_is_not_the_criterion():
    cfg = _cfg(synth.TINY)
    w = synth.layer_weights(synth.TINY, seed=0)
    x = synth.hidden_states(synth.TINY, 0, (1, 16))
    exact, _, _ = O.layer_prefill(cfg, w, x)
    emu, _, _ = O.layer_prefill(cfg, w, x, emulate_fp16=True)
    rms = np.sqrt(np.mean(exact * exact, axis=-1, keepdims=True))
    assert np.max(np.abs(emu - exact) / rms) < 5e-3


def test_synth_is_reproducible_and_distributed_as_stated():
    a = synth.layer_tensor(synth.TINY, 0, 0, "wq")
    b = synth.layer_tensor(synth.TINY, 0, 0, "wq")
    np.testing.assert_array_equal(a, b)
    assert a.dtype == np.float16 and a.shape == (256, 256)
    assert abs(float(a.astype(np.float64).std()) - 0.02) < 1e-3
    g = synth.layer_tensor(synth.TINY, 0, 0, "attn_norm").astype(np.float64)
    assert abs(g.mean() - 1.0) < 0.01
    assert not np.array_equal(a, synth.layer_tensor(synth.TINY, 0, 1, "wq"))
    assert not np.array_equal(synth.layer_tensor(synth.TINY, 0, 0, "wk"), synth.layer_tensor(synth.TINY, 0, 0, "wv"))
    ids = synth.token_ids(synth.LLAMA_7B, 0, (4, 16))
    assert ids.min() >= 0 and ids.max() < 32000 and ids.dtype == np.int32
