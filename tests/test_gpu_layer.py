"""The layer and stack through the C ABI (thinfer_create / prefill / decode_step)
against the oracle on the same seeded inputs (run with -m gpu on a B200).

Per-layer checks are chained: the oracle is fed the same FP16 inputs as the GPU.
Tolerance: max |err| <= 2e-2 x row RMS and cosine >= 0.999 (tests/parity.py)."""
import dataclasses

import numpy as np
import pytest

from oracle import oracle as O
from paper_2605_25655_b200 import synth
from tests.parity import assert_rows_close, oracle_config

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def T():
    import torch
    from paper_2605_25655_b200 import thinfer
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    thinfer.lib()
    return torch, thinfer


def _ctx(T, shape, np_layers, max_batch, max_seq, stack=None, buf_slots=1):
    torch, thinfer = T
    layers = thinfer.to_device_layers(np_layers)
    st = {k: torch.from_numpy(v).cuda() for k, v in stack.items() if k != "layers"} if stack else None
    return thinfer.Context(shape, layers, st, max_batch=max_batch, max_seq=max_seq, buf_slots=buf_slots)


def _layer_case(T, shape, batch, seq, n_decode, seed=0, check_batches=None, max_seq=None, check_prefill=True,
                launch_mode=None):
    """Prefill `seq` tokens then `n_decode` decode steps on seeded hidden states; compare everything."""
    torch, thinfer = T
    cfg = oracle_config(shape)
    w = synth.layer_weights(shape, seed)
    x = synth.hidden_states(shape, seed, (batch, seq + n_decode))
    ctx = _ctx(T, shape, [w], batch, max_seq or (seq + n_decode))
    if launch_mode is not None:
        ctx.set_launch_mode(launch_mode)
    xd = torch.from_numpy(x).cuda()
    out = ctx.prefill(xd[:, :seq].contiguous())
    dec = [ctx.decode_step(xd[:, seq + i].contiguous()) for i in range(n_decode)]
    torch.cuda.synchronize()
    assert ctx.status() == 0
    assert ctx.slot_state(0) == (batch, seq + n_decode)
    bs = list(range(batch)) if check_batches is None else check_batches
    stats = []
    kg = ctx.kv_view(0, 0, 0).cpu().numpy()[bs]
    vg = ctx.kv_view(0, 0, 1).cpu().numpy()[bs]
    if check_prefill:
        ref, kc, vc = O.layer_prefill(cfg, w, x[bs, :seq])
        got = out.cpu().numpy()[bs]
        stats.append(assert_rows_close(got, ref, f"prefill B={batch} S={seq}"))
        assert_rows_close(kg[:, :, :seq], kc, "K cache after prefill", max_err=6e-3)
        assert_rows_close(vg[:, :, :seq], vc, "V cache after prefill", max_err=6e-3)
    else:
        assert np.all(np.isfinite(out.cpu().numpy().astype(np.float32)))
    # decode: the oracle continues from the GPU's own FP16 cache (chained check)
    k_run = kg[:, :, :seq].astype(np.float64)
    v_run = vg[:, :, :seq].astype(np.float64)
    for i in range(n_decode):
        r, k_run, v_run = O.layer_decode(cfg, w, x[bs, seq + i], k_run, v_run, seq + i)
        stats.append(assert_rows_close(dec[i].cpu().numpy()[bs], r, f"decode step {i} B={batch}"))
        kg = ctx.kv_view(0, 0, 0).cpu().numpy()[bs]
        vg = ctx.kv_view(0, 0, 1).cpu().numpy()[bs]
        assert_rows_close(kg[:, :, seq + i], k_run[:, :, seq + i], f"K append {i}", max_err=6e-3)
        assert_rows_close(vg[:, :, seq + i], v_run[:, :, seq + i], f"V append {i}", max_err=6e-3)
        k_run[:, :, seq + i] = kg[:, :, seq + i]
        v_run[:, :, seq + i] = vg[:, :, seq + i]
    ctx.close()
    return stats


def test_tiny_config_prefill_then_decode(T):
    # configuration 1: hidden 256, 4 x 64 heads, FFN 688, batch 1, prompt 32, 8 decode steps
    _layer_case(T, synth.TINY, batch=1, seq=32, n_decode=8)


@pytest.mark.parametrize("batch,seq,n_decode", [(2, 1, 6), (3, 130, 3), (4, 77, 2), (16, 40, 2)])
def test_tiny_shapes_ragged(T, batch, seq, n_decode):
    _layer_case(T, synth.TINY, batch=batch, seq=seq, n_decode=n_decode, seed=batch)


# the same small layer with every dimension a multiple of 64: decode of up to 16 requests runs on the skinny
# projections (shares smaller than one 16-row tile, K shorter than the 8 warp slices, 1 .. 16 tokens, GQA)
@pytest.mark.parametrize("batch,seq,n_decode,hkv", [(1, 32, 8, 4), (2, 1, 6, 4), (3, 130, 3, 2), (5, 77, 2, 1),
                                                    (8, 33, 3, 4), (9, 20, 3, 2), (16, 40, 2, 4)])
def test_small_layer_on_skinny_projections(T, batch, seq, n_decode, hkv):
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=hkv, head_dim=64, ffn=704)
    _layer_case(T, shape, batch=batch, seq=seq, n_decode=n_decode, seed=batch)


# ---- launch mode 2: the whole decode step in one cooperative persistent kernel ---------------------
@pytest.mark.parametrize("batch,seq,n_decode", [(1, 32, 8), (2, 1, 6), (3, 130, 3), (16, 40, 3), (7, 5, 12)])
def test_unified_decode_kernel_tiny(T, batch, seq, n_decode):
    _layer_case(T, synth.TINY, batch=batch, seq=seq, n_decode=n_decode, seed=batch, launch_mode=2)


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 128), (8, 4, 64), (6, 2, 64), (8, 1, 128)])
def test_unified_decode_kernel_gqa(T, hq, hkv, d):
    shape = synth.Shape(hidden=512, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, ffn=1024)
    _layer_case(T, shape, batch=3, seq=150, n_decode=3, seed=4, launch_mode=2)


@pytest.mark.parametrize("batch", [1, 4, 16])
def test_unified_decode_kernel_llama7b_layer(T, batch):
    _layer_case(T, synth.LLAMA_7B_LAYER, batch=batch, seq=512, n_decode=3, check_batches=[0, batch - 1], max_seq=640,
                check_prefill=False, launch_mode=2)


def test_unified_decode_kernel_multi_layer_stack(T):
    # four layers in one launch: residual ping-pong, the next layer's norm folded into the down projection
    torch, thinfer = T
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=688, n_layers=4, vocab=1000)
    cfg = oracle_config(shape)
    sw = synth.stack_weights(shape, 5)
    ids = synth.token_ids(shape, 5, (3, 14))
    ctx = _ctx(T, shape, sw["layers"], 3, 16, stack=sw)
    ctx.set_launch_mode(2)
    idd = torch.from_numpy(ids).cuda()
    nxt, logits = ctx.prefill(idd[:, :9].contiguous(), want_logits=True)
    ref_logits, _, caches, _ = O.stack_prefill(cfg, sw, ids[:, :9])
    assert_rows_close(logits.cpu().numpy(), ref_logits, "prefill logits")
    for t in range(9, 14):
        nxt, logits = ctx.decode_step(idd[:, t].contiguous(), want_logits=True)
        ref_logits, _, caches, _ = O.stack_decode(cfg, sw, ids[:, t], caches, t)
        assert_rows_close(logits.cpu().numpy(), ref_logits, f"decode logits t={t}")
        _check_greedy(nxt.cpu().numpy(), logits.cpu().numpy(), ref_logits)
        for l in (0, 3):                                       # caches of the first and last layer
            kg = ctx.kv_view(0, l, 0).cpu().numpy()[:3, :, :t + 1]
            assert_rows_close(kg, caches[l][0], f"K cache layer {l} t={t}", max_err=8e-3)
    assert ctx.status() == 0
    ctx.close()


def test_unified_decode_kernel_is_deterministic(T):
    torch, thinfer = T
    shape = synth.TINY
    w = synth.layer_weights(shape, 6)
    x = torch.from_numpy(synth.hidden_states(shape, 6, (5, 40))).cuda()
    outs = []
    for rep in range(2):
        ctx = _ctx(T, shape, [w], 5, 48)
        ctx.set_launch_mode(2)
        res = [ctx.prefill(x[:, :33].contiguous())] + [ctx.decode_step(x[:, 33 + i].contiguous()) for i in range(7)]
        torch.cuda.synchronize()
        assert ctx.status() == 0
        outs.append([r.cpu().numpy() for r in res])
        ctx.close()
    for a, b in zip(*outs):
        np.testing.assert_array_equal(a, b)


@pytest.mark.parametrize("batch", [17, 33, 64])
def test_decode_with_more_than_16_requests(T, batch):
    # token tiles of 32 and 64 in the stream-K decode projections; launch mode 2 falls back to per-unit kernels
    for mode in (1, 2):
        _layer_case(T, synth.TINY, batch=batch, seq=9, n_decode=2, seed=batch, launch_mode=mode,
                    check_batches=[0, batch // 2, batch - 1])


def test_gqa_layer(T):
    shape = synth.Shape(hidden=512, n_q_heads=8, n_kv_heads=2, head_dim=128, ffn=1024)
    _layer_case(T, shape, batch=2, seq=150, n_decode=3, seed=4)


def test_decode_equals_last_row_of_prefill(T):
    # the cache is built one token at a time; each step must equal the oracle's full prefill row
    torch, thinfer = T
    shape = synth.TINY
    cfg = oracle_config(shape)
    w = synth.layer_weights(shape, 2)
    x = synth.hidden_states(shape, 2, (2, 20))
    ref, _, _ = O.layer_prefill(cfg, w, x)
    ctx = _ctx(T, shape, [w], 2, 32)
    xd = torch.from_numpy(x).cuda()
    first = ctx.prefill(xd[:, :1].contiguous())
    assert_rows_close(first.cpu().numpy(), ref[:, :1], "prefill of one token")
    for t in range(1, 20):
        out = ctx.decode_step(xd[:, t].contiguous())
        assert_rows_close(out.cpu().numpy(), ref[:, t], f"incremental decode t={t}")
    ctx.close()


def test_batch_independence(T):
    torch, thinfer = T
    shape = synth.TINY
    w = synth.layer_weights(shape, 0)
    x = synth.hidden_states(shape, 0, (3, 24))
    ctx = _ctx(T, shape, [w], 3, 32)
    xd = torch.from_numpy(x).cuda()
    base = ctx.prefill(xd.contiguous()).cpu().numpy()
    ctx.release_slot(0)
    x2 = x.copy()
    x2[1] = -x2[1]
    other = ctx.prefill(torch.from_numpy(x2).cuda()).cpu().numpy()
    np.testing.assert_array_equal(other[0], base[0])
    np.testing.assert_array_equal(other[2], base[2])
    assert not np.array_equal(other[1], base[1])
    ctx.close()


def test_llama7b_layer_batch1_full(T):
    # configuration 2 at batch 1: 512-token prompt, decode steps at T = 512, 513, 514
    _layer_case(T, synth.LLAMA_7B_LAYER, batch=1, seq=512, n_decode=3, max_seq=640)


@pytest.mark.parametrize("batch", [4, 16])
def test_llama7b_layer_batched_subset(T, batch):
    # configuration 2 at batch 4 / 16: first and last request checked (batch independence covers the rest)
    _layer_case(T, synth.LLAMA_7B_LAYER, batch=batch, seq=512, n_decode=2, check_batches=[0, batch - 1], max_seq=640)


def test_llama7b_layer_long_kv_decode(T):
    # decode attention over 1279 .. 1281 cached keys (the KV length configuration 4 reaches); the prompt is
    # processed on the GPU only, the decode steps are checked against the oracle continuing from that cache
    _layer_case(T, synth.LLAMA_7B_LAYER, batch=2, seq=1279, n_decode=2, max_seq=1281, check_prefill=False, seed=3)


def test_llama13b_layer_reduced_budget(T):
    # configuration 4's layer shape (hidden 5120, 40 x 128 heads, FFN 13824) on a reduced token budget
    shape = dataclasses.replace(synth.LLAMA_13B, n_layers=1, vocab=0)
    _layer_case(T, shape, batch=2, seq=64, n_decode=2, seed=13)


def test_llama70b_layer_reduced_budget(T):
    # configuration 5's layer shape (hidden 8192, 64 query / 8 KV heads, FFN 28672) on a reduced token budget
    # (batch 2 x 64 tokens of every one of the 80 layers is covered by tests/test_gpu_full_depth.py)
    shape = dataclasses.replace(synth.LLAMA_70B, n_layers=1, vocab=0)
    _layer_case(T, shape, batch=1, seq=3, n_decode=2, seed=71)        # batch 1: the FMA streaming path with 8:1 GQA


def test_llama7b_two_layer_stack_with_32000_vocab(T):
    # configuration 3's shapes at reduced depth: embedding, 2 layers, final norm, 32000-way head, greedy pick
    torch, thinfer = T
    shape = dataclasses.replace(synth.LLAMA_7B, n_layers=2)
    cfg = oracle_config(shape)
    sw = synth.stack_weights(shape, 3)
    for batch in (2, 1):
        ids = synth.token_ids(shape, 3, (batch, 34))
        ctx = _ctx(T, shape, sw["layers"], batch, 40, stack=sw)
        idd = torch.from_numpy(ids).cuda()
        nxt, logits = ctx.prefill(idd[:, :32].contiguous(), want_logits=True)
        ref_logits, _, caches, _ = O.stack_prefill(cfg, sw, ids[:, :32])
        assert_rows_close(logits.cpu().numpy(), ref_logits, "prefill logits")
        _check_greedy(nxt.cpu().numpy(), logits.cpu().numpy(), ref_logits)
        for t in range(32, 34):
            nxt, logits = ctx.decode_step(idd[:, t].contiguous(), want_logits=True)
            ref_logits, _, caches, _ = O.stack_decode(cfg, sw, ids[:, t], caches, t)
            assert_rows_close(logits.cpu().numpy(), ref_logits, f"decode logits t={t}")
            _check_greedy(nxt.cpu().numpy(), logits.cpu().numpy(), ref_logits)
        assert ctx.status() == 0
        ctx.close()


def test_stack_teacher_forced(T):
    torch, thinfer = T
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=688, n_layers=3, vocab=1000)
    cfg = oracle_config(shape)
    sw = synth.stack_weights(shape, 1)
    ids = synth.token_ids(shape, 1, (2, 20))
    ctx = _ctx(T, shape, sw["layers"], 2, 32, stack=sw)
    idd = torch.from_numpy(ids).cuda()
    nxt, logits = ctx.prefill(idd[:, :16].contiguous(), want_logits=True)
    ref_logits, ref_next, caches, _ = O.stack_prefill(cfg, sw, ids[:, :16])
    assert_rows_close(logits.cpu().numpy(), ref_logits, "prefill logits")
    _check_greedy(nxt.cpu().numpy(), logits.cpu().numpy(), ref_logits)
    for t in range(16, 20):                                   # teacher forced: both sides consume the same ids
        nxt, logits = ctx.decode_step(idd[:, t].contiguous(), want_logits=True)
        ref_logits, ref_next, caches, _ = O.stack_decode(cfg, sw, ids[:, t], caches, t)
        assert_rows_close(logits.cpu().numpy(), ref_logits, f"decode logits t={t}")
        _check_greedy(nxt.cpu().numpy(), logits.cpu().numpy(), ref_logits)
    assert ctx.status() == 0
    ctx.close()


def _check_greedy(ids, gpu_logits, ref_logits):
    # the GPU's pick is the lowest-index argmax of its own logits (bit exact), and agrees with the
    # oracle wherever the oracle's top-2 gap is larger than 4x the logit error
    np.testing.assert_array_equal(ids, np.argmax(gpu_logits, axis=-1))
    err = np.max(np.abs(gpu_logits - ref_logits), axis=-1)
    top2 = np.sort(ref_logits, axis=-1)[:, -2:]
    clear = (top2[:, 1] - top2[:, 0]) > 4 * err
    np.testing.assert_array_equal(ids[clear], np.argmax(ref_logits, axis=-1)[clear])


def test_errors_and_slots(T):
    torch, thinfer = T
    shape = synth.TINY
    w = synth.layer_weights(shape, 0)
    ctx = _ctx(T, shape, [w], 2, 8, buf_slots=2)
    x = torch.from_numpy(synth.hidden_states(shape, 0, (2, 8))).cuda()
    with pytest.raises(thinfer.ThinferError) as e:
        ctx.decode_step(x[:, 0].contiguous())                  # empty slot
    assert e.value.code == thinfer.EINVAL
    with pytest.raises(thinfer.ThinferError) as e:
        ctx.prefill(torch.cat([x, x], dim=1))                  # 16 > max_seq
    assert e.value.code == thinfer.ECAPACITY
    with pytest.raises(thinfer.ThinferError) as e:
        ctx.prefill(torch.cat([x, x, x], dim=0))               # batch 6 > max_batch
    assert e.value.code == thinfer.ECAPACITY
    a = ctx.prefill(x[:, :7].contiguous(), slot=0)
    with pytest.raises(thinfer.ThinferError) as e:
        ctx.prefill(x[:, :7].contiguous(), slot=0)             # back-pressure: slot not released
    assert e.value.code == thinfer.EBUSY
    b = ctx.prefill(x[:, :7].contiguous(), slot=1)             # the second slot is free
    np.testing.assert_array_equal(a.cpu().numpy(), b.cpu().numpy())
    ctx.decode_step(x[:, 7].contiguous(), slot=0)
    with pytest.raises(thinfer.ThinferError) as e:
        ctx.decode_step(x[:, 7].contiguous(), slot=0)          # slot full
    assert e.value.code == thinfer.ECAPACITY
    with pytest.raises(thinfer.ThinferError) as e:
        ctx.prefill(x, slot=5)
    assert e.value.code == thinfer.EINVAL
    ctx.release_slot(0)
    assert ctx.slot_state(0) == (0, 0)
    ctx.prefill(x[:, :3].contiguous(), slot=0)
    assert ctx.slot_state(0) == (2, 3) and ctx.slot_state(1) == (2, 7)
    assert ctx.launch_count() > 0 and ctx.status() == 0
    ctx.close()


def test_host_buffer_calls_match_device_calls(T):
    torch, thinfer = T
    shape = synth.TINY
    w = synth.layer_weights(shape, 3)
    x = torch.from_numpy(synth.hidden_states(shape, 3, (2, 12)))
    ctx = _ctx(T, shape, [w], 2, 16, buf_slots=2)
    dev = ctx.prefill(x[:, :11].contiguous().cuda(), slot=0)
    dev2 = ctx.decode_step(x[:, 11].contiguous().cuda(), slot=0)
    hin = x[:, :11].contiguous().pin_memory()
    hout = torch.empty_like(hin).pin_memory()
    ctx.prefill_host(hin, hout, slot=1)
    hin2 = x[:, 11].contiguous().pin_memory()
    hout2 = torch.empty_like(hin2).pin_memory()
    ctx.decode_step_host(hin2, hout2, slot=1)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(hout.numpy(), dev.cpu().numpy())
    np.testing.assert_array_equal(hout2.numpy(), dev2.cpu().numpy())
    ctx.close()


@pytest.mark.parametrize("batch", [1, 5])
def test_launch_modes_agree_bit_for_bit(T, batch):
    # plain launches and programmatic dependent launch (kernels start early and wait on the device)
    # run the same arithmetic in the same order: outputs and caches must be identical
    torch, thinfer = T
    shape = synth.TINY
    w = synth.layer_weights(shape, 6)
    x = torch.from_numpy(synth.hidden_states(shape, 6, (batch, 40))).cuda()
    outs = []
    for mode in (0, 1):
        ctx = _ctx(T, shape, [w], batch, 48)
        ctx.set_launch_mode(mode)
        res = [ctx.prefill(x[:, :33].contiguous())]
        res += [ctx.decode_step(x[:, 33 + i].contiguous()) for i in range(7)]
        torch.cuda.synchronize()
        assert ctx.status() == 0
        outs.append([r.cpu().numpy() for r in res] + [ctx.kv_view(0, 0, 0).cpu().numpy()[:, :, :40],
                                                      ctx.kv_view(0, 0, 1).cpu().numpy()[:, :, :40]])
        ctx.close()
    for a, b in zip(*outs):
        np.testing.assert_array_equal(a, b)


@pytest.mark.parametrize("ffn", [688, 704])
def test_prefill_and_decode_stages_on_two_streams(T, ffn):
    # the Prefill -> Buffer -> Decode schedule on one device: slot 1 is being prefilled on one stream while slot 0
    # decodes on another; the hand-off events order each slot's stages; results equal the serial run bit for bit
    torch, thinfer = T
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64, ffn=ffn)
    w = synth.layer_weights(shape, 9)
    x = torch.from_numpy(synth.hidden_states(shape, 9, (2, 3, 40))).cuda()     # two micro-batches of 3 requests

    # every input is materialised and the device synchronised before the streams start: a temporary made on
    # torch's current stream would neither be ordered with, nor kept alive for, work on the other streams
    pin = {"p0": x[0, :, :30].contiguous(), "p1": x[1, :, :30].contiguous(), "p0b": x[1, :, :25].contiguous(),
           "d0b": x[1, :, 25].contiguous()}
    d0 = [x[0, :, 30 + i].contiguous() for i in range(6)]
    d1 = [x[1, :, 30 + i].contiguous() for i in range(4)]

    def run(two_streams):
        ctx = _ctx(T, shape, [w], 3, 48, buf_slots=2)
        sp = torch.cuda.Stream() if two_streams else torch.cuda.current_stream()
        sd = torch.cuda.Stream() if two_streams else torch.cuda.current_stream()
        torch.cuda.synchronize()
        outs = {}
        outs["p0"] = ctx.prefill(pin["p0"], slot=0, stream=sp)
        outs["p1"] = ctx.prefill(pin["p1"], slot=1, stream=sp)      # runs while slot 0 decodes
        for i in range(6):
            outs[f"d0_{i}"] = ctx.decode_step(d0[i], slot=0, stream=sd)
        ctx.release_slot(0, stream=sd)
        outs["p0b"] = ctx.prefill(pin["p0b"], slot=0, stream=sp)    # waits for the release on the device
        for i in range(4):
            outs[f"d1_{i}"] = ctx.decode_step(d1[i], slot=1, stream=sd)
        outs["d0b"] = ctx.decode_step(pin["d0b"], slot=0, stream=sd)
        torch.cuda.synchronize()
        assert ctx.status() == 0
        res = {k: v.cpu().numpy() for k, v in outs.items()}
        ctx.close()
        return res

    serial, overlapped = run(False), run(True)
    for k in serial:
        np.testing.assert_array_equal(serial[k], overlapped[k], err_msg=k)


# ffn 688 is not a multiple of 64: decode runs on the FMA GEMV (one request) / stream-K tensor-core path;
# ffn 704 puts the same small layer on the skinny projections (per-request positions in their epilogue)
@pytest.mark.parametrize("ffn", [688, 704])
@pytest.mark.parametrize("lens,n_decode,mode", [((5, 17, 32), 4, 1), ((1, 64, 33, 7, 20), 3, 2), ((130,), 2, 1)])
def test_ragged_prompts_layer(T, lens, n_decode, mode, ffn):
    # prompts of different lengths in one batch: every request must equal the oracle run on that request alone
    torch, thinfer = T
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=4, head_dim=64, ffn=ffn)
    cfg = oracle_config(shape)
    w = synth.layer_weights(shape, 12)
    batch, pad = len(lens), max(lens)
    x = synth.hidden_states(shape, 12, (batch, pad + n_decode))
    ctx = _ctx(T, shape, [w], batch, pad + n_decode)
    ctx.set_launch_mode(mode)
    xd = torch.from_numpy(x).cuda()
    out = ctx.prefill_ragged(xd[:, :pad].contiguous(), lens).cpu().numpy()
    # decode inputs: request b consumes x[b, lens[b] + i] at step i (its own continuation)
    dec = []
    for i in range(n_decode):
        step_in = np.stack([x[b, lens[b] + i] for b in range(batch)])
        dec.append(ctx.decode_step(torch.from_numpy(step_in).cuda()).cpu().numpy())
        assert ctx.slot_lengths(0) == [l + i + 1 for l in lens]
    assert ctx.status() == 0
    for b in range(batch):
        ref, k, v = O.layer_prefill(cfg, w, x[b:b + 1, :lens[b]])
        assert_rows_close(out[b, :lens[b]], ref[0], f"request {b} prefill ({lens[b]} tokens)")
        kg = ctx.kv_view(0, 0, 0).cpu().numpy()[b, :, :lens[b]]
        assert_rows_close(kg, k[0], f"request {b} K cache", max_err=6e-3)
        for i in range(n_decode):
            r, k, v = O.layer_decode(cfg, w, x[b:b + 1, lens[b] + i], k, v, lens[b] + i)
            assert_rows_close(dec[i][b], r[0], f"request {b} decode step {i}")
    ctx.close()


@pytest.mark.parametrize("ffn", [688, 704])
def test_ragged_prompts_stack_logits(T, ffn):
    torch, thinfer = T
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=ffn, n_layers=2, vocab=1000)
    cfg = oracle_config(shape)
    sw = synth.stack_weights(shape, 13)
    lens = (9, 3, 14)
    ids = synth.token_ids(shape, 13, (3, 16))
    ctx = _ctx(T, shape, sw["layers"], 3, 20, stack=sw)
    nxt, logits = ctx.prefill_ragged(torch.from_numpy(ids[:, :14].copy()).cuda(), lens, want_logits=True)
    step_ids = np.array([ids[b, lens[b]] for b in range(3)], dtype=np.int32)
    nxt2, logits2 = ctx.decode_step(torch.from_numpy(step_ids).cuda(), want_logits=True)
    for b in range(3):
        ref, _, caches, _ = O.stack_prefill(cfg, sw, ids[b:b + 1, :lens[b]])
        assert_rows_close(logits.cpu().numpy()[b:b + 1], ref, f"request {b}: logits of its own last prompt token")
        ref2, _, _, _ = O.stack_decode(cfg, sw, ids[b:b + 1, lens[b]], caches, lens[b])
        assert_rows_close(logits2.cpu().numpy()[b:b + 1], ref2, f"request {b}: first decode step")
    with pytest.raises(thinfer.ThinferError) as e:
        ctx.release_slot(0)
        ctx.prefill_ragged(torch.from_numpy(ids[:, :14].copy()).cuda(), (9, 0, 14))
    assert e.value.code == thinfer.EINVAL
    ctx.close()


# ---- free-running greedy generation (Section 3.4.2: the prefill emits the first token, decode the rest) ----------
def _greedy_case(T, shape, seed, batch, prompt, n_new):
    """Generates n_new tokens per request with the ids fed back ON THE DEVICE (no host synchronisation inside the
    loop) and follows the oracle's own greedy run.  A request counts as agreeing until the first step at which
    the two picks differ; that may only happen where the oracle's top-2 gap is below 4x the logit error (both
    picks are then correct answers).  Returns (steps compared, steps agreeing, requests that ever diverged)."""
    torch, thinfer = T
    cfg = oracle_config(shape)
    sw = synth.stack_weights(shape, seed)
    ids0 = synth.token_ids(shape, seed, (batch, prompt))
    ctx = _ctx(T, shape, sw["layers"], batch, prompt + n_new, stack=sw)
    cur, lg = ctx.prefill(torch.from_numpy(ids0).cuda(), want_logits=True)
    gpu_ids, gpu_logits = [cur], [lg]
    for _ in range(n_new - 1):
        cur, lg = ctx.decode_step(cur, want_logits=True)       # the previous step's device tensor is the input
        gpu_ids.append(cur)
        gpu_logits.append(lg)
    torch.cuda.synchronize()
    assert ctx.status() == 0
    assert ctx.slot_state(0) == (batch, prompt + n_new - 1)
    gpu_ids = [t.cpu().numpy() for t in gpu_ids]
    gpu_logits = [t.cpu().numpy() for t in gpu_logits]
    ctx.close()

    ref_logits, ref_next, caches, _ = O.stack_prefill(cfg, sw, ids0)
    alive = np.ones(batch, dtype=bool)
    compared = agreed = 0
    for step in range(n_new):
        # the GPU's pick is always the lowest-index argmax of its own logits
        np.testing.assert_array_equal(gpu_ids[step], np.argmax(gpu_logits[step], axis=-1))
        for b in np.nonzero(alive)[0]:
            compared += 1
            err = np.max(np.abs(gpu_logits[step][b] - ref_logits[b]))
            top2 = np.sort(ref_logits[b])[-2:]
            if gpu_ids[step][b] == ref_next[b]:
                agreed += 1
                assert err <= 2e-2 * np.sqrt(np.mean(ref_logits[b] ** 2)), f"step {step} request {b}: logits off"
            else:
                assert top2[1] - top2[0] <= 4 * err, (f"step {step} request {b}: picks differ although the oracle's "
                                                      f"top-2 gap {top2[1] - top2[0]:.3e} > 4 x logit error {err:.3e}")
                alive[b] = False
        if step + 1 < n_new:
            ref_logits, ref_next, caches, _ = O.stack_decode(cfg, sw, ref_next.astype(np.int32), caches, prompt + step)
    return compared, agreed, int((~alive).sum())


def test_greedy_generation_small_stack_ids_fed_back_on_device(T):
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=704, n_layers=3, vocab=1000)
    compared, agreed, diverged = _greedy_case(T, shape, seed=41, batch=4, prompt=12, n_new=24)
    print(f"greedy, small stack: {agreed}/{compared} request-steps agree with the oracle's greedy run, "
          f"{diverged}/4 requests met a near-tie")
    assert agreed >= compared // 2


def test_greedy_generation_llama7b_dims_two_layers(T):
    shape = dataclasses.replace(synth.LLAMA_7B, n_layers=2)
    compared, agreed, diverged = _greedy_case(T, shape, seed=42, batch=2, prompt=16, n_new=8)
    print(f"greedy, 2-layer 7B shapes, 32000-way head: {agreed}/{compared} request-steps agree, "
          f"{diverged}/2 requests met a near-tie")
    assert agreed >= compared // 2


def test_exact_tie_in_the_vocabulary_projection_goes_to_the_lowest_index(T):
    # rows 8 and 9 of the head are identical and dominate: their logits are bit-identical, the pick must be 8
    torch, thinfer = T
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=704, n_layers=1, vocab=1000)
    sw = synth.stack_weights(shape, 43)
    ids = synth.token_ids(shape, 43, (3, 6))
    for batch in (3, 1):
        head = sw["lm_head"].copy()
        ctx0 = _ctx(T, shape, sw["layers"], batch, 8, stack=sw)
        cap = torch.zeros(batch * 5, shape.hidden, dtype=torch.float16, device="cuda")
        ctx0.capture_hidden({0: cap})
        ctx0.prefill(torch.from_numpy(ids[:batch, :5].copy()).cuda())
        last = cap.view(batch, 5, -1)[:, -1].float().cpu().numpy()          # final hidden state of the last position
        ctx0.close()
        # a head row aligned with request 0's normalised state wins by a wide margin; duplicate it
        direction = (last[0] * sw["final_norm"].astype(np.float32))
        direction = (direction / np.linalg.norm(direction)).astype(np.float16)
        head[8] = direction
        head[9] = direction
        sw2 = dict(sw, lm_head=head)
        ctx = _ctx(T, shape, sw["layers"], batch, 8, stack=sw2)
        nxt, logits = ctx.prefill(torch.from_numpy(ids[:batch, :5].copy()).cuda(), want_logits=True)
        lg = logits.cpu().numpy()
        assert lg[0, 8] == lg[0, 9] and lg[0, 8] == lg[0].max()
        assert int(nxt.cpu()[0]) == 8
        ctx.close()


def test_bounded_wait_runs_out_and_the_context_recovers(T):
    # a wait that nothing satisfies gives up after its limit: the kernel returns, the status word reports
    # THINFER_ETIMEOUT, and after thinfer_clear_status the context computes as before
    torch, thinfer = T
    shape = synth.TINY
    w = synth.layer_weights(shape, 0)
    x = torch.from_numpy(synth.hidden_states(shape, 0, (2, 12))).cuda()
    ctx = _ctx(T, shape, [w], 2, 16)
    before = ctx.prefill(x[:, :11].contiguous()).cpu().numpy()
    step_before = ctx.decode_step(x[:, 11].contiguous()).cpu().numpy()
    ctx.release_slot(0)
    assert ctx.status() == 0
    ctx.selftest_bounded_wait(limit_ns=2_000_000)                    # 2 ms
    torch.cuda.synchronize()
    assert ctx.status() == thinfer.ETIMEOUT
    ctx.clear_status()
    assert ctx.status() == 0
    for mode in (1, 2):
        ctx.set_launch_mode(mode)
        after = ctx.prefill(x[:, :11].contiguous()).cpu().numpy()
        step_after = ctx.decode_step(x[:, 11].contiguous()).cpu().numpy()
        ctx.release_slot(0)
        torch.cuda.synchronize()
        assert ctx.status() == 0
        np.testing.assert_array_equal(after, before)
        if mode == 1:
            np.testing.assert_array_equal(step_after, step_before)
    with pytest.raises(thinfer.ThinferError):
        ctx.selftest_bounded_wait(limit_ns=10**10)                    # limits above 100 ms are refused
    ctx.close()


def test_two_stream_stages_with_vocabulary_and_batches_above_16(T):
    # both stages use the stream-K tensor-core path here (32 requests): the prefill stage's vocabulary projection
    # and the decode stage's projections have separate partial-sum areas, so slot 1 may be prefilled while slot 0
    # decodes.  Results: equal to the serial run bit for bit, and to the oracle within tolerance.
    torch, thinfer = T
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=704, n_layers=2, vocab=1000)
    cfg = oracle_config(shape)
    sw = synth.stack_weights(shape, 44)
    B = 32
    ids = synth.token_ids(shape, 44, (2, B, 14))
    dev = torch.from_numpy(ids).cuda()
    p = [dev[s, :, :10].contiguous() for s in range(2)]
    d = [[dev[s, :, 10 + i].contiguous() for i in range(4)] for s in range(2)]

    def run(two_streams):
        ctx = _ctx(T, shape, sw["layers"], B, 16, stack=sw, buf_slots=2)
        sp = torch.cuda.Stream() if two_streams else torch.cuda.current_stream()
        sd = torch.cuda.Stream() if two_streams else torch.cuda.current_stream()
        torch.cuda.synchronize()
        out = {}
        out["p0"] = ctx.prefill(p[0], slot=0, stream=sp, want_logits=True)[1]
        for rep in range(3):                                          # keep the prefill stream busy meanwhile
            out[f"p1_{rep}"] = ctx.prefill(p[1], slot=1, stream=sp, want_logits=True)[1]
            if rep < 2:
                ctx.release_slot(1, stream=sp)
        for i in range(4):
            out[f"d0_{i}"] = ctx.decode_step(d[0][i], slot=0, stream=sd, want_logits=True)[1]
        for i in range(4):
            out[f"d1_{i}"] = ctx.decode_step(d[1][i], slot=1, stream=sd, want_logits=True)[1]
        torch.cuda.synchronize()
        assert ctx.status() == 0
        res = {k: v.cpu().numpy() for k, v in out.items()}
        ctx.close()
        return res

    serial, overlapped = run(False), run(True)
    for k in serial:
        np.testing.assert_array_equal(serial[k], overlapped[k], err_msg=k)
    for s in range(2):
        ref, _, caches, _ = O.stack_prefill(cfg, sw, ids[s, :, :10])
        assert_rows_close(overlapped["p0" if s == 0 else "p1_2"], ref, f"slot {s}: prefill logits")
        for i in range(4):
            ref, _, caches, _ = O.stack_decode(cfg, sw, ids[s, :, 10 + i], caches, 10 + i)
            assert_rows_close(overlapped[f"d{s}_{i}"], ref, f"slot {s}: decode logits step {i}")


@pytest.mark.parametrize("hq,hkv,d", [(8, 1, 64), (8, 2, 128), (16, 2, 128)])
@pytest.mark.parametrize("mode", [1])
def test_ragged_prompts_grouped_query_attention(T, hq, hkv, d, mode):
    # 4 or 8 query heads per KV head: decode attention runs on the tensor-core kernel; ragged lengths put the end
    # of a request's keys in the middle of a 16-key block, and long prompts spread one pair over several CTAs
    torch, thinfer = T
    shape = synth.Shape(hidden=512, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, ffn=1024)
    cfg = oracle_config(shape)
    w = synth.layer_weights(shape, 15)
    lens, n_decode = (1, 17, 300, 1029), 3
    batch, pad = len(lens), max(lens)
    x = synth.hidden_states(shape, 15, (batch, pad + n_decode))
    ctx = _ctx(T, shape, [w], batch, pad + n_decode)
    ctx.set_launch_mode(mode)
    xd = torch.from_numpy(x).cuda()
    ctx.prefill_ragged(xd[:, :pad].contiguous(), lens)
    dec = []
    for i in range(n_decode):
        step_in = np.stack([x[b, lens[b] + i] for b in range(batch)])
        dec.append(ctx.decode_step(torch.from_numpy(step_in).cuda()).cpu().numpy())
    assert ctx.status() == 0
    for b in range(batch):
        # the oracle continues from the GPU's own cache of the request (chained; the prefill is checked elsewhere)
        k = ctx.kv_view(0, 0, 0).cpu().numpy()[b:b + 1, :, :lens[b]].astype(np.float64)
        v = ctx.kv_view(0, 0, 1).cpu().numpy()[b:b + 1, :, :lens[b]].astype(np.float64)
        for i in range(n_decode):
            r, k, v = O.layer_decode(cfg, w, x[b:b + 1, lens[b] + i], k, v, lens[b] + i)
            assert_rows_close(dec[i][b], r[0], f"request {b} ({lens[b]} keys) decode step {i}")
            kg = ctx.kv_view(0, 0, 0).cpu().numpy()[b, :, lens[b] + i]
            k[0, :, lens[b] + i] = kg
            v[0, :, lens[b] + i] = ctx.kv_view(0, 0, 1).cpu().numpy()[b, :, lens[b] + i]
    ctx.close()
