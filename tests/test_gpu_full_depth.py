"""The three full-stack configurations at their real depth against the oracle (run with -m gpu on a B200):
Llama-7B x 32 layers, Llama-13B x 40 layers, Llama-2-70B x 80 layers (GQA 64/8), each with the 32000-way head.

The weights are drawn on the device tensor by tensor (synth.device_stack_weights; the 70B set is 138 GB and
never exists on the host); the oracle sees one layer at a time, widened to float64 on the device and copied
into reusable pinned host buffers.

Per configuration:
  (i)   full depth, reduced token budget (2 requests, 64-token prompt, 4 decode steps, teacher forced), end to
        end - the oracle runs on its own states, nothing is chained: final hidden state cosine >= 0.999 per
        token and logits within the row-RMS tolerance, for the per-unit decode path and for the unified kernel;
  (ii)  the configuration's real batch and prompt length: per-layer chained checks of layers {0, L/2, L-1}
        on the first and the last request (the oracle layer is fed the GPU's own FP16 input of that layer,
        captured with thinfer_capture_hidden), for the prefill and for the first decode step, K/V cache
        contents included;
  (iii) decode steps of one layer at the real batch and the KV length the configuration ends at.
Tolerance: max |err| <= 2e-2 x row RMS and cosine >= 0.999 (tests/parity.py)."""
import dataclasses
import gc

import numpy as np
import pytest

from oracle import oracle as O
from paper_2605_25655_b200 import synth
from tests.parity import assert_rows_close, oracle_config, row_stats
from tests.test_gpu_layer import _check_greedy, _layer_case

pytestmark = pytest.mark.gpu

# name -> (shape, batch, prompt, generated tokens) of configurations 3, 4 and 5
CONFIGS = {
    "llama7b": (synth.LLAMA_7B, 8, 512, 256),
    "llama13b": (synth.LLAMA_13B, 16, 1024, 256),
    "llama70b": (synth.LLAMA_70B, 4, 512, 128),
}


@pytest.fixture(scope="module")
def T():
    import torch
    from paper_2605_25655_b200 import thinfer
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    thinfer.lib()
    return torch, thinfer


class HostLayers:
    """What the oracle iterates over as sw["layers"]: per layer a dict of float64 numpy arrays.  The arrays are
    views of pinned buffers that are reused from layer to layer (the oracle is done with a layer's weights
    when it asks for the next), filled by an exact FP16 -> float64 widening on the device and one copy."""

    def __init__(self, torch, dev_layers):
        self.torch, self.dev_layers = torch, dev_layers
        self.bufs = {n: torch.empty(tuple(t.shape), dtype=torch.float64, pin_memory=True)
                     for n, t in dev_layers[0].items()}

    def fetch(self, l):
        for n, t in self.dev_layers[l].items():
            self.bufs[n].copy_(t.double())
        self.torch.cuda.synchronize()
        return {n: b.numpy() for n, b in self.bufs.items()}

    def __len__(self):
        return len(self.dev_layers)

    def __iter__(self):
        for l in range(len(self.dev_layers)):
            yield self.fetch(l)


@pytest.fixture(scope="module", params=list(CONFIGS))
def model(request, T):
    torch, thinfer = T
    shape, batch, prompt, gen = CONFIGS[request.param]
    gc.collect()
    torch.cuda.empty_cache()
    free, _ = torch.cuda.mem_get_info()
    need = synth.model_bytes(shape) + (12 << 30)
    assert free > need, f"{request.param}: {free >> 30} GiB free on the device, {need >> 30} GiB needed"
    sw = synth.device_stack_weights(shape, seed=5)
    host = HostLayers(torch, sw["layers"])
    stack64 = {n: sw[n].double().cpu().numpy() for n in ("embed", "final_norm", "lm_head")}
    m = dict(name=request.param, shape=shape, batch=batch, prompt=prompt, gen=gen, sw=sw, host=host, stack64=stack64)
    yield m
    m.clear()
    del sw, host, stack64
    gc.collect()
    torch.cuda.empty_cache()


def _context(T, m, max_batch, max_seq):
    torch, thinfer = T
    sw = m["sw"]
    return thinfer.Context(m["shape"], sw["layers"], {n: sw[n] for n in ("embed", "final_norm", "lm_head")},
                           max_batch=max_batch, max_seq=max_seq)


def test_full_depth_end_to_end_on_a_reduced_token_budget(T, model):
    torch, thinfer = T
    shape, L = model["shape"], model["shape"].n_layers
    cfg = oracle_config(shape)
    B, S, n_dec = 2, 64, 4
    ids = synth.token_ids(shape, 31, (B, S + n_dec))
    # One pass of the oracle's own stack loop over all S + n_dec tokens.  Row t of a prefill equals the
    # incremental decode of token t (pinned on the CPU), so its rows are the reference for every decode step.
    sw_host = dict(model["stack64"], layers=model["host"])
    _, _, _, hid = O.stack_prefill(cfg, sw_host, ids)
    final = hid[-1]                                                    # [B, S + n_dec, D], float64
    ref_logits = {t: O.head_logits(cfg, sw_host, final[:, t]) for t in range(S - 1, S + n_dec)}
    del hid

    idd = torch.from_numpy(ids).cuda()
    report = []
    for mode in (1, 2):
        ctx = _context(T, model, B, S + n_dec + 4)
        ctx.set_launch_mode(mode)
        cap = torch.zeros(B * S, shape.hidden, dtype=torch.float16, device="cuda")
        ctx.capture_hidden({L - 1: cap})
        nxt, logits = ctx.prefill(idd[:, :S].contiguous(), want_logits=True)
        got_final = cap.view(B, S, shape.hidden).cpu().numpy()
        err_h, cos_h = row_stats(got_final, final[:, :S])
        assert cos_h >= 0.999, f"mode {mode}: final hidden state after {L} layers, cosine {cos_h:.6f}"
        err_l, cos_l = assert_rows_close(logits.cpu().numpy(), ref_logits[S - 1], f"mode {mode}: prefill logits after {L} layers")
        _check_greedy(nxt.cpu().numpy(), logits.cpu().numpy(), ref_logits[S - 1])
        report.append((mode, "prefill", err_h, cos_h, err_l, cos_l))
        for t in range(S, S + n_dec):
            nxt, logits = ctx.decode_step(idd[:, t].contiguous(), want_logits=True)
            got = cap[:B].cpu().numpy()
            err_h, cos_h = row_stats(got, final[:, t])
            assert cos_h >= 0.999, f"mode {mode}: final hidden state of decode step t={t}, cosine {cos_h:.6f}"
            err_l, cos_l = assert_rows_close(logits.cpu().numpy(), ref_logits[t], f"mode {mode}: decode logits t={t}")
            _check_greedy(nxt.cpu().numpy(), logits.cpu().numpy(), ref_logits[t])
            report.append((mode, f"decode t={t}", err_h, cos_h, err_l, cos_l))
        assert ctx.status() == 0
        ctx.close()
    for r in report:
        print(f"{model['name']} x{L} mode {r[0]} {r[1]}: hidden max|err|/rms {r[2]:.2e} cos {r[3]:.6f}; "
              f"logits max|err|/rms {r[4]:.2e} cos {r[5]:.6f}")


def test_chained_per_layer_checks_at_the_real_batch_and_prompt(T, model):
    torch, thinfer = T
    shape, L, B, S = model["shape"], model["shape"].n_layers, model["batch"], model["prompt"]
    cfg = oracle_config(shape)
    ids = synth.token_ids(shape, 32, (B, S + 1))
    idd = torch.from_numpy(ids).cuda()
    probe = sorted({0, L // 2, L - 1})
    wanted = sorted({l - 1 for l in probe} | set(probe))               # input and output of every probed layer
    ctx = _context(T, model, B, S + 8)
    pre = {l: torch.zeros(B * S, shape.hidden, dtype=torch.float16, device="cuda") for l in wanted}
    ctx.capture_hidden(pre)
    ctx.prefill(idd[:, :S].contiguous())
    dec = {l: torch.zeros(B, shape.hidden, dtype=torch.float16, device="cuda") for l in wanted}
    ctx.capture_hidden(dec)
    ctx.decode_step(idd[:, S].contiguous())
    ctx.capture_hidden(None)
    torch.cuda.synchronize()
    assert ctx.status() == 0

    # the embedding gather is exact
    emb = model["sw"]["embed"]
    assert torch.equal(pre[-1].view(B, S, -1), emb[idd[:, :S].long()])
    assert torch.equal(dec[-1], emb[idd[:, S].long()])

    reqs = sorted({0, B - 1})
    for l in probe:
        w = model["host"].fetch(l)
        x_in = pre[l - 1].view(B, S, -1)[reqs].cpu().numpy()
        ref, kc, vc = O.layer_prefill(cfg, w, x_in)
        got = pre[l].view(B, S, -1)[reqs].cpu().numpy()
        e, c = assert_rows_close(got, ref, f"layer {l}: prefill output at batch {B}, prompt {S}")
        kg = ctx.kv_view(0, l, 0)[reqs].cpu().numpy()
        vg = ctx.kv_view(0, l, 1)[reqs].cpu().numpy()
        assert_rows_close(kg[:, :, :S], kc, f"layer {l}: K cache after prefill", max_err=6e-3)
        assert_rows_close(vg[:, :, :S], vc, f"layer {l}: V cache after prefill", max_err=6e-3)
        # first decode step, continued from the GPU's own FP16 cache
        x_dec = dec[l - 1][reqs].cpu().numpy()
        r, k_run, v_run = O.layer_decode(cfg, w, x_dec, kg[:, :, :S].astype(np.float64), vg[:, :, :S].astype(np.float64), S)
        e2, c2 = assert_rows_close(dec[l][reqs].cpu().numpy(), r, f"layer {l}: decode step at {S} cached keys")
        assert_rows_close(kg[:, :, S], k_run[:, :, S], f"layer {l}: K append", max_err=6e-3)
        assert_rows_close(vg[:, :, S], v_run[:, :, S], f"layer {l}: V append", max_err=6e-3)
        print(f"{model['name']} layer {l}: prefill max|err|/rms {e:.2e} cos {c:.6f}; decode {e2:.2e} cos {c2:.6f}")
    ctx.close()


@pytest.mark.parametrize("name", list(CONFIGS))
def test_decode_at_the_final_kv_length_and_real_batch(T, name):
    # (iii) one layer of the configuration, its real batch, the last two decode steps of its run
    shape, batch, prompt, gen = CONFIGS[name]
    layer = dataclasses.replace(shape, n_layers=1, vocab=0)
    t_end = prompt + gen - 1                                           # keys the last decode step attends
    _layer_case(T, layer, batch=batch, seq=t_end - 2, n_decode=2, seed=17, check_batches=sorted({0, batch - 1}),
                max_seq=t_end, check_prefill=False)
