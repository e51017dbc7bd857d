"""The BF16 storage build (libthinfer_bf16.so: the same kernels compiled with BF16 as the 16-bit storage type,
Section 3.2.4's operator variants) against the oracle (run with -m gpu on a B200).

Inputs are drawn as BF16 values; the oracle receives their exact float32 widening, so both sides start from the
same numbers.  Bounds: those of the FP16 tests times 8, the ratio of the two unit roundoffs (tests/parity.py)."""
import numpy as np
import pytest

from oracle import oracle as O
from paper_2605_25655_b200 import synth
from tests.parity import BF16_FACTOR, BF16_MIN_COSINE, MAX_ERR_OVER_RMS, assert_rows_close, oracle_config

pytestmark = pytest.mark.gpu
TOL = dict(max_err=MAX_ERR_OVER_RMS * BF16_FACTOR, min_cos=BF16_MIN_COSINE)
OP_TOL = dict(max_err=4e-3 * BF16_FACTOR, min_cos=BF16_MIN_COSINE)


@pytest.fixture(scope="module")
def T():
    import torch
    from paper_2605_25655_b200 import thinfer
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    assert thinfer.lib("bf16").thinfer_storage_type() == 1
    return torch, thinfer


def _bf16(torch, rng, shape, std):
    return torch.from_numpy((rng.standard_normal(shape) * std).astype(np.float32)).bfloat16()


def _np(t):
    return t.float().cpu().numpy()          # exact: every BF16 value is a float32 value


@pytest.mark.parametrize("rows,n_out,k", [(32, 256, 688), (300, 1376, 256), (512, 384, 4096), (5, 130, 72), (16, 1000, 1024)])
@pytest.mark.parametrize("out_fp32", [False, True])
def test_linear_tensor_core_path_bf16(T, rows, n_out, k, out_fp32):
    torch, thinfer = T
    rng = np.random.default_rng(rows + n_out)
    x, w = _bf16(torch, rng, (rows, k), 1.0), _bf16(torch, rng, (n_out, k), 0.05)
    y = thinfer.op_linear(x.cuda(), w.cuda(), out_fp32=out_fp32, path=0)
    assert y.dtype == (torch.float32 if out_fp32 else torch.bfloat16)
    assert_rows_close(_np(y), O.linear(_np(x), _np(w)), f"bf16 linear tc {rows}x{n_out}x{k}", **OP_TOL)


@pytest.mark.parametrize("rows,n_out,k,path", [(1, 256, 256, 1), (3, 1376, 688, 1), (4, 4096, 4096, 2), (16, 512, 1024, 2),
                                               (9, 12288, 4096, 2), (8, 32000, 512, 2)])
def test_linear_streaming_paths_bf16(T, rows, n_out, k, path):
    torch, thinfer = T
    rng = np.random.default_rng(rows * 3 + k)
    x, w = _bf16(torch, rng, (rows, k), 1.0), _bf16(torch, rng, (n_out, k), 0.05)
    for fp32 in (False, True):
        y = thinfer.op_linear(x.cuda(), w.cuda(), out_fp32=fp32, path=path)
        assert_rows_close(_np(y), O.linear(_np(x), _np(w)), f"bf16 linear path {path} {rows}x{n_out}x{k}", **OP_TOL)


@pytest.mark.parametrize("b,hq,hkv,s,d", [(2, 4, 2, 128, 128), (1, 2, 1, 77, 64), (1, 4, 4, 1024, 128)])
def test_attention_prefill_bf16(T, b, hq, hkv, s, d):
    torch, thinfer = T
    rng = np.random.default_rng(s + d)
    q, k, v = (_bf16(torch, rng, (b, h, s, d), 1.0) for h in (hq, hkv, hkv))
    out = thinfer.op_attention_prefill(q.cuda(), k.cuda(), v.cuda())
    for i in range(b):
        ref = O.causal_attention(_np(q[i]), _np(k[i]), _np(v[i]))
        assert_rows_close(_np(out[i]), ref, f"bf16 attention b={i}", max_err=6e-3 * BF16_FACTOR, min_cos=BF16_MIN_COSINE)


def test_rmsnorm_bf16(T):
    torch, thinfer = T
    rng = np.random.default_rng(3)
    x, g = _bf16(torch, rng, (37, 1024), 2.0), _bf16(torch, rng, (1024,), 0.1) + 1
    y = thinfer.op_rmsnorm(x.cuda(), g.cuda(), 1e-5)
    assert_rows_close(_np(y), O.rmsnorm(_np(x), _np(g), 1e-5), "bf16 rmsnorm", max_err=3e-3 * BF16_FACTOR,
                      min_cos=BF16_MIN_COSINE)


def _weights_np(w):
    return {n: _np(t) for n, t in w.items()}


def _layer_case_bf16(T, shape, batch, seq, n_decode, seed, launch_mode=None, check=None):
    torch, thinfer = T
    cfg = oracle_config(shape)
    w = synth.device_layer_weights(shape, seed, 0, dtype=torch.bfloat16)
    g = torch.Generator(device="cuda").manual_seed(seed)
    x = torch.randn(batch, seq + n_decode, shape.hidden, device="cuda", generator=g).bfloat16()
    ctx = thinfer.Context(shape, [w], None, max_batch=batch, max_seq=seq + n_decode)
    assert ctx.storage == "bf16"
    if launch_mode is not None:
        ctx.set_launch_mode(launch_mode)
    out = ctx.prefill(x[:, :seq].contiguous())
    dec = [ctx.decode_step(x[:, seq + i].contiguous()) for i in range(n_decode)]
    torch.cuda.synchronize()
    assert ctx.status() == 0 and out.dtype == torch.bfloat16
    bs = list(range(batch)) if check is None else check
    wn, xn = _weights_np(w), _np(x)
    ref, kc, vc = O.layer_prefill(cfg, wn, xn[bs, :seq])
    stats = [assert_rows_close(_np(out)[bs], ref, f"bf16 prefill B={batch} S={seq}", **TOL)]
    kg, vg = _np(ctx.kv_view(0, 0, 0))[bs], _np(ctx.kv_view(0, 0, 1))[bs]
    assert kg.dtype == np.float32
    assert_rows_close(kg[:, :, :seq], kc, "bf16 K cache", max_err=6e-3 * BF16_FACTOR, min_cos=BF16_MIN_COSINE)
    assert_rows_close(vg[:, :, :seq], vc, "bf16 V cache", max_err=6e-3 * BF16_FACTOR, min_cos=BF16_MIN_COSINE)
    k_run, v_run = kg[:, :, :seq].astype(np.float64), vg[:, :, :seq].astype(np.float64)
    for i in range(n_decode):                      # chained: the oracle continues from the GPU's own cache
        r, k_run, v_run = O.layer_decode(cfg, wn, xn[bs, seq + i], k_run, v_run, seq + i)
        stats.append(assert_rows_close(_np(dec[i])[bs], r, f"bf16 decode step {i} B={batch}", **TOL))
        kg, vg = _np(ctx.kv_view(0, 0, 0))[bs], _np(ctx.kv_view(0, 0, 1))[bs]
        k_run[:, :, seq + i], v_run[:, :, seq + i] = kg[:, :, seq + i], vg[:, :, seq + i]
    ctx.close()
    return stats


@pytest.mark.parametrize("batch,seq,n_decode,hkv,ffn", [(1, 32, 4, 4, 704), (3, 130, 3, 2, 704), (16, 40, 2, 1, 704),
                                                        (2, 33, 3, 4, 688), (20, 9, 2, 2, 704)])
def test_small_layer_bf16(T, batch, seq, n_decode, hkv, ffn):
    # skinny projections (ffn 704), FMA / stream-K paths (ffn 688, batch 20), MHA and grouped-query attention
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=hkv, head_dim=64, ffn=ffn)
    _layer_case_bf16(T, shape, batch, seq, n_decode, seed=batch)


def test_unified_decode_kernel_bf16(T):
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=704)
    _layer_case_bf16(T, shape, 5, 40, 3, seed=9, launch_mode=2)


def test_llama7b_layer_bf16(T):
    stats = _layer_case_bf16(T, synth.LLAMA_7B_LAYER, batch=4, seq=256, n_decode=2, seed=7, check=[0, 3])
    print("bf16 7B layer: max|err|/rms, cosine per stage:", [(f"{e:.2e}", f"{c:.6f}") for e, c in stats])


def test_llama70b_layer_shapes_bf16(T):
    import dataclasses
    shape = dataclasses.replace(synth.LLAMA_70B, n_layers=1, vocab=0)        # GQA 8:1: tensor-core decode attention
    _layer_case_bf16(T, shape, batch=2, seq=80, n_decode=2, seed=70)


def test_stack_teacher_forced_bf16(T):
    torch, thinfer = T
    shape = synth.Shape(hidden=256, n_q_heads=4, n_kv_heads=2, head_dim=64, ffn=704, n_layers=3, vocab=1000)
    cfg = oracle_config(shape)
    sw = synth.device_stack_weights(shape, 5, dtype=torch.bfloat16)
    swn = {"layers": [_weights_np(w) for w in sw["layers"]], **{n: _np(sw[n]) for n in ("embed", "final_norm", "lm_head")}}
    ids = synth.token_ids(shape, 5, (2, 20))
    ctx = thinfer.Context(shape, sw["layers"], {n: sw[n] for n in ("embed", "final_norm", "lm_head")}, max_batch=2, max_seq=24)
    idd = torch.from_numpy(ids).cuda()
    nxt, logits = ctx.prefill(idd[:, :16].contiguous(), want_logits=True)
    ref, _, caches, _ = O.stack_prefill(cfg, swn, ids[:, :16])
    assert_rows_close(logits.cpu().numpy(), ref, "bf16 prefill logits", **TOL)
    np.testing.assert_array_equal(nxt.cpu().numpy(), np.argmax(logits.cpu().numpy(), axis=-1))
    for t in range(16, 20):
        nxt, logits = ctx.decode_step(idd[:, t].contiguous(), want_logits=True)
        ref, _, caches, _ = O.stack_decode(cfg, swn, ids[:, t], caches, t)
        assert_rows_close(logits.cpu().numpy(), ref, f"bf16 decode logits t={t}", **TOL)
    assert ctx.status() == 0
    ctx.close()


def test_fp16_and_bf16_builds_coexist_in_one_process(T):
    torch, thinfer = T
    rng = np.random.default_rng(11)
    x32 = (rng.standard_normal((8, 512))).astype(np.float32)
    w32 = (rng.standard_normal((256, 512)) * 0.05).astype(np.float32)
    for dt in (torch.float16, torch.bfloat16, torch.float16):
        x, w = torch.from_numpy(x32).to(dt), torch.from_numpy(w32).to(dt)
        y = thinfer.op_linear(x.cuda(), w.cuda(), path=2)
        assert y.dtype == dt
        assert_rows_close(_np(y), O.linear(_np(x), _np(w)), f"linear in {dt}", **OP_TOL)
    with pytest.raises(thinfer.ThinferError):
        thinfer.op_linear(torch.zeros(2, 64, device="cuda"), torch.zeros(4, 64, device="cuda"))      # float32 storage
