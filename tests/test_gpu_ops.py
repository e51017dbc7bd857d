"""Single operators through the C ABI against the oracle (run with -m gpu on a B200)."""
import numpy as np
import pytest

from oracle import oracle as O
from tests.parity import assert_rows_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def T():
    import torch
    from paper_2605_25655_b200 import thinfer
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    thinfer.lib()
    return torch, thinfer


def _rand16(rng, shape, std):
    return (rng.standard_normal(shape) * std).astype(np.float16)


# rows, n_out, k: multi-tile with ragged tails in every dimension; k = 688 is not a multiple of 64
LINEAR_SHAPES = [(32, 256, 256), (32, 256, 688), (5, 130, 72), (300, 1376, 256), (512, 384, 4096), (1, 4096, 4096),
                 (16, 1000, 1024), (129, 128, 64), (700, 300, 520)]


@pytest.mark.parametrize("rows,n_out,k", LINEAR_SHAPES)
@pytest.mark.parametrize("out_fp32", [False, True])
def test_linear_tensor_core_path(T, rows, n_out, k, out_fp32):
    torch, thinfer = T
    rng = np.random.default_rng(rows * 7 + n_out)
    x, w = _rand16(rng, (rows, k), 1.0), _rand16(rng, (n_out, k), 0.05)
    y = thinfer.op_linear(torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda(), out_fp32=out_fp32, path=0)
    torch.cuda.synchronize()
    assert_rows_close(y.cpu().numpy(), O.linear(x, w), f"linear tc {rows}x{n_out}x{k}", max_err=4e-3)


@pytest.mark.parametrize("rows,n_out,k", [(1, 256, 256), (2, 130, 72), (3, 1376, 688), (4, 4096, 4096), (7, 256, 11008),
                                          (16, 512, 1024)])
def test_linear_streaming_path(T, rows, n_out, k):
    torch, thinfer = T
    rng = np.random.default_rng(rows * 11 + k)
    x, w = _rand16(rng, (rows, k), 1.0), _rand16(rng, (n_out, k), 0.05)
    for fp32 in (False, True):
        y = thinfer.op_linear(torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda(), out_fp32=fp32, path=1)
        torch.cuda.synchronize()
        assert_rows_close(y.cpu().numpy(), O.linear(x, w), f"linear gemv {rows}x{n_out}x{k}", max_err=4e-3)


# K is a multiple of 64 here.  Covered: fewer features than one 16-row tile per CTA share, K shorter than
# the 8 warp slices, block counts that do not divide by 8, shares of 1 .. 5 tiles, 9..16 tokens (two token
# tiles), the 7B projection shapes and a vocabulary-sized output
@pytest.mark.parametrize("rows,n_out,k", [(1, 256, 256), (2, 130, 64), (3, 1376, 704), (4, 4096, 4096), (7, 256, 11008),
                                          (16, 512, 1024), (9, 12288, 4096), (16, 4096, 11008), (13, 2, 64),
                                          (8, 6, 192), (16, 32000, 512), (5, 9472, 320), (11, 18944, 128),
                                          (16, 22016, 4096)])
def test_linear_skinny_tensor_core_path(T, rows, n_out, k):
    torch, thinfer = T
    rng = np.random.default_rng(rows * 13 + k)
    x, w = _rand16(rng, (rows, k), 1.0), _rand16(rng, (n_out, k), 0.05)
    for fp32 in (False, True):
        y = thinfer.op_linear(torch.from_numpy(x).cuda(), torch.from_numpy(w).cuda(), out_fp32=fp32, path=2)
        torch.cuda.synchronize()
        assert_rows_close(y.cpu().numpy(), O.linear(x, w), f"linear skinny {rows}x{n_out}x{k}", max_err=4e-3)


def test_linear_skinny_rejects_what_it_does_not_cover(T):
    torch, thinfer = T
    x = torch.zeros(17, 64, dtype=torch.float16, device="cuda")
    w = torch.zeros(8, 64, dtype=torch.float16, device="cuda")
    with pytest.raises(thinfer.ThinferError):
        thinfer.op_linear(x, w, path=2)            # more than 16 tokens
    with pytest.raises(thinfer.ThinferError):
        thinfer.op_linear(x[:4, :40].contiguous(), w[:, :40].contiguous(), path=2)  # K not a multiple of 64


def test_linear_identity_weight_is_exact(T):
    torch, thinfer = T
    rng = np.random.default_rng(5)
    x = _rand16(rng, (40, 192), 1.0)
    w = np.eye(192, dtype=np.float16)
    for path in (0, 1, 2):
        xs = x[:16] if path >= 1 else x
        y = thinfer.op_linear(torch.from_numpy(xs).cuda(), torch.from_numpy(w).cuda(), path=path)
        np.testing.assert_array_equal(y.cpu().numpy(), xs)


@pytest.mark.parametrize("rows,n", [(1, 256), (37, 4096), (300, 8192), (9, 688)])
def test_rmsnorm(T, rows, n):
    torch, thinfer = T
    rng = np.random.default_rng(n)
    x = _rand16(rng, (rows, n), 2.0)
    g = (1.0 + 0.1 * rng.standard_normal(n)).astype(np.float16)
    y = thinfer.op_rmsnorm(torch.from_numpy(x).cuda(), torch.from_numpy(g).cuda(), 1e-5)
    assert_rows_close(y.cpu().numpy(), O.rmsnorm(x, g, 1e-5), f"rmsnorm {rows}x{n}", max_err=3e-3)


# batch, q heads, kv heads, seq, cache stride, head_dim
ATTN_SHAPES = [(1, 4, 4, 32, 40, 64), (2, 4, 2, 128, 128, 128), (1, 2, 2, 129, 200, 128), (2, 8, 2, 300, 384, 64),
               (1, 32, 32, 512, 640, 128), (1, 1, 1, 1, 8, 128), (1, 2, 1, 77, 77, 64),
               (1, 2, 2, 1024, 1024, 128), (1, 2, 1, 4096, 4096, 128), (1, 1, 1, 2049, 2100, 64),
               # eight query heads per KV head; 40 (request, head) pairs walked longest first in two chunks (32 + 8)
               (1, 16, 2, 700, 704, 128), (1, 40, 40, 2048, 2048, 128)]


@pytest.mark.parametrize("b,hq,hkv,s,t,d", ATTN_SHAPES)
def test_attention_prefill(T, b, hq, hkv, s, t, d):
    torch, thinfer = T
    rng = np.random.default_rng(s * 3 + d)
    q, k, v = _rand16(rng, (b, hq, s, d), 1.0), _rand16(rng, (b, hkv, t, d), 1.0), _rand16(rng, (b, hkv, t, d), 1.0)
    # positions past the sequence hold garbage the kernel must never let through
    k[:, :, s:, :] = np.float16(np.nan)
    v[:, :, s:, :] = np.float16(np.inf)
    out = thinfer.op_attention_prefill(torch.from_numpy(q).cuda(), torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda())
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    for bi in range(b):
        ref = O.causal_attention(q[bi], k[bi, :, :s], v[bi, :, :s])
        assert_rows_close(got[bi], ref, f"attention b{bi} S={s} d={d}", max_err=6e-3)


def test_attention_first_row_returns_v0_and_uniform_keys_give_running_mean(T):
    torch, thinfer = T
    rng = np.random.default_rng(9)
    s, d = 200, 128
    q = _rand16(rng, (1, 2, s, d), 1.0)
    k = np.broadcast_to(_rand16(rng, (1, 2, 1, d), 1.0), (1, 2, s, d)).copy()
    v = _rand16(rng, (1, 2, s, d), 1.0)
    out = thinfer.op_attention_prefill(torch.from_numpy(q).cuda(), torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda())
    got = out.cpu().numpy().reshape(s, 2, d).astype(np.float64)
    np.testing.assert_allclose(got[0], v[0, :, 0, :].astype(np.float64), rtol=2e-3, atol=2e-3)
    mean = np.cumsum(v[0].astype(np.float64), axis=1) / np.arange(1, s + 1)[None, :, None]
    np.testing.assert_allclose(got, mean.transpose(1, 0, 2), rtol=0, atol=4e-3)


@pytest.mark.parametrize("s,d", [(600, 128), (333, 64)])
def test_attention_prefill_rescales_while_the_row_maximum_keeps_growing(T, s, d):
    """Scores that rise by more than 2^8 from one 64-key tile to the next: the running maximum of every row is
    replaced and the accumulated output rescaled in (nearly) every tile (Section 3.3.2's online form)."""
    torch, thinfer = T
    rng = np.random.default_rng(s + d)
    q, k, v = _rand16(rng, (1, 2, s, d), 0.25), _rand16(rng, (1, 2, s, d), 0.25), _rand16(rng, (1, 2, s, d), 1.0)
    # 0.2 * sqrt(d) / log2(e) per key in raw score units = 0.2 per key in the kernel's base-2 units: 12.8 per tile
    slope = 0.2 * np.sqrt(d) / np.log2(np.e)
    q[..., 0] = np.float16(4.0)
    k[..., 0] = (np.arange(s) * slope / 4.0).astype(np.float16)[None, None, :]
    out = thinfer.op_attention_prefill(torch.from_numpy(q).cuda(), torch.from_numpy(k).cuda(), torch.from_numpy(v).cuda())
    torch.cuda.synchronize()
    assert_rows_close(out.cpu().numpy()[0], O.causal_attention(q[0], k[0], v[0]), f"growing maximum S={s} d={d}", max_err=6e-3)


def test_argmax_exact_ties_go_to_the_lowest_index(T):
    torch, thinfer = T
    n = 32000
    rng = np.random.default_rng(5)
    lg = rng.standard_normal((6, n)).astype(np.float32)
    lg[0, [31999, 17, 20000]] = 9.0                 # three equal maxima far apart (different threads and warps)
    lg[1, [1024, 1025]] = 7.5                       # neighbours across a thread-stride boundary
    lg[2, :] = 1.25                                 # everything ties: index 0
    lg[3, [5, 31998]] = np.inf                      # infinite maxima tie as well
    lg[4, :] = -np.inf
    lg[4, [123, 30000]] = -3.0                      # the rest is -inf
    lg[5, 31999] = 50.0                             # unique maximum in the last column
    ids = thinfer.op_argmax(torch.from_numpy(lg).cuda()).cpu().numpy()
    np.testing.assert_array_equal(ids, [17, 1024, 0, 5, 123, 31999])
    np.testing.assert_array_equal(ids, O.argmax_lowest(lg))
    # odd row length, fewer columns than threads
    small = np.array([[0.0, 2.0, 2.0, -1.0, 2.0]], dtype=np.float32)
    assert int(thinfer.op_argmax(torch.from_numpy(small).cuda()).cpu()[0]) == 1


# heads, KV heads, head_dim: FMA kernel with 1 and 2 query heads per KV head, tensor-core kernel with 4 and 8;
# 16 query heads per KV head (two groups of 8 read the same keys), 6 (groups of 2), 3 (odd: one head per pass)
@pytest.mark.parametrize("hq,hkv,d", [(4, 4, 128), (8, 4, 64), (8, 2, 128), (8, 1, 64), (16, 2, 128), (32, 32, 128),
                                      (16, 1, 64), (12, 2, 64), (3, 1, 128)])
def test_decode_attention_schedules(T, hq, hkv, d):
    # the split-KV schedules of decode attention on their own, over many (batch, key count) combinations: one
    # segment per pair, equal segments merged in a thread-block cluster (2 .. 8 CTAs), equal segments merged through
    # a ticket, exactly balanced runs that cross pair boundaries, ragged key counts, single keys
    from paper_2605_25655_b200 import synth
    torch, thinfer = T
    shape = synth.Shape(hidden=hq * d, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, ffn=64)
    max_b, max_t = 16, 2100
    w = {n: torch.zeros(synth.layer_tensor_shape(shape, n), dtype=torch.float16, device="cuda") for n in synth.LAYER_TENSORS}
    ctx = thinfer.Context(shape, [w], None, max_batch=max_b, max_seq=max_t)
    rng = np.random.default_rng(hq * 1000 + hkv * 10 + d)
    k_np = rng.standard_normal((max_b, hkv, max_t, d)).astype(np.float16)
    v_np = rng.standard_normal((max_b, hkv, max_t, d)).astype(np.float16)
    ctx.kv_view(0, 0, 0).copy_(torch.from_numpy(k_np))
    ctx.kv_view(0, 0, 1).copy_(torch.from_numpy(v_np))
    cases = [(1, 1), (1, 33), (2, 64), (3, 65), (16, 31), (5, 129), (1, 2100), (16, 640), (7, 1023), (16, 1279), (4, 528),
             (9, 257), (2, 2047), (12, 96)]
    cases += [(int(rng.integers(1, 17)), int(rng.integers(1, max_t + 1))) for _ in range(10)]
    for batch, t_len in cases:
        q_np = (rng.standard_normal((batch, hq, d)) * 1.5).astype(np.float16)
        ragged = (batch * 7 + t_len) % 3 == 0
        lens = [int(rng.integers(1, t_len + 1)) for _ in range(batch)] if ragged else None
        qd = torch.from_numpy(q_np).cuda()
        out = ctx.attention_decode(qd, t_len, seq_lens=lens).cpu().numpy()
        again = ctx.attention_decode(qd, t_len, seq_lens=lens).cpu().numpy()
        np.testing.assert_array_equal(out, again)       # segments are merged in a fixed order: no run-to-run noise
        for b in range(batch):
            n = lens[b] if ragged else t_len
            ref = O.decode_attention(q_np[b], k_np[b, :, :n], v_np[b, :, :n])
            assert_rows_close(out[b].reshape(hq, d), ref.reshape(hq, d),
                              f"decode attention {hq}q/{hkv}kv d={d} batch {batch} keys {n} (request {b})", max_err=6e-3)
    assert ctx.status() == 0
    ctx.close()


def test_decode_attention_schedules_up_to_64_requests(T):
    # the same sweep with the largest slots the library accepts (17 .. 64 requests: more pairs than CTA slots, so
    # the exactly balanced runs cross pair boundaries), MHA and 4 query heads per KV head
    from paper_2605_25655_b200 import synth
    torch, thinfer = T
    for hq, hkv, d in ((8, 8, 128), (8, 2, 64)):
        shape = synth.Shape(hidden=hq * d, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, ffn=64)
        max_b, max_t = 64, 700
        w = {n: torch.zeros(synth.layer_tensor_shape(shape, n), dtype=torch.float16, device="cuda") for n in synth.LAYER_TENSORS}
        ctx = thinfer.Context(shape, [w], None, max_batch=max_b, max_seq=max_t)
        rng = np.random.default_rng(hq + d)
        k_np = rng.standard_normal((max_b, hkv, max_t, d)).astype(np.float16)
        v_np = rng.standard_normal((max_b, hkv, max_t, d)).astype(np.float16)
        ctx.kv_view(0, 0, 0).copy_(torch.from_numpy(k_np))
        ctx.kv_view(0, 0, 1).copy_(torch.from_numpy(v_np))
        for batch, t_len, ragged in ((17, 300, False), (64, 700, False), (33, 129, True), (64, 65, True), (48, 1, False)):
            q_np = (rng.standard_normal((batch, hq, d)) * 1.5).astype(np.float16)
            lens = [int(rng.integers(1, t_len + 1)) for _ in range(batch)] if ragged else None
            out = ctx.attention_decode(torch.from_numpy(q_np).cuda(), t_len, seq_lens=lens).cpu().numpy()
            for b in (0, batch // 2, batch - 1):
                n = lens[b] if ragged else t_len
                ref = O.decode_attention(q_np[b], k_np[b, :, :n], v_np[b, :, :n])
                assert_rows_close(out[b].reshape(hq, d), ref.reshape(hq, d),
                                  f"decode attention {hq}q/{hkv}kv batch {batch} keys {n} (request {b})", max_err=6e-3)
        assert ctx.status() == 0
        ctx.close()
