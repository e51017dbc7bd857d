"""Shared helpers of the parity tests: the pass criterion and oracle plumbing."""
import numpy as np

from oracle import oracle as O

# The criterion the target states for floating-point parity: per-layer hidden
# state max |gpu - oracle| <= 2e-2 x RMS of the oracle's row, and cosine
# similarity >= 0.999 per token.
MAX_ERR_OVER_RMS = 2e-2
MIN_COSINE = 0.999
# The BF16 storage build rounds every stored value to 8 significant bits instead of FP16's 11: a unit roundoff of
# 2^-8 against 2^-11.  Every bound of the FP16 tests is a multiple of the storage roundoff (accumulation is FP32 in
# both builds), so the BF16 tests use the same bounds times 8; the cosine bound loosens with the square of that.
BF16_FACTOR = 8.0
BF16_MIN_COSINE = 1.0 - (1.0 - MIN_COSINE) * 16   # 0.984: well inside the factor-64 the scaling would allow


def oracle_config(shape):
    return O.Config(hidden=shape.hidden, n_q_heads=shape.n_q_heads, n_kv_heads=shape.n_kv_heads,
                    head_dim=shape.head_dim, ffn=shape.ffn, n_layers=shape.n_layers, vocab=shape.vocab,
                    rms_eps=shape.rms_eps, rope_base=shape.rope_base)


def row_stats(got, ref):
    """got, ref: [..., n].  Returns (max |err| / row rms, min cosine) over all rows."""
    got = np.asarray(got, dtype=np.float64).reshape(-1, ref.shape[-1])
    ref = np.asarray(ref, dtype=np.float64).reshape(-1, ref.shape[-1])
    rms = np.sqrt(np.mean(ref * ref, axis=-1))
    err = np.max(np.abs(got - ref), axis=-1) / np.maximum(rms, 1e-30)
    cos = np.sum(got * ref, axis=-1) / np.maximum(np.linalg.norm(got, axis=-1) * np.linalg.norm(ref, axis=-1), 1e-30)
    return float(err.max()), float(cos.min())


def assert_rows_close(got, ref, what="", max_err=MAX_ERR_OVER_RMS, min_cos=MIN_COSINE):
    assert np.all(np.isfinite(np.asarray(got, dtype=np.float64))), f"{what}: non-finite values"
    err, cos = row_stats(got, ref)
    assert err <= max_err, f"{what}: max|err|/rms = {err:.3e} > {max_err}"
    assert cos >= min_cos, f"{what}: cosine = {cos:.6f} < {min_cos}"
    return err, cos
