"""The allocation-free linear entry point against the ordinary one and the oracle (collected last).

thinfer_op_linear_noalloc serves hosts that cannot allocate device memory at the call site
(a capture in progress elsewhere in the process, a real-time loop, a fixed arena): its split-K
scratch is a fixed array inside the library.  Every call shares that array and it keeps what
the last call left, so the check runs two different products back to back, and must hold both
in a fresh process and after the rest of the suite."""
import numpy as np
import pytest

from oracle import oracle as O
from tests.parity import assert_rows_close

pytestmark = pytest.mark.gpu


def _case(torch, thinfer, rows, n_out, k, seed, fp32):
    rng = np.random.default_rng(seed)
    x_np = (rng.standard_normal((rows, k))).astype(np.float16)
    w_np = (rng.standard_normal((n_out, k)) * 0.05).astype(np.float16)
    x, w = torch.from_numpy(x_np).cuda(), torch.from_numpy(w_np).cuda()
    want = thinfer.op_linear(x, w, out_fp32=fp32, path=0)           # existing entry point
    y = torch.full((rows, n_out), float("nan"), dtype=torch.float32 if fp32 else torch.float16, device="cuda")
    thinfer.op_linear_noalloc(x, w, y)                                # caller-provided output, nothing allocated inside
    torch.cuda.synchronize()
    # same tolerance as the linear parity tests: the two differ only in the order of the FP32 partial sums
    assert_rows_close(y.float().cpu().numpy(), want.float().cpu().numpy().astype(np.float64),
                      f"no-alloc linear {rows}x{n_out}x{k}", max_err=4e-3)
    # and against the definition itself, with the tolerance of the other linear parity tests
    assert_rows_close(y.float().cpu().numpy(), O.linear(x_np, w_np), f"no-alloc linear {rows}x{n_out}x{k} vs oracle",
                      max_err=4e-3)


def test_noalloc_linear_matches_the_ordinary_entry_point_twice_in_a_row():
    import torch
    from paper_2605_25655_b200 import thinfer
    assert torch.cuda.is_available()
    _case(torch, thinfer, 16, 4096, 4096, seed=1, fp32=False)       # many tiles, every tile split over several CTAs
    _case(torch, thinfer, 5, 1000, 11008, seed=2, fp32=True)        # ragged rows and features, long contraction
    _case(torch, thinfer, 16, 4096, 4096, seed=3, fp32=False)       # first shape again on reused scratch


def test_noalloc_linear_rejects_sizes_beyond_its_scratch():
    import torch
    from paper_2605_25655_b200 import thinfer
    x = torch.zeros(17, 64, dtype=torch.float16, device="cuda")
    w = torch.zeros(128, 64, dtype=torch.float16, device="cuda")
    with pytest.raises(thinfer.ThinferError) as e:
        thinfer.op_linear_noalloc(x, w, torch.empty(17, 128, dtype=torch.float16, device="cuda"))
    assert e.value.code == thinfer.ECAPACITY and "limit" in str(e.value)
    x = torch.zeros(4, 64, dtype=torch.float16, device="cuda")
    w = torch.zeros(16386, 64, dtype=torch.float16, device="cuda")
    with pytest.raises(thinfer.ThinferError) as e:
        thinfer.op_linear_noalloc(x, w, torch.empty(4, 16386, dtype=torch.float16, device="cuda"))
    assert e.value.code == thinfer.ECAPACITY
