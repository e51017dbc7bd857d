"""The C-ABI library loads and exports every symbol the header declares; host
side validation answers with error codes (no GPU needed, no compute calls)."""
import ctypes as C
import os
import re

import pytest

from paper_2605_25655_b200 import _build, synth, thinfer

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    _build.build()          # cross-compiles for sm_100a; a no-op when the library is current
    return thinfer.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "thinfer.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(thinfer_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert set(names) == set(thinfer.EXPORTS)
    for storage, code in (("f16", 0), ("bf16", 1)):          # one build per storage type, the same exports
        L = thinfer.lib(storage)
        for n in names:
            assert hasattr(L, n), (storage, n)
        assert L.thinfer_storage_type() == code
    for n in ("thinfer_create", "thinfer_prefill", "thinfer_decode_step", "thinfer_destroy"):
        assert n in names


def test_header_compiles_as_plain_c(tmp_path):
    src = tmp_path / "t.c"
    src.write_text('#include "thinfer.h"\nint main(void){thinfer_config c; (void)c; return THINFER_OK;}\n')
    assert os.system(f"gcc -std=c99 -Wall -Werror -I{ROOT}/include -c {src} -o {tmp_path}/t.o") == 0


def test_workspace_bytes_validates_and_sizes(lib):
    cfg = thinfer.make_config(synth.TINY, max_batch=2, max_seq=64, buf_slots=3)
    kv, sc = thinfer.workspace_bytes(cfg)
    per = 2 * synth.TINY.n_kv_heads * 64 * synth.TINY.head_dim * 2      # one of K/V, one layer, one slot
    assert kv >= 3 * 1 * 2 * per and kv % 1024 == 0
    assert sc > 0
    bad = thinfer.make_config(synth.TINY, max_batch=2, max_seq=64)
    bad.head_dim = 96
    with pytest.raises(thinfer.ThinferError) as e:
        thinfer.workspace_bytes(bad)
    assert e.value.code == thinfer.EUNSUPPORTED
    bad = thinfer.make_config(synth.TINY, max_batch=0, max_seq=64)
    with pytest.raises(thinfer.ThinferError) as e:
        thinfer.workspace_bytes(bad)
    assert e.value.code == thinfer.EINVAL
    bad = thinfer.make_config(synth.TINY, max_batch=1, max_seq=64)
    bad.n_kv_heads = 3
    with pytest.raises(thinfer.ThinferError) as e:
        thinfer.workspace_bytes(bad)
    assert e.value.code == thinfer.EUNSUPPORTED
    assert lib.thinfer_workspace_bytes(None, None, None) == thinfer.EINVAL


def test_null_context_calls_return_einval(lib):
    assert lib.thinfer_prefill(None, 0, None, 1, 1, None, None, None) == thinfer.EINVAL
    assert lib.thinfer_decode_step(None, 0, None, None, None, None) == thinfer.EINVAL
    assert lib.thinfer_release_slot(None, 0, None) == thinfer.EINVAL
    assert lib.thinfer_status(None, None) == thinfer.EINVAL
    assert lib.thinfer_op_linear(None, None, None, 1, 2, 8, 0, 0, None) == thinfer.EINVAL
    assert lib.thinfer_launch_count(None) == 0
    lib.thinfer_destroy(None)                  # a no-op


def test_70b_sizes_fit_one_gpu():
    # KV of the largest configuration (batch 4, 512 + 128 positions) and its scratch stay far below 180 GB
    cfg = thinfer.make_config(synth.LLAMA_70B, max_batch=4, max_seq=640)
    kv, sc = thinfer.workspace_bytes(cfg)
    assert kv == 80 * 2 * 4 * 8 * 640 * 128 * 2
    assert kv + sc < 8e9
