"""ctypes binding over libthinfer.so (include/thinfer.h).

Argument marshalling only: torch supplies device memory and streams, every step
of the path runs in the library's CUDA kernels.  There is no CPU fallback: if
the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libthinfer.so")
# one build per 16-bit storage type, same exports (include/thinfer.h)
LIB_PATHS = {"f16": LIB_PATH, "bf16": os.path.join(_HERE, "libthinfer_bf16.so")}

OK, EINVAL, EUNSUPPORTED, ECAPACITY, EBUSY, ECUDA, ETIMEOUT = 0, -1, -2, -3, -4, -5, -6
ERR_NAMES = {OK: "THINFER_OK", EINVAL: "THINFER_EINVAL", EUNSUPPORTED: "THINFER_EUNSUPPORTED",
             ECAPACITY: "THINFER_ECAPACITY", EBUSY: "THINFER_EBUSY", ECUDA: "THINFER_ECUDA",
             ETIMEOUT: "THINFER_ETIMEOUT"}
K_RMSNORM, K_QKV, K_ATTN, K_ATTN_COMBINE, K_OPROJ, K_GATEUP, K_DOWN, K_HEAD, K_EMBED, K_ARGMAX, K_DECODE_UNIFIED = range(11)

EXPORTS = (
    "thinfer_storage_type", "thinfer_workspace_bytes", "thinfer_create", "thinfer_prefill", "thinfer_prefill_ragged", "thinfer_slot_lengths",
    "thinfer_decode_step",
    "thinfer_prefill_host", "thinfer_decode_step_host", "thinfer_release_slot", "thinfer_slot_state",
    "thinfer_kv_pointer", "thinfer_status", "thinfer_clear_status", "thinfer_capture_hidden", "thinfer_set_launch_mode", "thinfer_profile_select",
    "thinfer_profile_read", "thinfer_trace_unified", "thinfer_launch_count", "thinfer_last_error", "thinfer_destroy",
    "thinfer_op_linear", "thinfer_op_linear_noalloc", "thinfer_op_attention_prefill", "thinfer_op_rmsnorm",
    "thinfer_op_argmax", "thinfer_op_attention_decode", "thinfer_selftest_bounded_wait",
)


class ThinferError(RuntimeError):
    def __init__(self, code, what=""):
        self.code = code
        super().__init__(f"{ERR_NAMES.get(code, code)}: {what}")


class Config(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("ffn", C.c_int32), ("n_layers", C.c_int32), ("vocab", C.c_int32),
                ("rms_eps", C.c_float), ("rope_base", C.c_float), ("max_batch", C.c_int32),
                ("max_seq", C.c_int32), ("buf_slots", C.c_int32)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")]


class Weights(C.Structure):
    _fields_ = [("layers", C.POINTER(LayerWeights)), ("embed", C.c_void_p), ("final_norm", C.c_void_p),
                ("lm_head", C.c_void_p)]


_libs = {}


def storage_of(tensor) -> str:
    """'f16' or 'bf16' for a torch tensor of a storage type the library is built for."""
    import torch
    if tensor.dtype == torch.float16:
        return "f16"
    if tensor.dtype == torch.bfloat16:
        return "bf16"
    raise ThinferError(EUNSUPPORTED, f"storage type {tensor.dtype}: the library is built for float16 and bfloat16")


def lib(storage="f16"):
    """Loads the shared library of a storage type (once).  Fails loudly when it has not been built."""
    if storage in _libs:
        return _libs[storage]
    path = LIB_PATHS[storage]
    if not os.path.exists(path):
        raise ThinferError(ECUDA, f"{path} is missing: build it with "
                                  "`python -m paper_2605_25655_b200._build` (needs nvcc)")
    L = C.CDLL(path)
    L.thinfer_storage_type.argtypes = []
    assert L.thinfer_storage_type() == {"f16": 0, "bf16": 1}[storage], path
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    L.thinfer_workspace_bytes.argtypes = [C.POINTER(Config), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    L.thinfer_create.argtypes = [C.POINTER(Config), C.POINTER(Weights), vp, C.c_size_t, vp, C.c_size_t, C.POINTER(vp)]
    L.thinfer_prefill.argtypes = [vp, i32, vp, i32, i32, vp, vp, vp]
    L.thinfer_prefill_ragged.argtypes = [vp, i32, vp, i32, i32, C.POINTER(i32), vp, vp, vp]
    L.thinfer_slot_lengths.argtypes = [vp, i32, C.POINTER(i32)]
    L.thinfer_decode_step.argtypes = [vp, i32, vp, vp, vp, vp]
    L.thinfer_prefill_host.argtypes = [vp, i32, vp, i32, i32, vp, vp, vp]
    L.thinfer_decode_step_host.argtypes = [vp, i32, vp, vp, vp, vp]
    L.thinfer_release_slot.argtypes = [vp, i32, vp]
    L.thinfer_slot_state.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(i32)]
    L.thinfer_kv_pointer.argtypes = [vp, i32, i32, i32, C.POINTER(vp)]
    L.thinfer_status.argtypes = [vp, C.POINTER(i32)]
    L.thinfer_clear_status.argtypes = [vp]
    L.thinfer_capture_hidden.argtypes = [vp, i32, C.POINTER(i32), C.POINTER(vp)]
    L.thinfer_set_launch_mode.argtypes = [vp, i32]
    L.thinfer_profile_select.argtypes = [vp, i32]
    L.thinfer_profile_read.argtypes = [vp, C.POINTER(i32), C.POINTER(C.c_float)]
    L.thinfer_trace_unified.argtypes = [vp, i32, C.POINTER(C.c_uint64), i32]
    L.thinfer_launch_count.argtypes = [vp]
    L.thinfer_launch_count.restype = i64
    L.thinfer_last_error.argtypes = [vp]
    L.thinfer_last_error.restype = C.c_char_p
    L.thinfer_destroy.argtypes = [vp]
    L.thinfer_destroy.restype = None
    L.thinfer_op_linear.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp]
    L.thinfer_op_linear_noalloc.argtypes = [vp, vp, vp, i32, i32, i32, i32, vp]
    L.thinfer_op_attention_prefill.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp]
    L.thinfer_op_rmsnorm.argtypes = [vp, vp, vp, i32, i32, C.c_float, vp]
    L.thinfer_op_argmax.argtypes = [vp, vp, i32, i32, vp]
    L.thinfer_op_attention_decode.argtypes = [vp, i32, i32, vp, vp, i32, i32, C.POINTER(i32), vp]
    L.thinfer_selftest_bounded_wait.argtypes = [vp, i64, vp]
    _libs[storage] = L
    return L


def _check(rc, ctx=None, storage="f16"):
    if rc != OK:
        msg = lib(storage).thinfer_last_error(ctx)
        raise ThinferError(rc, msg.decode() if msg else "")


def _stream_ptr(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def make_config(shape, max_batch, max_seq, buf_slots=1) -> Config:
    """shape: any object with the fields of synth.Shape."""
    return Config(shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn, shape.n_layers,
                  shape.vocab, shape.rms_eps, shape.rope_base, max_batch, max_seq, buf_slots)


def workspace_bytes(cfg: Config, storage="f16"):
    kv, sc = C.c_size_t(0), C.c_size_t(0)
    _check(lib(storage).thinfer_workspace_bytes(C.byref(cfg), C.byref(kv), C.byref(sc)), None, storage)
    return kv.value, sc.value


class Context:
    """One thinfer_ctx plus the torch tensors that back its caller-owned memory.

    layers: list of dicts name -> CUDA float16 (or bfloat16) tensor (names of thinfer_layer_weights);
    stack:  dict with embed / final_norm / lm_head when shape.vocab > 0.
    """

    def __init__(self, shape, layers, stack=None, max_batch=1, max_seq=128, buf_slots=1, device="cuda:0"):
        import torch
        self.torch = torch
        self.shape = shape
        self.device = torch.device(device)
        self.cfg = make_config(shape, max_batch, max_seq, buf_slots)
        self.storage = storage_of(layers[0]["wq"])         # the weights decide which build serves this context
        self.dtype = layers[0]["wq"].dtype
        self.L = lib(self.storage)
        kv_bytes, scratch_bytes = workspace_bytes(self.cfg, self.storage)
        with torch.cuda.device(self.device):
            self.kv = torch.empty(kv_bytes, dtype=torch.uint8, device=self.device)
            self.scratch = torch.empty(scratch_bytes, dtype=torch.uint8, device=self.device)
            self._keep = (layers, stack)
            arr = (LayerWeights * shape.n_layers)()
            for l, w in enumerate(layers):
                for name, _ in LayerWeights._fields_:
                    t = w[name]
                    assert t.is_cuda and t.dtype == self.dtype and t.is_contiguous(), name
                    setattr(arr[l], name, t.data_ptr())
            wts = Weights(arr, None, None, None)
            if shape.vocab > 0:
                wts.embed, wts.final_norm, wts.lm_head = (stack[n].data_ptr() for n in ("embed", "final_norm", "lm_head"))
            h = C.c_void_p(None)
            _check(self.L.thinfer_create(C.byref(self.cfg), C.byref(wts), self.kv.data_ptr(), kv_bytes,
                                         self.scratch.data_ptr(), scratch_bytes, C.byref(h)), None, self.storage)
        self.h = h

    # -- device-buffer calls ------------------------------------------------
    def prefill(self, inp, slot=0, stream=None, want_logits=False, out=None):
        torch = self.torch
        batch, seq = int(inp.shape[0]), int(inp.shape[1])
        assert inp.is_cuda and inp.is_contiguous()
        if self.shape.vocab == 0:
            assert inp.dtype == self.dtype
            out = torch.empty_like(inp)
            _check(self.L.thinfer_prefill(self.h, slot, inp.data_ptr(), batch, seq, out.data_ptr(), None,
                                         _stream_ptr(stream)), self.h, self.storage)
            return out
        assert inp.dtype == torch.int32
        ids = torch.empty(batch, dtype=torch.int32, device=self.device) if out is None else out
        logits = torch.empty(batch, self.shape.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        _check(self.L.thinfer_prefill(self.h, slot, inp.data_ptr(), batch, seq, ids.data_ptr(),
                                     logits.data_ptr() if want_logits else None, _stream_ptr(stream)), self.h, self.storage)
        return (ids, logits) if want_logits else ids

    def prefill_ragged(self, inp, seq_lens, slot=0, stream=None, want_logits=False):
        """Prompts of different lengths, padded to inp.shape[1]; seq_lens: one length per request."""
        torch = self.torch
        batch, seq = int(inp.shape[0]), int(inp.shape[1])
        lens = (C.c_int32 * batch)(*[int(v) for v in seq_lens])
        assert inp.is_cuda and inp.is_contiguous()
        if self.shape.vocab == 0:
            out = torch.empty_like(inp)
            _check(self.L.thinfer_prefill_ragged(self.h, slot, inp.data_ptr(), batch, seq, lens, out.data_ptr(), None,
                                                _stream_ptr(stream)), self.h, self.storage)
            return out
        ids = torch.empty(batch, dtype=torch.int32, device=self.device)
        logits = torch.empty(batch, self.shape.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        _check(self.L.thinfer_prefill_ragged(self.h, slot, inp.data_ptr(), batch, seq, lens, ids.data_ptr(),
                                            logits.data_ptr() if want_logits else None, _stream_ptr(stream)), self.h, self.storage)
        return (ids, logits) if want_logits else ids

    def slot_lengths(self, slot=0):
        b, _ = self.slot_state(slot)
        buf = (C.c_int32 * max(b, 1))()
        _check(self.L.thinfer_slot_lengths(self.h, slot, buf), self.h, self.storage)
        return list(buf)[:b]

    def decode_step(self, inp, slot=0, stream=None, want_logits=False, out=None):
        torch = self.torch
        assert inp.is_cuda and inp.is_contiguous()
        if self.shape.vocab == 0:
            out = torch.empty_like(inp) if out is None else out
            _check(self.L.thinfer_decode_step(self.h, slot, inp.data_ptr(), out.data_ptr(), None,
                                             _stream_ptr(stream)), self.h, self.storage)
            return out
        batch = int(inp.shape[0])
        ids = torch.empty(batch, dtype=torch.int32, device=self.device) if out is None else out
        logits = torch.empty(batch, self.shape.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        _check(self.L.thinfer_decode_step(self.h, slot, inp.data_ptr(), ids.data_ptr(),
                                         logits.data_ptr() if want_logits else None, _stream_ptr(stream)), self.h, self.storage)
        return (ids, logits) if want_logits else ids

    # -- host-buffer calls (pinned tensors make the copies asynchronous) -----
    def prefill_host(self, host_in, host_out, slot=0, stream=None, host_logits=None):
        batch, seq = int(host_in.shape[0]), int(host_in.shape[1])
        _check(self.L.thinfer_prefill_host(self.h, slot, host_in.data_ptr(), batch, seq, host_out.data_ptr(),
                                          host_logits.data_ptr() if host_logits is not None else None,
                                          _stream_ptr(stream)), self.h, self.storage)

    def decode_step_host(self, host_in, host_out, slot=0, stream=None, host_logits=None):
        _check(self.L.thinfer_decode_step_host(self.h, slot, host_in.data_ptr(), host_out.data_ptr(),
                                              host_logits.data_ptr() if host_logits is not None else None,
                                              _stream_ptr(stream)), self.h, self.storage)

    # -- bookkeeping ----------------------------------------------------------
    def release_slot(self, slot=0, stream=None):
        _check(self.L.thinfer_release_slot(self.h, slot, _stream_ptr(stream)), self.h, self.storage)

    def slot_state(self, slot=0):
        b, n = C.c_int32(0), C.c_int32(0)
        _check(self.L.thinfer_slot_state(self.h, slot, C.byref(b), C.byref(n)), self.h, self.storage)
        return b.value, n.value

    def kv_view(self, slot, layer, which):
        """Strided torch view [max_batch][n_kv_heads][max_seq][head_dim] of K (0) or V (1)."""
        p = C.c_void_p(None)
        _check(self.L.thinfer_kv_pointer(self.h, slot, layer, which, C.byref(p)), self.h, self.storage)
        off = p.value - self.kv.data_ptr()
        n = self.cfg.max_batch * self.cfg.n_kv_heads * self.cfg.max_seq * self.cfg.head_dim
        return self.kv[off:off + 2 * n].view(self.dtype).view(
            self.cfg.max_batch, self.cfg.n_kv_heads, self.cfg.max_seq, self.cfg.head_dim)

    def status(self):
        v = C.c_int32(0)
        _check(self.L.thinfer_status(self.h, C.byref(v)), self.h, self.storage)
        return v.value

    def clear_status(self):
        _check(self.L.thinfer_clear_status(self.h), self.h, self.storage)

    def attention_decode(self, q, t_len, slot=0, layer=0, seq_lens=None, stream=None):
        """Decode attention alone over the cache of (slot, layer): q [batch, n_q_heads, head_dim] -> [batch, n_q_heads*d]."""
        batch = int(q.shape[0])
        out = self.torch.empty(batch, self.shape.n_q_heads * self.shape.head_dim, dtype=q.dtype, device=q.device)
        lens = (C.c_int32 * batch)(*[int(v) for v in seq_lens]) if seq_lens is not None else None
        _check(self.L.thinfer_op_attention_decode(self.h, slot, layer, q.data_ptr(), out.data_ptr(), batch, int(t_len),
                                                  lens, _stream_ptr(stream)), self.h, self.storage)
        return out

    def selftest_bounded_wait(self, limit_ns=1_000_000, stream=None):
        _check(self.L.thinfer_selftest_bounded_wait(self.h, int(limit_ns), _stream_ptr(stream)), self.h, self.storage)

    def capture_hidden(self, captures):
        """captures: dict layer index (-1 = input of layer 0) -> CUDA FP16 tensor that receives the hidden
        state behind that layer on every later prefill / decode step; {} or None removes all captures."""
        captures = captures or {}
        n = len(captures)
        layers = (C.c_int32 * max(n, 1))(*[int(l) for l in captures])
        bufs = (C.c_void_p * max(n, 1))(*[t.data_ptr() for t in captures.values()])
        self._captures = captures                      # keeps the tensors alive
        _check(self.L.thinfer_capture_hidden(self.h, n, layers, bufs), self.h, self.storage)

    def set_launch_mode(self, mode):
        _check(self.L.thinfer_set_launch_mode(self.h, mode), self.h, self.storage)

    def profile_select(self, kernel_id):
        _check(self.L.thinfer_profile_select(self.h, kernel_id), self.h, self.storage)

    def profile_read(self):
        n, ms = C.c_int32(0), C.c_float(0)
        _check(self.L.thinfer_profile_read(self.h, C.byref(n), C.byref(ms)), self.h, self.storage)
        return n.value, ms.value

    def trace_unified(self, enable=True, read=0):
        """Switches the unit-boundary trace of the unified decode kernel on/off; returns `read` entries (ns)."""
        buf = (C.c_uint64 * max(read, 1))()
        _check(self.L.thinfer_trace_unified(self.h, int(enable), buf if read else None, read), self.h, self.storage)
        return list(buf)[:read]

    def launch_count(self):
        return int(self.L.thinfer_launch_count(self.h))

    def close(self):
        if self.h is not None and self.h.value:
            self.L.thinfer_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ---------------------------------------------------------------- operators
def op_linear(x, w, out_fp32=False, path=0, stream=None, out=None):
    import torch
    rows, k = x.shape
    n_out = w.shape[0]
    if out is not None:
        y, out_fp32 = out, out.dtype == torch.float32
    else:
        y = torch.empty(rows, n_out, dtype=torch.float32 if out_fp32 else x.dtype, device=x.device)
    st = storage_of(x)
    _check(lib(st).thinfer_op_linear(x.data_ptr(), w.data_ptr(), y.data_ptr(), rows, n_out, k, int(out_fp32), path,
                                     _stream_ptr(stream)), None, st)
    return y


def op_linear_noalloc(x, w, y, stream=None):
    """y[rows, n_out] = x w^T through the entry point that allocates nothing: the caller passes
    the output (FP16 or FP32 tensor); the split-K scratch is a fixed array inside the library.
    For hosts that cannot call cudaMalloc where they need the product.  rows <= 16, n_out <= 16384."""
    import torch
    rows, k = x.shape
    n_out = w.shape[0]
    assert y.shape == (rows, n_out) and y.is_contiguous()
    st = storage_of(x)
    _check(lib(st).thinfer_op_linear_noalloc(x.data_ptr(), w.data_ptr(), y.data_ptr(), rows, n_out, k,
                                             int(y.dtype == torch.float32), _stream_ptr(stream)), None, st)
    return y


def op_attention_prefill(q, k, v, seq=None, stream=None, out=None):
    """q [B, Hq, S, d]; k, v [B, Hkv, T, d] with T >= S (the first S positions are used) -> [B, S, Hq*d]."""
    import torch
    b, hq, s, d = q.shape
    hkv, t = k.shape[1], k.shape[2]
    if out is None:
        out = torch.empty(b, s, hq * d, dtype=q.dtype, device=q.device)
    st = storage_of(q)
    _check(lib(st).thinfer_op_attention_prefill(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), b, hq, hkv,
                                                s, t, d, _stream_ptr(stream)), None, st)
    return out


def op_rmsnorm(x, gain, eps, stream=None):
    import torch
    rows, n = x.shape
    y = torch.empty_like(x)
    st = storage_of(x)
    _check(lib(st).thinfer_op_rmsnorm(x.data_ptr(), gain.data_ptr(), y.data_ptr(), rows, n, eps, _stream_ptr(stream)), None, st)
    return y


def op_argmax(logits, stream=None):
    import torch
    rows, n = logits.shape
    ids = torch.empty(rows, dtype=torch.int32, device=logits.device)
    _check(lib().thinfer_op_argmax(logits.data_ptr(), ids.data_ptr(), rows, n, _stream_ptr(stream)))
    return ids


def to_device_layers(np_layers, device="cuda:0"):
    """numpy FP16 weight dicts (synth.layer_weights) -> torch CUDA tensors."""
    import torch
    return [{k: torch.from_numpy(v).to(device) for k, v in w.items()} for w in np_layers]
