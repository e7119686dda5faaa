"""ctypes binding of libfastmtp.so: argument marshalling only.

Function names mirror the C ABI (include/fastmtp.h). Tensors are torch tensors (device memory
for the device entry points, CPU tensors for the *_host ones); the binding passes their
data pointers and sizes and never computes anything itself. There is no fallback: if the
shared library is missing or fails to load, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

from . import build as _build

_LIB_PATH = os.environ.get("FASTMTP_LIB", _build.LIB)     # override: a library built elsewhere
if not os.path.exists(_LIB_PATH):
    raise ImportError(f"{_LIB_PATH} not built: run `python -m paper_2509_18362_b200.build` "
                      "(there is no CPU fallback)")
lib = C.CDLL(_LIB_PATH)

FMTP_OK = 0
DEV_BAD_TOKEN, DEV_BAD_PAGE, DEV_BAD_POS, DEV_TIMEOUT, DEV_ALL_NAN = 1, 2, 4, 8, 16

EXPORTS = ["fmtp_create", "fmtp_destroy", "fmtp_workspace_bytes", "fmtp_set_workspace", "fmtp_strerror",
           "fmtp_last_cuda_error", "fmtp_launch_count", "fmtp_tmem_launch_count", "fmtp_selftest_wait_timeout", "fmtp_selftest_inject_wait_timeout",
           "fastmtp_draft", "fastmtp_draft_host",
           "fastmtp_verify_accept", "fastmtp_verify_accept_host", "fastmtp_verify_accept_static", "fastmtp_accept_ids",
           "fastmtp_target_step"]

_p = C.c_void_p


class fmtp_shape(C.Structure):
    _fields_ = [("d", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("ffn", C.c_int32), ("vocab", C.c_int32), ("n_layers", C.c_int32), ("rms_eps", C.c_float),
                ("rope_theta", C.c_float), ("page_size", C.c_int32), ("max_rows", C.c_int32),
                ("max_K", C.c_int32), ("max_ctx", C.c_int32)]


class fmtp_layer_w(C.Structure):
    _fields_ = [(n, _p) for n in ("g_in", "wq", "wk", "wv", "wo", "g_post", "w_gate", "w_up", "w_down")]


class fmtp_mtp_w(C.Structure):
    _fields_ = [(n, _p) for n in ("embed", "lm_head", "g_hnorm", "g_enorm", "w_proj", "g_final")] + \
               [("layer", fmtp_layer_w)]


class fmtp_target_w(C.Structure):
    _fields_ = [("embed", _p), ("lm_head", _p), ("g_final", _p), ("layers", C.POINTER(fmtp_layer_w))]


class fmtp_kv(C.Structure):
    _fields_ = [("k_pages", _p), ("v_pages", _p), ("block_table", _p), ("seq_lens", _p),
                ("num_pages", C.c_int32), ("max_pages_per_seq", C.c_int32)]


lib.fmtp_create.argtypes = [C.POINTER(fmtp_shape), C.POINTER(_p)]
lib.fmtp_create.restype = C.c_int
lib.fmtp_destroy.argtypes = [_p]
lib.fmtp_destroy.restype = C.c_int
lib.fmtp_workspace_bytes.argtypes = [_p]
lib.fmtp_workspace_bytes.restype = C.c_size_t
lib.fmtp_set_workspace.argtypes = [_p, _p, C.c_size_t]
lib.fmtp_set_workspace.restype = C.c_int
lib.fmtp_strerror.argtypes = [C.c_int]
lib.fmtp_strerror.restype = C.c_char_p
lib.fmtp_last_cuda_error.argtypes = [_p]
lib.fmtp_last_cuda_error.restype = C.c_int
lib.fmtp_launch_count.argtypes = [_p]
lib.fmtp_launch_count.restype = C.c_longlong
lib.fmtp_tmem_launch_count.argtypes = [_p]
lib.fmtp_tmem_launch_count.restype = C.c_longlong
lib.fmtp_selftest_wait_timeout.argtypes = [_p, C.c_int, _p, _p]
lib.fmtp_selftest_wait_timeout.restype = C.c_int
lib.fmtp_selftest_inject_wait_timeout.argtypes = [_p, C.c_int, C.c_int]
lib.fmtp_selftest_inject_wait_timeout.restype = C.c_int
lib.fastmtp_draft.argtypes = [_p, C.POINTER(fmtp_mtp_w), _p, _p, _p, C.c_int, C.POINTER(fmtp_kv), C.c_int, C.c_int, _p,
                              C.c_int, _p, _p, _p, _p, _p]
lib.fastmtp_draft.restype = C.c_int
lib.fastmtp_draft_host.argtypes = [_p, C.POINTER(fmtp_mtp_w), _p, _p, _p, C.c_int, C.POINTER(fmtp_kv), C.c_int, C.c_int,
                                   _p, C.c_int, _p, _p]
lib.fastmtp_draft_host.restype = C.c_int
lib.fastmtp_verify_accept.argtypes = [_p, _p, _p, C.c_int, C.c_int, C.c_int, _p, _p, _p, _p, _p]
lib.fastmtp_verify_accept.restype = C.c_int
lib.fastmtp_verify_accept_host.argtypes = [_p, _p, _p, C.c_int, C.c_int, C.c_int, _p, _p, _p]
lib.fastmtp_verify_accept_host.restype = C.c_int
lib.fastmtp_accept_ids.argtypes = [_p, _p, _p, C.c_int, C.c_int, _p, _p, _p]
lib.fastmtp_accept_ids.restype = C.c_int
lib.fastmtp_verify_accept_static.argtypes = [_p, _p, C.c_int, C.c_int, C.c_int, _p, _p, _p, _p, _p]
lib.fastmtp_verify_accept_static.restype = C.c_int
lib.fastmtp_target_step.argtypes = [_p, C.POINTER(fmtp_target_w), _p, C.POINTER(fmtp_kv), C.c_int, C.c_int,
                                    _p, _p, _p, _p, _p]
lib.fastmtp_target_step.restype = C.c_int


class FastMTPError(RuntimeError):
    def __init__(self, code: int, where: str, cuda: int = 0):
        self.code = code
        msg = lib.fmtp_strerror(code).decode()
        super().__init__(f"{where}: {msg} (status {code}" + (f", cudaError {cuda}" if cuda else "") + ")")


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def layer_w(t: dict) -> fmtp_layer_w:
    """Pointer struct over a dict of device tensors named like the C fields."""
    return fmtp_layer_w(**{n: t[n].data_ptr() for n, _ in fmtp_layer_w._fields_})


def mtp_w(t: dict) -> fmtp_mtp_w:
    w = fmtp_mtp_w(**{n: t[n].data_ptr() for n in ("embed", "lm_head", "g_hnorm", "g_enorm", "w_proj", "g_final")})
    w.layer = layer_w(t["layer"])
    return w


def target_w(t: dict):
    """Returns (struct, keepalive): the layer array must outlive the struct's use."""
    n = len(t["layers"])
    arr = (fmtp_layer_w * n)(*[layer_w(l) for l in t["layers"]])
    w = fmtp_target_w(t["embed"].data_ptr(), t["lm_head"].data_ptr(), t["g_final"].data_ptr(),
                      C.cast(arr, C.POINTER(fmtp_layer_w)))
    return w, arr


def kv(t: dict) -> fmtp_kv:
    return fmtp_kv(t["k_pages"].data_ptr(), t["v_pages"].data_ptr(), t["block_table"].data_ptr(),
                   t["seq_lens"].data_ptr(), int(t["k_pages"].shape[0]), int(t["block_table"].shape[1]))


def fmtp_selftest_wait_timeout(dev_status, limit_ms, dev_waited_ns=None, stream=None):
    """Launches the bounded-wait probe (a wait that must run out); see include/fastmtp.h."""
    rc = lib.fmtp_selftest_wait_timeout(_ptr(dev_status), int(limit_ms), _ptr(dev_waited_ns), _stream(stream))
    if rc != FMTP_OK:
        raise FastMTPError(rc, "fmtp_selftest_wait_timeout")


STATIC_VERIFY_MAX_ROWS = 1024


def fastmtp_verify_accept_static(target_logits, drafts, B, K, V, out_accept_len, out_bonus, out_argmax=None,
                                 dev_status=None, stream=None):
    """Verification through the entry point that needs no context and allocates nothing (its scratch
    is a fixed array inside the library). Same arguments as Context.fastmtp_verify_accept."""
    rc = lib.fastmtp_verify_accept_static(_ptr(target_logits), _ptr(drafts), B, K, V, _ptr(out_accept_len),
                                          _ptr(out_bonus), _ptr(out_argmax), _ptr(dev_status), _stream(stream))
    if rc != FMTP_OK:
        raise FastMTPError(rc, "fastmtp_verify_accept_static")


class Context:
    """Owns an fmtp_ctx and the torch-allocated workspace handed to it."""

    def __init__(self, shape, max_rows: int = 8, max_K: int = 8, max_ctx: int = 8704, n_layers=None):
        self.shape = shape
        cs = fmtp_shape(shape.d, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn, shape.vocab,
                        shape.n_layers if n_layers is None else n_layers, shape.rms_eps, shape.rope_theta,
                        shape.page_size, max_rows, max_K, max_ctx)
        h = _p()
        rc = lib.fmtp_create(C.byref(cs), C.byref(h))
        if rc != FMTP_OK:
            raise FastMTPError(rc, "fmtp_create")
        self.handle = h
        nbytes = lib.fmtp_workspace_bytes(h)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        self._check(lib.fmtp_set_workspace(h, C.c_void_p(base), nbytes), "fmtp_set_workspace")

    def _check(self, rc, where):
        if rc != FMTP_OK:
            raise FastMTPError(rc, where, lib.fmtp_last_cuda_error(self.handle))

    def close(self):
        if self.handle:
            lib.fmtp_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def fmtp_selftest_inject_wait_timeout(self, limit_ms, which):
        self._check(lib.fmtp_selftest_inject_wait_timeout(self.handle, int(limit_ms), int(which)),
                    "fmtp_selftest_inject_wait_timeout")

    @property
    def launch_count(self) -> int:
        return int(lib.fmtp_launch_count(self.handle))

    @property
    def tmem_launch_count(self) -> int:
        return int(lib.fmtp_tmem_launch_count(self.handle))

    # -- entry points (same names and argument order as the C ABI)
    def fastmtp_draft(self, w: fmtp_mtp_w, h_last, tok_last, mtp_kv: fmtp_kv, B, K, vocab_subset, out_drafts,
                      out_h=None, out_logits=None, dev_status=None, stream=None, n_ext=None, max_ext=1):
        """h_last [B, max_ext, d] / tok_last [B, max_ext]; n_ext (device int32 [B]) and max_ext follow tok_last in
        the C argument list and default to the plain one-pair-per-sequence form."""
        N = 0 if vocab_subset is None else int(vocab_subset.numel())
        self._check(lib.fastmtp_draft(self.handle, C.byref(w), _ptr(h_last), _ptr(tok_last), _ptr(n_ext), int(max_ext),
                                      C.byref(mtp_kv), B, K, _ptr(vocab_subset), N, _ptr(out_drafts), _ptr(out_h),
                                      _ptr(out_logits), _ptr(dev_status), _stream(stream)), "fastmtp_draft")

    def fastmtp_draft_host(self, w: fmtp_mtp_w, h_last_host, tok_last_host, mtp_kv: fmtp_kv, B, K, vocab_subset,
                           out_drafts_host, stream=None, n_ext_host=None, max_ext=1):
        N = 0 if vocab_subset is None else int(vocab_subset.numel())
        self._check(lib.fastmtp_draft_host(self.handle, C.byref(w), _ptr(h_last_host), _ptr(tok_last_host),
                                           _ptr(n_ext_host), int(max_ext), C.byref(mtp_kv), B, K, _ptr(vocab_subset), N,
                                           _ptr(out_drafts_host), _stream(stream)), "fastmtp_draft_host")

    def fastmtp_verify_accept(self, target_logits, drafts, B, K, V, out_accept_len, out_bonus, out_argmax=None,
                              dev_status=None, stream=None):
        self._check(lib.fastmtp_verify_accept(self.handle, _ptr(target_logits), _ptr(drafts), B, K, V,
                                              _ptr(out_accept_len), _ptr(out_bonus), _ptr(out_argmax),
                                              _ptr(dev_status), _stream(stream)), "fastmtp_verify_accept")

    def fastmtp_accept_ids(self, target_argmax, drafts, B, K, out_accept_len, out_bonus, stream=None):
        self._check(lib.fastmtp_accept_ids(self.handle, _ptr(target_argmax), _ptr(drafts), B, K, _ptr(out_accept_len),
                                           _ptr(out_bonus), _stream(stream)), "fastmtp_accept_ids")

    def fastmtp_verify_accept_host(self, logits_host, drafts_host, B, K, V, out_accept_host, out_bonus_host,
                                   stream=None):
        self._check(lib.fastmtp_verify_accept_host(self.handle, _ptr(logits_host), _ptr(drafts_host), B, K, V,
                                                   _ptr(out_accept_host), _ptr(out_bonus_host), _stream(stream)),
                    "fastmtp_verify_accept_host")

    def fastmtp_target_step(self, w: fmtp_target_w, tokens, layer_kvs, B, M, out_h=None, out_logits=None,
                            out_argmax=None, dev_status=None, stream=None):
        n = len(layer_kvs)
        arr = (fmtp_kv * n)(*layer_kvs)
        self._check(lib.fastmtp_target_step(self.handle, C.byref(w), _ptr(tokens), arr, B, M, _ptr(out_h),
                                            _ptr(out_logits), _ptr(out_argmax), _ptr(dev_status), _stream(stream)),
                    "fastmtp_target_step")


# ---- conversions between the generators' numpy arrays and torch tensors (no arithmetic) ------

def bf16_tensor(bits, device="cuda"):
    """numpy uint16 bf16 bit patterns -> torch.bfloat16 tensor on `device`."""
    import numpy as np
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(device) if device != "cpu" else t


def bf16_bits(t):
    """torch.bfloat16 tensor -> numpy uint16 bit patterns."""
    import numpy as np
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def to_device(tree, device="cuda"):
    """Moves a (nested) dict of generator outputs to the device: uint16 arrays become bf16 tensors,
    int32 arrays int32 tensors; ints are kept."""
    import numpy as np
    if isinstance(tree, dict):
        return {k: to_device(v, device) for k, v in tree.items()}
    if isinstance(tree, list):
        return [to_device(v, device) for v in tree]
    if isinstance(tree, np.ndarray):
        if tree.dtype == np.uint16:
            return bf16_tensor(tree, device)
        return torch.from_numpy(np.ascontiguousarray(tree)).to(device)
    return tree
