"""ctypes binding of the C ABI in include/lola.h.

The functions named `lola_*` mirror the C entry points one to one and only marshal arguments.
`LolaLayer` is a convenience holder that owns the torch tensors the library needs (state buffer,
W, host arrays of the state view); every step of the method runs in the CUDA library.

There is no CPU path: importing this module without the built library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblola_b200.so")

LOLA_OK = 0
LOLA_ERR_ARG, LOLA_ERR_SHAPE, LOLA_ERR_ALIGN, LOLA_ERR_SIZE = -1, -2, -3, -4
LOLA_ERR_UNSUPPORTED, LOLA_ERR_CUDA, LOLA_ERR_DEVICE = -5, -6, -7
LOLA_F32, LOLA_BF16 = 0, 1
LOLA_PHI_SOFTMAX, LOLA_PHI_EXP = 0, 1


class lola_config(C.Structure):
    _fields_ = [("batch", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("feat_half", C.c_int32), ("window", C.c_int32),
                ("sparse", C.c_int32), ("max_chunk", C.c_int32), ("dtype", C.c_int32),
                ("phi_kind", C.c_int32), ("softmax_scale", C.c_float), ("flags", C.c_uint32)]


class lola_state_view(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("H", "s", "sparse_count", "sparse_pos", "sparse_k", "sparse_v", "sparse_score", "threshold",
                 "window_count", "window_pos", "window_k", "window_v", "n_seen", "status")]


class lola_call_info(C.Structure):
    _fields_ = [("paths", C.c_uint32), ("launches", C.c_int32), ("ctas", C.c_int32 * 8)]


PATH_BITS = ["attend_tma", "attend_mma", "attend_generic", "score_tma", "score_mma", "score_generic", "select_kernel",
             "apply_tma", "update_generic", "decode_fused", "decode_fused_long", "h_image_rebuild"]
LOLA_STATUS_SELFTEST = 128
LOLA_FLAG_GENERIC_KERNELS, LOLA_FLAG_QUERY_NO_LINEAR, LOLA_FLAG_QUERY_NO_SPARSE = 1, 4, 8


class LolaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {lola_strerror(code)} ({code})")


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_23666_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    cfgp, viewp = C.POINTER(lola_config), C.POINTER(lola_state_view)
    sig = {
        "lola_state_bytes": (sz, [cfgp]),
        "lola_init_state": (C.c_int, [cfgp, vp, vp, sz, vp, C.POINTER(vp)]),
        "lola_prefill_chunk": (C.c_int, [vp, vp, vp, vp, i32, vp, vp]),
        "lola_prefill_chunks": (C.c_int, [vp, vp, vp, vp, i32, i32, vp, vp]),
        "lola_decode_step": (C.c_int, [vp, vp, vp, vp, vp, vp]),
        "lola_decode_step_static": (C.c_int, [vp, vp, vp, vp, vp, vp]),
        "lola_staging_bytes": (sz, [cfgp, i32]),
        "lola_prefill_chunk_host": (C.c_int, [vp, vp, vp, vp, i32, vp, vp, sz, vp]),
        "lola_prefill_host": (C.c_int, [vp, vp, vp, vp, i32, i32, vp, vp, sz, vp]),
        "lola_decode_step_host": (C.c_int, [vp, vp, vp, vp, vp, vp, sz, vp]),
        "lola_read_state": (C.c_int, [vp, viewp, vp]),
        "lola_write_state": (C.c_int, [vp, viewp, vp]),
        "lola_reset_state": (C.c_int, [vp, vp]),
        "lola_profile_enable": (C.c_int, [vp, C.c_int]),
        "lola_profile_read": (C.c_int, [vp, C.POINTER(C.c_double), C.POINTER(C.c_int64), vp]),
        "lola_last_call_info": (C.c_int, [vp, C.POINTER(lola_call_info)]),
        "lola_selftest_wait_timeout": (C.c_int, [vp, i32, vp]),
        "lola_launch_count": (i64, [vp]),
        "lola_tokens_seen": (i64, [vp]),
        "lola_set_tokens_seen": (C.c_int, [vp, i64]),
        "lola_destroy_state": (C.c_int, [vp]),
        "lola_strerror": (C.c_char_p, [C.c_int]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    return lib


_lib = _load()
EXPORTS = ["lola_state_bytes", "lola_init_state", "lola_prefill_chunk", "lola_prefill_chunks", "lola_decode_step", "lola_decode_step_static", "lola_staging_bytes",
           "lola_prefill_chunk_host", "lola_decode_step_host", "lola_prefill_host", "lola_read_state", "lola_write_state",
           "lola_reset_state", "lola_profile_enable", "lola_profile_read", "lola_last_call_info", "lola_selftest_wait_timeout",
           "lola_launch_count", "lola_tokens_seen", "lola_set_tokens_seen", "lola_destroy_state", "lola_strerror"]


# ---- one-to-one wrappers (pointers are integers: tensor.data_ptr(), stream.cuda_stream) ----
def lola_strerror(code: int) -> str:
    return _lib.lola_strerror(int(code)).decode()


def lola_state_bytes(cfg: lola_config) -> int:
    return int(_lib.lola_state_bytes(C.byref(cfg)))


def lola_staging_bytes(cfg: lola_config, n_tokens: int) -> int:
    return int(_lib.lola_staging_bytes(C.byref(cfg), int(n_tokens)))


def lola_init_state(cfg: lola_config, W_dev: int, state_dev: int, state_bytes: int, stream: int) -> int:
    """Returns the handle (an integer) or raises LolaError."""
    h = C.c_void_p()
    rc = _lib.lola_init_state(C.byref(cfg), W_dev, state_dev, state_bytes, stream, C.byref(h))
    if rc != LOLA_OK:
        raise LolaError(rc, "lola_init_state")
    return h.value


def lola_prefill_chunk(st: int, q: int, k: int, v: int, n_tokens: int, out: int, stream: int) -> int:
    return _lib.lola_prefill_chunk(st, q or None, k, v, int(n_tokens), out or None, stream)


def lola_prefill_chunks(st: int, q: int, k: int, v: int, n_chunks: int, n_tokens: int, out: int, stream: int) -> int:
    return _lib.lola_prefill_chunks(st, q or None, k, v, int(n_chunks), int(n_tokens), out or None, stream)


def lola_decode_step(st: int, q: int, k: int, v: int, out: int, stream: int) -> int:
    return _lib.lola_decode_step(st, q, k, v, out, stream)


def lola_decode_step_static(st: int, q: int, k: int, v: int, out: int, stream: int) -> int:
    """lola_decode_step with the step's work lists in the library's own static device array (for callers
    that cannot supply scratch memory); limited to LOLA_STATIC_MAX_UNITS units."""
    return _lib.lola_decode_step_static(st, q, k, v, out, stream)


def lola_prefill_chunk_host(st, q_host, k_host, v_host, n_tokens, out_host, staging_dev, staging_bytes, stream) -> int:
    return _lib.lola_prefill_chunk_host(st, q_host or None, k_host, v_host, int(n_tokens), out_host or None,
                                        staging_dev, staging_bytes, stream)


def lola_prefill_host(st, q_host, k_host, v_host, n_chunks, n_tokens, out_host, staging_dev, staging_bytes, stream) -> int:
    return _lib.lola_prefill_host(st, q_host or None, k_host, v_host, int(n_chunks), int(n_tokens), out_host or None,
                                  staging_dev, staging_bytes, stream)


def lola_decode_step_host(st, q_host, k_host, v_host, out_host, staging_dev, staging_bytes, stream) -> int:
    return _lib.lola_decode_step_host(st, q_host, k_host, v_host, out_host, staging_dev, staging_bytes, stream)


def lola_read_state(st: int, view: lola_state_view, stream: int) -> int:
    return _lib.lola_read_state(st, C.byref(view), stream)


def lola_write_state(st: int, view: lola_state_view, stream: int) -> int:
    return _lib.lola_write_state(st, C.byref(view), stream)


def lola_reset_state(st: int, stream: int) -> int:
    return _lib.lola_reset_state(st, stream)


KERNEL_KINDS = ["attend", "score", "select", "update", "decode", "kind5", "kind6", "kind7"]


def lola_profile_enable(st: int, enable: bool) -> int:
    return _lib.lola_profile_enable(st, 1 if enable else 0)


def lola_profile_read(st: int, stream: int):
    """Returns ({kind: ms}, {kind: launches}) accumulated since the last read."""
    ms = (C.c_double * 8)()
    n = (C.c_int64 * 8)()
    rc = _lib.lola_profile_read(st, ms, n, stream)
    if rc != LOLA_OK:
        raise LolaError(rc, "lola_profile_read")
    return ({k: ms[i] for i, k in enumerate(KERNEL_KINDS) if n[i]}, {k: n[i] for i, k in enumerate(KERNEL_KINDS) if n[i]})


def lola_last_call_info(st: int) -> dict:
    """{"paths": [names of the LOLA_PATH_* bits], "launches": n, "ctas": {kind: blocks}} of the last call."""
    info = lola_call_info()
    rc = _lib.lola_last_call_info(st, C.byref(info))
    if rc != LOLA_OK:
        raise LolaError(rc, "lola_last_call_info")
    return {"paths": [n for i, n in enumerate(PATH_BITS) if info.paths >> i & 1], "launches": int(info.launches),
            "ctas": {k: int(info.ctas[i]) for i, k in enumerate(KERNEL_KINDS) if info.ctas[i]}}


def lola_selftest_wait_timeout(st: int, limit_us: int, stream: int) -> int:
    return _lib.lola_selftest_wait_timeout(st, int(limit_us), stream)


def lola_launch_count(st: int) -> int:
    return int(_lib.lola_launch_count(st))


def lola_tokens_seen(st: int) -> int:
    return int(_lib.lola_tokens_seen(st))


def lola_set_tokens_seen(st: int, n_seen: int) -> int:
    return _lib.lola_set_tokens_seen(st, int(n_seen))


def lola_destroy_state(st: int) -> int:
    return _lib.lola_destroy_state(st)


# ---- convenience holder --------------------------------------------------------------------
def make_config(batch, n_q_heads, n_kv_heads, head_dim, feat_half, window, sparse, max_chunk,
                dtype="bf16", phi_kind="softmax", softmax_scale=0.0, generic_kernels=False, flags=0) -> lola_config:
    return lola_config(batch, n_q_heads, n_kv_heads, head_dim, feat_half, window, sparse, max_chunk,
                       LOLA_BF16 if dtype == "bf16" else LOLA_F32,
                       LOLA_PHI_EXP if phi_kind == "exp" else LOLA_PHI_SOFTMAX, float(softmax_scale),
                       int(flags) | (1 if generic_kernels else 0))


def _check(rc: int, where: str):
    if rc != LOLA_OK:
        raise LolaError(rc, where)


class LolaLayer:
    """Owns the device buffers of one layer's state and calls the library on torch's current stream."""

    def __init__(self, cfg: lola_config, W, device="cuda:0"):
        self.cfg = cfg
        self.device = torch.device(device)
        self.tdtype = torch.bfloat16 if cfg.dtype == LOLA_BF16 else torch.float32
        W = torch.as_tensor(np.asarray(W, dtype=np.float32)) if not torch.is_tensor(W) else W
        assert tuple(W.shape) == (cfg.n_kv_heads, cfg.head_dim, cfg.feat_half), W.shape
        self.W = W.to(self.device, self.tdtype).contiguous()
        self.nbytes = lola_state_bytes(cfg)
        if self.nbytes == 0:
            raise LolaError(LOLA_ERR_SHAPE, "lola_state_bytes")
        self.state = torch.empty(self.nbytes, dtype=torch.uint8, device=self.device)
        with torch.cuda.device(self.device):
            self.handle = lola_init_state(cfg, self.W.data_ptr(), self.state.data_ptr(), self.nbytes, self._stream())
        self._staging = None

    def _stream(self) -> int:
        return torch.cuda.current_stream(self.device).cuda_stream

    def close(self):
        if getattr(self, "handle", None):
            lola_destroy_state(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- device tensors in, device tensor out
    def prefill_chunk(self, q, k, v, out=None, want_out=True):
        """q [B, n, Hq, d] (or None), k, v [B, n, Hkv, d] device tensors of the state's dtype."""
        n = k.shape[1]
        if want_out and out is None:
            out = torch.empty_like(q)
        _check(lola_prefill_chunk(self.handle, q.data_ptr() if (want_out and q is not None) else 0, k.data_ptr(),
                                  v.data_ptr(), n, out.data_ptr() if want_out else 0, self._stream()),
               "lola_prefill_chunk")
        return out if want_out else None

    def prefill_chunks(self, q, k, v, out=None, want_out=True):
        """q, k, v (and out): device tensors [n_chunks, B, n_tokens, heads, d], the chunks in order."""
        nch, n = k.shape[0], k.shape[2]
        if want_out and out is None:
            out = torch.empty_like(q)
        _check(lola_prefill_chunks(self.handle, q.data_ptr() if want_out else 0, k.data_ptr(), v.data_ptr(), nch, n,
                                   out.data_ptr() if want_out else 0, self._stream()), "lola_prefill_chunks")
        return out if want_out else None

    def decode_step(self, q, k, v, out=None):
        if out is None:
            out = torch.empty_like(q)
        _check(lola_decode_step(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), self._stream()),
               "lola_decode_step")
        return out

    # -- host tensors in, host tensor out (copies inside the call)
    def _staging_for(self, n):
        need = lola_staging_bytes(self.cfg, n)
        if self._staging is None or self._staging.numel() < need:
            self._staging = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._staging

    def prefill_chunk_host(self, q, k, v, out=None, want_out=True):
        n = k.shape[1]
        stg = self._staging_for(n)
        _check(lola_prefill_chunk_host(self.handle, q.data_ptr() if want_out else 0, k.data_ptr(), v.data_ptr(), n,
                                       out.data_ptr() if want_out else 0, stg.data_ptr(), stg.numel(), self._stream()),
               "lola_prefill_chunk_host")
        return out

    def prefill_host(self, q, k, v, out=None, want_out=True):
        """q, k, v (and out): host tensors [n_chunks, B, n_tokens, heads, d], the chunks in order."""
        nch, n = k.shape[0], k.shape[2]
        need = 2 * lola_staging_bytes(self.cfg, n)
        if self._staging is None or self._staging.numel() < need:
            self._staging = torch.empty(need, dtype=torch.uint8, device=self.device)
        stg = self._staging
        _check(lola_prefill_host(self.handle, q.data_ptr() if want_out else 0, k.data_ptr(), v.data_ptr(), nch, n,
                                 out.data_ptr() if want_out else 0, stg.data_ptr(), stg.numel(), self._stream()),
               "lola_prefill_host")
        return out

    def decode_step_host(self, q, k, v, out):
        stg = self._staging_for(1)
        _check(lola_decode_step_host(self.handle, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                     stg.data_ptr(), stg.numel(), self._stream()), "lola_decode_step_host")
        return out

    # -- state view
    def _view_tensors(self, fields=None) -> Dict[str, torch.Tensor]:
        c = self.cfg
        U, d, D, lam, eta = c.batch * c.n_kv_heads, c.head_dim, 2 * c.feat_half, c.sparse, c.window
        spec = {
            "H": ((U, D, d), torch.float32), "s": ((U, D), torch.float32),
            "sparse_count": ((U,), torch.int32), "sparse_pos": ((U, lam), torch.int32),
            "sparse_k": ((U, lam, d), self.tdtype), "sparse_v": ((U, lam, d), self.tdtype),
            "sparse_score": ((U, lam), torch.float32), "threshold": ((U, 2), torch.float32),
            "window_count": ((U,), torch.int32), "window_pos": ((U, eta), torch.int32),
            "window_k": ((U, eta, d), self.tdtype), "window_v": ((U, eta, d), self.tdtype),
            "n_seen": ((c.batch,), torch.int64), "status": ((1,), torch.int32),
        }
        if fields is not None:
            spec = {k: v for k, v in spec.items() if k in fields}
        return {k: torch.zeros(shape, dtype=dt) for k, (shape, dt) in spec.items()}

    def read_state(self, fields=None, check=True) -> Dict[str, np.ndarray]:
        """Host copy of the three memories as numpy arrays, shaped [B, Hkv, ...] (float32 for bf16 data)."""
        t = self._view_tensors(fields)
        view = lola_state_view(**{k: (v.data_ptr() if v.numel() else None) for k, v in t.items()})
        rc = lola_read_state(self.handle, view, self._stream())
        if rc != LOLA_OK and (check or rc != LOLA_ERR_DEVICE):
            raise LolaError(rc, "lola_read_state")
        c = self.cfg
        out = {}
        for k, v in t.items():
            a = v.float().numpy() if v.dtype == torch.bfloat16 else v.numpy()
            out[k] = a.reshape((c.batch, c.n_kv_heads) + a.shape[1:]) if k not in ("n_seen", "status") else a
        return out

    def write_state(self, st: Dict[str, np.ndarray]):
        """Imports a state given in the layout `read_state` returns (window rows in any order)."""
        c = self.cfg
        t = self._view_tensors()
        keep = {}
        for k, buf in t.items():
            if k == "status" or k not in st:
                continue
            a = np.asarray(st[k])
            if k.startswith("window_") and k != "window_count" or k in ("sparse_pos", "sparse_k", "sparse_v", "sparse_score"):
                slots = buf.shape[1]                      # pad or cut the slot axis to the state's capacity
                a = a.reshape((buf.shape[0], -1) + tuple(a.shape[3:]))
                if a.shape[1] > slots:
                    a = a[:, :slots]
                elif a.shape[1] < slots:
                    fill = -1 if k.endswith("_pos") else (np.nan if k == "sparse_score" else 0)
                    pad = np.full((a.shape[0], slots - a.shape[1]) + a.shape[2:], fill, dtype=a.dtype)
                    a = np.concatenate([a, pad], axis=1)
            a = torch.as_tensor(np.ascontiguousarray(a))
            if k in ("sparse_score", "threshold", "H", "s"):
                a = a.to(torch.float32)
            a = a.to(buf.dtype).reshape(buf.shape).contiguous()
            keep[k] = a
        view = lola_state_view(**{k: (v.data_ptr() if v.numel() else None) for k, v in keep.items()})
        _check(lola_write_state(self.handle, view, self._stream()), "lola_write_state")

    def reset(self):
        _check(lola_reset_state(self.handle, self._stream()), "lola_reset_state")

    def profile(self, enable: bool):
        _check(lola_profile_enable(self.handle, enable), "lola_profile_enable")

    def profile_read(self):
        return lola_profile_read(self.handle, self._stream())

    def last_call_info(self) -> dict:
        return lola_last_call_info(self.handle)

    @property
    def launches(self) -> int:
        return lola_launch_count(self.handle)

    @property
    def tokens_seen(self) -> int:
        return lola_tokens_seen(self.handle)

    def to_device(self, a: np.ndarray) -> torch.Tensor:
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(self.device, self.tdtype)
