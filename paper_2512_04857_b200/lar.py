"""Thin ctypes binding of the C ABI in include/lar.h (same names; argument marshalling only).

Every step of the hot path runs in the CUDA kernels of liblar.so.  There is no fallback: if the
library has not been built (python -m paper_2512_04857_b200.build) loading raises.
PyTorch is used by callers for device memory and streams; this module only needs raw addresses.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblar.so")

LAR_OK, LAR_ERR_INVALID_ARG, LAR_ERR_BAD_STATE, LAR_ERR_CAPACITY, LAR_ERR_CUDA, LAR_ERR_NOMEM, \
    LAR_ERR_DEVICE_CHECK = range(7)
LAR_BF16, LAR_FP32 = 0, 1
LAR_FLAG_NO_HOST_CHECKS, LAR_FLAG_PDL, LAR_FLAG_SHUFFLE_PAGES, LAR_FLAG_TILE_RANGES = 0x1, 0x2, 0x4, 0x8
LAR_FLAG_SCORE_CACHE_NORM = 0x10
LAR_FLAG_HOST_DEFER_OUT = 0x20
LAR_FLAG_SCORE_ACCUM = 0x40
LAR_FLAG_SLOT_REUSE = 0x80
LAR_FLAG_TEST_STALL = 0x100


class lar_config_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_layers", C.c_int32), ("batch", C.c_int32),
                ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("dtype", C.c_int32), ("cond_len", C.c_int32), ("line_width", C.c_int32),
                ("n_lines", C.c_int32), ("anchor_len", C.c_int32), ("recent_lines", C.c_int32),
                ("budget_lines", C.c_int32), ("softmax_scale", C.c_float), ("page_tokens", C.c_int32),
                ("flags", C.c_uint32), ("kv_splits", C.c_int32), ("warps_per_cta", C.c_int32),
                ("stages", C.c_int32), ("page_seed", C.c_uint32), ("decode_ctas", C.c_int32)]


class lar_plan_t(C.Structure):
    _fields_ = [("capacity", C.c_int32), ("pages_per_unit", C.c_int32), ("page_tokens", C.c_int32),
                ("mid_len", C.c_int32), ("kv_splits", C.c_int32), ("warps_per_cta", C.c_int32),
                ("stages", C.c_int32), ("decode_smem_bytes", C.c_int32), ("line_end_smem_bytes", C.c_int32),
                ("compressing", C.c_int32), ("slab_bytes", C.c_uint64), ("decode_ctas", C.c_int32),
                ("max_segments", C.c_int32), ("scratch_bytes", C.c_uint64)]


class LarError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = lib().lar_status_str(status).decode()
        extra = f" (cudaError {lib().lar_last_cuda_error()})" if status == LAR_ERR_CUDA else ""
        super().__init__(f"{what}: {msg}{extra}")


_LIB = None


def lib():
    """Load liblar.so (once).  Raises if the CUDA library has not been built."""
    global _LIB
    if _LIB is not None:
        return _LIB
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2512_04857_b200.build` "
                           "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, ip, cfgp, planp = C.c_void_p, C.c_int, C.POINTER(lar_config_t), C.POINTER(lar_plan_t)
    sigs = {
        "lar_plan_query": (C.c_int, [cfgp, planp]),
        "lar_cache_slab_bytes": (C.c_size_t, [cfgp]),
        "lar_cache_create": (C.c_int, [cfgp, vp, C.c_size_t, C.POINTER(vp)]),
        "lar_cache_reset": (C.c_int, [vp, vp]),
        "lar_append_kv": (C.c_int, [vp, ip, vp, vp, ip, vp]),
        "lar_decode_attn": (C.c_int, [vp, ip, vp, vp, vp]),
        "lar_decode_step": (C.c_int, [vp, ip, vp, vp, vp, vp, vp]),
        "lar_decode_step_strided": (C.c_int, [vp, ip, vp, vp, vp, vp, C.c_int64, C.c_int64, C.c_int64, C.c_int64, vp]),
        "lar_decode_step_rope": (C.c_int, [vp, ip, vp, vp, vp, vp, C.c_int64, C.c_int64, C.c_int64, C.c_int64, vp, ip, vp]),
        "lar_decode_step_host": (C.c_int, [vp, ip, vp, vp, vp, vp, vp]),
        "lar_cache_host_join": (C.c_int, [vp, vp]),
        "lar_line_end_score_evict": (C.c_int, [vp, ip, vp]),
        "lar_line_end_score_evict_all": (C.c_int, [vp, vp]),
        "lar_cache_destroy": (C.c_int, [vp]),
        "lar_cache_get_state": (C.c_int, [vp, ip, vp, vp, vp, vp]),
        "lar_cache_poll_device_status": (C.c_int, [vp, C.POINTER(C.c_uint32), vp]),
        "lar_cache_set_host_checks": (C.c_int, [vp, ip]),
        "lar_cache_launch_count": (C.c_uint64, [vp]),
        "lar_cache_get_plan": (C.c_int, [vp, planp]),
        "lar_attend_dense_noalloc": (C.c_int, [vp, vp, vp, vp, ip, ip, ip, ip, C.c_float, vp]),
        "lar_status_str": (C.c_char_p, [C.c_int]),
        "lar_last_cuda_error": (C.c_int, []),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(L, name)
        fn.restype, fn.argtypes = res, args
    _LIB = L
    return L


def make_config(*, n_layers, batch, n_q_heads, n_kv_heads, head_dim, dtype, cond_len, line_width, n_lines,
                anchor_len, recent_lines, budget_lines, softmax_scale=0.0, page_tokens=0, flags=0,
                kv_splits=0, warps_per_cta=0, stages=0, page_seed=0, decode_ctas=0) -> lar_config_t:
    dt = {"bf16": LAR_BF16, "fp32": LAR_FP32}.get(dtype, dtype)
    return lar_config_t(C.sizeof(lar_config_t), n_layers, batch, n_q_heads, n_kv_heads, head_dim, dt,
                        cond_len, line_width, n_lines, anchor_len, recent_lines, budget_lines,
                        float(softmax_scale), page_tokens, flags, kv_splits, warps_per_cta, stages, page_seed,
                        decode_ctas)


def config_from_workload(w, **overrides) -> lar_config_t:
    kw = dict(n_layers=w.n_layers, batch=w.batch, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
              head_dim=w.head_dim, dtype=w.dtype, cond_len=w.cond_len, line_width=w.line_width,
              n_lines=w.n_lines, anchor_len=w.anchor_len, recent_lines=w.recent_lines,
              budget_lines=w.budget_lines)
    kw.update(overrides)
    if getattr(w, "score_norm", "mid") == "cache":
        kw["flags"] = kw.get("flags", 0) | LAR_FLAG_SCORE_CACHE_NORM
    if getattr(w, "score_norm", "mid") == "accum":
        kw["flags"] = kw.get("flags", 0) | LAR_FLAG_SCORE_ACCUM
    return make_config(**kw)


def _chk(status: int, what: str):
    if status != LAR_OK:
        raise LarError(status, what)


def _ptr(x) -> Optional[int]:
    """Raw address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(type(x))


# ---- the C entry points, same names --------------------------------------------------------------
def lar_plan_query(cfg: lar_config_t) -> lar_plan_t:
    plan = lar_plan_t()
    _chk(lib().lar_plan_query(C.byref(cfg), C.byref(plan)), "lar_plan_query")
    return plan


def lar_cache_slab_bytes(cfg: lar_config_t) -> int:
    return int(lib().lar_cache_slab_bytes(C.byref(cfg)))


def lar_cache_create(cfg: lar_config_t, dev_slab, slab_bytes: int) -> int:
    out = C.c_void_p()
    _chk(lib().lar_cache_create(C.byref(cfg), _ptr(dev_slab), slab_bytes, C.byref(out)), "lar_cache_create")
    return out.value


def lar_cache_reset(cache, stream=None):
    _chk(lib().lar_cache_reset(cache, stream), "lar_cache_reset")


def lar_append_kv(cache, layer, k, v, n_tokens, stream=None):
    _chk(lib().lar_append_kv(cache, layer, _ptr(k), _ptr(v), n_tokens, stream), "lar_append_kv")


def lar_decode_attn(cache, layer, q, out, stream=None):
    _chk(lib().lar_decode_attn(cache, layer, _ptr(q), _ptr(out), stream), "lar_decode_attn")


def lar_decode_step(cache, layer, q, k, v, out, stream=None):
    _chk(lib().lar_decode_step(cache, layer, _ptr(q), _ptr(k), _ptr(v), _ptr(out), stream), "lar_decode_step")


def lar_decode_step_strided(cache, layer, q, k, v, out, q_seq_stride, k_seq_stride, v_seq_stride, out_seq_stride,
                            stream=None):
    _chk(lib().lar_decode_step_strided(cache, layer, _ptr(q), _ptr(k), _ptr(v), _ptr(out), q_seq_stride, k_seq_stride,
                                       v_seq_stride, out_seq_stride, stream), "lar_decode_step_strided")


def lar_decode_step_rope(cache, layer, q, k, v, out, q_seq_stride, k_seq_stride, v_seq_stride, out_seq_stride, cos_sin,
                         interleaved, stream=None):
    _chk(lib().lar_decode_step_rope(cache, layer, _ptr(q), _ptr(k), _ptr(v), _ptr(out), q_seq_stride, k_seq_stride,
                                    v_seq_stride, out_seq_stride, _ptr(cos_sin), int(interleaved), stream),
         "lar_decode_step_rope")


def lar_decode_step_host(cache, layer, q, k, v, out, stream=None):
    _chk(lib().lar_decode_step_host(cache, layer, _ptr(q), _ptr(k), _ptr(v), _ptr(out), stream),
         "lar_decode_step_host")


def lar_cache_host_join(cache, stream=None):
    _chk(lib().lar_cache_host_join(cache, stream), "lar_cache_host_join")


def lar_line_end_score_evict(cache, layer, stream=None):
    _chk(lib().lar_line_end_score_evict(cache, layer, stream), "lar_line_end_score_evict")


def lar_line_end_score_evict_all(cache, stream=None):
    _chk(lib().lar_line_end_score_evict_all(cache, stream), "lar_line_end_score_evict_all")


def lar_cache_destroy(cache):
    _chk(lib().lar_cache_destroy(cache), "lar_cache_destroy")


def lar_cache_get_state(cache, layer, lens=None, index_map=None, scores=None, stream=None):
    _chk(lib().lar_cache_get_state(cache, layer, _ptr(lens), _ptr(index_map), _ptr(scores), stream),
         "lar_cache_get_state")


def lar_cache_poll_device_status(cache, stream=None) -> int:
    """Returns the device status bits (0 = clean); does not raise on a recorded check."""
    bits = C.c_uint32(0)
    st = lib().lar_cache_poll_device_status(cache, C.byref(bits), stream)
    if st not in (LAR_OK, LAR_ERR_DEVICE_CHECK):
        raise LarError(st, "lar_cache_poll_device_status")
    return int(bits.value)


def lar_cache_set_host_checks(cache, enabled: bool):
    _chk(lib().lar_cache_set_host_checks(cache, int(bool(enabled))), "lar_cache_set_host_checks")


def lar_cache_launch_count(cache) -> int:
    return int(lib().lar_cache_launch_count(cache))


def lar_cache_get_plan(cache) -> lar_plan_t:
    plan = lar_plan_t()
    _chk(lib().lar_cache_get_plan(cache, C.byref(plan)), "lar_cache_get_plan")
    return plan


def lar_attend_dense_noalloc(q, k, v, out, n_units, group, head_dim, length, softmax_scale=0.0, stream=None):
    """Decode attention over dense bf16 K/V; the split-KV scratch is a static device array of the library."""
    _chk(lib().lar_attend_dense_noalloc(_ptr(q), _ptr(k), _ptr(v), _ptr(out), n_units, group, head_dim, length,
                                        float(softmax_scale), stream), "lar_attend_dense_noalloc")


class Cache:
    """Owns the device slab (a torch uint8 tensor) and the C handle; methods mirror the C calls."""

    def __init__(self, cfg: lar_config_t, device="cuda:0"):
        import numpy as np
        import torch
        self._np, self._torch = np, torch
        self.cfg = cfg
        self.device = torch.device(device)
        nbytes = lar_cache_slab_bytes(cfg)
        if nbytes == 0:
            raise LarError(LAR_ERR_INVALID_ARG, "lar_cache_slab_bytes")
        with torch.cuda.device(self.device):
            self.slab = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.slab.data_ptr()
            self._slab_ptr = (base + 255) // 256 * 256
            torch.cuda.synchronize(self.device)
            self.handle = lar_cache_create(cfg, self._slab_ptr, nbytes)
        self.plan = lar_cache_get_plan(self.handle)
        self.units = cfg.batch * cfg.n_kv_heads

    def _stream(self):
        return self._torch.cuda.current_stream(self.device).cuda_stream

    def close(self):
        if getattr(self, "handle", None):
            lar_cache_destroy(self.handle)
            self.handle = None
            self.slab = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        lar_cache_reset(self.handle, self._stream())

    def append_kv(self, layer, k, v, n_tokens):
        lar_append_kv(self.handle, layer, k, v, n_tokens, self._stream())

    def decode_attn(self, layer, q, out):
        lar_decode_attn(self.handle, layer, q, out, self._stream())

    def decode_step(self, layer, q, k, v, out):
        lar_decode_step(self.handle, layer, q, k, v, out, self._stream())

    def decode_step_strided(self, layer, q, k, v, out, q_seq_stride, k_seq_stride, v_seq_stride, out_seq_stride):
        lar_decode_step_strided(self.handle, layer, q, k, v, out, q_seq_stride, k_seq_stride, v_seq_stride,
                                out_seq_stride, self._stream())

    def decode_step_rope(self, layer, q, k, v, out, q_seq_stride, k_seq_stride, v_seq_stride, out_seq_stride, cos_sin,
                         interleaved=False):
        lar_decode_step_rope(self.handle, layer, q, k, v, out, q_seq_stride, k_seq_stride, v_seq_stride, out_seq_stride,
                             cos_sin, interleaved, self._stream())

    def decode_step_host(self, layer, q, k, v, out):
        lar_decode_step_host(self.handle, layer, q, k, v, out, self._stream())

    def host_join(self):
        lar_cache_host_join(self.handle, self._stream())

    def line_end_score_evict(self, layer):
        lar_line_end_score_evict(self.handle, layer, self._stream())

    def line_end_score_evict_all(self):
        lar_line_end_score_evict_all(self.handle, self._stream())

    def set_host_checks(self, enabled):
        lar_cache_set_host_checks(self.handle, enabled)

    def poll_device_status(self) -> int:
        return lar_cache_poll_device_status(self.handle, self._stream())

    def launch_count(self) -> int:
        return lar_cache_launch_count(self.handle)

    def get_state(self, layer, want_scores=False):
        np = self._np
        lens = np.zeros(self.units, dtype=np.int32)
        imap = np.zeros((self.units, self.plan.capacity), dtype=np.int32)
        scores = np.zeros((self.units, max(self.plan.mid_len, 1)), dtype=np.float32) if want_scores else None
        lar_cache_get_state(self.handle, layer, lens, imap, scores, self._stream())
        return (lens, imap, scores) if want_scores else (lens, imap)
