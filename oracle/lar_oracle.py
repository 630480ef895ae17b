"""ctypes access to the C oracle (oracle/lar_oracle.c).  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the benchmark's cpu-baseline leg may import this module.  It does
argument marshalling and nothing else: every number it returns is computed by the C file.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

from . import build as _build

_LIB = None


class Cfg(C.Structure):
    _fields_ = [("cond_len", C.c_int), ("line_width", C.c_int), ("n_lines", C.c_int),
                ("budget_lines", C.c_int), ("anchor_len", C.c_int), ("recent_lines", C.c_int),
                ("group", C.c_int), ("head_dim", C.c_int), ("scale", C.c_double), ("score_norm", C.c_int)]


def lib():
    global _LIB
    if _LIB is None:
        path = _build.build()
        L = C.CDLL(path)
        dp, fp, ip = C.POINTER(C.c_double), C.POINTER(C.c_float), C.POINTER(C.c_int)
        L.lar_oracle_attention.argtypes = [dp, dp, dp, C.c_int, C.c_int, C.c_double, dp, dp]
        L.lar_oracle_attention.restype = None
        L.lar_oracle_saliency.argtypes = [dp, C.c_int, dp, C.c_int, C.c_int, C.c_double, dp]
        L.lar_oracle_saliency.restype = None
        L.lar_oracle_saliency_cache.argtypes = [dp, C.c_int, C.c_int, dp, ip, C.c_int, C.c_int, C.c_double,
                                                C.c_int, ip, C.c_int, dp]
        L.lar_oracle_saliency_cache.restype = None
        L.lar_oracle_bottomk.argtypes = [dp, ip, C.c_int, C.c_int, ip]
        L.lar_oracle_bottomk.restype = None
        L.lar_oracle_unit_create.argtypes = [C.POINTER(Cfg)]
        L.lar_oracle_unit_create.restype = C.c_void_p
        L.lar_oracle_unit_destroy.argtypes = [C.c_void_p]
        L.lar_oracle_unit_destroy.restype = None
        for name in ("lar_oracle_unit_len", "lar_oracle_unit_n_visual", "lar_oracle_unit_line_end_due"):
            getattr(L, name).argtypes = [C.c_void_p]
            getattr(L, name).restype = C.c_int
        L.lar_oracle_unit_positions.argtypes = [C.c_void_p, ip]
        L.lar_oracle_unit_positions.restype = None
        L.lar_oracle_unit_accumulated.argtypes = [C.c_void_p, dp]
        L.lar_oracle_unit_accumulated.restype = None
        L.lar_oracle_unit_prefill.argtypes = [C.c_void_p, fp, fp]
        L.lar_oracle_unit_prefill.restype = C.c_int
        L.lar_oracle_unit_step.argtypes = [C.c_void_p, fp, fp, fp, dp, dp]
        L.lar_oracle_unit_step.restype = C.c_int
        L.lar_oracle_unit_mid_scores.argtypes = [C.c_void_p, dp, ip]
        L.lar_oracle_unit_mid_scores.restype = C.c_int
        L.lar_oracle_unit_evict.argtypes = [C.c_void_p, ip, C.c_int]
        L.lar_oracle_unit_evict.restype = C.c_int
        L.lar_oracle_unit_line_end.argtypes = [C.c_void_p, dp, ip, ip, dp]
        L.lar_oracle_unit_line_end.restype = C.c_int
        L.lar_oracle_run_units.argtypes = [C.POINTER(Cfg), C.c_int, fp, fp, fp, fp, fp, C.c_int, dp, ip,
                                           C.c_int, C.c_int]
        L.lar_oracle_run_units.restype = C.c_int
        _LIB = L
    return _LIB


def _d(a):
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _f(a):
    return a.ctypes.data_as(C.POINTER(C.c_float))


def _i(a):
    return a.ctypes.data_as(C.POINTER(C.c_int))


def _f32(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float32))


def _f64(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


# Eq. 9 as written / softmax over the whole live cache / attention accumulated over all history
SCORE_NORM = {"mid": 0, "cache": 1, "accum": 2}


def make_cfg(cond_len, line_width, n_lines, budget_lines, anchor_len, recent_lines, group, head_dim,
             scale=0.0, score_norm=0) -> Cfg:
    return Cfg(cond_len, line_width, n_lines, budget_lines, anchor_len, recent_lines, group, head_dim,
               float(scale), int(score_norm))


def cfg_from_workload(w) -> Cfg:
    return make_cfg(w.cond_len, w.line_width, w.n_lines, w.budget_lines, w.anchor_len, w.recent_lines,
                    w.group, w.head_dim, score_norm=SCORE_NORM[getattr(w, "score_norm", "mid")])


def attention(q, K, V, scale, want_probs=False):
    """Eq. 2 for one query row: returns out [d] (and probs [len])."""
    q, K, V = _f64(q), _f64(K), _f64(V)
    n, d = K.shape
    out = np.zeros(d)
    probs = np.zeros(n) if want_probs else None
    lib().lar_oracle_attention(_d(q), _d(K), _d(V), n, d, float(scale), _d(out),
                               _d(probs) if want_probs else None)
    return (out, probs) if want_probs else out


def saliency(Qg, Kmid, scale):
    """Eq. 9: mean over the guide queries of the softmax over the mid keys."""
    Qg, Kmid = _f64(Qg), _f64(Kmid)
    nq, d = Qg.shape
    M = Kmid.shape[0]
    S = np.zeros(M)
    lib().lar_oracle_saliency(_d(Qg), nq, _d(Kmid), M, d, float(scale), _d(S))
    return S


def saliency_cache(Qg, K, pos, first_qpos, mid_slot, scale):
    """Variant of Eq. 9: Qg [n][G][d]; every query normalised over the entries it attended to."""
    Qg, K = _f64(Qg), _f64(K)
    n, G, d = Qg.shape
    pos = np.ascontiguousarray(np.asarray(pos, dtype=np.int32))
    mid_slot = np.ascontiguousarray(np.asarray(mid_slot, dtype=np.int32))
    S = np.zeros(len(mid_slot))
    lib().lar_oracle_saliency_cache(_d(Qg), n, G, _d(K), _i(pos), K.shape[0], d, float(scale), int(first_qpos),
                                    _i(mid_slot), len(mid_slot), _d(S))
    return S


def bottomk(S, pos, k):
    """Eq. 10: indices of the k least salient entries, least salient first."""
    S = _f64(S)
    pos = np.ascontiguousarray(np.asarray(pos, dtype=np.int32))
    ev = np.zeros(k, dtype=np.int32)
    lib().lar_oracle_bottomk(_d(S), _i(pos), len(S), k, _i(ev))
    return ev


class Unit:
    """One independent (layer, sequence, KV head) unit of the oracle."""

    def __init__(self, cfg: Cfg):
        self.cfg = cfg
        self._h = lib().lar_oracle_unit_create(C.byref(cfg))
        if not self._h:
            raise ValueError("oracle rejected the configuration")

    def close(self):
        if self._h:
            lib().lar_oracle_unit_destroy(self._h)
            self._h = None

    def __del__(self):
        self.close()

    @property
    def len(self) -> int:
        return lib().lar_oracle_unit_len(self._h)

    @property
    def n_visual(self) -> int:
        return lib().lar_oracle_unit_n_visual(self._h)

    def positions(self) -> np.ndarray:
        p = np.zeros(max(self.len, 1), dtype=np.int32)
        lib().lar_oracle_unit_positions(self._h, _i(p))
        return p[: self.len]

    def accumulated(self) -> np.ndarray:
        """Attention mass each live entry has received since it was appended (cache order; sum over the G heads)."""
        a = np.zeros(max(self.len, 1))
        lib().lar_oracle_unit_accumulated(self._h, _d(a))
        return a[: self.len]

    def prefill(self, kc, vc):
        kc, vc = _f32(kc), _f32(vc)
        assert kc.shape == (self.cfg.cond_len, self.cfg.head_dim) and vc.shape == kc.shape
        rc = lib().lar_oracle_unit_prefill(self._h, _f(kc), _f(vc))
        if rc:
            raise RuntimeError(f"prefill rc={rc}")

    def step(self, q, k, v, want_probs=False):
        q, k, v = _f32(q), _f32(k), _f32(v)
        G, d = self.cfg.group, self.cfg.head_dim
        assert q.shape == (G, d) and k.shape == (d,) and v.shape == (d,)
        out = np.zeros((G, d))
        probs = np.zeros((G, self.len + 1)) if want_probs else None
        rc = lib().lar_oracle_unit_step(self._h, _f(q), _f(k), _f(v), _d(out),
                                        _d(probs) if want_probs else None)
        if rc:
            raise RuntimeError(f"step rc={rc}")
        return (out, probs) if want_probs else out

    def line_end_due(self) -> int:
        return lib().lar_oracle_unit_line_end_due(self._h)

    def mid_scores(self):
        S = np.zeros(self.len)
        mp = np.zeros(self.len, dtype=np.int32)
        M = lib().lar_oracle_unit_mid_scores(self._h, _d(S), _i(mp))
        if M < 0:
            raise RuntimeError("no compression due")
        return S[:M].copy(), mp[:M].copy()

    def evict(self, positions):
        p = np.ascontiguousarray(np.asarray(positions, dtype=np.int32))
        rc = lib().lar_oracle_unit_evict(self._h, _i(p), len(p))
        if rc:
            raise RuntimeError(f"evict rc={rc}")

    def line_end(self):
        """Returns None for a no-op line end, else dict(scores, mid_pos, evicted_pos, boundary)."""
        n = self.cfg.line_width
        S = np.zeros(self.len)
        mp = np.zeros(self.len, dtype=np.int32)
        ev = np.zeros(n, dtype=np.int32)
        bd = np.zeros(2)
        len_before = self.len
        rc = lib().lar_oracle_unit_line_end(self._h, _d(S), _i(mp), _i(ev), _d(bd))
        if rc < 0:
            raise RuntimeError(f"line_end rc={rc}")
        if rc == 0:
            return None
        M = self.cfg.budget_lines * n - self.cfg.anchor_len - self.cfg.recent_lines * n
        assert self.len == len_before - n
        return {"scores": S[:M].copy(), "mid_pos": mp[:M].copy(), "evicted_pos": ev, "boundary": bd}


def run_units(cfg: Cfg, q, k, v, kc, vc, n_steps: Optional[int] = None, want_out=True, want_kept=True,
              n_threads: int = 0):
    """Whole generations of U independent units (OpenMP over units).

    q [U,N,G,d], k,v [U,N,d], kc,vc [U,C,d] float32.  Returns (out [U,n_steps,G,d] float64 | None,
    kept [U,n_line_ends,stride] int32 | None, threads_used).
    """
    q, k, v, kc, vc = _f32(q), _f32(k), _f32(v), _f32(kc), _f32(vc)
    U, N, G, d = q.shape
    n = cfg.line_width
    assert N == n * cfg.n_lines and G == cfg.group and d == cfg.head_dim
    n_steps = N if n_steps is None else n_steps
    out = np.zeros((U, n_steps, G, d)) if want_out else None
    stride = cfg.cond_len + min(cfg.budget_lines, cfg.n_lines) * n
    n_le = n_steps // n
    kept = np.full((U, max(n_le, 1), stride), -1, dtype=np.int32) if want_kept else None
    rc = lib().lar_oracle_run_units(C.byref(cfg), U, _f(q), _f(k), _f(v), _f(kc), _f(vc), n_steps,
                                    _d(out) if want_out else None, _i(kept) if want_kept else None,
                                    stride, n_threads)
    if rc < 0:
        raise RuntimeError(f"run_units rc={rc}")
    return out, kept, rc
