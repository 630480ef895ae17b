"""Parity driver shared by the GPU tests, the smoke check and nothing else.

Runs a workload through the C ABI (CUDA kernels) line by line and, for a sample of independent
units (layer, sequence, KV head), drives the CPU oracle on the very same input values.  Compares
every decode output element by element and every line end's kept-token positions bit-exactly;
a kept-set difference is tolerated only as a *near-tie* (all positions in the symmetric difference
have an oracle score within 1e-5 relative of the oracle's eviction boundary); it is counted, and the
oracle is then re-synchronised by evicting the GPU's choice so later steps compare like with like.
"""
from __future__ import annotations

import os
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

from oracle import lar_oracle as O
from paper_2512_04857_b200 import lar
from paper_2512_04857_b200 import workloads as W

TOL = {"bf16": 2e-2, "fp32": 1e-4}       # max-abs tolerance of attention outputs
NEAR_TIE_REL = 1e-5
# per test file: what the parity runs of this session compared (printed at the end of a pytest run)
TOTALS: Dict[str, Dict[str, float]] = {}


def _account(rep: "ParityReport") -> None:
    where = os.environ.get("PYTEST_CURRENT_TEST", "outside pytest").split("::")[0]
    t = TOTALS.setdefault(where, {"runs": 0, "outputs": 0, "line_ends": 0, "compressions": 0, "near_ties": 0,
                                  "max_abs_err_bf16": 0.0, "max_abs_err_fp32": 0.0})
    t["runs"] += 1
    t["outputs"] += rep.outputs_compared
    t["line_ends"] += rep.line_ends_compared
    t["compressions"] += rep.compressions
    t["near_ties"] += rep.near_ties
    key = "max_abs_err_" + rep.dtype
    t[key] = max(t[key], rep.max_abs_err)


@dataclass
class ParityReport:
    max_abs_err: float = 0.0
    outputs_compared: int = 0
    line_ends_compared: int = 0
    compressions: int = 0
    near_ties: int = 0
    max_score_rel_err: float = 0.0
    mismatches: List[str] = field(default_factory=list)
    dtype: str = "bf16"

    def ok(self, tol: float) -> bool:
        return not self.mismatches and self.max_abs_err <= tol


def pick_units(w: W.Workload, n: int, seed: int = 0) -> List[Tuple[int, int, int]]:
    """A deterministic sample of (layer, sequence, kv head) triples incl. the first and last unit."""
    rng = np.random.default_rng(seed)
    picks = {(0, 0, 0), (w.n_layers - 1, w.batch - 1, w.n_kv_heads - 1)}
    while len(picks) < min(n, w.n_layers * w.batch * w.n_kv_heads):
        picks.add((int(rng.integers(w.n_layers)), int(rng.integers(w.batch)), int(rng.integers(w.n_kv_heads))))
    return sorted(picks)


def run_parity(w: W.Workload, *, units: Optional[Sequence[Tuple[int, int, int]]] = None, fused: bool = True,
               gen_device: str = "cpu", n_steps: Optional[int] = None, cfg_overrides: Optional[Dict] = None,
               check_scores: bool = True, device: str = "cuda:0", line_end_all: bool = False) -> ParityReport:
    dev = torch.device(device)
    cfg = lar.config_from_workload(w, **(cfg_overrides or {}))
    cache = lar.Cache(cfg, device=device)
    # without compaction the slots do not follow positions: the live SET is what Eq. 5-7 define
    reuse = bool(cfg.flags & lar.LAR_FLAG_SLOT_REUSE)
    rep = ParityReport(dtype=w.dtype)
    L, S, Hq, Hkv, d, G, n, C = (w.n_layers, w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.group,
                                 w.line_width, w.cond_len)
    N = w.n_visual if n_steps is None else n_steps
    if units is None:
        units = [(l, s, h) for l in range(L) for s in range(S) for h in range(Hkv)]
    ocfg = O.cfg_from_workload(w)
    orc = {u: O.Unit(ocfg) for u in units}
    layers_sampled = sorted({u[0] for u in units})
    tol = TOL[w.dtype]

    def to_dev(x):
        return x.to(dev) if x.device != dev else x

    # ---- prefill
    for layer in range(L):
        if C > 0:
            kc, vc = W.gen_prefix(w, layer, gen_device)
            kc, vc = to_dev(kc), to_dev(vc)
            cache.append_kv(layer, kc, vc, C)
            for (l, s, h) in units:
                if l == layer:
                    orc[(l, s, h)].prefill(kc[s, h].float().cpu().numpy(), vc[s, h].float().cpu().numpy())
        else:
            for (l, s, h) in units:
                if l == layer:
                    orc[(l, s, h)].prefill(np.zeros((0, d), np.float32), np.zeros((0, d), np.float32))
    torch.cuda.synchronize(dev)

    out_line = torch.empty((n, L, S, Hq, d), dtype=w.torch_dtype, device=dev)
    for t0 in range(0, N, n):
        t1 = min(t0 + n, N)
        ins = []
        for layer in range(L):
            q, k, v = W.gen_tokens(w, layer, t0, t1, gen_device)
            ins.append((to_dev(q), to_dev(k), to_dev(v)))
        for t in range(t1 - t0):
            for layer in range(L):
                q, k, v = ins[layer]
                if fused:
                    cache.decode_step(layer, q[t], k[t], v[t], out_line[t, layer])
                else:
                    cache.append_kv(layer, k[t], v[t], 1)
                    cache.decode_attn(layer, q[t], out_line[t, layer])
        torch.cuda.synchronize(dev)
        # ---- compare the line's outputs
        for (l, s, h) in units:
            q, k, v = ins[l]
            qs = q[:, s, h * G:(h + 1) * G].float().cpu().numpy()
            ks = k[:, s, h].float().cpu().numpy()
            vs = v[:, s, h].float().cpu().numpy()
            got = out_line[: t1 - t0, l, s, h * G:(h + 1) * G].float().cpu().numpy().astype(np.float64)
            u = orc[(l, s, h)]
            for t in range(t1 - t0):
                ref = u.step(qs[t], ks[t], vs[t])
                err = float(np.max(np.abs(got[t] - ref)))
                if not np.isfinite(got[t]).all():
                    err = float("inf")
                rep.max_abs_err = max(rep.max_abs_err, err)
                rep.outputs_compared += got[t].size
                if err > tol and len(rep.mismatches) < 10:
                    rep.mismatches.append(f"out layer {l} seq {s} head {h} token {t0 + t + 1}: max abs err {err:.3e}")
        # ---- line end
        if (t1 - t0) == n and t1 < w.n_visual:
            if line_end_all:
                cache.line_end_score_evict_all()           # one launch for every layer
            else:
                for layer in range(L):
                    cache.line_end_score_evict(layer)
            for layer in layers_sampled:
                lens, imap, gscores = cache.get_state(layer, want_scores=True)
                for (l, s, h) in units:
                    if l != layer:
                        continue
                    u = orc[(l, s, h)]
                    ui = s * Hkv + h
                    due = u.line_end_due()
                    assert due >= 0
                    rep.line_ends_compared += 1
                    if due == 0:
                        u.line_end()
                    else:
                        rep.compressions += 1
                        S_o, mid_pos = u.mid_scores()
                        ev_idx = O.bottomk(S_o, mid_pos, n)
                        ev_o = set(int(p) for p in mid_pos[ev_idx])
                        kept_gpu = set(int(p) for p in imap[ui, : lens[ui]])
                        ev_g = set(int(p) for p in mid_pos) - kept_gpu
                        if check_scores:
                            rel = np.max(np.abs(gscores[ui, : len(S_o)] - S_o) / np.maximum(np.abs(S_o), 1e-30))
                            rep.max_score_rel_err = max(rep.max_score_rel_err, float(rel))
                        if ev_g != ev_o:
                            order = sorted(range(len(S_o)), key=lambda m: (S_o[m], -mid_pos[m]))
                            b_hi_evicted, b_lo_kept = S_o[order[n - 1]], S_o[order[n]] if len(order) > n else S_o[order[n - 1]]
                            score_of = {int(p): S_o[i] for i, p in enumerate(mid_pos)}
                            sym = ev_g ^ ev_o
                            near = len(ev_g) == n and all(
                                min(abs(score_of[p] - b_hi_evicted), abs(score_of[p] - b_lo_kept))
                                <= NEAR_TIE_REL * max(abs(b_hi_evicted), abs(b_lo_kept)) for p in sym)
                            if near:
                                rep.near_ties += 1
                            elif len(rep.mismatches) < 10:
                                rep.mismatches.append(
                                    f"kept set layer {l} seq {s} head {h} line {t1 // n}: gpu-only evictions "
                                    f"{sorted(ev_g - ev_o)[:8]} oracle-only {sorted(ev_o - ev_g)[:8]}")
                            u.evict(sorted(ev_g) if len(ev_g) == n else sorted(ev_o))
                        else:
                            u.evict(sorted(ev_o))
                    pos_o = u.positions()
                    live = imap[ui, : lens[ui]]
                    same = (np.array_equal(np.sort(live), pos_o) and len(set(live.tolist())) == len(live)) if reuse \
                        else np.array_equal(live, pos_o)
                    if lens[ui] != len(pos_o) or not same:
                        if len(rep.mismatches) < 10:
                            rep.mismatches.append(f"index map layer {l} seq {s} head {h} line {t1 // n}: "
                                                  f"len gpu {lens[ui]} oracle {len(pos_o)}")
    bits = cache.poll_device_status()
    if bits:
        rep.mismatches.append(f"device status bits {bits:#x}")
    for u in orc.values():
        u.close()
    cache.close()
    _account(rep)
    return rep
