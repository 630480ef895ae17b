"""Synthetic workloads: shapes of the paper's models and the seeded input generator.

This module holds *no* arithmetic of the method (no attention, no scoring, no
selection).  It only describes problem shapes and draws the random Q/K/V values
that both the CUDA path and the CPU oracle consume, so that the two sides see
bit-identical inputs without sharing any code of the method itself.

Shapes follow the models evaluated in the paper's experimental set-up
(LlamaGen-XL, Janus-Pro-7B, Lumina-mGPT-768/1024: 576, 2352 and 4160 visual
tokens) and the batch sizes of its efficiency table; the values are synthetic
because the trained models, prompts and datasets are not available.

Generator
---------
Every value is a pure function of (seed, stream, layer, sequence, head, token,
dim): a 64-bit mixing hash of the flattened counter yields two 32-bit uniforms,
a Box-Muller transform turns them into one N(0,1) sample (fp64).  Keys and
queries of *visual* tokens additionally receive a 2-D sinusoidal positional
term of amplitude 1 (first half of the head dimension encodes the row, second
half the column), so that logits favour tokens of neighbouring rows/columns,
like the locally concentrated attention the paper observes.  Prefix keys can be
scaled (config "janus_pro_7b": x1.5) to make the prefix an attention sink.
Values are rounded once to the storage dtype (bf16 RNE, or fp32) and handed out
in that dtype; the oracle widens them exactly.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass
from typing import Dict, Tuple

import torch

# stream ids of the counter-based generator
_Q, _K, _V, _KC, _VC = 0, 1, 2, 3, 4


@dataclass(frozen=True)
class Workload:
    name: str
    n_layers: int            # L
    batch: int               # S: sequences after classifier-free-guidance doubling
    images: int              # images per batch (= batch / 2 with CFG)
    n_q_heads: int           # Hq
    n_kv_heads: int          # Hkv
    head_dim: int            # d
    dtype: str               # "bf16" | "fp32"
    cond_len: int            # C: conditional prefix, always kept, not counted in B
    line_width: int          # n: tokens per raster line (incl. a line-end token if any)
    n_lines: int             # h
    budget_lines: int        # B / n
    anchor_len: int          # N_init
    recent_lines: int        # r
    seed: int
    prefix_key_scale: float = 1.0
    note: str = ""
    score_norm: str = "mid"  # scoring at a line end: Eq. 9 over the "mid" keys (as written), over the whole live "cache"
                             # (variant), or "accum": attention accumulated over all decode steps (the paper's ablation)

    @property
    def n_visual(self) -> int:            # N
        return self.line_width * self.n_lines

    @property
    def group(self) -> int:               # G
        return self.n_q_heads // self.n_kv_heads

    @property
    def budget_tokens(self) -> int:       # B
        return self.budget_lines * self.line_width

    @property
    def is_full_cache(self) -> bool:
        return self.budget_lines >= self.n_lines

    @property
    def mid_len(self) -> int:             # M at a compressing line end
        return self.budget_tokens - self.anchor_len - self.recent_lines * self.line_width

    @property
    def n_units(self) -> int:             # independent (sequence, kv head) units per layer
        return self.batch * self.n_kv_heads

    @property
    def elt_bytes(self) -> int:
        return 2 if self.dtype == "bf16" else 4

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    def full_cache(self) -> "Workload":
        """Same inputs, cache never compressed (the 'Full' rows of the paper's tables)."""
        return dataclasses.replace(self, name=self.name + "_full", budget_lines=self.n_lines)

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)

    # ---- trajectory of the live length (closed form; used for byte accounting) ----
    def live_len_at_step(self, i: int) -> int:
        """Live cache length (prefix + visual) seen by the attention of visual token i (1-based)."""
        n, B = self.line_width, self.budget_tokens
        if self.is_full_cache or i <= B:
            return self.cond_len + i
        j = (i - 1) % n + 1               # j-th token of its line
        return self.cond_len + B - n + j

    def kv_bytes_per_generation(self) -> int:
        """Algorithmic bytes of live K and V read by decode attention over one whole image, all layers."""
        tot = sum(self.live_len_at_step(i) for i in range(1, self.n_visual + 1))
        return tot * self.head_dim * 2 * self.elt_bytes * self.n_units * self.n_layers


def _mk(**kw) -> Workload:
    return Workload(**kw)


WORKLOADS: Dict[str, Workload] = {
    # fp32 sanity case; post-compression occupancy = prefix + first-line anchor + 4 recent lines,
    # i.e. B - n = 16 + 64 => budget 6 lines (the paper's toy ratio 3/8), mid = one line.
    "tiny": _mk(name="tiny", n_layers=1, batch=1, images=1, n_q_heads=8, n_kv_heads=8, head_dim=64,
                dtype="fp32", cond_len=16, line_width=16, n_lines=16, budget_lines=6, anchor_len=16,
                recent_lines=4, seed=0),
    # same inputs, budget 8 lines: mid = 48 tokens, 32 survive -> selection is non-trivial
    "tiny_b": _mk(name="tiny_b", n_layers=1, batch=1, images=1, n_q_heads=8, n_kv_heads=8, head_dim=64,
                  dtype="fp32", cond_len=16, line_width=16, n_lines=16, budget_lines=8, anchor_len=16,
                  recent_lines=4, seed=0),
    "llamagen_xl": _mk(name="llamagen_xl", n_layers=36, batch=64, images=32, n_q_heads=20, n_kv_heads=20,
                       head_dim=64, dtype="bf16", cond_len=1, line_width=24, n_lines=24, budget_lines=4,
                       anchor_len=24, recent_lines=1, seed=2),
    "janus_pro_7b": _mk(name="janus_pro_7b", n_layers=30, batch=32, images=16, n_q_heads=32, n_kv_heads=32,
                        head_dim=128, dtype="bf16", cond_len=64, line_width=24, n_lines=24, budget_lines=4,
                        anchor_len=24, recent_lines=1, seed=3, prefix_key_scale=1.5),
    "lumina_768": _mk(name="lumina_768", n_layers=32, batch=8, images=4, n_q_heads=32, n_kv_heads=32,
                      head_dim=128, dtype="bf16", cond_len=128, line_width=49, n_lines=48, budget_lines=6,
                      anchor_len=49, recent_lines=2, seed=4, note="48 columns + 1 line-end token per row"),
    # further shapes of the paper's tables (same generator; not the headline): LlamaGen-XXL (class-conditional, Table 2)
    # and Janus-Pro-1B (Table 1, ablations)
    "llamagen_xxl": _mk(name="llamagen_xxl", n_layers=48, batch=64, images=32, n_q_heads=24, n_kv_heads=24,
                        head_dim=64, dtype="bf16", cond_len=1, line_width=24, n_lines=24, budget_lines=4,
                        anchor_len=24, recent_lines=1, seed=6),
    "janus_pro_1b": _mk(name="janus_pro_1b", n_layers=24, batch=32, images=16, n_q_heads=16, n_kv_heads=16,
                        head_dim=128, dtype="bf16", cond_len=64, line_width=24, n_lines=24, budget_lines=4,
                        anchor_len=24, recent_lines=1, seed=7, prefix_key_scale=1.5),
    "gqa_1024": _mk(name="gqa_1024", n_layers=32, batch=16, images=8, n_q_heads=32, n_kv_heads=8,
                    head_dim=128, dtype="bf16", cond_len=128, line_width=65, n_lines=64, budget_lines=8,
                    anchor_len=65, recent_lines=3, seed=5, note="64 columns + 1 line-end token per row"),
}


# --------------------------------------------------------------------------------------
# counter-based generator
# --------------------------------------------------------------------------------------
_M64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Python int -> the int64 two's-complement value with the same low 64 bits."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_C1 = _s64(0xBF58476D1CE4E5B9)
_C2 = _s64(0x94D049BB133111EB)
_GOLD = _s64(0x9E3779B97F4A7C15)


def _lsr(x: torch.Tensor, k: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor."""
    return (x >> k) & ((1 << (64 - k)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    """Bijective 64-bit finaliser (xor-shift-multiply rounds); int64 arithmetic wraps."""
    x = (x ^ _lsr(x, 30)) * _C1
    x = (x ^ _lsr(x, 27)) * _C2
    return x ^ _lsr(x, 31)


def _normal_from_counter(counter: torch.Tensor, seed: int) -> torch.Tensor:
    """N(0,1) fp64 sample per int64 counter value."""
    hsh = _mix64(counter * _GOLD + _s64(seed * 0xD6E8FEB86659FD93 + 0x2545F4914F6CDD1D))
    hsh = _mix64(hsh ^ _GOLD)
    hi = _lsr(hsh, 32).to(torch.float64)
    lo = (hsh & 0xFFFFFFFF).to(torch.float64)
    u1 = (hi + 0.5) * (1.0 / 4294967296.0)
    u2 = (lo + 0.5) * (1.0 / 4294967296.0)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def _positional(w: Workload, tok: torch.Tensor, device) -> torch.Tensor:
    """2-D sinusoidal term, amplitude 1: [T, d] fp64 for 0-based visual token indices `tok`."""
    d = w.head_dim
    half = d // 2
    row = (tok // w.line_width).to(torch.float64)[:, None]
    col = (tok % w.line_width).to(torch.float64)[:, None]
    dim = torch.arange(half, device=device)
    pair = (dim // 2).to(torch.float64)
    omega = torch.pow(torch.tensor(10000.0, dtype=torch.float64, device=device), -2.0 * pair / half)[None, :]
    is_sin = (dim % 2 == 0)[None, :]
    pe_row = torch.where(is_sin, torch.sin(row * omega), torch.cos(row * omega))
    pe_col = torch.where(is_sin, torch.sin(col * omega), torch.cos(col * omega))
    return torch.cat([pe_row, pe_col], dim=1)


def _field(w: Workload, stream: int, layer: int, seqs: torch.Tensor, heads: torch.Tensor,
           toks: torch.Tensor, n_heads_total: int, n_tok_total: int) -> torch.Tensor:
    """fp64 N(0,1) samples of shape [len(toks), len(seqs), len(heads), d] for the given indices."""
    dev = toks.device
    d = w.head_dim
    dims = torch.arange(d, device=dev, dtype=torch.int64)
    base = (stream * 4096 + layer)
    c = ((base * w.batch + seqs[None, :, None, None]) * n_heads_total + heads[None, None, :, None])
    c = (c * n_tok_total + toks[:, None, None, None]) * d + dims[None, None, None, :]
    return _normal_from_counter(c, w.seed)


def _round(w: Workload, x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.float32).to(w.torch_dtype) if w.dtype == "bf16" else x.to(torch.float32)


def gen_tokens(w: Workload, layer: int, t0: int, t1: int, device="cpu",
               seqs: torch.Tensor | None = None, q_heads: torch.Tensor | None = None,
               kv_heads: torch.Tensor | None = None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Per-step inputs of visual tokens t0..t1-1 (0-based) of one layer.

    Returns q [T, S, Hq, d], k [T, S, Hkv, d], v [T, S, Hkv, d] in the storage dtype
    (all sequences / heads unless index subsets are given).
    """
    dev = torch.device(device)
    toks = torch.arange(t0, t1, device=dev, dtype=torch.int64)
    seqs = torch.arange(w.batch, device=dev) if seqs is None else seqs.to(dev)
    qh = torch.arange(w.n_q_heads, device=dev) if q_heads is None else q_heads.to(dev)
    kh = torch.arange(w.n_kv_heads, device=dev) if kv_heads is None else kv_heads.to(dev)
    pe = _positional(w, toks, dev)[:, None, None, :]
    q = _field(w, _Q, layer, seqs, qh, toks, w.n_q_heads, w.n_visual) + pe
    k = _field(w, _K, layer, seqs, kh, toks, w.n_kv_heads, w.n_visual) + pe
    v = _field(w, _V, layer, seqs, kh, toks, w.n_kv_heads, w.n_visual)
    return _round(w, q), _round(w, k), _round(w, v)


def gen_prefix(w: Workload, layer: int, device="cpu", seqs: torch.Tensor | None = None,
               kv_heads: torch.Tensor | None = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Conditional-prefix K, V of one layer: [S, Hkv, C, d] in the storage dtype."""
    dev = torch.device(device)
    toks = torch.arange(w.cond_len, device=dev, dtype=torch.int64)
    seqs = torch.arange(w.batch, device=dev) if seqs is None else seqs.to(dev)
    kh = torch.arange(w.n_kv_heads, device=dev) if kv_heads is None else kv_heads.to(dev)
    n_tok_total = max(w.cond_len, 1)
    k = _field(w, _KC, layer, seqs, kh, toks, w.n_kv_heads, n_tok_total) * w.prefix_key_scale
    v = _field(w, _VC, layer, seqs, kh, toks, w.n_kv_heads, n_tok_total)
    # [C, S, Hkv, d] -> [S, Hkv, C, d]
    return (_round(w, k).permute(1, 2, 0, 3).contiguous(), _round(w, v).permute(1, 2, 0, 3).contiguous())


def gen_unit(w: Workload, layer: int, seq: int, kv_head: int, device="cpu"):
    """All inputs of ONE independent unit (layer, sequence, kv head), as fp32 CPU-friendly tensors.

    Returns dict with q [N, G, d], k [N, d], v [N, d], kc [C, d], vc [C, d] (float32, exact widening
    of the storage dtype).  The same values appear at the matching indices of gen_tokens/gen_prefix.
    """
    G = w.group
    s = torch.tensor([seq])
    kh = torch.tensor([kv_head])
    qh = torch.arange(kv_head * G, (kv_head + 1) * G)
    q, k, v = gen_tokens(w, layer, 0, w.n_visual, device, seqs=s, q_heads=qh, kv_heads=kh)
    kc, vc = gen_prefix(w, layer, device, seqs=s, kv_heads=kh)
    f = lambda x: x.to(torch.float32).cpu().contiguous()
    return {"q": f(q[:, 0]), "k": f(k[:, 0, 0]), "v": f(v[:, 0, 0]), "kc": f(kc[0, 0]), "vc": f(vc[0, 0])}
