"""CPU-only checks of the C ABI: the library loads, exports every declared symbol, and the host-side
logic (config validation, derived plan, slab sizing, argument checks) behaves as documented."""
import ctypes as C
import os
import re

import pytest

from paper_2512_04857_b200 import lar, workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(lar_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_loads_and_exports_every_declared_symbol():
    L = lar.lib()
    names = _declared_symbols()
    assert {"lar_cache_create", "lar_append_kv", "lar_decode_attn", "lar_line_end_score_evict",
            "lar_cache_destroy"} <= names
    for n in sorted(names):
        assert hasattr(L, n), f"liblar.so does not export {n}"


def test_status_strings():
    L = lar.lib()
    assert L.lar_status_str(0) == b"ok"
    assert len({L.lar_status_str(i) for i in range(7)}) == 7


@pytest.mark.parametrize("name", list(W.WORKLOADS))
def test_plan_of_each_workload(name):
    w = W.WORKLOADS[name]
    p = lar.lar_plan_query(lar.config_from_workload(w))
    assert p.capacity == w.cond_len + w.budget_tokens
    assert p.mid_len == w.mid_len and p.compressing == 1
    assert p.pages_per_unit * p.page_tokens >= p.capacity
    assert p.kv_splits in (1, 2, 4, 8) and 1 <= p.warps_per_cta <= 8 and 1 <= p.stages <= 32
    assert p.decode_ctas >= 1 and 1 <= p.max_segments <= p.decode_ctas and p.scratch_bytes < p.slab_bytes
    if w.dtype == "bf16":
        assert p.stages % p.warps_per_cta == 0 and p.stages >= 2 * p.warps_per_cta
        assert p.decode_ctas <= 444 and (w.n_units >= 148 or p.decode_ctas % w.n_units == 0)
    assert p.decode_smem_bytes <= 227 * 1024 and p.line_end_smem_bytes <= 227 * 1024
    kv = 2 * w.n_layers * w.n_units * p.pages_per_unit * p.page_tokens * w.head_dim * w.elt_bytes
    assert kv <= p.slab_bytes <= kv * 1.3 + (1 << 22)
    assert lar.lar_cache_slab_bytes(lar.config_from_workload(w)) == p.slab_bytes
    pf = lar.lar_plan_query(lar.config_from_workload(w.full_cache()))
    assert pf.compressing == 0 and pf.mid_len == 0 and pf.capacity == w.cond_len + w.n_visual


def _cfg(**kw):
    base = dict(n_layers=1, batch=1, n_q_heads=4, n_kv_heads=4, head_dim=64, dtype="bf16", cond_len=4,
                line_width=8, n_lines=8, anchor_len=8, recent_lines=1, budget_lines=4)
    base.update(kw)
    return lar.make_config(**base)


@pytest.mark.parametrize("bad", [
    dict(n_q_heads=6, n_kv_heads=4),          # Hq % Hkv != 0
    dict(n_q_heads=12, n_kv_heads=4),         # group 3
    dict(head_dim=96),
    dict(dtype=7),
    dict(recent_lines=0),
    dict(budget_lines=2),                     # B - N_init - r n = 0 < n
    dict(anchor_len=17, budget_lines=4),      # mid would be 7 < n
    dict(page_tokens=24),
    dict(kv_splits=3),
    dict(warps_per_cta=9),
    dict(stages=33),
    dict(stages=1),                           # bf16 ring needs two stages
    dict(dtype="fp32", stages=5),
    dict(dtype="fp32", warps_per_cta=9),
    dict(decode_ctas=-1),
    dict(decode_ctas=2000),
    dict(n_layers=0),
    dict(cond_len=-1),
    dict(softmax_scale=-1.0),
])
def test_invalid_configs_are_rejected(bad):
    cfg = _cfg(**bad)
    plan = lar.lar_plan_t()
    assert lar.lib().lar_plan_query(C.byref(cfg), C.byref(plan)) == lar.LAR_ERR_INVALID_ARG
    assert lar.lar_cache_slab_bytes(cfg) == 0


def test_struct_size_is_checked_and_null_arguments():
    L = lar.lib()
    cfg = _cfg()
    cfg.struct_size = 8
    assert L.lar_plan_query(C.byref(cfg), None) == lar.LAR_ERR_INVALID_ARG
    assert L.lar_plan_query(None, None) == lar.LAR_ERR_INVALID_ARG
    cfg = _cfg()
    assert L.lar_plan_query(C.byref(cfg), None) == lar.LAR_OK
    out = C.c_void_p()
    # no slab / misaligned slab / too small: rejected before any CUDA work
    assert L.lar_cache_create(C.byref(cfg), None, 1 << 30, C.byref(out)) == lar.LAR_ERR_INVALID_ARG
    assert L.lar_cache_create(C.byref(cfg), 4096 + 8, 1 << 30, C.byref(out)) == lar.LAR_ERR_INVALID_ARG
    assert L.lar_cache_create(C.byref(cfg), 4096, 16, C.byref(out)) == lar.LAR_ERR_NOMEM
    assert L.lar_cache_create(C.byref(cfg), 4096, 1 << 30, None) == lar.LAR_ERR_INVALID_ARG
    for fn, args in [(L.lar_cache_destroy, (None,)), (L.lar_cache_reset, (None, None)),
                     (L.lar_append_kv, (None, 0, None, None, 1, None)),
                     (L.lar_decode_attn, (None, 0, None, None, None)),
                     (L.lar_line_end_score_evict, (None, 0, None))]:
        assert fn(*args) == lar.LAR_ERR_INVALID_ARG
    assert L.lar_cache_launch_count(None) == 0


def test_a_mid_region_too_large_to_stage_with_the_guide_rows_still_gets_a_plan():
    """1024-px shape at a quarter of the tokens: 520 mid keys + 260 guide rows of 272 B exceed 227 KB; the plan then reads
    the guide rows from global memory (8 warps) instead of refusing the configuration."""
    w = W.WORKLOADS["gqa_1024"]
    quarter = w.scaled(budget_lines=16, recent_lines=7, anchor_len=w.line_width)
    assert quarter.mid_len == 520
    p = lar.lar_plan_query(lar.config_from_workload(quarter))
    assert 520 * 272 < p.line_end_smem_bytes <= 227 * 1024
    assert p.line_end_smem_bytes < lar.lar_plan_query(lar.config_from_workload(w.scaled(budget_lines=12, recent_lines=5))).line_end_smem_bytes


def test_full_cache_budget_and_overrides():
    p = lar.lar_plan_query(_cfg(budget_lines=8))
    assert p.compressing == 0 and p.capacity == 4 + 64
    p = lar.lar_plan_query(_cfg(budget_lines=100))
    assert p.compressing == 0 and p.capacity == 4 + 64
    p = lar.lar_plan_query(_cfg(dtype="fp32", kv_splits=4, warps_per_cta=8, stages=2, page_tokens=32))
    assert (p.kv_splits, p.warps_per_cta, p.stages, p.page_tokens) == (4, 8, 2, 32)
    p = lar.lar_plan_query(_cfg(warps_per_cta=3, stages=9, decode_ctas=40, page_tokens=64))
    assert (p.warps_per_cta, p.stages, p.decode_ctas, p.page_tokens) == (3, 6, 40, 64)   # ring depth: multiple of 3 consumers and 2 producers
    # 4 units of up to 2 tiles (36 slots, 32-row tiles) dealt to 40 CTAs: every tile may sit in a CTA of its own
    assert p.max_segments == 2


def test_cache_normalised_scoring_plan():
    """LAR_FLAG_SCORE_CACHE_NORM stages C + B keys per unit in the line-end kernel: the plan's shared-memory figure
    grows accordingly, every benchmark shape still fits, and a cache that cannot be staged is refused."""
    for name, w in W.WORKLOADS.items():
        base = lar.lar_plan_query(lar.config_from_workload(w))
        var = lar.lar_plan_query(lar.config_from_workload(w.scaled(score_norm="cache")))
        assert var.line_end_smem_bytes > base.line_end_smem_bytes, name
        assert var.line_end_smem_bytes <= 227 * 1024, name
        assert var.decode_smem_bytes == base.decode_smem_bytes and var.slab_bytes == base.slab_bytes
        extra_rows = (w.cond_len + w.budget_tokens + 7) // 8 * 8 + 8 - (w.mid_len + 7) // 8 * 8
        if w.dtype == "bf16":   # keys grow by extra_rows padded rows; the staged guide rows go away
            nq16 = (w.line_width * w.group + 15) // 16 * 16
            row = w.head_dim * 2 + 16
            # (a short line against a small mid region runs 2 or 4 warps in the written form, 8 in the variant: one row of
            # M column sums per warp)
            small = w.line_width * w.group <= 32 and w.mid_len <= 64
            warps_base = (2 if w.head_dim * 2 <= 128 else 4) if small else None
            colsums = (8 - warps_base) * w.mid_len * 4 if small else 0
            assert abs((var.line_end_smem_bytes - base.line_end_smem_bytes) - (extra_rows - nq16) * row - colsums) <= 16, name
    big = W.WORKLOADS["gqa_1024"].scaled(score_norm="cache", cond_len=512)     # 1032 keys of 272 B > 227 KB
    with pytest.raises(lar.LarError) as e:
        lar.lar_plan_query(lar.config_from_workload(big))
    assert e.value.status == lar.LAR_ERR_INVALID_ARG
    lar.lar_plan_query(lar.config_from_workload(big.scaled(score_norm="mid")))  # the written form still fits
