"""GPU parity: CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.

Bars: attention outputs max-abs 1e-4 (fp32) / 2e-2 (bf16); kept-token positions bit-exact, except
near-ties within 1e-5 relative of the eviction boundary, which are counted."""
import numpy as np
import pytest
import torch

from paper_2512_04857_b200 import lar, workloads as W
from _harness import TOL, pick_units, run_parity

pytestmark = pytest.mark.gpu


def _check(rep, w, allow_near_ties=0):
    assert not rep.mismatches, rep.mismatches
    assert rep.max_abs_err <= TOL[w.dtype], rep.max_abs_err
    assert rep.near_ties <= allow_near_ties, rep.near_ties
    assert rep.outputs_compared > 0


# ------------------------------------------------------------------ the tiny fp32 configs, every unit
@pytest.mark.parametrize("name", ["tiny", "tiny_b"])
@pytest.mark.parametrize("fused", [True, False])
def test_tiny_configs_all_units(name, fused):
    w = W.WORKLOADS[name]
    rep = run_parity(w, fused=fused)
    _check(rep, w)
    assert rep.compressions == 8 * (w.n_lines - w.budget_lines)
    assert rep.max_score_rel_err < 1e-4


def test_tiny_full_cache_path():
    w = W.WORKLOADS["tiny"].full_cache()
    rep = run_parity(w)
    _check(rep, w)
    assert rep.compressions == 0


@pytest.mark.parametrize("splits,warps,stages", [(1, 1, 1), (1, 8, 3), (2, 2, 2), (4, 1, 4), (8, 4, 1), (8, 8, 2)])
def test_launch_shapes(splits, warps, stages):
    w = W.WORKLOADS["tiny_b"]
    rep = run_parity(w, cfg_overrides=dict(kv_splits=splits, warps_per_cta=warps, stages=stages))
    _check(rep, w)


@pytest.mark.parametrize("ctas,warps,stages", [(1, 1, 2), (3, 2, 3), (7, 4, 5), (40, 3, 12), (148, 4, 0), (296, 1, 16), (148, 5, 10), (74, 6, 12),
                                               (1024, 4, 2)])
@pytest.mark.parametrize("fused", [True, False])
def test_stream_launch_shapes_bf16(ctas, warps, stages, fused):
    """bf16 streaming decode kernel: any grid size / ring depth / consumer count gives the same result,
    including grids that cut every unit into many segments (scratch partials + ticket merge) and grids
    with more CTAs than tiles."""
    w = W.WORKLOADS["tiny_b"].scaled(dtype="bf16", n_q_heads=4, n_kv_heads=2, n_layers=2, cond_len=37)
    rep = run_parity(w, fused=fused, cfg_overrides=dict(decode_ctas=ctas, warps_per_cta=warps, stages=stages,
                                                        flags=lar.LAR_FLAG_PDL))
    _check(rep, w, allow_near_ties=1)


@pytest.mark.parametrize("page_tokens", [16, 32, 64])
def test_shuffled_pages(page_tokens):
    w = W.WORKLOADS["tiny_b"]
    rep = run_parity(w, cfg_overrides=dict(page_tokens=page_tokens, flags=lar.LAR_FLAG_SHUFFLE_PAGES, page_seed=7))
    _check(rep, w)


def test_pdl_flag_multi_layer():
    w = W.WORKLOADS["tiny_b"].scaled(n_layers=3)
    rep = run_parity(w, cfg_overrides=dict(flags=lar.LAR_FLAG_PDL))
    _check(rep, w)


# ------------------------------------------------------------------ scaled-down shapes of the paper's models
SMALL = {
    "llamagen": W.WORKLOADS["llamagen_xl"].scaled(n_layers=2, batch=2, n_q_heads=4, n_kv_heads=4),
    "janus": W.WORKLOADS["janus_pro_7b"].scaled(n_layers=2, batch=2, n_q_heads=4, n_kv_heads=4),
    "lumina": W.WORKLOADS["lumina_768"].scaled(n_layers=1, batch=1, n_q_heads=4, n_kv_heads=4, n_lines=16),
    "gqa": W.WORKLOADS["gqa_1024"].scaled(n_layers=1, batch=2, n_q_heads=8, n_kv_heads=2, n_lines=14),
}


@pytest.mark.parametrize("name", list(SMALL))
def test_small_bf16_shapes_all_units(name):
    w = SMALL[name]
    rep = run_parity(w)
    _check(rep, w, allow_near_ties=2)
    assert rep.compressions > 0


@pytest.mark.parametrize("name", ["janus", "gqa"])
def test_line_end_of_all_layers_in_one_launch(name):
    w = SMALL[name].scaled(n_layers=3)
    rep = run_parity(w, line_end_all=True, cfg_overrides=dict(flags=lar.LAR_FLAG_PDL))
    _check(rep, w, allow_near_ties=2)
    assert rep.compressions > 0


def test_line_end_of_all_layers_fp32_and_protocol():
    w = W.WORKLOADS["tiny_b"].scaled(n_layers=2)
    rep = run_parity(w, line_end_all=True)
    _check(rep, w)
    # every layer must have finished the line
    cfg = lar.config_from_workload(w)
    c = lar.Cache(cfg)
    with pytest.raises(lar.LarError) as e:
        c.line_end_score_evict_all()
    assert e.value.status == lar.LAR_ERR_BAD_STATE
    c.close()


# ------------------------------------------------------------------ edge cases
@pytest.mark.parametrize("kw", [
    dict(cond_len=0),                                        # no prefix
    dict(anchor_len=0),                                      # no anchor
    dict(anchor_len=5, recent_lines=2, budget_lines=5),      # anchor not a whole line
    dict(n_q_heads=8, n_kv_heads=4),                         # G = 2
    dict(n_q_heads=8, n_kv_heads=1),                         # G = 8
    dict(head_dim=128),                                      # fp32, 512-byte rows
    dict(line_width=7, n_lines=9, anchor_len=7, recent_lines=1, budget_lines=3, cond_len=3),  # odd sizes
    dict(line_width=1, n_lines=40, anchor_len=1, recent_lines=2, budget_lines=6),             # 1-token lines
    dict(dtype="bf16", head_dim=64, n_q_heads=4, n_kv_heads=2),
    dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=1),                               # bf16, G = 8
    dict(dtype="bf16", head_dim=64, n_q_heads=8, n_kv_heads=1, flags=0x8),                     # G = 8, tile ranges
])
def test_edge_shapes(kw):
    kw = dict(kw)
    flags = kw.pop("flags", 0)
    w = W.WORKLOADS["tiny_b"].scaled(**kw)
    rep = run_parity(w, cfg_overrides=dict(flags=flags, decode_ctas=5 if flags else 0))
    _check(rep, w, allow_near_ties=1)


def test_partial_generation_stops_mid_line():
    w = W.WORKLOADS["tiny_b"]
    rep = run_parity(w, n_steps=w.line_width * 9 + 5)
    _check(rep, w)


# ------------------------------------------------------------------ full-size shapes, sampled units
FULL = [("llamagen_xl", 2, 6), ("janus_pro_7b", 2, 6), ("lumina_768", 1, 4), ("gqa_1024", 1, 4)]


@pytest.mark.parametrize("name,layers,n_units", FULL)
def test_full_size_shapes_sampled_units(name, layers, n_units):
    """Full batch / heads / grid / budget of the benchmark shapes in the launch configuration the
    benchmark times (fused step, default plan, PDL); fewer layers (layers are independent and
    identically shaped), oracle on a sample of units."""
    w = W.WORKLOADS[name].scaled(n_layers=layers)
    rep = run_parity(w, units=pick_units(w, n_units, seed=1), gen_device="cuda",
                     cfg_overrides=dict(flags=lar.LAR_FLAG_PDL))
    _check(rep, w, allow_near_ties=2)
    assert rep.compressions == n_units * (w.n_lines - w.budget_lines)


def _with_budget(w, lines):
    """The benchmark's budget sweep: N_init = n, r = (budget_lines - 2) / 2 (at least 1)."""
    return w.scaled(budget_lines=lines, recent_lines=max(1, (lines - 2) // 2), anchor_len=w.line_width)


# every configuration a benchmark number is quoted on: the efficiency table's batch sizes (256 / 64 / 12 images) and
# budget ratios (1/4, 1/6, 1/8), the batch-sweep end points of the 1024-px shape, and the two added model shapes
QUOTED = {
    "janus_pro_7b at 64 images": lambda: W.WORKLOADS["janus_pro_7b"].scaled(batch=128, images=64),
    "gqa_1024 at 64 images": lambda: W.WORKLOADS["gqa_1024"].scaled(batch=128, images=64),
    "gqa_1024 at 1 image": lambda: W.WORKLOADS["gqa_1024"].scaled(batch=2, images=1),
    "llamagen_xl at 256 images": lambda: W.WORKLOADS["llamagen_xl"].scaled(batch=512, images=256),
    "lumina_768 at 12 images": lambda: W.WORKLOADS["lumina_768"].scaled(batch=24, images=12),
    "llamagen_xxl": lambda: W.WORKLOADS["llamagen_xxl"],
    "janus_pro_1b": lambda: W.WORKLOADS["janus_pro_1b"],
    "janus_pro_7b budget 6 lines (1/4)": lambda: _with_budget(W.WORKLOADS["janus_pro_7b"], 6),
    "janus_pro_7b budget 3 lines (1/8)": lambda: _with_budget(W.WORKLOADS["janus_pro_7b"], 3),
    "llamagen_xl budget 6 lines (1/4)": lambda: _with_budget(W.WORKLOADS["llamagen_xl"], 6),
    "lumina_768 budget 12 lines (1/4)": lambda: _with_budget(W.WORKLOADS["lumina_768"], 12),
    "lumina_768 budget 8 lines (1/6)": lambda: _with_budget(W.WORKLOADS["lumina_768"], 8),
    # M = 520 mid keys and 260 guide rows do not fit into shared memory together: the guide rows are read from global
    "gqa_1024 budget 16 lines (1/4)": lambda: _with_budget(W.WORKLOADS["gqa_1024"], 16),
}


@pytest.mark.parametrize("which", sorted(QUOTED))
def test_quoted_configurations_sampled_units(which):
    """One layer (layers are independent and identically shaped; the launch plan does not depend on their number), the
    whole generation in the benchmark's launch configuration, the oracle on a sample of units."""
    w = QUOTED[which]().scaled(n_layers=1)
    n_units = 3
    rep = run_parity(w, units=pick_units(w, n_units, seed=5), gen_device="cuda",
                     cfg_overrides=dict(flags=lar.LAR_FLAG_PDL), line_end_all=True)
    _check(rep, w, allow_near_ties=2)
    assert rep.compressions == min(n_units, w.batch * w.n_kv_heads) * (w.n_lines - w.budget_lines)


@pytest.mark.parametrize("name,steps", [("janus_pro_7b", None), ("gqa_1024", 65 * 20)])
def test_full_cache_path_full_size_sampled(name, steps):
    w = W.WORKLOADS[name].scaled(n_layers=1).full_cache()
    rep = run_parity(w, units=pick_units(w, 3, seed=2), gen_device="cuda", n_steps=steps)
    _check(rep, w)


def test_generator_gpu_matches_cpu():
    w = W.WORKLOADS["janus_pro_7b"].scaled(batch=2)
    a = W.gen_tokens(w, 1, 10, 14, "cpu")
    b = W.gen_tokens(w, 1, 10, 14, "cuda")
    for x, y in zip(a, b):
        diff = (x.float() != y.float().cpu()).float().mean().item()
        assert diff < 1e-4


# ------------------------------------------------------------------ Eq. 9 normalised over the whole live cache (variant)
@pytest.mark.parametrize("kw", [
    dict(),                                                   # fp32, M = 48
    dict(n_q_heads=8, n_kv_heads=1),                          # fp32, G = 8
    dict(cond_len=0, anchor_len=0),                           # nothing in front of the mid region
    dict(line_width=7, n_lines=9, anchor_len=7, recent_lines=1, budget_lines=3, cond_len=3),  # odd sizes, mid_off not a multiple of 8
    dict(line_width=1, n_lines=40, anchor_len=1, recent_lines=2, budget_lines=6),             # 1-token lines
    dict(dtype="bf16", head_dim=64, n_q_heads=4, n_kv_heads=2),
    dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=1),
    dict(dtype="bf16", head_dim=64, n_q_heads=4, n_kv_heads=4, cond_len=3, anchor_len=5, recent_lines=2, budget_lines=5),
])
@pytest.mark.parametrize("score_norm", ["cache", "accum"])
def test_cache_normalised_scoring(kw, score_norm):
    """The two scoring variants that soft-max over the whole live cache: the line's own decode probabilities ("cache"),
    and those probabilities accumulated over every step since a token was appended ("accum", the paper's ablation)."""
    w = W.WORKLOADS["tiny_b"].scaled(score_norm=score_norm, **kw)
    rep = run_parity(w)
    _check(rep, w, allow_near_ties=1)
    assert rep.compressions > 0
    assert rep.max_score_rel_err < (2e-3 if w.dtype == "bf16" else 1e-4)


def test_cache_normalised_scoring_one_launch_for_all_layers():
    """The flag must reach the kernel on the all-layers launch too: the exported scores match the oracle's variant
    (whose scores of a unit sum to well below one, unlike Eq. 9 as written)."""
    w = W.WORKLOADS["tiny_b"].scaled(score_norm="cache")
    cfg = lar.config_from_workload(w)
    assert cfg.flags & lar.LAR_FLAG_SCORE_CACHE_NORM
    rep = run_parity(w, line_end_all=True)
    _check(rep, w, allow_near_ties=1)
    assert rep.max_score_rel_err < 1e-4


def test_accumulated_attention_scoring_one_launch_for_all_layers_and_unfused_appends():
    w = W.WORKLOADS["tiny_b"].scaled(score_norm="accum", n_layers=3, dtype="bf16", n_q_heads=4, n_kv_heads=2)
    assert lar.config_from_workload(w).flags & lar.LAR_FLAG_SCORE_ACCUM
    for fused in (True, False):
        rep = run_parity(w, line_end_all=True, fused=fused)
        _check(rep, w, allow_near_ties=1)
        assert rep.compressions > 0 and rep.max_score_rel_err < 2e-3


@pytest.mark.parametrize("score_norm", ["cache", "accum"])
@pytest.mark.parametrize("name,layers,n_units", [("janus_pro_7b", 2, 4), ("gqa_1024", 1, 3)])
def test_cache_normalised_scoring_full_size_sampled(name, layers, n_units, score_norm):
    w = W.WORKLOADS[name].scaled(n_layers=layers, score_norm=score_norm)
    rep = run_parity(w, units=pick_units(w, n_units, seed=3), gen_device="cuda", cfg_overrides=dict(flags=lar.LAR_FLAG_PDL),
                     line_end_all=True)
    _check(rep, w, allow_near_ties=2)
    assert rep.compressions == n_units * (w.n_lines - w.budget_lines)


# ------------------------------------------------------------------ no compaction: evicted slots are refilled
@pytest.mark.parametrize("kw", [
    dict(),                                                             # fp32, G = 1
    dict(dtype="bf16", head_dim=64, n_q_heads=4, n_kv_heads=2),
    dict(dtype="bf16", head_dim=128, n_q_heads=8, n_kv_heads=1, cond_len=0),
    dict(dtype="bf16", head_dim=64, n_q_heads=4, n_kv_heads=4, cond_len=3, anchor_len=5, recent_lines=2, budget_lines=5),
    dict(dtype="bf16", head_dim=64, n_q_heads=2, n_kv_heads=2, anchor_len=0, recent_lines=3, budget_lines=6),
])
@pytest.mark.parametrize("score_norm", ["mid", "cache", "accum"])
def test_slot_reuse_keeps_the_same_sets_and_outputs(kw, score_norm):
    """Under LAR_FLAG_SLOT_REUSE the live set after every line end, every output and every score equal the oracle's;
    only the order of the slots differs (the harness compares the index map as a set and rejects duplicates)."""
    w = W.WORKLOADS["tiny_b"].scaled(score_norm=score_norm, **kw)
    for line_end_all in (False, True):
        rep = run_parity(w, cfg_overrides=dict(flags=lar.LAR_FLAG_SLOT_REUSE | lar.LAR_FLAG_PDL), line_end_all=line_end_all)
        _check(rep, w, allow_near_ties=1)
        assert rep.compressions > 0
        assert rep.max_score_rel_err < (2e-3 if w.dtype == "bf16" else 1e-4)


@pytest.mark.parametrize("name,layers,n_units", [("janus_pro_7b", 2, 4), ("gqa_1024", 1, 3), ("llamagen_xl", 1, 3), ("lumina_768", 1, 3)])
def test_slot_reuse_full_size_sampled(name, layers, n_units):
    w = W.WORKLOADS[name].scaled(n_layers=layers)
    rep = run_parity(w, units=pick_units(w, n_units, seed=4), gen_device="cuda",
                     cfg_overrides=dict(flags=lar.LAR_FLAG_PDL | lar.LAR_FLAG_SLOT_REUSE), line_end_all=True)
    _check(rep, w, allow_near_ties=2)
    assert rep.compressions == n_units * (w.n_lines - w.budget_lines)


def test_bf16_mid_region_smaller_than_one_key_tile():
    # M = 6 < 8: some lanes of the scoring warp see no valid key at all in the only tile
    w = W.WORKLOADS["tiny_b"].scaled(dtype="bf16", head_dim=64, n_q_heads=4, n_kv_heads=2, line_width=3, n_lines=12,
                                     anchor_len=3, recent_lines=2, budget_lines=5)
    assert w.mid_len == 6
    for sn in ("mid", "cache"):
        rep = run_parity(w.scaled(score_norm=sn))
        _check(rep, w, allow_near_ties=1)
        assert rep.compressions > 0


# ------------------------------------------------------------------ every layer of the deepest shapes
@pytest.mark.parametrize("name", ["janus_pro_7b", "gqa_1024", "llamagen_xl", "lumina_768"])
def test_every_layer_of_the_full_size_shape(name):
    """All layers, full batch, whole generation in the benchmark's launch configuration (fused step, PDL, one
    line-end launch for all layers); the oracle follows one unit of every layer (sequence and head vary with the layer)."""
    w = W.WORKLOADS[name]
    units = [(layer, (7 * layer + 3) % w.batch, (5 * layer + 1) % w.n_kv_heads) for layer in range(w.n_layers)]
    rep = run_parity(w, units=units, gen_device="cuda", cfg_overrides=dict(flags=lar.LAR_FLAG_PDL), line_end_all=True)
    _check(rep, w, allow_near_ties=3)
    assert rep.compressions == w.n_layers * (w.n_lines - w.budget_lines)
