"""GPU parity of the launch mode the benchmark times: one CUDA graph per line (fused append + decode steps of every
layer) and one per line end, captured once and replayed for a second generation.  The decode kernel receives the live
length from the host at capture time, so this also checks that replaying the graphs in capture order reproduces the
lengths (device status bit 16 stays clear) and the oracle's outputs and kept sets."""
import argparse

import numpy as np
import pytest
import torch

import bench
from oracle import lar_oracle as O
from paper_2512_04857_b200 import lar, workloads as W
from _harness import TOL

pytestmark = pytest.mark.gpu


def _args(**kw):
    base = dict(no_pdl=False, tile_ranges=False, kv_splits=0, warps=0, stages=0, page_tokens=0, ctas=0)
    base.update(kw)
    return argparse.Namespace(**base)


@pytest.mark.parametrize("shape,kw", [
    ("janus_pro_7b", dict(n_layers=3, batch=2, n_q_heads=4, n_kv_heads=4)),
    ("gqa_1024", dict(n_layers=2, batch=2, n_q_heads=8, n_kv_heads=2, n_lines=12)),
])
@pytest.mark.parametrize("tile_ranges,score_norm", [(False, "mid"), (True, "mid"), (False, "cache"), (False, "accum")])
def test_graph_replay_of_a_second_generation_matches_the_oracle(shape, kw, tile_ranges, score_norm):
    w = W.WORKLOADS[shape].scaled(score_norm=score_norm, **kw)
    dev = torch.device("cuda:0")
    r = bench.Runner(w, dev, _args(tile_ranges=tile_ranges))
    r.capture()
    r.generation()                     # first replay
    r.generation()                     # second replay of the same graphs: lengths must come out the same
    torch.cuda.synchronize(dev)
    assert r.cache.poll_device_status() == 0
    n, L, G, Hkv = w.line_width, w.n_layers, w.group, w.n_kv_heads
    last = r.out[:, :, :, :, :].float().cpu().numpy()          # outputs of the last line: [n, L, S, Hq, d]
    ocfg = O.cfg_from_workload(w)
    worst = 0.0
    for layer in range(L):
        lens, imap = r.cache.get_state(layer)
        for s in range(w.batch):
            for h in range(Hkv):
                u = W.gen_unit(w, layer, s, h)
                out, kept, _ = O.run_units(ocfg, *[u[k].numpy()[None] for k in ("q", "k", "v", "kc", "vc")])
                ref = out[0, -n:]                                 # [n, G, d]
                got = last[:, layer, s, h * G:(h + 1) * G]
                worst = max(worst, float(np.abs(got - ref).max()))
                # live positions after the last token: what the last line end kept + the last line itself
                ui = s * Hkv + h
                pos_gpu = imap[ui, : lens[ui]]
                k_last = kept[0, w.n_lines - 2]
                k_last = k_last[k_last >= 0]
                pos_ref = np.concatenate([k_last, w.cond_len + np.arange(w.n_visual - n, w.n_visual)])
                assert np.array_equal(pos_gpu, pos_ref), (layer, s, h)
    assert worst <= TOL[w.dtype], worst
    r.close()


def test_two_runs_give_bit_identical_outputs_and_kept_sets():
    """No result depends on the order in which CTAs or warps happen to finish: scores are summed in a fixed order, the
    cross-CTA merge reads its partials in segment order."""
    w = W.WORKLOADS["gqa_1024"].scaled(n_layers=2, batch=2, n_q_heads=8, n_kv_heads=2, n_lines=12)
    dev = torch.device("cuda:0")
    outs, maps = [], []
    for tile_ranges in (False, True):
        for _ in range(2):
            r = bench.Runner(w, dev, _args(tile_ranges=tile_ranges))
            r.generation()                 # eager launches
            torch.cuda.synchronize(dev)
            assert r.cache.poll_device_status() == 0
            outs.append(r.out.clone())
            maps.append([r.cache.get_state(layer)[1].copy() for layer in range(w.n_layers)])
            r.close()
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[2], outs[3])
    for a, b in ((maps[0], maps[1]), (maps[2], maps[3]), (maps[0], maps[2])):
        for x, y in zip(a, b):
            assert np.array_equal(x, y)
