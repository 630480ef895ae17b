"""GPU tests of the call protocol, error reporting and the host-buffer entry point."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2512_04857_b200 import lar, workloads as W

pytestmark = pytest.mark.gpu


def _small(**kw):
    base = dict(n_layers=2, batch=2, n_q_heads=4, n_kv_heads=4, head_dim=64, dtype="bf16", cond_len=4,
                line_width=8, n_lines=8, anchor_len=8, recent_lines=1, budget_lines=4)
    base.update(kw)
    return lar.make_config(**base)


def _bufs(cfg, dev="cuda:0"):
    dt = torch.bfloat16 if cfg.dtype == lar.LAR_BF16 else torch.float32
    g = torch.Generator(device="cpu").manual_seed(1)
    mk = lambda *s: torch.randn(*s, generator=g).to(dt).to(dev)
    return dict(q=mk(cfg.batch, cfg.n_q_heads, cfg.head_dim), k=mk(cfg.batch, cfg.n_kv_heads, cfg.head_dim),
                v=mk(cfg.batch, cfg.n_kv_heads, cfg.head_dim),
                kc=mk(cfg.batch, cfg.n_kv_heads, max(cfg.cond_len, 1), cfg.head_dim),
                vc=mk(cfg.batch, cfg.n_kv_heads, max(cfg.cond_len, 1), cfg.head_dim),
                out=torch.zeros(cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=dt, device=dev))


def _status(fn, *a):
    try:
        fn(*a)
        return lar.LAR_OK
    except lar.LarError as e:
        return e.status


def test_call_order_errors():
    cfg = _small()
    c = lar.Cache(cfg)
    b = _bufs(cfg)
    # visual append before the prefill, decode without an append, wrong prefix length
    assert _status(c.decode_step, 0, b["q"], b["k"], b["v"], b["out"]) == lar.LAR_ERR_BAD_STATE
    assert _status(c.decode_attn, 0, b["q"], b["out"]) == lar.LAR_ERR_BAD_STATE
    assert _status(c.append_kv, 0, b["kc"], b["vc"], 3) == lar.LAR_ERR_INVALID_ARG
    c.append_kv(0, b["kc"], b["vc"], 4)
    assert _status(c.append_kv, 0, b["k"], b["v"], 2) == lar.LAR_ERR_INVALID_ARG
    assert _status(c.line_end_score_evict, 0) == lar.LAR_ERR_BAD_STATE       # no line finished
    c.append_kv(0, b["k"], b["v"], 1)
    assert _status(c.append_kv, 0, b["k"], b["v"], 1) == lar.LAR_ERR_BAD_STATE   # decode is due
    assert _status(c.line_end_score_evict, 0) == lar.LAR_ERR_BAD_STATE
    c.decode_attn(0, b["q"], b["out"])
    assert _status(c.decode_attn, 0, b["q"], b["out"]) == lar.LAR_ERR_BAD_STATE
    for _ in range(7):
        c.decode_step(0, b["q"], b["k"], b["v"], b["out"])
    # the line is complete: the n-token buffer is exhausted until the line-end call
    assert _status(c.decode_step, 0, b["q"], b["k"], b["v"], b["out"]) == lar.LAR_ERR_CAPACITY
    c.line_end_score_evict(0)
    c.decode_step(0, b["q"], b["k"], b["v"], b["out"])
    assert _status(c.decode_step, 5, b["q"], b["k"], b["v"], b["out"]) == lar.LAR_ERR_INVALID_ARG
    assert _status(c.decode_step, 0, None, b["k"], b["v"], b["out"]) == lar.LAR_ERR_INVALID_ARG
    assert c.poll_device_status() == 0
    # layers are independent: layer 1 still needs its prefill
    assert _status(c.decode_step, 1, b["q"], b["k"], b["v"], b["out"]) == lar.LAR_ERR_BAD_STATE
    lens, imap = c.get_state(0)
    assert (lens == 4 + 9).all() and (imap[:, :13] == np.arange(13)).all() and (imap[:, 13:] == -1).all()
    c.reset()
    lens, _ = c.get_state(0)
    assert (lens == 0).all()
    assert c.launch_count() > 0
    c.close()


def test_device_side_checks_record_status_instead_of_faulting():
    cfg = _small(flags=lar.LAR_FLAG_NO_HOST_CHECKS)
    c = lar.Cache(cfg)
    b = _bufs(cfg)
    c.append_kv(0, b["kc"], b["vc"], 4)
    for _ in range(3):
        c.decode_step(0, b["q"], b["k"], b["v"], b["out"])
    c.line_end_score_evict(0)                       # off a line boundary -> recorded, nothing touched
    assert c.poll_device_status() & 2
    lens, _ = c.get_state(0)
    assert (lens == 7).all()
    for _ in range(29):                             # fill to capacity C + B = 36 without line ends
        c.decode_step(0, b["q"], b["k"], b["v"], b["out"])
    assert c.poll_device_status() == 0
    c.decode_step(0, b["q"], b["k"], b["v"], b["out"])   # one more: no room, row is not stored
    assert c.poll_device_status() & 1
    lens, _ = c.get_state(0)
    assert (lens == 36).all()
    assert torch.isfinite(b["out"].float()).all()
    assert c.poll_device_status() == 0              # polling clears the word
    c.close()


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_a_key_that_is_not_finite_is_recorded_and_the_line_end_still_evicts_n(dtype):
    """A NaN key gives NaN scores: they rank lowest, the kept count stays M - n (the length trajectory is unchanged, the
    index map has no duplicate) and status bit 32 tells the host."""
    cfg = _small(n_layers=1, dtype=dtype, budget_lines=4, n_lines=8)     # B = 32, N_init = 8, r = 1: M = 16, evict 8
    c = lar.Cache(cfg)
    b = _bufs(cfg)
    c.append_kv(0, b["kc"], b["vc"], 4)
    g = torch.Generator(device="cpu").manual_seed(7)
    for t in range(32):
        k = torch.randn(cfg.batch, cfg.n_kv_heads, cfg.head_dim, generator=g).to(b["k"].dtype).to("cuda:0")
        if t == 12:                                    # a mid token (visual index 13: behind the anchor, before the last line)
            k[0, 1, 5] = float("nan")
        c.decode_step(0, b["q"], k, b["v"], b["out"])
        if t % 8 == 7:
            c.line_end_score_evict(0)
    bits = c.poll_device_status()
    assert bits == 32, bits
    lens, imap = c.get_state(0)
    assert (lens == 4 + 32 - 8).all()
    for u in range(cfg.batch * cfg.n_kv_heads):
        live = imap[u, : lens[u]]
        assert len(set(live.tolist())) == len(live) and (np.diff(live) > 0).all()
    # (a NaN key poisons the softmax of every guide row of its unit: all its scores tie at the bottom, so the n
    # newest mid tokens go, as for any tie)
    assert imap[1, : lens[1]].tolist() == list(range(4 + 16)) + list(range(4 + 24, 4 + 32))
    c.close()


@pytest.mark.parametrize("n_q_heads,n_kv_heads,head_dim", [(4, 4, 64), (8, 2, 128)])
def test_strided_views_of_a_fused_qkv_buffer_give_the_same_as_dense_tensors(n_q_heads, n_kv_heads, head_dim):
    """q, k, v as column ranges of one [batch, (Hq + 2 Hkv) d] buffer and out as a view of a wider buffer: outputs are
    bit-equal to the dense call's, the caches end in the same state (two line ends, one of them compressing)."""
    kw = dict(n_layers=1, batch=3, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim, budget_lines=3, n_lines=6)
    cfg = _small(**kw)
    ca, cb = lar.Cache(cfg), lar.Cache(cfg)
    b = _bufs(cfg)
    for c in (ca, cb):
        c.append_kv(0, b["kc"], b["vc"], 4)
    S, d = cfg.batch, head_dim
    nq, nk = n_q_heads * d, n_kv_heads * d
    row = nq + 2 * nk
    g = torch.Generator(device="cpu").manual_seed(3)
    out_wide = torch.zeros(S, nq + 64, dtype=torch.bfloat16, device="cuda:0")
    for t in range(4 * 8):
        qkv = torch.randn(S, row, generator=g).to(torch.bfloat16).to("cuda:0")
        q, k, v = qkv[:, :nq], qkv[:, nq:nq + nk], qkv[:, nq + nk:]
        dense_out = torch.zeros(S, n_q_heads, d, dtype=torch.bfloat16, device="cuda:0")
        ca.decode_step(0, q.contiguous().view(S, n_q_heads, d), k.contiguous().view(S, n_kv_heads, d),
                       v.contiguous().view(S, n_kv_heads, d), dense_out)
        out_wide.fill_(float("nan"))
        cb.decode_step_strided(0, q, k, v, out_wide[:, 32:], row, row, row, nq + 64)
        torch.cuda.synchronize()
        assert torch.equal(out_wide[:, 32:32 + nq].reshape(S, n_q_heads, d), dense_out)
        assert torch.isnan(out_wide[:, :32]).all() and torch.isnan(out_wide[:, 32 + nq:]).all()   # nothing written outside the view
        if t % 8 == 7:
            ca.line_end_score_evict(0)
            cb.line_end_score_evict(0)
    (la, ia), (lb, ib) = ca.get_state(0), cb.get_state(0)
    assert (la == lb).all() and (ia == ib).all() and (la == 4 + 3 * 8 - 8).all()   # C + B - n after a compressing line end
    assert ca.poll_device_status() == 0 and cb.poll_device_status() == 0
    # strides that are not 16-byte multiples, or shorter than a sequence's heads, are refused
    assert _status(cb.decode_step_strided, 0, q, k, v, out_wide, row + 4, row, row, nq + 64) == lar.LAR_ERR_INVALID_ARG
    assert _status(cb.decode_step_strided, 0, q, k, v, out_wide, row, nk - 8, row, nq + 64) == lar.LAR_ERR_INVALID_ARG
    ca.close()
    cb.close()


def _rotate(x, cos, sin, interleaved):
    """Rotary embedding of x [S, H, d] (bf16) with cos, sin [S, d/2] (fp32), rounded like the kernel: fp32 products and
    sums, each rounded, result to bf16."""
    S, H, d = x.shape
    xf = x.float()
    a, b = (xf[..., 0::2], xf[..., 1::2]) if interleaved else (xf[..., : d // 2], xf[..., d // 2:])
    c, s_ = cos[:, None, :], sin[:, None, :]
    ra, rb = a * c - b * s_, b * c + a * s_
    out = torch.empty_like(xf)
    if interleaved:
        out[..., 0::2], out[..., 1::2] = ra, rb
    else:
        out[..., : d // 2], out[..., d // 2:] = ra, rb
    return out.to(torch.bfloat16)


@pytest.mark.parametrize("n_q_heads,n_kv_heads,head_dim,interleaved", [(4, 4, 64, False), (8, 2, 128, False), (4, 2, 128, True)])
def test_fused_rotary_embedding_equals_rotating_first(n_q_heads, n_kv_heads, head_dim, interleaved):
    """lar_decode_step_rope on raw q, k against lar_decode_step on q, k rotated beforehand with the same arithmetic:
    outputs bit-equal, the caches evict the same tokens (the guide queue and the cached keys hold rotated rows)."""
    kw = dict(n_layers=1, batch=3, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim, budget_lines=3, n_lines=6)
    cfg = _small(**kw)
    ca, cb = lar.Cache(cfg), lar.Cache(cfg)
    b = _bufs(cfg)
    for c in (ca, cb):
        c.append_kv(0, b["kc"], b["vc"], 4)
    S, d = cfg.batch, head_dim
    g = torch.Generator(device="cpu").manual_seed(11)
    mk = lambda *s: torch.randn(*s, generator=g).to(torch.bfloat16).to("cuda:0")
    inv_freq = 1.0 / (10000.0 ** (torch.arange(d // 2, dtype=torch.float32) / (d // 2)))
    for t in range(5 * 8):
        q, k, v = mk(S, n_q_heads, d), mk(S, n_kv_heads, d), mk(S, n_kv_heads, d)
        pos = torch.tensor([t + 3 * s_ for s_ in range(S)], dtype=torch.float32)      # a position per sequence
        ang = pos[:, None] * inv_freq[None, :]
        cos, sin = torch.cos(ang).to("cuda:0"), torch.sin(ang).to("cuda:0")
        cos_sin = torch.cat([cos, sin], dim=1).contiguous()
        oa = torch.zeros(S, n_q_heads, d, dtype=torch.bfloat16, device="cuda:0")
        ob = torch.zeros_like(oa)
        ca.decode_step(0, _rotate(q, cos, sin, interleaved), _rotate(k, cos, sin, interleaved), v, oa)
        cb.decode_step_rope(0, q, k, v, ob, n_q_heads * d, n_kv_heads * d, n_kv_heads * d, n_q_heads * d, cos_sin, interleaved)
        torch.cuda.synchronize()
        assert torch.equal(oa, ob), f"step {t}: max diff {(oa.float() - ob.float()).abs().max().item()}"
        if t % 8 == 7:
            ca.line_end_score_evict(0)
            cb.line_end_score_evict(0)
    (la, ia), (lb, ib) = ca.get_state(0), cb.get_state(0)
    assert (la == lb).all() and (ia == ib).all()
    assert ca.poll_device_status() == 0 and cb.poll_device_status() == 0
    assert _status(cb.decode_step_rope, 0, q, k, v, ob, n_q_heads * d, n_kv_heads * d, n_kv_heads * d, n_q_heads * d, None,
                   interleaved) == lar.LAR_ERR_INVALID_ARG
    ca.close()
    cb.close()


def test_strided_entry_point_is_refused_for_fp32_caches():
    cfg = _small(n_layers=1, dtype="fp32")
    c = lar.Cache(cfg)
    b = _bufs(cfg)
    c.append_kv(0, b["kc"], b["vc"], 4)
    assert _status(c.decode_step_strided, 0, b["q"], b["k"], b["v"], b["out"], 4 * 64, 4 * 64, 4 * 64, 4 * 64) == lar.LAR_ERR_INVALID_ARG
    c.close()


def test_reset_forgets_deferred_host_copies():
    cfg = _small(n_layers=1, flags=lar.LAR_FLAG_HOST_DEFER_OUT)
    c = lar.Cache(cfg)
    b = _bufs(cfg)
    hq = torch.cat([b["q"].flatten(), b["k"].flatten(), b["v"].flatten()]).cpu().pin_memory()
    ho = torch.empty(b["out"].shape, dtype=b["out"].dtype).pin_memory()
    for _ in range(2):                                 # second round: the slots' bookkeeping starts afresh
        c.append_kv(0, b["kc"], b["vc"], 4)
        for _ in range(3):
            c.decode_step_host(0, hq, None, None, ho)
        torch.cuda.synchronize()
        c.reset()
    assert c.poll_device_status() == 0
    c.close()


def test_host_buffer_entry_point_matches_device_entry_point():
    cfg = _small(n_layers=1)
    b = _bufs(cfg)
    outs = []
    for host in (False, True):
        c = lar.Cache(cfg)
        c.append_kv(0, b["kc"], b["vc"], 4)
        if host:
            pin = {k: b[k].cpu().pin_memory() for k in ("q", "k", "v")}
            out = torch.zeros_like(b["out"], device="cpu").pin_memory()
        res = []
        for i in range(8):
            if host:
                c.decode_step_host(0, pin["q"], pin["k"], pin["v"], out)
                torch.cuda.synchronize()
                res.append(out.clone())
            else:
                c.decode_step(0, b["q"], b["k"], b["v"], b["out"])
                torch.cuda.synchronize()
                res.append(b["out"].cpu().clone())
        outs.append(torch.stack(res))
        assert c.poll_device_status() == 0
        c.close()
    assert torch.equal(outs[0], outs[1])


def _host_pipeline_inputs(cfg, steps, packed):
    """Distinct pinned q, k, v per (step, layer); packed: q | k | v of a call adjacent in one buffer."""
    L, S, Hq, Hkv, d = cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    g = torch.Generator(device="cpu").manual_seed(7)
    nq, nk = S * Hq * d, S * Hkv * d
    buf = torch.randn(steps, L, nq + 2 * nk, generator=g).to(torch.bfloat16).pin_memory()
    if packed:
        q, k, v = buf[..., :nq], buf[..., nq:nq + nk], buf[..., nq + nk:]
    else:
        q, k, v = (buf[..., :nq].contiguous().pin_memory(), buf[..., nq:nq + nk].contiguous().pin_memory(),
                   buf[..., nq + nk:].contiguous().pin_memory())
    return q, k, v


def _device_path(cfg, b, q, k, v, steps):
    """The same calls through the device-pointer entry point, synchronised after every call."""
    L, S, Hq, Hkv, d, n = cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.line_width
    c = lar.Cache(cfg)
    for layer in range(L):
        c.append_kv(layer, b["kc"], b["vc"], cfg.cond_len)
    outs = torch.zeros(steps, L, S * Hq * d, dtype=torch.bfloat16)
    for t in range(steps):
        for layer in range(L):
            c.decode_step(layer, q[t, layer].cuda().view(S, Hq, d), k[t, layer].cuda().view(S, Hkv, d),
                          v[t, layer].cuda().view(S, Hkv, d), b["out"])
            torch.cuda.synchronize()
            outs[t, layer] = b["out"].cpu().view(-1)
        if (t + 1) % n == 0:
            for layer in range(L):
                c.line_end_score_evict(layer)
    assert c.poll_device_status() == 0
    c.close()
    return outs


@pytest.mark.parametrize("packed,flags", [(False, 0), (True, 0), (True, lar.LAR_FLAG_PDL),
                                          (True, lar.LAR_FLAG_PDL | lar.LAR_FLAG_HOST_DEFER_OUT)])
def test_host_buffer_calls_back_to_back_without_synchronising(packed, flags):
    """The copies of consecutive calls overlap each other's kernels (two staging slots, library-owned copy streams):
    distinct inputs per call, no synchronisation in between, line ends in the middle; results must be those of the
    device-pointer entry point, bit for bit."""
    cfg = _small(n_layers=3, flags=flags)
    b = _bufs(cfg)
    steps = 3 * cfg.line_width + 5
    q, k, v = _host_pipeline_inputs(cfg, steps, packed)
    ref = _device_path(_small(n_layers=3), b, q, k, v, steps)
    c = lar.Cache(cfg)
    for layer in range(cfg.n_layers):
        c.append_kv(layer, b["kc"], b["vc"], cfg.cond_len)
    outs = torch.zeros_like(ref).pin_memory()
    for t in range(steps):
        for layer in range(cfg.n_layers):
            if packed:
                c.decode_step_host(layer, q[t, layer], None, None, outs[t, layer])
            else:
                c.decode_step_host(layer, q[t, layer], k[t, layer], v[t, layer], outs[t, layer])
        if (t + 1) % cfg.line_width == 0:
            for layer in range(cfg.n_layers):
                c.line_end_score_evict(layer)
    c.host_join()                                   # (a no-op unless the copy-outs are deferred)
    torch.cuda.synchronize()
    assert c.poll_device_status() == 0
    c.close()
    assert torch.equal(outs, ref)


def test_host_buffer_calls_inside_cuda_graphs_then_eagerly():
    """A line of host-buffer calls captured into a graph (the copy streams join the capture and re-join the capturing
    stream by the end of every call), replayed line after line, followed by eager calls and a second capture."""
    cfg = _small(n_layers=2, flags=lar.LAR_FLAG_NO_HOST_CHECKS)
    b = _bufs(cfg)
    n, L = cfg.line_width, cfg.n_layers
    lines = 5
    steps = lines * n
    q, k, v = _host_pipeline_inputs(cfg, steps, True)
    ref = _device_path(_small(n_layers=2), b, q, k, v, steps)
    c = lar.Cache(cfg)
    outs = torch.zeros_like(ref).pin_memory()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for layer in range(L):
            c.append_kv(layer, b["kc"], b["vc"], cfg.cond_len)

        def line(t0):
            for t in range(t0, t0 + n):
                for layer in range(L):
                    c.decode_step_host(layer, q[t, layer], None, None, outs[t, layer])
            for layer in range(L):
                c.line_end_score_evict(layer)

        graphs = []
        for ln in range(2):                       # lines 0 and 1: one graph each (different host addresses)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                line(ln * n)
            graphs.append(g)
        graphs[0].replay()
        graphs[1].replay()
        line(2 * n)                               # line 2 eagerly, right behind the graphs
        g = torch.cuda.CUDAGraph()                # lines 3 and 4 in one more graph
        with torch.cuda.graph(g, stream=s):
            line(3 * n)
            line(4 * n)
        g.replay()
    torch.cuda.synchronize()
    assert c.poll_device_status() == 0
    c.close()
    assert torch.equal(outs, ref)


def test_host_buffer_calls_with_deferred_copy_out():
    """LAR_FLAG_HOST_DEFER_OUT: the caller's stream does not wait for a call's copy-out until lar_cache_host_join (or
    the second call after it).  Eager calls, then a graph per line with the join before the capture ends; a capture
    that starts while copy-outs are pending is refused."""
    cfg = _small(n_layers=2, flags=lar.LAR_FLAG_NO_HOST_CHECKS | lar.LAR_FLAG_HOST_DEFER_OUT)
    b = _bufs(cfg)
    n, L = cfg.line_width, cfg.n_layers
    steps = 4 * n
    q, k, v = _host_pipeline_inputs(cfg, steps, True)
    ref = _device_path(_small(n_layers=2), b, q, k, v, steps)
    c = lar.Cache(cfg)
    outs = torch.zeros_like(ref).pin_memory()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for layer in range(L):
            c.append_kv(layer, b["kc"], b["vc"], cfg.cond_len)

        def line(t0, join):
            for t in range(t0, t0 + n):
                for layer in range(L):
                    c.decode_step_host(layer, q[t, layer], None, None, outs[t, layer])
            for layer in range(L):
                c.line_end_score_evict(layer)
            if join:
                c.host_join()

        line(0, False)                            # eagerly; the last two copy-outs stay pending
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):       # pending copy-outs do not cross into a capture
            st = _status(c.decode_step_host, 0, q[n, 0], None, None, outs[n, 0])
        assert st == lar.LAR_ERR_BAD_STATE
        c.host_join()
        c.host_join()                             # nothing pending: no-op
        graphs = []
        for ln in range(1, 4):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                line(ln * n, True)
            graphs.append(g)
        for g in graphs:
            g.replay()
    torch.cuda.synchronize()
    assert c.poll_device_status() == 0
    c.close()
    assert torch.equal(outs, ref)


def test_softmax_scale_override_and_single_row_cache():
    # C = 0 and the very first token: attention over one entry returns v exactly
    cfg = _small(n_layers=1, cond_len=0, softmax_scale=0.37, dtype="fp32")
    c = lar.Cache(cfg)
    b = _bufs(cfg)
    c.decode_step(0, b["q"], b["k"], b["v"], b["out"])
    torch.cuda.synchronize()
    assert torch.allclose(b["out"], b["v"], atol=1e-6)
    # second token: two-entry softmax with the overridden scale
    k2, v2 = b["k"] * 0.5, b["v"] + 1.0
    c.decode_step(0, b["q"], k2, v2, b["out"])
    torch.cuda.synchronize()
    logit = torch.stack([(b["q"] * b["k"]).sum(-1), (b["q"] * k2).sum(-1)], -1).double() * 0.37
    p = torch.softmax(logit, -1)
    ref = p[..., :1] * b["v"].double() + p[..., 1:] * v2.double()
    assert torch.allclose(b["out"].double(), ref, atol=1e-5)
    c.close()


def test_a_wait_that_runs_out_ends_the_launch_with_a_status_bit_and_leaves_the_device_usable():
    """Failure detection without a fault: with the test hook the producer warps request no tile, every consumer's
    bounded wait for its first tile runs out (~1 s), the roles of each CTA give up and the launch returns by itself;
    the host reads status bit 4.  A cache created afterwards works as usual."""
    import time
    cfg = _small(n_layers=1, flags=lar.LAR_FLAG_TEST_STALL)
    c = lar.Cache(cfg)
    b = _bufs(cfg)
    c.append_kv(0, b["kc"], b["vc"], 4)
    torch.cuda.synchronize()
    t0 = time.time()
    c.decode_step(0, b["q"], b["k"], b["v"], b["out"])
    torch.cuda.synchronize()
    dt = time.time() - t0
    assert 0.5 < dt < 20.0, dt                       # the limit, not a hang and not an immediate return
    bits = c.poll_device_status()
    assert bits & 4, bits
    c.close()
    # the same device, a cache without the hook: a fused step agrees with the unfused append + attention of another cache
    cfg2 = _small(n_layers=1)
    c1, c2 = lar.Cache(cfg2), lar.Cache(cfg2)
    o1, o2 = torch.zeros_like(b["out"]), torch.zeros_like(b["out"])
    for cc in (c1, c2):
        cc.append_kv(0, b["kc"], b["vc"], 4)
    c1.decode_step(0, b["q"], b["k"], b["v"], o1)
    c2.append_kv(0, b["k"], b["v"], 1)
    c2.decode_attn(0, b["q"], o2)
    torch.cuda.synchronize()
    assert c1.poll_device_status() == 0 and c2.poll_device_status() == 0
    assert torch.isfinite(o1.float()).all() and (o1.float() - o2.float()).abs().max().item() < 2e-2
    c1.close()
    c2.close()
