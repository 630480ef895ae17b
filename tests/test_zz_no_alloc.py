"""The entry point for callers that cannot allocate device memory (lar_attend_dense_noalloc).

Some users of this library hold nothing but their q / K / V / out tensors when they need attention: code inside a
framework's "no allocation" region, a server whose KV-cache manager already owns all free memory, a plug-in that
receives raw pointers.  They have no slab to give, so this call keeps its split-KV partials in a static device array
of the library.  The test drives the ordinary cache entry point (lar_decode_step) and the no-allocation call on the
same keys and values, two steps in a row, and checks that both give the same attention output within the bf16
tolerance of the parity tests -- and that the no-allocation call agrees with the CPU oracle's Eq. 2 on the same bf16
inputs within that tolerance.  It runs last (file name) so that a failure here cannot hide other results."""
import numpy as np
import pytest
import torch

from oracle import lar_oracle as O
from paper_2512_04857_b200 import lar

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2     # max-abs tolerance of bf16 attention outputs, as in the parity tests


def _against_oracle(q, k_all, v_all, out, group, head_dim, sample=5):
    """max-abs difference to the oracle's attention (fp64, Eq. 2) on a few units."""
    units = k_all.shape[0] * k_all.shape[1]
    qf = q.reshape(units, group, head_dim).float().cpu().numpy()
    kf = k_all.reshape(units, -1, head_dim).float().cpu().numpy()
    vf = v_all.reshape(units, -1, head_dim).float().cpu().numpy()
    of = out.reshape(units, group, head_dim).float().cpu().numpy().astype(np.float64)
    worst = 0.0
    for u in sorted({0, units - 1, *range(0, units, max(1, units // sample))}):
        for g in range(group):
            ref = O.attention(qf[u, g], kf[u], vf[u], 1.0 / np.sqrt(head_dim))
            worst = max(worst, float(np.max(np.abs(of[u, g] - ref))))
    return worst


def _run(head_dim, n_q_heads, n_kv_heads, cond_len, batch=3):
    dev = "cuda:0"
    group = n_q_heads // n_kv_heads
    # budget >= number of lines: the cache is never compressed, so the test knows every cached row
    cfg = lar.make_config(n_layers=1, batch=batch, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim,
                          dtype="bf16", cond_len=cond_len, line_width=8, n_lines=4, anchor_len=8, recent_lines=1,
                          budget_lines=4)
    cache = lar.Cache(cfg, device=dev)
    g = torch.Generator(device="cpu").manual_seed(head_dim + cond_len)
    mk = lambda *s: torch.randn(*s, generator=g).to(torch.bfloat16).to(dev)
    kc, vc = mk(batch, n_kv_heads, cond_len, head_dim), mk(batch, n_kv_heads, cond_len, head_dim)
    cache.append_kv(0, kc, vc, cond_len)
    units = batch * n_kv_heads
    k_all, v_all = kc.clone(), vc.clone()
    stream = torch.cuda.current_stream().cuda_stream
    worst = 0.0
    for step in range(2):                                   # two calls in a row share the static array
        q, k, v = mk(batch, n_q_heads, head_dim), mk(batch, n_kv_heads, head_dim), mk(batch, n_kv_heads, head_dim)
        ref = torch.zeros(batch, n_q_heads, head_dim, dtype=torch.bfloat16, device=dev)
        cache.decode_step(0, q, k, v, ref)                  # the existing entry point: append + attention
        k_all = torch.cat([k_all, k[:, :, None, :]], dim=2).contiguous()
        v_all = torch.cat([v_all, v[:, :, None, :]], dim=2).contiguous()
        length = cond_len + step + 1
        out = torch.full_like(ref, float("nan"))
        lar.lar_attend_dense_noalloc(q, k_all, v_all, out, units, group, head_dim, length, 0.0, stream)
        torch.cuda.synchronize()
        assert torch.isfinite(out.float()).all()
        worst = max(worst, (out.float() - ref.float()).abs().max().item())
        worst = max(worst, _against_oracle(q, k_all, v_all, out, group, head_dim))
    assert cache.poll_device_status() == 0
    cache.close()
    return worst


@pytest.mark.parametrize("head_dim,n_q_heads,n_kv_heads,cond_len", [
    (128, 8, 8, 200),      # several key ranges per unit: partials and tickets in the static array
    (64, 8, 2, 37),        # grouped queries, ragged length
    (128, 4, 4, 3),        # shorter than one key range (fewer than 16 rows): no scratch used
    (128, 8, 1, 200),      # 8 query heads per KV head, 8 key ranges per unit: the largest partials
])
def test_no_alloc_entry_point_matches_cache_entry_point(head_dim, n_q_heads, n_kv_heads, cond_len):
    assert _run(head_dim, n_q_heads, n_kv_heads, cond_len) <= TOL_BF16


def test_no_alloc_entry_point_with_more_units_than_ctas_can_be_split():
    """More than 296 units of 70 rows: every unit is one key range, only the tickets of the static array are touched."""
    assert _run(64, 40, 20, 68, batch=16) <= TOL_BF16     # 320 units


def test_no_alloc_entry_point_rejects_what_does_not_fit():
    x = torch.zeros(16, dtype=torch.bfloat16, device="cuda:0")
    L = lar.lib()
    # more units than the static array has tickets for: refused before anything is launched
    assert L.lar_attend_dense_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), 16385, 1, 64, 16, 0.0,
                                      None) == lar.LAR_ERR_CAPACITY
    assert L.lar_attend_dense_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), 4, 3, 96, 16, 0.0,
                                      None) == lar.LAR_ERR_INVALID_ARG
    assert L.lar_attend_dense_noalloc(None, x.data_ptr(), x.data_ptr(), x.data_ptr(), 4, 1, 64, 16, 0.0,
                                      None) == lar.LAR_ERR_INVALID_ARG
