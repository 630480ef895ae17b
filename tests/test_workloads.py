"""The seeded input generator: determinism, index consistency, distribution, byte accounting."""
import numpy as np
import torch

from paper_2512_04857_b200 import workloads as W


def test_generator_is_deterministic_and_index_consistent():
    w = W.WORKLOADS["tiny"]
    q1, k1, v1 = W.gen_tokens(w, 0, 0, 40)
    q2, k2, v2 = W.gen_tokens(w, 0, 16, 40)
    assert torch.equal(q1[16:], q2) and torch.equal(k1[16:], k2) and torch.equal(v1[16:], v2)
    u = W.gen_unit(w, 0, 0, 3)
    qa, ka, va = W.gen_tokens(w, 0, 0, w.n_visual)
    assert torch.equal(u["q"][:, 0], qa[:, 0, 3]) and torch.equal(u["k"], ka[:, 0, 3])
    assert torch.equal(u["v"], va[:, 0, 3])
    kc, vc = W.gen_prefix(w, 0)
    assert torch.equal(u["kc"], kc[0, 3]) and torch.equal(u["vc"], vc[0, 3])
    # different layers / streams are different draws
    qb, _, _ = W.gen_tokens(w, 1 if w.n_layers > 1 else 0, 0, 8)
    assert not torch.equal(k1[:8], v1[:8])


def test_gqa_unit_slices_query_group():
    w = W.WORKLOADS["gqa_1024"].scaled(n_lines=2, batch=2)
    u = W.gen_unit(w, 3, 1, 2)
    q, k, v = W.gen_tokens(w, 3, 0, w.n_visual)
    G = w.group
    assert u["q"].shape == (w.n_visual, G, w.head_dim)
    assert torch.equal(u["q"], q[:, 1, 2 * G:(2 + 1) * G].float())
    assert torch.equal(u["k"], k[:, 1, 2].float())


def test_values_are_unit_normal_and_bf16_exact():
    w = W.WORKLOADS["janus_pro_7b"].scaled(batch=2)
    _, _, v = W.gen_tokens(w, 0, 0, 16)
    x = v.double().flatten().numpy()
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    assert v.dtype == torch.bfloat16
    kc, _ = W.gen_prefix(w, 0)
    assert abs(kc.double().std().item() - 1.5) < 0.03       # prefix keys scaled by 1.5
    # the positional term makes same-position q.k larger than distant ones on average
    q, k, _ = W.gen_tokens(w, 0, 0, w.line_width * 4)
    qd, kd = q.double()[:, 0, 0], k.double()[:, 0, 0]
    logits = qd @ kd.T
    near = torch.diagonal(logits).mean()
    far = logits[0, -1]
    assert near > far + 10


def test_budgets_follow_the_efficiency_table():
    # B = rho N with n | B (efficiency table: 576 -> 96 at 1/6; 2352 -> 294 at 1/8)
    assert W.WORKLOADS["llamagen_xl"].budget_tokens == 96 == 576 // 6
    assert W.WORKLOADS["janus_pro_7b"].budget_tokens == 96
    assert W.WORKLOADS["lumina_768"].budget_tokens == 294 == 2352 // 8
    assert W.WORKLOADS["gqa_1024"].budget_tokens == 520 == 4160 // 8
    for w in W.WORKLOADS.values():
        assert w.budget_tokens % w.line_width == 0 and w.mid_len >= w.line_width


def test_live_length_closed_form():
    w = W.WORKLOADS["janus_pro_7b"]
    n, B, C = w.line_width, w.budget_tokens, w.cond_len
    lens = [w.live_len_at_step(i) for i in range(1, w.n_visual + 1)]
    assert lens[0] == C + 1 and lens[B - 1] == C + B and lens[B] == C + B - n + 1
    assert max(lens) == C + B
    assert w.full_cache().live_len_at_step(w.n_visual) == C + w.n_visual
