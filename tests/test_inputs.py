"""The seeded workload generator: determinism, independence of chunking, shapes, statistics."""
import numpy as np
import torch

import usv_inputs as ui


def test_counter_based_generator_is_deterministic_and_chunk_independent():
    a = ui.sin_field(7, 3, (2, 5, 6), 16, 64, chunk_tokens=7)
    b = ui.sin_field(7, 3, (2, 5, 6), 16, 64, chunk_tokens=1000)
    assert torch.equal(a, b)
    assert not torch.equal(a, ui.sin_field(8, 3, (2, 5, 6), 16, 64))
    assert not torch.equal(a, ui.sin_field(7, 4, (2, 5, 6), 16, 64))
    padded = ui.sin_field(7, 3, (2, 5, 6), 16, 64, n_rows=64)
    assert torch.equal(padded[:60], a) and torch.all(padded[60:] == 0)


def test_uniform_and_normal_moments():
    c = torch.arange(200000, dtype=torch.int64)
    u = ui.uniform01(12345, c)
    assert 0 < u.min() and u.max() < 1 and abs(u.mean() - 0.5) < 5e-3
    n = ui.normal(999, c)
    assert abs(n.mean()) < 1e-2 and abs(n.std() - 1) < 1e-2


def test_workload_table_matches_the_stated_shapes():
    w = {x.name: x for x in ui.WORKLOADS}
    assert (w["tiny"].N, w["tiny"].NB, w["tiny"].k_per_head()) == (1024, 16, [4, 4])
    assert (w["wan1.3b_480p"].N, w["wan1.3b_480p"].NB) == (32760, 512)
    assert w["wan1.3b_480p"].k_per_head() == [52] * 12
    m = w["wan1.3b_480p_merge50"]
    assert (m.r, m.N_attn, m.NB, m.k_per_head()[0]) == (16380, 16380, 256, 26)
    assert (w["wan14b_720p"].N, w["wan14b_720p"].NB, w["wan14b_720p"].k_per_head()[0]) == (75600, 1182, 60)
    h = w["hunyuan_720p"]
    assert (h.N, h.r, h.N_attn, h.NB) == (118800, 29700, 89100, 1393)
    assert h.k_per_head()[:4] == [1393, 349, 140, 70]
    for pct, k in ((100, 1393), (25, 349), (10, 140), (5, 70)):
        u = w["hunyuan_720p_keep%d" % pct]
        assert (u.B, u.H, u.N_attn, u.NB, u.k_per_head()) == (2, 24, 89100, 1393, [k] * 24)
    for name, n, nb, k in (("seq_99k", 99840, 1560, 78), ("seq_131k", 131040, 2048, 103), ("seq_193k", 193440, 3023, 152)):
        assert (w[name].N, w[name].NB, w[name].k_per_head()[0]) == (n, nb, k)


def test_tiny_qkv_layouts_hold_the_same_values():
    wl = ui.workload("tiny")
    q1, k1, v1 = ui.make_qkv(wl, layout="bhnd")
    q2, k2, v2 = ui.make_qkv(wl, layout="bnhd")
    assert q1.shape == (1, 2, 1024, 64) and q1.is_contiguous() and not q2.is_contiguous()
    assert torch.equal(q1, q2) and torch.equal(k1, k2) and torch.equal(v1, v2)
    assert not torch.equal(q1, k1)
    # magnitude: eight unit-variance-amplitude sinusoids (power 1/2 each) + 0.25 noise power
    expected = np.sqrt(8 * 0.5 + 0.25) * 64 ** -0.25
    assert abs(q1.float().std().item() / expected - 1) < 0.25
