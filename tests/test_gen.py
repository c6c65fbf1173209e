"""Seeded input generators: determinism, ranges, tree shapes."""

import numpy as np

import gen


def test_draws_are_reproducible_and_keyed():
    cfg = gen.get_config(1)
    a = gen.prefill_inputs(cfg, 3, 64)
    b = gen.prefill_inputs(cfg, 3, 64)
    c = gen.prefill_inputs(cfg, 4, 64)
    for u, v in zip(a, b):
        assert np.array_equal(u, v)
    assert not np.array_equal(a[0], c[0])
    assert not np.array_equal(a[0], a[1])
    n = gen.node_inputs(cfg, 3, 0, 64)
    assert not np.array_equal(a[0], n[0])


def test_bf16_rounding_is_exact_and_nearest_even():
    cfg = gen.get_config(1)
    x = gen.prefill_inputs(cfg, 0, 128)[0]
    assert np.array_equal(gen.from_bf16_bits(gen.bf16_bits(x)), x)          # already representable
    one = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7], dtype=np.float32)
    got = gen.from_bf16_bits(gen.bf16_bits(one))
    assert np.array_equal(got, np.array([1.0, 1.0, 1.0 + 2 ** -6, 1.0 + 2 ** -7], dtype=np.float32))


def test_step_size_range():
    # softplus(dt + bias) must stay in [1e-3, 1e-1] (checked with numpy, independent of the oracle)
    for cid in (0, 1):
        cfg = gen.get_config(cid)
        dt = gen.prefill_inputs(cfg, 0, 512)[2].astype(np.float64)
        p = gen.layer_params(cfg, 0)
        delta = np.log1p(np.exp(dt + p.dt_bias.astype(np.float64)[None]))
        assert delta.min() >= 1e-3 and delta.max() <= 1e-1
        assert np.array_equal(p.A[0], -np.arange(1, cfg.d_state + 1, dtype=np.float32))
        assert np.all(p.A == p.A[0]) and np.all(p.D == 1)


def test_tree_shapes():
    t0 = gen.config_tree(gen.get_config(0))
    assert t0.n_nodes == 15 and list(t0.level_offsets) == [0, 1, 3, 7, 15]
    assert list(t0.parents[:7]) == [-1, 0, 0, 1, 1, 2, 2]
    t2 = gen.config_tree(gen.get_config(2), rnd=3)
    assert t2.n_nodes == 150 and list(t2.level_offsets) == [0, 1, 5, 21, 53, 117, 150]
    t3 = gen.config_tree(gen.get_config(3))
    assert t3.n_nodes == 16 and list(t3.parents) == list(range(-1, 15))
    # the paper's configurations: generation i holds N_1*...*N_i nodes (Section 4.1)
    assert list(np.diff(gen.paper_tree((3, 3, 2, 1)).level_offsets)) == [1, 3, 9, 18, 18]
    assert list(np.diff(gen.paper_tree((3, 2, 2, 1, 1)).level_offsets)) == [1, 3, 6, 12, 12, 12]
    assert list(np.diff(gen.paper_tree((2, 2, 2, 1, 1, 1)).level_offsets)) == [1, 2, 4, 8, 8, 8, 8]
    for s in range(32):
        for r in range(4):
            t = gen.config_tree(gen.get_config(4), r, s)
            assert t.n_nodes == 32 and t.n_levels <= 5
            d = t.depth()
            assert np.all(np.diff(d) >= 0) and np.all(np.diff(t.parents) >= 0)       # BFS order
            assert np.all(t.parents[1:] < np.arange(1, 32)) and t.parents[0] == -1
            assert np.bincount(t.parents[1:]).max() <= 3
            for l in range(t.n_levels):
                assert np.all(d[t.level_offsets[l]:t.level_offsets[l + 1]] == l)


def test_accepted_node_is_on_a_root_path():
    cfg = gen.get_config(2)
    t = gen.config_tree(cfg)
    seen = set()
    for r in range(40):
        v = gen.random_accepted_node(t, 0, cfg.cid, r)
        assert 0 <= v < t.n_nodes and t.path_to(v)[0] == 0
        seen.add(int(t.depth()[v]))
    assert len(seen) >= 4


def test_seq_lengths():
    cu = gen.seq_lengths(gen.get_config(4))
    lens = np.diff(cu)
    assert cu[0] == 0 and len(lens) == 32 and lens.min() >= 1024 and lens.max() <= 8192
    assert list(gen.seq_lengths(gen.get_config(1))) == [0, 2048]
