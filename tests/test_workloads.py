import numpy as np

from workloads import TINY_EAGLE
from workloads.generate import (MEDUSA_ALPHA, WeightStore, clipped_poisson_mean, forced_lengths,
                                medusa_static_tree, normal_f64, prompts, weight_shapes)


def test_generator_is_a_pure_function_of_seed_name_index():
    a = normal_f64(3, "x", 1000, "cpu")
    b = normal_f64(3, "x", 1000, "cpu", chunk=128)          # chunking must not change values
    assert np.array_equal(a.numpy(), b.numpy())
    assert not np.array_equal(a.numpy(), normal_f64(4, "x", 1000, "cpu").numpy())
    assert not np.array_equal(a.numpy(), normal_f64(3, "y", 1000, "cpu").numpy())


def test_normal_moments():
    z = normal_f64(0, "moments", 400000, "cpu").numpy()
    assert abs(z.mean()) < 0.01 and abs(z.std() - 1.0) < 0.01
    assert abs(np.mean(z ** 3)) < 0.03 and abs(np.mean(z ** 4) - 3.0) < 0.08


def test_weight_recipe():
    ws = WeightStore(TINY_EAGLE)
    assert set(ws.tensors) == set(weight_shapes(TINY_EAGLE))
    wq = ws.host("layers.0.wq")
    assert wq.shape == (256, 256) and abs(wq.std() - 0.02) < 1e-3
    g = ws.host("layers.1.ffn_norm")
    assert abs(g.mean() - 1.0) < 0.01 and abs(g.std() - 0.02) < 5e-3
    assert ws.host("fc_w").shape == (256, 512)


def test_prompt_is_uniform_ids():
    p = prompts(TINY_EAGLE)[0]
    assert p.shape == (64,) and p.min() >= 0 and p.max() < 1024


def test_forced_schedule_matches_closed_form_mean():
    # mean of Poisson(3) clipped to [1, 6], summed term by term
    assert abs(clipped_poisson_mean() - 2.99908) < 1e-4
    f = forced_lengths(2002, 20000)
    assert f.min() == 1 and f.max() == 6
    assert abs(f.mean() - clipped_poisson_mean()) < 0.05


def test_static_tree_shape():
    # the first three weights are the single-layer Medusa head's 1/2/3-alpha on the 7B target
    # (Table 1 of the paper), see tests/golden/medusa_alpha_table1.txt
    gold = [float(x) for x in open(__file__.rsplit("/", 1)[0] + "/golden/medusa_alpha_table1.txt")
            .read().split("\n")[-2].split()]
    assert tuple(gold) == MEDUSA_ALPHA[:3]
    parent, level, rank = medusa_static_tree(64)
    assert len(parent) == 64 and parent[0] == -1
    assert list(np.bincount(level)) == [1, 10, 31, 17, 5]
    for u in range(1, 64):
        assert 0 <= parent[u] < u and level[u] == level[parent[u]] + 1
    # prefix- and left-sibling-closed
    paths = {}
    for u in range(64):
        paths[u] = () if u == 0 else paths[parent[u]] + (int(rank[u]),)
    have = set(paths.values())
    for p in have:
        if p:
            assert p[:-1] in have
            if p[-1] > 0:
                assert p[:-1] + (p[-1] - 1,) in have
    # sibling tokens come from distinct ranks
    for u in range(64):
        kids = [int(rank[v]) for v in range(64) if parent[v] == u]
        assert len(kids) == len(set(kids))
