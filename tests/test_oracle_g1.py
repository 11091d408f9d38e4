"""Pins of the oracle's routing and forward with g1 clusters per token (Sec. 3.3, "Top-g1 groups") against what
does not go through them: the pinned g1 = 1 functions, brute-force enumeration on independently computed logits,
a dense evaluation with numpy on independently decoded weights, the full soft mixture (g1 = G, k = K) and a
hand-worked two-cluster token."""
import itertools
import math

import numpy as np
import pytest
from scipy.special import softmax

from oracle import ref
from paper_2510_02345_b200 import inputs
from test_oracle_pins import gelu64, np_weights


def _layer(seed=5, **kw):
    s = inputs.small_shape(**kw)
    L = inputs.make_layer(s, seed)
    rng = np.random.default_rng(seed + 100)
    L["b_c"] = (rng.standard_normal(s.G) * 0.1).astype(np.float32)
    L["b_e"] = (rng.standard_normal((s.G, s.K)) * 0.1).astype(np.float32)
    return L


def test_one_cluster_is_the_pinned_routing_and_forward():
    L = _layer(T=40, d=64, d_ff=32, E=12, G=3, k=2, r=4)
    o = ref.Layer(L)
    a, b = o.route(L["x"]), o.route_g1(L["x"], 1)
    assert np.array_equal(a["cluster_id"], b["cluster_id"][:, 0])
    assert np.array_equal(a["expert_slot"], b["expert_slot"][:, 0])
    assert np.array_equal(a["gates"], b["gates"][:, 0])
    np.testing.assert_allclose(o.forward_g1(L["x"], 1), o.forward(L["x"]), rtol=0, atol=1e-6)


@pytest.mark.parametrize("kw,g1", [(dict(E=12, G=3, k=2), 2), (dict(E=16, G=4, k=3), 3), (dict(E=8, G=2, k=1), 2)])
def test_routes_by_enumeration(kw, g1):
    L = _layer(T=64, d=64, d_ff=32, r=0, **kw)
    s = L["shape"]
    r = ref.Layer(L).route_g1(L["x"], g1)
    x64 = L["x"].astype(np.float64)
    z = x64 @ L["C"].astype(np.float64) + L["b_c"]
    for t in range(s.T):
        # the g1 clusters of largest z, by enumeration of all subsets
        best = max(itertools.combinations(range(s.G), g1), key=lambda c: sum(z[t][g] for g in c))
        got = [int(g) for g in r["cluster_id"][t]]
        assert sorted(got) == sorted(best) and len(set(got)) == g1
        assert all(z[t][got[i]] >= z[t][got[i + 1]] for i in range(g1 - 1))        # descending z
        pg = softmax(z[t])[got]
        pg = pg / pg.sum()                                  # Eq. 9 over all clusters, renormalised over the kept ones
        total = 0.0
        for c, g in enumerate(got):
            l = x64[t] @ L["R"][g].astype(np.float64) + L["b_e"][g]
            kept = max(itertools.combinations(range(s.K), s.k), key=lambda q: sum(l[i] for i in q))
            ids = [int(v) - g * s.K for v in r["expert_slot"][t, c]]
            assert sorted(ids) == sorted(kept)
            assert all(l[ids[i]] >= l[ids[i + 1]] for i in range(s.k - 1))
            pi = softmax(l)[ids]
            pi = pi / pi.sum()                              # Eq. 10 renormalised over the kept experts
            np.testing.assert_allclose(r["gates"][t, c], pg[c] * pi, atol=1e-6)
            total += float(r["gates"][t, c].astype(np.float64).sum())
        assert abs(total - 1.0) < 1e-6


def test_forward_against_a_dense_evaluation():
    L = _layer(seed=9, T=24, d=64, d_ff=96, E=8, G=4, k=2, r=8)
    s = L["shape"]
    o = ref.Layer(L)
    g1 = 2
    r = o.route_g1(L["x"], g1)              # routes pinned above; weights decoded independently, FFN by numpy
    y = o.forward_g1(L["x"], g1)
    x64 = L["x"].astype(np.float64)
    W = {}
    for t in range(s.T):
        want = np.zeros(s.d)
        for c in range(g1):
            for j in range(s.k):
                e = int(r["expert_slot"][t, c, j])
                if e not in W:
                    W[e] = np_weights(L, e)
                want += float(r["gates"][t, c, j]) * (gelu64(x64[t] @ W[e][0]) @ W[e][1])
        np.testing.assert_allclose(y[t], want, rtol=1e-5, atol=1e-5)
    # listed tokens give the same rows
    idx = np.array([5, 0, 17], np.int32)
    np.testing.assert_allclose(o.forward_g1(L["x"], g1, idx), y[idx], rtol=0, atol=1e-6)


def test_all_clusters_and_all_experts_is_the_full_soft_mixture():
    # g1 = G and k = K: nothing is dropped, every expert weighs softmax(z)_g softmax(l_g)_i
    L = _layer(seed=3, T=10, d=32, d_ff=48, E=6, G=3, k=2, r=4)
    s = L["shape"]
    assert s.K == s.k
    y = ref.Layer(L).forward_g1(L["x"], s.G)
    x64 = L["x"].astype(np.float64)
    z = x64 @ L["C"].astype(np.float64) + L["b_c"]
    for t in range(s.T):
        pg = softmax(z[t])
        want = np.zeros(s.d)
        for g in range(s.G):
            pi = softmax(x64[t] @ L["R"][g].astype(np.float64) + L["b_e"][g])
            for i in range(s.K):
                W1, W2 = np_weights(L, g * s.K + i)
                want += pg[g] * pi[i] * (gelu64(x64[t] @ W1) @ W2)
        np.testing.assert_allclose(y[t], want, rtol=1e-5, atol=1e-5)


def test_hand_worked_token():
    # d = 2, three clusters of one expert: x = (1, 0), z = (ln 3, 0, -5) -> kept clusters 0 and 1 with
    # weights 3/4 and 1/4 (e^{ln 3} : e^0 = 3 : 1); each cluster's only expert has gate 1 inside it
    s = inputs.small_shape(T=1, d=32, d_ff=32, E=3, G=3, k=1, r=0)
    L = inputs.make_layer(s, 0)
    L["x"] = np.zeros((1, 32), np.float16); L["x"][0, 0] = 1.0
    L["C"] = np.zeros((32, 3), np.float32); L["C"][0] = [math.log(3.0), 0.0, -5.0]
    L["b_c"] = None; L["b_e"] = None
    r = ref.Layer(L).route_g1(L["x"], 2)
    assert r["cluster_id"].tolist() == [[0, 1]]
    assert r["expert_slot"].reshape(-1).tolist() == [0, 1]
    np.testing.assert_allclose(r["gates"].reshape(-1), [0.75, 0.25], atol=1e-6)


def test_ties_and_bad_arguments():
    s = inputs.small_shape(T=3, d=32, d_ff=32, E=8, G=4, k=1, r=0)
    L = inputs.make_layer(s, 1)
    L["C"] = np.zeros_like(L["C"])                          # all z equal: the lowest indices win, in order
    L["b_c"] = None
    r = ref.Layer(L).route_g1(L["x"], 3)
    assert np.array_equal(r["cluster_id"], np.tile([0, 1, 2], (3, 1)))
    np.testing.assert_allclose(r["gates"].sum(axis=(1, 2)), 1.0, atol=1e-6)
    np.testing.assert_allclose(r["gates"].sum(axis=2), 1.0 / 3.0, atol=1e-6)
    with pytest.raises(ValueError):
        ref.Layer(L).route_g1(L["x"], 0)
    with pytest.raises(ValueError):
        ref.Layer(L).route_g1(L["x"], 5)
