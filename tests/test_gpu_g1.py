"""GPU parity of the layer with two clusters per token (cmoe_options.clusters_per_token = 2; Sec. 3.3, "Top-g1
groups") against the oracle's route_g1 / forward_g1.

Routes: bit-exact for every token whose decisions are not near-ties (margins of the logits, computed here in fp64,
above 1e-4: first against second against third cluster, and around the k-th expert of either kept cluster); gates to
1e-5.  y: max|y - y_ref| <= 1e-2 max|y_ref| + 1e-3 on every such token (a near-tie token may take another valid route
and is left out of the row comparison; they are counted and must stay rare)."""
import numpy as np
import pytest

from oracle import ref
from paper_2510_02345_b200 import inputs

pytestmark = pytest.mark.gpu

BAND = 1e-4


def _clear_tokens(L, g1=2):
    """Tokens none of whose routing decisions is a near-tie (margins in fp64)."""
    s = L["shape"]
    x64 = L["x"].astype(np.float64)
    z = x64 @ L["C"].astype(np.float64)
    if L.get("b_c") is not None:
        z = z + L["b_c"]
    order = np.argsort(-z, axis=1, kind="stable")
    zs = np.take_along_axis(z, order, axis=1)
    ok = np.ones(x64.shape[0], bool)
    for c in range(min(g1, s.G - 1)):
        ok &= (zs[:, c] - zs[:, c + 1]) > BAND
    for c in range(g1):
        g = order[:, c]
        l = np.einsum("td,tdk->tk", x64, L["R"].astype(np.float64)[g])
        if L.get("b_e") is not None:
            l = l + L["b_e"][g]
        ls = -np.sort(-l, axis=1)
        for j in range(min(s.k, s.K - 1)):
            ok &= (ls[:, j] - ls[:, j + 1]) > BAND
    return ok


def _check(L, options=None, expect_path=None):
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    s = L["shape"]
    o = ref.Layer(L)
    want_r = o.route_g1(L["x"], 2)
    want_y = o.forward_g1(L["x"], 2)
    m = ClusteredMoELayer(L, options=dict(options or {}, clusters_per_token=2))
    if expect_path is not None:
        assert m.info.path == expect_path
    x = torch.from_numpy(L["x"]).cuda()
    cid, eid, gates = m.route(x)
    y = m.forward(x)
    torch.cuda.synchronize()
    assert m.status() == 0
    cid, eid, gates, y = cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), y.float().cpu().numpy()
    ok = _clear_tokens(L)
    assert ok.mean() > 0.97, "too many near-tie tokens for this check to mean anything"
    assert np.array_equal(cid[ok], want_r["cluster_id"][ok])
    assert np.array_equal(eid[ok], want_r["expert_slot"][ok])         # labels are the identity in these layers
    assert np.abs(gates[ok] - want_r["gates"][ok]).max() <= 1e-5
    np.testing.assert_allclose(gates.reshape(gates.shape[0], -1).sum(axis=1), 1.0, atol=1e-5)
    assert (cid[:, 0] != cid[:, 1]).all()
    tol = 1e-2 * np.abs(want_y).max() + 1e-3
    err = np.abs(y[ok] - want_y[ok]).max()
    assert err <= tol, (err, tol)
    # a second call gives the same rows (scratch is rewritten, nothing accumulates across calls)
    y2 = m.forward(x).float().cpu().numpy()
    assert np.abs(y2[ok] - want_y[ok]).max() <= tol
    m.close()
    return dict(err=float(err), tol=float(tol), near_ties=int((~ok).sum()))


@pytest.mark.parametrize("kw,path", [
    (dict(T=64, d=256, d_ff=384, E=8, G=4, r=8, k=2), 2),          # 128 virtual tokens: weight-streaming path
    (dict(T=40, d=128, d_ff=128, E=6, G=2, r=4, k=1), 2),          # G = 2: both clusters kept
    (dict(T=300, d=128, d_ff=256, E=8, G=4, r=16, k=2), 1),        # pair path, per-token router (600 virtual tokens)
    (dict(T=700, d=256, d_ff=512, E=12, G=3, r=16, k=2), 1),       # pair path, tensor-core router (1400 virtual tokens)
    (dict(T=333, d=96, d_ff=160, E=8, G=4, r=4, k=2), 0),          # generic path
    (dict(T=650, d=128, d_ff=256, E=8, G=2, r=0, k=2), 1),         # no residual factors
], ids=["stream", "stream_G2", "pairs_small", "pairs_tc_router", "generic", "r0"])
def test_two_clusters_per_token(kw, path):
    s = inputs.small_shape(**kw)
    L = inputs.make_layer(s, 41)
    _check(L, expect_path=path)


def test_two_clusters_with_the_fp32_tile_router():
    s = inputs.small_shape(T=900, d=256, d_ff=256, E=16, G=4, r=8, k=2)
    L = inputs.make_layer(s, 42)
    _check(L, options=dict(router_fp32=1))


def test_two_clusters_on_the_bert_shape():
    # BERT-base-shaped layer, 2048 tokens = 4096 virtual tokens
    s = inputs.CONFIGS["bert"]
    L = inputs.make_layer(s, 0, T=2048)
    assert L["x"].shape[0] == 2048
    res = _check(L, expect_path=1)
    assert res["err"] / res["tol"] < 0.5


def test_loads_count_both_clusters_and_limits():
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer, CmoeError
    s = inputs.small_shape(T=500, d=128, d_ff=128, E=8, G=4, r=4, k=2)
    L = inputs.make_layer(s, 43)
    m = ClusteredMoELayer(L, options=dict(clusters_per_token=2))
    x = torch.from_numpy(L["x"]).cuda()
    loads, _, _ = m.expert_stats(x)
    torch.cuda.synchronize()
    want = np.bincount(ref.Layer(L).route_g1(L["x"], 2)["expert_slot"].reshape(-1), minlength=s.E)
    got = loads.cpu().numpy()
    assert got.sum() == 2 * s.k * s.T
    assert np.abs(got - want).sum() <= 2 * int((~_clear_tokens(L)).sum()) * s.k      # only near-tie tokens may differ
    # more tokens than T_max as the caller counts them
    with pytest.raises(CmoeError):
        m.forward(torch.zeros((s.T + 1, s.d), dtype=torch.float16, device="cuda"))
    m.close()
    # one cluster in all: two per token is not possible
    s1 = inputs.small_shape(T=16, d=128, d_ff=128, E=4, G=1, r=0, k=2)
    with pytest.raises(CmoeError):
        ClusteredMoELayer(inputs.make_layer(s1, 1), options=dict(clusters_per_token=2))
