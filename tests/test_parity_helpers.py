"""The parity helpers themselves, on the CPU: what they accept inside the near-tie band, what they
reject, and that a banded token's row is compared with the layer evaluated for the route it took."""
import numpy as np
import pytest

from oracle import ref
from paper_2510_02345_b200 import inputs
from parity import MARGIN, check_routes, compare, y_for_route


def _layer_with_a_tie():
    s = inputs.small_shape(T=24, d=64, d_ff=96, E=8, G=2, r=4, k=2)
    L = inputs.make_layer(s, 41)
    R = L["R"].copy()
    R[:, :, 1] = R[:, :, 0]            # experts 0 and 1 of every cluster: identical router vectors -> exact ties
    L["R"] = R
    return s, L


def test_exact_routes_pass_and_y_for_route_matches_the_oracle():
    s, L = _layer_with_a_tie()
    o = ref.Layer(L)
    r = o.route(L["x"])
    y = o.forward(L["x"])
    err, tol, ties = compare(L, o, L["x"], r["cluster_id"], r["expert_slot"], r["gates"], y)
    assert err == 0.0 and ties["expert_near_ties"] > 0
    t = 3
    alt = y_for_route(o, L["x"][t], [int(v) for v in r["expert_slot"][t]], [float(v) for v in r["gates"][t]])
    assert np.abs(alt - y[t]).max() <= 1e-5 * max(1.0, np.abs(y[t]).max())


def test_a_swap_inside_the_band_is_accepted_and_checked_against_its_own_route():
    s, L = _layer_with_a_tie()
    o = ref.Layer(L)
    r = o.route(L["x"])
    y = o.forward(L["x"])
    eid = r["expert_slot"].copy()
    gates = r["gates"].copy()
    y2 = y.copy()
    swapped = 0
    for t in range(s.T):
        loc = eid[t] % s.K
        if set(loc) == {0, 1}:                      # the tied pair was kept: the other order is as good
            eid[t] = eid[t][::-1]
            gates[t] = gates[t][::-1]
            swapped += 1
        elif 0 in loc:                              # only one of the tied pair kept: the other one is as good
            j = int(np.nonzero(loc == 0)[0][0])
            eid[t, j] += 1
            y2[t] = y_for_route(o, L["x"][t], [int(v) for v in eid[t]], [float(v) for v in gates[t]])
            swapped += 1
    assert swapped > 0
    err, tol, ties = compare(L, o, L["x"], r["cluster_id"], eid, gates, y2)
    assert err <= 1e-5
    # the same rows with the ORACLE's y must fail where the kept expert changed (the helper really re-evaluates)
    if np.abs(y2 - y).max() > 10 * tol:
        with pytest.raises(AssertionError):
            compare(L, o, L["x"], r["cluster_id"], eid, gates, y)


@pytest.mark.parametrize("what", ["outside_cluster", "repeated", "below_band", "bad_gates", "wrong_cluster"])
def test_invalid_routes_inside_the_band_are_rejected(what):
    s, L = _layer_with_a_tie()
    o = ref.Layer(L)
    r = o.route(L["x"])
    cid, eid, gates = r["cluster_id"].copy(), r["expert_slot"].copy(), r["gates"].copy()
    loc = eid % s.K
    t = int(np.nonzero(((loc == 0) | (loc == 1)).any(axis=1))[0][0])     # a banded token
    if what == "outside_cluster":
        eid[t, 0] = (eid[t, 0] + s.K) % s.E
    elif what == "repeated":
        eid[t, 1] = eid[t, 0]
    elif what == "below_band":
        l = r["l"][t]
        worst = int(np.argmin(l))
        assert l[worst] < np.sort(l)[::-1][s.k - 1] - MARGIN
        eid[t, 1] = cid[t] * s.K + worst
    elif what == "bad_gates":
        gates[t] = np.array([0.9, 0.1], np.float32) if abs(gates[t, 0] - 0.9) > 0.01 else np.array([0.5, 0.5], np.float32)
    elif what == "wrong_cluster":
        z = r["z"][t]
        assert abs(z[0] - z[1]) > MARGIN
        cid[t] = 1 - cid[t]
        eid[t] = cid[t] * s.K + eid[t] % s.K
    with pytest.raises(AssertionError):
        check_routes(s, r, cid, eid, gates, layer=L, x=L["x"])
