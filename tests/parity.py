"""Shared helpers of the GPU parity tests: compare the CUDA library's outputs with the CPU oracle's
on the same seeded inputs.  (Test infrastructure; imports nothing from the library.)

Routes (Eq. 9-10) must be bit-exact wherever the oracle's logit margins exceed MARGIN.  Inside that band
several routes are correct; what is checked there is that the route the library took is a valid one (its
cluster's logit within MARGIN of the best, its experts distinct, inside that cluster, none further than
MARGIN below the k-th largest logit, ordered by logit up to MARGIN, gates = softmax over the kept logits),
and its output row is compared with the layer evaluated for THAT route."""
from __future__ import annotations

import json
import os

import numpy as np

MARGIN = 1e-4          # routes must be bit-exact where the oracle's logit margins exceed this
Y_REL, Y_ABS = 1e-2, 1e-3   # max|y - y_ref| <= Y_REL * max|y_ref| + Y_ABS
GATE_ATOL = 1e-5
GATE_ATOL_BAND = 2e-5       # inside the band the two sides' logits differ by rounding at the 1e-6 level


def route_margins(ref_route: dict, k: int):
    """Per token: gap between the best and second cluster logit, and the smallest gap that decides
    the kept expert set or its order."""
    z = np.sort(ref_route["z"].astype(np.float64), axis=1)[:, ::-1]
    l = np.sort(ref_route["l"].astype(np.float64), axis=1)[:, ::-1]
    cm = z[:, 0] - z[:, 1] if z.shape[1] > 1 else np.full(z.shape[0], np.inf)
    last = min(k, l.shape[1] - 1)           # gaps between ranks 0..last
    em = np.min(l[:, :last] - l[:, 1:last + 1], axis=1) if last >= 1 else np.full(l.shape[0], np.inf)
    return cm, em


def _expert_logits(layer: dict, x_row: np.ndarray, g: int) -> np.ndarray:
    """fp64 logits of one token against the K experts of cluster g (validity check of a banded token
    whose cluster differs from the oracle's; the oracle reports logits of its own cluster only)."""
    l = x_row.astype(np.float64) @ layer["R"][g].astype(np.float64)
    if layer.get("b_e") is not None:
        l = l + layer["b_e"][g].astype(np.float64)
    return l


def check_routes(shape, ref_route: dict, cid, eid, gates, label=None, layer=None, x=None):
    """Bit-exact cluster and expert ids outside the near-tie band; gates to 1e-5.  Inside the band the
    library's route must be a valid one (module docstring; needs `layer` and `x`).

    Returns (decided, ties, banded): the boolean mask of tokens whose whole route is decided by the
    margins, the tie counts, and {token: (cluster, [slots], [gates])} for the banded tokens (the
    library's route, by slot index g*K+i)."""
    K, k = shape.K, shape.k
    cm, em = route_margins(ref_route, k)
    c_ok = cm > MARGIN
    e_ok = c_ok & (em > MARGIN)
    want_e = ref_route["expert_slot"] if label is None else label[ref_route["expert_slot"]]
    assert np.array_equal(cid[c_ok], ref_route["cluster_id"][c_ok]), "cluster ids differ outside the near-tie band"
    assert np.array_equal(eid[e_ok], want_e[e_ok]), "expert ids differ outside the near-tie band"
    assert np.allclose(gates[e_ok], ref_route["gates"][e_ok], atol=GATE_ATOL, rtol=0), "gates differ"
    assert np.all((cid >= 0) & (cid < shape.G))
    assert np.allclose(gates.sum(1), 1.0, atol=1e-5)
    inv = None
    if label is not None:
        inv = {int(v): i for i, v in enumerate(label)}
    banded = {}
    for t in np.nonzero(~e_ok)[0]:
        g = int(cid[t])
        z = ref_route["z"][t].astype(np.float64)
        assert z[g] >= z.max() - MARGIN, f"token {t}: cluster {g} is not within the band of the best cluster logit"
        slots = [int(e) if inv is None else inv[int(e)] for e in eid[t]]
        assert len(set(slots)) == k, f"token {t}: repeated experts {slots}"
        assert all(s // K == g for s in slots), f"token {t}: experts {slots} outside cluster {g}"
        if g == int(ref_route["cluster_id"][t]):
            l = ref_route["l"][t].astype(np.float64)
        else:
            assert layer is not None and x is not None, "a banded token changed cluster: pass layer and x"
            l = _expert_logits(layer, x[t], g)
        kth = np.sort(l)[::-1][k - 1]
        chosen = np.array([l[s - g * K] for s in slots])
        assert np.all(chosen >= kth - MARGIN), f"token {t}: a kept expert lies below the k-th logit by more than the band"
        assert np.all(chosen[:-1] >= chosen[1:] - MARGIN), f"token {t}: kept experts out of logit order"
        p = np.exp(chosen - chosen.max())
        p /= p.sum()
        assert np.allclose(gates[t], p, atol=GATE_ATOL_BAND, rtol=0), f"token {t}: gates are not the softmax of the kept logits"
        banded[int(t)] = (g, slots, [float(v) for v in gates[t]])
    ties = dict(cluster_near_ties=int((~c_ok).sum()), expert_near_ties=int((c_ok & ~e_ok).sum()))
    return e_ok, ties, banded


def y_for_route(oracle_layer, x_row: np.ndarray, slots, gates) -> np.ndarray:
    """The layer's output row for a GIVEN route, from the oracle's explicitly formed expert weights
    (W_e = B_g + U_e V_e, Eq. 7) in fp64: y = sum_j p_j GELU(x W1_e) W2_e."""
    from scipy.special import erf
    xr = x_row.astype(np.float64)
    y = np.zeros(oracle_layer.shape.d, np.float64)
    for e, p in zip(slots, gates):
        h = xr @ oracle_layer.weight(e, 1).astype(np.float64)
        a = 0.5 * h * (1.0 + erf(h / np.sqrt(2.0)))
        y += p * (a @ oracle_layer.weight(e, 2).astype(np.float64))
    return y.astype(np.float32)


def patch_banded_rows(oracle_layer, x, idx, y_ref, banded, ref_route):
    """Rows of y_ref (for the tokens idx) whose token is banded and whose library route differs from
    the oracle's are replaced by the layer evaluated for the library's route."""
    pos = {int(t): i for i, t in enumerate(idx)}
    n = 0
    for t, (g, slots, gates) in banded.items():
        if t not in pos:
            continue
        if g == int(ref_route["cluster_id"][t]) and slots == [int(s) for s in ref_route["expert_slot"][t]]:
            continue
        y_ref[pos[t]] = y_for_route(oracle_layer, x[t], slots, gates)
        n += 1
    return n


def check_y(y, y_ref, rows=None):
    y = np.asarray(y, np.float32)
    if rows is not None:
        y, y_ref = y[rows], y_ref[rows]
    if y_ref.size == 0:
        return 0.0, 0.0
    assert np.all(np.isfinite(y)), "non-finite outputs"
    tol = Y_REL * float(np.max(np.abs(y_ref))) + Y_ABS
    err = float(np.max(np.abs(y - y_ref)))
    assert err <= tol, f"max|y - y_ref| = {err:.3e} exceeds {tol:.3e}"
    return err, tol


def record(name: str, **facts):
    """Append one line of parity facts (near-tie counts, rows checked, max error) to the file named by
    CMOE_PARITY_LOG, if set: the kept summary of a test run."""
    path = os.environ.get("CMOE_PARITY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(dict(case=name, **facts)) + "\n")


def compare(layer: dict, oracle_layer, x, cid, eid, gates, y, idx=None, label=None, name=None):
    """Whole comparison of one library call with the oracle: routes of all tokens, then the output rows
    `idx` (default: all), every one of them - rows of banded tokens against the layer evaluated for the
    route the library took.  Returns (max error, tolerance, tie counts)."""
    s = layer["shape"]
    x = np.asarray(x)
    T = x.shape[0]
    r = oracle_layer.route(x)
    decided, ties, banded = check_routes(s, r, cid, eid, gates, label=label, layer=layer, x=x)
    if idx is None:
        idx = np.arange(T, dtype=np.int32)
    y_ref = oracle_layer.forward(x, idx)
    rerouted = patch_banded_rows(oracle_layer, x, idx, y_ref, banded, r)
    err, tol = check_y(np.asarray(y)[idx], y_ref)
    record(name or s.name, T=int(T), rows_checked=int(len(idx)), rerouted_rows=int(rerouted), max_err=err, tol=tol, **ties)
    return err, tol, ties
