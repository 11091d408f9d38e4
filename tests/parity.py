"""Shared helpers of the GPU parity tests: compare the CUDA library's outputs with the CPU oracle's
on the same seeded inputs.  (Test infrastructure; imports the oracle.)"""
from __future__ import annotations

import numpy as np

MARGIN = 1e-4          # routes must be bit-exact where the oracle's logit margins exceed this
Y_REL, Y_ABS = 1e-2, 1e-3   # max|y - y_ref| <= Y_REL * max|y_ref| + Y_ABS


def route_margins(ref_route: dict, k: int):
    """Per token: gap between the best and second cluster logit, and the smallest gap that decides
    the kept expert set or its order."""
    z = np.sort(ref_route["z"].astype(np.float64), axis=1)[:, ::-1]
    l = np.sort(ref_route["l"].astype(np.float64), axis=1)[:, ::-1]
    cm = z[:, 0] - z[:, 1] if z.shape[1] > 1 else np.full(z.shape[0], np.inf)
    last = min(k, l.shape[1] - 1)           # gaps between ranks 0..last
    em = np.min(l[:, :last] - l[:, 1:last + 1], axis=1) if last >= 1 else np.full(l.shape[0], np.inf)
    return cm, em


def check_routes(shape, ref_route: dict, cid, eid, gates, label=None):
    """Bit-exact cluster and expert ids outside the near-tie band; gates to 1e-5.  Returns the
    boolean mask of tokens whose whole route is decided (not a near-tie) and the tie counts."""
    cm, em = route_margins(ref_route, shape.k)
    c_ok = cm > MARGIN
    e_ok = c_ok & (em > MARGIN)
    want_e = ref_route["expert_slot"] if label is None else label[ref_route["expert_slot"]]
    assert np.array_equal(cid[c_ok], ref_route["cluster_id"][c_ok]), "cluster ids differ outside the near-tie band"
    assert np.array_equal(eid[e_ok], want_e[e_ok]), "expert ids differ outside the near-tie band"
    assert np.allclose(gates[e_ok], ref_route["gates"][e_ok], atol=1e-5, rtol=0), "gates differ"
    # inside the band either order is accepted, but the result must still be a valid route
    assert np.all((cid >= 0) & (cid < shape.G))
    assert np.allclose(gates.sum(1), 1.0, atol=1e-5)
    return e_ok, dict(cluster_near_ties=int((~c_ok).sum()), expert_near_ties=int((c_ok & ~e_ok).sum()))


def check_y(y, y_ref, decided=None):
    y = np.asarray(y, np.float32)
    if decided is not None:
        y, y_ref = y[decided], y_ref[decided]
    if y_ref.size == 0:
        return 0.0, 0.0
    assert np.all(np.isfinite(y)), "non-finite outputs"
    tol = Y_REL * float(np.max(np.abs(y_ref))) + Y_ABS
    err = float(np.max(np.abs(y - y_ref)))
    assert err <= tol, f"max|y - y_ref| = {err:.3e} exceeds {tol:.3e}"
    return err, tol
