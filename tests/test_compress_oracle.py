"""Pins for the CPU oracle of the offline compressor (oracle/compress_ref.py): what the paper and linear algebra fix
(Eq. 6, Eq. 7, the optimality of the truncated SVD, the INT4 storage format), computed by routes that do not go
through the oracle's own SVD call."""
import math

import numpy as np
import pytest

from oracle import compress_ref as cr
from paper_2510_02345_b200 import inputs


def test_mean_and_residual_by_hand():
    # one cluster of two 2 x 2 experts: base = [[2, 0], [1, 3]], residuals +-[[1, 0], [0, 1]] (rank 2, sigma = 1, 1)
    W = np.array([[[3, 0], [1, 4]], [[1, 0], [1, 2]]], np.float32)
    assert np.array_equal(cr.shared_base(W, 1)[0], np.array([[2, 0], [1, 3]], np.float16))
    A, Bt, S = cr.truncated_factors(W[0].astype(np.float64) - [[2, 0], [1, 3]], 2)
    assert np.allclose(S, [1, 1]) and np.allclose(A @ Bt, [[1, 0], [0, 1]], atol=1e-12)
    # two clusters: the mean runs over each cluster's own experts only (slot e = g K + i)
    W4 = np.stack([W[0], W[1], 10 * W[0], 10 * W[1]])
    B = cr.shared_base(W4, 2)
    assert np.array_equal(B[1], 10 * B[0])


def test_prescribed_singular_values_give_the_eckart_young_error():
    rng = np.random.default_rng(1)
    d_in, d_out = 48, 80
    s = np.array([5.0, 3.0, 2.0, 1.0, 0.5, 0.25, 0.125, 0.0625])
    P, _ = np.linalg.qr(rng.standard_normal((d_in, s.size)))
    Q, _ = np.linalg.qr(rng.standard_normal((d_out, s.size)))
    dW = (P * s) @ Q.T
    prev = np.inf
    for r in range(1, s.size + 1):
        A, Bt, S = cr.truncated_factors(dW, r)
        err = np.linalg.norm(dW - A @ Bt)
        assert abs(err - math.sqrt((s[r:] ** 2).sum())) < 1e-10          # closed form: the dropped singular values
        assert np.allclose(S, s[:r], atol=1e-10)
        assert err <= prev + 1e-12                                       # the error-versus-r curve never rises
        prev = err
        # the singular values are split evenly: both factors carry sqrt(sigma) per component
        assert np.allclose(np.linalg.norm(A, axis=0), np.sqrt(s[:r]), atol=1e-10)
        assert np.allclose(np.linalg.norm(Bt, axis=1), np.sqrt(s[:r]), atol=1e-10)


def test_known_low_rank_residuals_are_recovered():
    # two clusters of two experts C_g +- D_g with D_g of rank 4: the mean is C_g, the residuals are +-D_g exactly
    rng = np.random.default_rng(3)
    d_in, d_out, r = 64, 96, 4
    W = np.empty((4, d_in, d_out), np.float32)
    D = []
    for g in range(2):
        C = rng.standard_normal((d_in, d_out)) / 8
        P, _ = np.linalg.qr(rng.standard_normal((d_in, r)))
        Q, _ = np.linalg.qr(rng.standard_normal((d_out, r)))
        D.append((P * [0.5, 0.4, 0.3, 0.2]) @ Q.T)
        W[2 * g], W[2 * g + 1] = C + D[g], C - D[g]
    c = cr.compress(W, 2, r)
    assert np.array_equal(c["B"][1], W[2:4].astype(np.float64).mean(0).astype(np.float16))
    for e in range(4):
        dW = W[e].astype(np.float64) - c["B"][e // 2].astype(np.float64)
        # (the residual against the fp16 base carries the base's rounding, a full-rank term: 2^-12 |C| against |D| ~ 0.7)
        assert np.linalg.norm(dW - c["A"][e] @ c["Bt"][e]) <= 4e-3 * np.linalg.norm(dW)
        assert c["rel_err"][e] <= 4e-3
        assert np.allclose(c["sigma"][e], [0.5, 0.4, 0.3, 0.2], atol=2e-3)
        sign = 1.0 if e % 2 == 0 else -1.0
        assert np.linalg.norm(c["A"][e] @ c["Bt"][e] - sign * D[e // 2]) <= 4e-3 * np.linalg.norm(D[e // 2])
        # stored form: INT4 factors put about 1/14 relative error on each factor entry
        Wt = cr.reconstruct(c, e, 2, d_in, d_out, r)
        assert np.linalg.norm(Wt - W[e]) <= 0.15 * np.linalg.norm(dW)
    # the generator's correlated experts: the error-versus-r curve of the whole pipeline falls with r
    Wg = inputs.make_dense_experts(8, 2, 64, 96, seed=3)
    errs = [cr.compress(Wg, 2, rr)["rel_err"].mean() for rr in (4, 8, 16, 32)]
    assert all(a > b for a, b in zip(errs, errs[1:])) and errs[-1] < 0.35


def test_quantiser_format_and_round_trip():
    rng = np.random.default_rng(5)
    w = rng.standard_normal(32 * 40).astype(np.float32) * 0.3
    w[64:96] = 0.0                                                       # an all-zero group
    q, s = cr.quantize_int4_groups(w)
    assert q.dtype == np.uint8 and q.size == w.size // 2 and s.dtype == np.float16 and s.size == w.size // 32
    sf = s.astype(np.float32)
    assert sf[2] == 0 and not q[32:48].any()
    want_scale = (np.abs(w.reshape(-1, 32)).max(1) / np.float32(7)).astype(np.float16)
    assert np.array_equal(s, want_scale)
    back = cr.dequantize_int4_groups(q, s)
    step = np.repeat(sf, 32).astype(np.float64)
    assert np.all(np.abs(back - w) <= 0.5 * step + 1e-7)                 # within half a scale step
    # a hand-written group: values k * 0.5 for k = -7..7 then 3.5 again: scale 0.5, codes k
    hand = np.array([k * 0.5 for k in range(-7, 8)] + [3.5] * 17, np.float32)
    qh, sh = cr.quantize_int4_groups(hand)
    assert float(sh[0]) == 0.5
    codes = [(b & 0xF, b >> 4) for b in qh]
    flat = [c for pair in codes for c in pair]
    assert flat[:15] == [(k & 0xF) for k in range(-7, 8)] and all(c == 7 for c in flat[15:])


def test_cosine_gate():
    rng = np.random.default_rng(7)
    d = 32
    base = rng.standard_normal((d, d))
    ortho = rng.standard_normal((d, d))
    ortho -= (ortho * base).sum() / (base * base).sum() * base           # exactly orthogonal to the base: cosine 0
    # two experts base +- delta: their mean is the base, residuals +-delta, delta = 0.1 ortho + 0.05 base
    delta = 0.1 * ortho + 0.05 * base
    W = np.stack([base + delta, base - delta]).astype(np.float32)
    c = cr.compress(W, 1, 4, gamma=0.0)
    cos = (delta * base).sum() / (np.linalg.norm(delta) * np.linalg.norm(base))
    assert abs(c["cosine"][0] - cos) < 5e-3 and abs(c["cosine"][1] + cos) < 5e-3
    assert not c["pruned"].any() and c["Uq"].any()
    c = cr.compress(W, 1, 4, gamma=0.5 * cos)                            # expert 0 stays, expert 1 (negative cosine) goes
    assert list(c["pruned"]) == [0, 1] and c["Uq"][0].any() and not c["Uq"][1].any() and not c["Vs"][1].any()


# ---- planted mistakes: each must make one of the pins above fail ------------------------------------------------
_MUTANTS = {
    "sum_instead_of_mean": (".mean(axis=1).astype(np.float16)", ".sum(axis=1).astype(np.float16)"),
    "base_of_the_wrong_cluster": ("base = B[e // K].astype(np.float64)", "base = B[(e // K + 1) % G].astype(np.float64)"),
    "residual_sign": ("dW = W[e].astype(np.float64) - base", "dW = base - W[e].astype(np.float64)"),
    "smallest_singular_values": ("root = np.sqrt(S[:r])\n    return U[:, :r] * root[None, :], root[:, None] * Vt[:r], S[:r]",
                                 "root = np.sqrt(S[-r:])\n    return U[:, -r:] * root[None, :], root[:, None] * Vt[-r:], S[-r:]"),
    "singular_values_not_split": ("root = np.sqrt(S[:r])", "root = S[:r]"),
    "scale_over_8": ("scale = (absmax / np.float32(7.0)).astype(np.float16)", "scale = (absmax / np.float32(8.0)).astype(np.float16)"),
    "nibbles_swapped": ("packed = (nib[0::2] | (nib[1::2] << 4)).astype(np.uint8)", "packed = (nib[1::2] | (nib[0::2] << 4)).astype(np.uint8)"),
    "gate_keeps_what_it_should_prune": ("if gamma > 0.0 and cos < gamma:", "if gamma > 0.0 and cos > gamma:"),
    "factor_layouts_swapped": ("quantize_int4_groups(A.T)          # U layout [r][d_in]: d_in fastest", "quantize_int4_groups(A)"),
}


@pytest.mark.parametrize("name", sorted(_MUTANTS))
def test_planted_mistakes_are_caught(name, monkeypatch):
    import inspect
    import types
    src = inspect.getsource(cr)
    old, new = _MUTANTS[name]
    assert src.count(old) == 1, name
    mutant = types.ModuleType("compress_mutant")
    exec(compile(src.replace(old, new), "compress_mutant", "exec"), mutant.__dict__)
    for fn in ("quantize_int4_groups", "dequantize_int4_groups", "shared_base", "truncated_factors", "compress", "reconstruct"):
        monkeypatch.setattr(cr, fn, getattr(mutant, fn))
    caught = 0
    for pin in (test_mean_and_residual_by_hand, test_prescribed_singular_values_give_the_eckart_young_error,
                test_known_low_rank_residuals_are_recovered, test_quantiser_format_and_round_trip, test_cosine_gate):
        try:
            pin()
        except (AssertionError, ValueError, IndexError):
            caught += 1
    assert caught >= 1, f"no pin notices the planted mistake {name}"
