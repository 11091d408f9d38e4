"""GPU parity of the offline compressor (cmoe_compress, cmoe_quantize_int4) against its numpy oracle.

The INT4 quantiser is byte work: bit-exact on identical inputs.  The factors come from a randomised SVD, so they are
compared where the result is unique: the base (fp16 of the cluster mean, to one unit in the last place), the singular
values, the error of the rank-r product A B^T against the optimum the oracle's exact SVD attains (Eckart-Young) and,
when the spectrum has a gap behind sigma_r (only then is the truncation unique), the product itself.
Tolerances: sigma to 2e-3 relative (1e-2 without a gap), A B^T to 5e-3, error within 0.5 % of the optimum; stored form:
the Frobenius error of the oracle's stored form to 3 %."""
import numpy as np
import pytest

from oracle import compress_ref as cr
from paper_2510_02345_b200 import inputs

pytestmark = pytest.mark.gpu


def _omega(E, d_out, l, seed):
    return np.random.Generator(np.random.PCG64([seed, 0x0E6A])).standard_normal((E, d_out, l)).astype(np.float32)


def test_quantiser_is_bit_exact():
    import torch
    from paper_2510_02345_b200 import binding
    rng = np.random.default_rng(2)
    w = (rng.standard_normal(32 * 5000) * np.exp(rng.standard_normal(32 * 5000))).astype(np.float32)
    w[320:352] = 0.0
    w[0:32] = np.arange(32, dtype=np.float32) * 0.25 - 4.0          # ties of round-half-even on purpose
    q, s = binding.quantize_int4(torch.from_numpy(w).cuda())
    torch.cuda.synchronize()
    q_ref, s_ref = cr.quantize_int4_groups(w)
    assert np.array_equal(s.cpu().numpy().view(np.uint16), s_ref.view(np.uint16))
    assert np.array_equal(q.cpu().numpy(), q_ref)


def _pairs_with_a_gap(G, d_in, d_out, r, seed):
    """G clusters of two experts C_g +- D_g; D_g has r singular values 0.5 * 0.85^j, then a gap of a factor 8, then a
    decaying tail: the rank-r truncation is unique, so the products A B^T can be compared."""
    rng = np.random.default_rng(seed)
    n = min(d_in, d_out, r + 24)
    spec = np.concatenate([0.5 * 0.85 ** np.arange(r), 0.5 * 0.85 ** r / 8 * 0.8 ** np.arange(n - r)])
    W = np.empty((2 * G, d_in, d_out), np.float32)
    for g in range(G):
        C = rng.standard_normal((d_in, d_out)) / np.sqrt(d_in)
        P, _ = np.linalg.qr(rng.standard_normal((d_in, n)))
        Q, _ = np.linalg.qr(rng.standard_normal((d_out, n)))
        D = (P * spec) @ Q.T
        W[2 * g], W[2 * g + 1] = C + D, C - D
    return W


@pytest.mark.parametrize("kw", [
    dict(E=8, G=4, d_in=128, d_out=256, r=8, l=16, gap=True),
    dict(E=6, G=3, d_in=256, d_out=96, r=4, l=12, gap=True),
    dict(E=4, G=2, d_in=320, d_out=512, r=16, l=24, gap=True),
    dict(E=4, G=2, d_in=128, d_out=128, r=32, l=40, gap=True),
    dict(E=8, G=2, d_in=128, d_out=256, r=8, l=16, gap=False),       # the generator's experts: no gap in the spectrum
], ids=["r8", "r4_wide_in", "r16", "r32", "no_gap"])
def test_compressor_against_the_oracle(kw):
    import torch
    from paper_2510_02345_b200 import binding
    E, G, d_in, d_out, r, l = (kw[k] for k in ("E", "G", "d_in", "d_out", "r", "l"))
    K = E // G
    W = _pairs_with_a_gap(G, d_in, d_out, r, 11) if kw["gap"] else inputs.make_dense_experts(E, G, d_in, d_out, seed=11)
    ref = cr.compress(W, G, r)
    got = binding.compress(torch.from_numpy(W).cuda(), G, r, torch.from_numpy(_omega(E, d_out, l, 12)).cuda())
    torch.cuda.synchronize()
    g = {k_: v.cpu().numpy() for k_, v in got.items() if not k_.startswith("_")}
    # Eq. 6: fp16 of the mean (fp32 sums against fp64: at most one unit in the last place)
    Bg, Br = g["B"].astype(np.float32), ref["B"].astype(np.float32)
    assert np.all(np.abs(Bg - Br) <= np.spacing(np.abs(Br).astype(np.float16)).astype(np.float32))
    assert (Bg != Br).mean() < 0.01
    for e in range(E):
        dW = W[e].astype(np.float64) - ref["B"][e // K].astype(np.float64)
        P_g = g["A"][e].astype(np.float64) @ g["Bt"][e].astype(np.float64)
        P_r = ref["A"][e] @ ref["Bt"][e]
        # what is unique whatever the spectrum: the error of the best rank-r approximation (Eckart-Young), which the
        # library's product must attain, and the singular values up to the closeness of their neighbours
        assert np.linalg.norm(dW - P_g) <= (1 + 5e-3) * np.linalg.norm(dW - P_r) + 1e-6 * np.linalg.norm(dW)
        assert abs(g["rel_err"][e] - ref["rel_err"][e]) <= 3e-3
        assert np.allclose(g["sigma"][e], ref["sigma"][e], rtol=1e-2 if not kw["gap"] else 2e-3, atol=1e-5)
        if kw["gap"]:
            assert np.linalg.norm(P_g - P_r) <= 5e-3 * np.linalg.norm(P_r)   # a gap behind sigma_r: the truncation itself is unique
        # balanced split of the singular values between the two factors
        assert np.allclose(np.linalg.norm(g["A"][e], axis=0) ** 2, g["sigma"][e], rtol=5e-3)
        # the stored form reconstructs the expert as well as the oracle's stored form does
        err_g = np.linalg.norm(cr.reconstruct(g, e, K, d_in, d_out, r) - W[e])
        err_r = np.linalg.norm(cr.reconstruct(ref, e, K, d_in, d_out, r) - W[e])
        assert err_g <= 1.03 * err_r + 1e-6 * np.linalg.norm(dW)
        assert abs(g["cosine"][e] - ref["cosine"][e]) <= 2e-3
    # the quantised factors are the quantiser's image of the library's own fp32 factors (bit-exact)
    for e in range(E):
        q_ref, s_ref = cr.quantize_int4_groups(g["A"][e].T)
        assert np.array_equal(g["Uq"][e], q_ref) and np.array_equal(g["Us"][e].view(np.uint16), s_ref.view(np.uint16))
        q_ref, s_ref = cr.quantize_int4_groups(g["Bt"][e].T)
        assert np.array_equal(g["Vq"][e], q_ref) and np.array_equal(g["Vs"][e].view(np.uint16), s_ref.view(np.uint16))


def test_error_falls_with_the_rank_and_low_rank_residuals_are_exact():
    import torch
    from paper_2510_02345_b200 import binding
    E, G, d_in, d_out = 4, 2, 128, 192
    W = inputs.make_dense_experts(E, G, d_in, d_out, seed=13)
    Wd = torch.from_numpy(W).cuda()
    errs = []
    for r in (4, 8, 16, 32):
        got = binding.compress(Wd, G, r, torch.from_numpy(_omega(E, d_out, r + 8, 14)).cuda())
        torch.cuda.synchronize()
        errs.append(float(got["rel_err"].mean()))
        assert abs(errs[-1] - cr.compress(W, G, r)["rel_err"].mean()) < 2e-3
    assert all(a > b for a, b in zip(errs, errs[1:]))                       # the paper's error-versus-r curve (Sec. 3.2)
    # residuals of rank 4 compressed at rank 8: the surplus components are (numerically) zero, nothing blows up
    rng = np.random.default_rng(15)
    C = rng.standard_normal((d_in, d_out)) / 8
    P, _ = np.linalg.qr(rng.standard_normal((d_in, 4)))
    Q, _ = np.linalg.qr(rng.standard_normal((d_out, 4)))
    D = (P * [0.5, 0.4, 0.3, 0.2]) @ Q.T
    W2 = np.stack([C + D, C - D]).astype(np.float32)
    got = binding.compress(torch.from_numpy(W2).cuda(), 1, 8, torch.from_numpy(_omega(2, d_out, 16, 16)).cuda())
    torch.cuda.synchronize()
    sig = got["sigma"].cpu().numpy()
    assert np.allclose(sig[:, :4], [[0.5, 0.4, 0.3, 0.2]] * 2, atol=3e-3) and np.all(sig[:, 4:] < 5e-3)
    assert np.all(np.isfinite(got["A"].cpu().numpy())) and np.all(np.isfinite(got["Bt"].cpu().numpy()))
    assert float(got["rel_err"].max()) < 6e-3


def test_cosine_gate_and_the_layer_built_from_compressed_experts():
    """The gate zeroes the blocks the oracle zeroes; and the stored form the compressor writes is a valid layer
    descriptor: cmoe_forward on it agrees with the oracle evaluated on the same stored arrays."""
    import torch
    from oracle import ref
    from parity import compare
    from paper_2510_02345_b200 import binding
    s = inputs.small_shape(T=700, d=128, d_ff=256, E=8, G=2, r=8, k=2)
    W1 = inputs.make_dense_experts(s.E, s.G, s.d, s.d_ff, seed=21)
    W2 = inputs.make_dense_experts(s.E, s.G, s.d_ff, s.d, seed=22, base_std=1.0 / np.sqrt(s.d_ff))
    # give the residuals a part along their base (weights that sum to zero in each cluster, so the mean stays):
    # cosines of both signs and of sizes a threshold can separate
    K = s.K
    for g in range(s.G):
        Cg = W1[g * K:(g + 1) * K].mean(0)
        for i, a in enumerate([0.4, -0.15, 0.05, -0.3]):
            W1[g * K + i] += a * Cg
    ref1 = cr.compress(W1, s.G, s.r)
    pos = np.sort(ref1["cosine"][ref1["cosine"] > 0])
    gamma = float(0.5 * (pos[0] + pos[-1]))        # prunes every block of negative cosine and the small positive ones
    ref1 = cr.compress(W1, s.G, s.r, gamma=gamma)
    n_pruned = int(ref1["pruned"].sum())
    assert 0 < n_pruned < s.E and np.abs(ref1["cosine"] - gamma).min() > 2e-2       # no block sits near the threshold
    c1 = binding.compress(torch.from_numpy(W1).cuda(), s.G, s.r, torch.from_numpy(_omega(s.E, s.d_ff, 16, 23)).cuda(), gamma=gamma)
    c2 = binding.compress(torch.from_numpy(W2).cuda(), s.G, s.r, torch.from_numpy(_omega(s.E, s.d, 16, 24)).cuda())
    torch.cuda.synchronize()
    pr = c1["pruned"].cpu().numpy()
    assert np.array_equal(pr, ref1["pruned"])
    for e in np.nonzero(pr)[0]:
        assert not c1["Uq"][e].any() and not c1["Us"][e].view(torch.int16).any() and not c1["Vs"][e].view(torch.int16).any()
    base = inputs.make_layer(s, 25)
    L = dict(base, B1=c1["B"].cpu().numpy(), B2=c2["B"].cpu().numpy())
    for n, c, tag in (("U1", c1, "U"), ("V1", c1, "V"), ("U2", c2, "U"), ("V2", c2, "V")):
        L[n + "q"] = c[tag + "q"].cpu().numpy().reshape(-1)
        L[n + "s"] = c[tag + "s"].cpu().numpy().reshape(-1)
    m = binding.ClusteredMoELayer(L)
    assert m.info.pruned_blocks == n_pruned
    x = torch.from_numpy(L["x"]).cuda()
    cid, eid, gates = m.route(x)
    y = m.forward(x)
    torch.cuda.synchronize()
    compare(L, ref.Layer(L), L["x"], cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), y.float().cpu().numpy())
