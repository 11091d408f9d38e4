"""Pins for the CPU oracle: each test checks it against something the paper or the
mathematics fixes, computed by a route that shares nothing with the oracle's C code."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2510_02345_b200 import inputs

GOLD = os.path.join(os.path.dirname(__file__), "golden")
NIBBLE_VALUE = [0, 1, 2, 3, 4, 5, 6, 7, -8, -7, -6, -5, -4, -3, -2, -1]  # two's complement, by hand


def unpack_codes(packed: np.ndarray) -> np.ndarray:
    """Inverse of the nibble packing (even flat index in the low nibble, two's complement), codes as int8."""
    table = np.array(NIBBLE_VALUE, np.int8)
    out = np.empty(packed.size * 2, np.int8)
    out[0::2] = table[packed & 0xF]
    out[1::2] = table[packed >> 4]
    return out


def np_dequant(q, s, shape):
    """Independent decoder (numpy): codes from the packing inverse times the per-32 scale, fp64."""
    codes = unpack_codes(q).astype(np.float64)
    scale = np.repeat(s.astype(np.float64), 32)
    return (codes * scale).reshape(shape)


def np_weights(L, e):
    """W1_e, W2_e in fp64 via numpy matmul on independently decoded factors."""
    s = L["shape"]
    g = e // s.K
    B1 = L["B1"][g].astype(np.float64)
    B2 = L["B2"][g].astype(np.float64)
    if s.r == 0:
        return B1, B2
    U1 = np_dequant(L["U1q"], L["U1s"], (s.E, s.r, s.d))[e]       # [r][d]   -> U1_e = U1.T
    V1 = np_dequant(L["V1q"], L["V1s"], (s.E, s.d_ff, s.r))[e]    # [d_ff][r]-> V1_e = V1.T
    U2 = np_dequant(L["U2q"], L["U2s"], (s.E, s.r, s.d_ff))[e]
    V2 = np_dequant(L["V2q"], L["V2s"], (s.E, s.d, s.r))[e]
    return B1 + U1.T @ V1.T, B2 + U2.T @ V2.T


def gelu64(u):
    return torch.nn.functional.gelu(torch.from_numpy(np.asarray(u, np.float64))).numpy()


# ---------------------------------------------------------------- number formats
def test_half_decode_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    want = bits.view(np.float16).astype(np.float32)
    got = np.array([ref.half_to_float(int(b)) for b in bits], np.float32)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan].view(np.uint32), want[~nan].view(np.uint32))


def test_int4_every_byte_both_positions():
    one = np.array([1.0], np.float16)
    for byte in range(256):
        q = np.zeros(16, np.uint8)
        q[0] = byte
        assert ref.dequant(q, one, 0) == NIBBLE_VALUE[byte & 0xF]
        assert ref.dequant(q, one, 1) == NIBBLE_VALUE[byte >> 4]


def test_int4_hand_written_vector():
    # 64 elements = two scale groups; bytes written by hand.
    q = np.zeros(32, np.uint8)
    q[0] = 0x21   # elements 0,1 = 1, 2
    q[1] = 0xF8   # elements 2,3 = -8, -1
    q[15] = 0x7F  # elements 30,31 = -1, 7
    q[16] = 0x9A  # elements 32,33 = -6, -7   (second group)
    q[31] = 0x80  # elements 62,63 = 0, -8
    s = np.array([0.5, 0.25], np.float16)
    want = {0: 0.5, 1: 1.0, 2: -4.0, 3: -0.5, 30: -0.5, 31: 3.5, 32: -1.5, 33: -1.75, 62: 0.0, 63: -2.0, 7: 0.0}
    for idx, v in want.items():
        assert ref.dequant(q, s, idx) == v


def test_quantiser_roundtrip_bound():
    rng = np.random.default_rng(3)
    w = rng.standard_normal((4, 8, 64)).astype(np.float32) * 0.02
    q, s = inputs.quantize_int4(w)
    back = np.array([ref.dequant(q, s, i) for i in range(w.size)]).reshape(w.shape)
    step = np.repeat(s.astype(np.float32), 32).reshape(w.shape)
    assert np.all(np.abs(back - w) <= 0.5 * step * (1 + 1e-3) + 1e-9)
    assert np.array_equal(back, np_dequant(q, s, w.shape).astype(np.float32))


# ---------------------------------------------------------------- paper's closed forms
def test_parameter_ratio_closed_form():
    want = {"tiny": 3.459, "bert": 3.623, "gpt2m": 3.710, "skew": 3.710, "decode": 7.405}
    for name, s in inputs.CONFIGS.items():
        # descriptor-only call: no arrays needed
        o = ref.Layer(dict(shape=s))
        stored, dense = o.param_count()
        W = 2 * s.d * s.d_ff
        assert dense == s.E * W
        cr = s.E * W / (s.G * W + s.E * 2 * s.r * (s.d + s.d_ff))
        assert stored == s.G * W + s.E * 2 * s.r * (s.d + s.d_ff)
        assert abs(dense / stored - cr) < 1e-12
        assert abs(dense / stored - want[name]) < 5e-4
        # Eq. 8 per cluster and matrix: K dio / (dio + K r (di + do)); both matrices share di+do
        K = s.K
        eq8 = K * s.d * s.d_ff / (s.d * s.d_ff + K * s.r * (s.d + s.d_ff))
        assert abs(dense / stored - eq8) < 1e-12


def test_paper_worked_values():
    # Eq. 8 in its square form at the paper's example, and the routing ratio of Sec. 3.3
    d, K, r = 4096, 8, 16
    assert abs(K / (1 + 2 * K * r / d) - 7.5294) < 1e-4
    assert abs(128 / (16 + 8) - 5.3333) < 1e-4
    s = inputs.LayerShape("sq", T=1, d=4096, d_ff=4096, E=8, G=1, r=16, k=2)
    stored, dense = ref.Layer(dict(shape=s)).param_count()
    assert abs(dense / stored - 7.5294) < 1e-4


def test_hand_worked_layer():
    with open(os.path.join(GOLD, "hand_worked_layer.txt")) as f:
        row = [ln for ln in f if ln.startswith("y ")][0].split()
    want = np.array([float(row[1]), float(row[2])])
    s = inputs.LayerShape("hand", T=1, d=2, d_ff=2, E=2, G=2, r=0, k=1)
    L = dict(shape=s, C=np.eye(2, dtype=np.float32), R=np.zeros((2, 2, 1), np.float32),
             B1=np.array([[[9, 9], [9, 9]], [[1, 0], [0, -1]]], np.float16),
             B2=np.array([[[9, 9], [9, 9]], [[1, 1], [2, 0]]], np.float16))
    x = np.array([[1, 2]], np.float16)
    o = ref.Layer(L)
    r = o.route(x)
    assert r["cluster_id"][0] == 1 and r["expert_slot"][0, 0] == 1 and r["gates"][0, 0] == 1.0
    assert np.allclose(o.forward(x)[0], want, atol=2e-7)


# ---------------------------------------------------------------- reductions
@pytest.mark.parametrize("seed", [0, 1])
def test_rank_zero_is_dense_ffn_per_cluster(seed):
    s = inputs.small_shape(T=41, d=64, d_ff=96, E=6, G=3, r=0, k=2)
    L = inputs.make_layer(s, seed)
    o = ref.Layer(L)
    y = o.forward(L["x"])
    # cluster choice from an independent fp64 matmul
    g = np.argmax(L["x"].astype(np.float64) @ L["C"].astype(np.float64), axis=1)
    x = torch.from_numpy(L["x"].astype(np.float64))
    for t in range(s.T):
        B1 = torch.from_numpy(L["B1"][g[t]].astype(np.float64))
        B2 = torch.from_numpy(L["B2"][g[t]].astype(np.float64))
        want = torch.nn.functional.gelu(x[t] @ B1) @ B2      # gates sum to 1 -> plain dense FFN
        assert np.allclose(y[t], want.numpy(), rtol=1e-5, atol=1e-5)


@pytest.mark.parametrize("seed", [0, 2])
def test_one_expert_per_cluster_is_top1_moe(seed):
    s = inputs.small_shape(T=33, d=64, d_ff=96, E=5, G=5, r=4, k=1)
    L = inputs.make_layer(s, seed)
    o = ref.Layer(L)
    y = o.forward(L["x"])
    r = o.route(L["x"])
    x64 = L["x"].astype(np.float64)
    e_star = np.argmax(x64 @ L["C"].astype(np.float64), axis=1)
    assert np.array_equal(r["expert_slot"][:, 0], e_star)
    assert np.all(r["gates"] == 1.0)
    for t in range(s.T):
        W1, W2 = np_weights(L, int(e_star[t]))
        want = gelu64(x64[t] @ W1) @ W2
        assert np.allclose(y[t], want, rtol=1e-5, atol=1e-5)


# ---------------------------------------------------------------- routing by brute force
@pytest.mark.parametrize("shape_kw", [dict(E=8, G=2, k=2), dict(E=12, G=3, k=3), dict(E=8, G=1, k=1), dict(E=16, G=2, k=4)])
def test_routes_by_enumeration(shape_kw):
    s = inputs.small_shape(T=64, d=64, d_ff=32, r=0, **shape_kw)
    L = inputs.make_layer(s, 5)
    rng = np.random.default_rng(1)
    L["b_c"] = rng.standard_normal(s.G).astype(np.float32) * 0.1
    L["b_e"] = rng.standard_normal((s.G, s.K)).astype(np.float32) * 0.1
    r = ref.Layer(L).route(L["x"])
    x64 = L["x"].astype(np.float64)
    z = x64 @ L["C"].astype(np.float64) + L["b_c"]
    assert np.allclose(r["z"], z, atol=1e-6)
    for t in range(s.T):
        g = int(np.argmax(z[t]))
        assert r["cluster_id"][t] == g
        l = x64[t] @ L["R"][g].astype(np.float64) + L["b_e"][g]
        assert np.allclose(r["l"][t], l, atol=1e-6)
        best = max(itertools.combinations(range(s.K), s.k), key=lambda c: sum(l[i] for i in c))
        got = [int(v) - g * s.K for v in r["expert_slot"][t]]
        assert sorted(got) == sorted(best)
        assert all(l[got[i]] >= l[got[i + 1]] for i in range(s.k - 1))      # descending logits
        p = r["gates"][t].astype(np.float64)
        assert np.all(p > 0) and abs(p.sum() - 1) < 1e-6
        for a in range(s.k):
            for b in range(s.k):
                assert abs(p[a] / p[b] - math.exp(l[got[a]] - l[got[b]])) < 1e-5
        # Eq. 10 over all K experts, then top-k, then renormalise == softmax over the kept logits
        full = np.exp(l - l.max()); full /= full.sum()
        assert np.allclose(p, full[got] / full[got].sum(), atol=1e-6)


def test_ties_take_lowest_index():
    s = inputs.LayerShape("tie", T=2, d=4, d_ff=4, E=8, G=2, r=0, k=2)
    L = dict(shape=s, C=np.zeros((4, 2), np.float32), R=np.zeros((2, 4, 4), np.float32),
             B1=np.zeros((2, 4, 4), np.float16), B2=np.zeros((2, 4, 4), np.float16))
    r = ref.Layer(L).route(np.ones((2, 4), np.float16))
    assert list(r["cluster_id"]) == [0, 0]
    assert r["expert_slot"].tolist() == [[0, 1], [0, 1]]
    assert np.allclose(r["gates"], 0.5)


# ---------------------------------------------------------------- the factored identity and the residual
def np_layer(L, x, route):
    """Independent fp64 layer that uses the factored form x B + (x U) V (reuse identity after Eq. 7)."""
    s = L["shape"]
    x64 = x.astype(np.float64)
    y = np.zeros((x.shape[0], s.d))
    dq = {n: np_dequant(L[n + "q"], L[n + "s"], shp) for n, shp in (
        ("U1", (s.E, s.r, s.d)), ("V1", (s.E, s.d_ff, s.r)), ("U2", (s.E, s.r, s.d_ff)), ("V2", (s.E, s.d, s.r)))}
    for t in range(x.shape[0]):
        g = route["cluster_id"][t]
        hb = x64[t] @ L["B1"][g].astype(np.float64)                  # shared by the token's experts
        for j in range(s.k):
            e = route["expert_slot"][t, j]
            h = hb + (dq["U1"][e] @ x64[t]) @ dq["V1"][e].T
            a = gelu64(h)
            y[t] += route["gates"][t, j] * (a @ L["B2"][g].astype(np.float64) + (dq["U2"][e] @ a) @ dq["V2"][e].T)
    return y


@pytest.mark.parametrize("name,seed", [("tiny", 0), ("tiny", 1)])
def test_explicit_weights_match_factored_form(name, seed):
    L = inputs.make_layer(inputs.CONFIGS[name], seed)
    o = ref.Layer(L)
    r = o.route(L["x"])
    y = o.forward(L["x"])
    want = np_layer(L, L["x"], r)
    assert np.max(np.abs(y - want)) <= 1e-5 * np.max(np.abs(want))


def test_residual_only_layer():
    # zero bases: the whole output comes from the rank-r factors, so a residual bug shows at full scale
    s = inputs.small_shape(T=29, d=64, d_ff=128, E=8, G=2, r=8, k=2)
    L = inputs.make_layer(s, 7)
    L["B1"] = np.zeros_like(L["B1"]); L["B2"] = np.zeros_like(L["B2"])
    # make the factors large so that activations are O(1)
    for n in ("U1s", "V1s", "U2s", "V2s"):
        L[n] = (L[n].astype(np.float32) * 25).astype(np.float16)
    o = ref.Layer(L)
    y = o.forward(L["x"])
    want = np_layer(L, L["x"], o.route(L["x"]))
    assert np.max(np.abs(want)) > 0.05
    assert np.max(np.abs(y - want)) <= 1e-5 * np.max(np.abs(want))
    for e in (0, 5):
        W1, W2 = np_weights(L, e)
        assert np.allclose(o.weight(e, 1), W1, rtol=1e-6, atol=1e-7)
        assert np.allclose(o.weight(e, 2), W2, rtol=1e-6, atol=1e-7)


def test_formed_weights_orientation():
    # non-square, distinct r/d/d_ff so a transposed factor cannot pass
    s = inputs.small_shape(T=4, d=32, d_ff=96, E=4, G=2, r=8, k=1)
    L = inputs.make_layer(s, 11)
    o = ref.Layer(L)
    for e in range(s.E):
        W1, W2 = np_weights(L, e)
        assert np.allclose(o.weight(e, 1), W1, rtol=1e-6, atol=1e-7)
        assert np.allclose(o.weight(e, 2), W2, rtol=1e-6, atol=1e-7)


# ---------------------------------------------------------------- invariants
def test_invariants():
    s = inputs.small_shape(T=48, d=64, d_ff=96, E=8, G=2, r=4, k=2)
    L = inputs.make_layer(s, 2)
    o = ref.Layer(L)
    x = L["x"]
    y = o.forward(x)
    # permuting tokens permutes rows; a duplicated token duplicates its row
    perm = np.random.default_rng(0).permutation(s.T)
    assert np.array_equal(o.forward(x[perm]), y[perm])
    x2 = np.concatenate([x, x[:3]])
    assert np.array_equal(o.forward(x2)[-3:], y[:3])
    # a token subset equals the same rows of the full result
    idx = np.array([5, 0, 47, 5], np.int32)
    assert np.array_equal(o.forward(x, idx), y[idx])
    # y is linear in the down-projection: doubling B2 and the V2 scales doubles y
    L2 = dict(L); L2["B2"] = (L["B2"].astype(np.float32) * 2).astype(np.float16)
    L2["V2s"] = (L["V2s"].astype(np.float32) * 2).astype(np.float16)
    assert np.allclose(ref.Layer(L2).forward(x), 2 * y, rtol=1e-6, atol=1e-7)
    # a constant added to all in-cluster logits changes nothing
    L3 = dict(L); L3["b_e"] = np.full((s.G, s.K), 0.75, np.float32)
    r0, r3 = o.route(x), ref.Layer(L3).route(x)
    assert np.array_equal(r0["expert_slot"], r3["expert_slot"])
    assert np.allclose(r0["gates"], r3["gates"], atol=1e-6)
    # gates are a distribution over the kept experts of one cluster
    assert np.allclose(r0["gates"].sum(1), 1, atol=1e-6)
    assert np.all(r0["expert_slot"] // s.K == r0["cluster_id"][:, None])
    assert np.all(r0["expert_slot"][:, 0] != r0["expert_slot"][:, 1])


def test_skewed_workload_recipe():
    s = inputs.LayerShape("skew_small", T=4096, d=64, d_ff=32, E=32, G=8, r=0, k=2, skew=True)
    L = inputs.make_layer(s, 0)
    r = ref.Layer(L).route(L["x"])
    share = np.bincount(r["cluster_id"], minlength=8) / s.T
    assert np.max(np.abs(share - inputs.zipf_shares(8, 1.2))) < 0.01
    assert abs(inputs.zipf_shares(8, 1.2)[0] - 0.429) < 1e-3
    # the +1.0 bias pulls expert 0 of every cluster into most top-2 sets
    frac0 = np.mean(np.any(r["expert_slot"] % s.K == 0, axis=1))
    assert frac0 > 0.75


def test_bad_descriptor_rejected():
    s = inputs.LayerShape("bad", T=1, d=4, d_ff=4, E=6, G=4, r=0, k=1)
    with pytest.raises(ValueError):
        ref.Layer(dict(shape=s, C=np.zeros((4, 4), np.float32))).route(np.zeros((1, 4), np.float16))


# ---- routing by-products: loads, mean routed token, Eq. 5, load CoV ------------------------------------
def _hand_stats_layer():
    s = inputs.small_shape(T=5, d=4, d_ff=2, E=4, G=2, r=0, k=1)
    C = np.zeros((4, 2), np.float32); C[0, 0] = 1; C[1, 1] = 1
    R = np.zeros((2, 4, 2), np.float32); R[:, 2, 0] = 1; R[:, 3, 1] = 1
    L = dict(shape=s, C=C, R=R, b_c=None, b_e=None, B1=np.zeros((2, 4, 2), np.float16), B2=np.zeros((2, 2, 4), np.float16))
    x = np.array([[2, 0, 1, 0], [4, 0, 3, 0], [1, 0, 0, 2], [0, 1, 2, 0], [1, 0, 0, 4]], np.float16)
    return L, x


def test_expert_stats_hand_counted():
    gold = {}
    for line in open(os.path.join(GOLD, "hand_worked_stats.txt")):
        if line.startswith("#") or not line.strip():
            continue
        key, *vals = line.split()
        gold[key] = np.array([float(v) for v in vals])
    L, x = _hand_stats_layer()
    mu = np.ones((4, 4), np.float32)
    loads, xbar, cov = ref.Layer(L).expert_stats(x, mu=mu, beta=0.25)
    assert np.array_equal(loads, gold["loads"].astype(np.int32))
    assert np.allclose(xbar.reshape(-1), gold["xbar"], atol=1e-6)
    assert np.allclose(mu.reshape(-1), gold["mu"], atol=1e-6)
    assert abs(cov - gold["cov"][0]) < 1e-6


def test_expert_stats_conservation_and_numpy_counts():
    L = inputs.make_layer(inputs.small_shape(T=301, d=64, d_ff=32, E=12, G=3, r=0, k=2), 51)
    s, x = L["shape"], L["x"]
    o = ref.Layer(L)
    mu0 = np.random.default_rng(0).standard_normal((s.E, s.d)).astype(np.float32)
    mu = mu0.copy()
    loads, xbar, cov = o.expert_stats(x, mu=mu, beta=0.05)
    # every token is counted once per kept expert
    assert loads.sum() == s.k * s.T
    # sum_e load_e xbar_e = k * (sum of all tokens): every token enters k expert means
    lhs = (loads[:, None].astype(np.float64) * xbar.astype(np.float64)).sum(0)
    rhs = s.k * x.astype(np.float64).sum(0)
    assert np.allclose(lhs, rhs, atol=1e-3)
    # counts and means again from the routes with numpy
    slots = o.route(x)["expert_slot"]
    assert np.array_equal(loads, np.bincount(slots.reshape(-1), minlength=s.E))
    for e in range(s.E):
        rows = np.nonzero((slots == e).any(axis=1))[0]
        want = x[rows].astype(np.float64).mean(0) if rows.size else np.zeros(s.d)
        assert np.allclose(xbar[e], want, atol=1e-6)
        want_mu = 0.95 * mu0[e].astype(np.float64) + 0.05 * want if rows.size else mu0[e]
        assert np.allclose(mu[e], want_mu, atol=1e-6)
    assert abs(cov - np.std(loads.astype(np.float64)) / np.mean(loads)) < 1e-6
    # an expert without tokens keeps its centroid: close cluster 1
    L["b_c"] = np.array([0.0, -50.0, 0.0], np.float32)
    mu = mu0.copy()
    loads, xbar, _ = ref.Layer(L).expert_stats(x, mu=mu, beta=0.5)
    assert loads[s.K:2 * s.K].sum() == 0 and np.array_equal(mu[s.K:2 * s.K], mu0[s.K:2 * s.K]) and not xbar[s.K:2 * s.K].any()


# ---- bfloat16 bases (a variant of the paper's FP16 storage) ---------------------------------------------------
def test_bf16_decode_all_bit_patterns():
    """All 65536 bfloat16 patterns against the format's definition worked out with Python integers: sign, 8
    exponent bits (bias 127), 7 mantissa bits; subnormals, infinities and NaNs included."""
    for bits in range(65536):
        sign = -1.0 if bits >> 15 else 1.0
        expo = (bits >> 7) & 0xFF
        mant = bits & 0x7F
        got = ref.bf16_to_float(bits)
        if expo == 255:
            if mant:
                assert math.isnan(got)
            else:
                assert got == sign * math.inf
            continue
        want = sign * (mant / 128.0) * 2.0 ** -126 if expo == 0 else sign * (1.0 + mant / 128.0) * 2.0 ** (expo - 127)
        assert got == want, (bits, got, want)


def test_bf16_bases_are_decoded_as_bf16():
    """A layer with bf16 bases and r = 0 is the dense FFN of the decoded bases (torch fp64): the decode path of the
    base and nothing else differs from the fp16 layer."""
    s = inputs.small_shape(T=9, d=32, d_ff=64, E=4, G=2, r=0, k=2)
    L = inputs.make_layer(s, 77, base_dtype="bf16")
    o = ref.Layer(L)
    y = o.forward(L["x"])
    r = o.route(L["x"])
    dec = lambda a: torch.from_numpy((a.astype(np.uint32) << 16).view(np.float32).astype(np.float64))
    B1, B2 = dec(L["B1"]), dec(L["B2"])
    x = torch.from_numpy(L["x"].astype(np.float64))
    for t in range(s.T):
        g = int(r["cluster_id"][t])
        h = x[t] @ B1[g]
        a = 0.5 * h * (1.0 + torch.erf(h / math.sqrt(2.0)))
        want = (a @ B2[g]).numpy()
        assert np.allclose(y[t], want, atol=1e-5, rtol=1e-5)
    # the same bits read as fp16 give something else: the flag matters
    L16 = dict(L, base_dtype="fp16", B1=L["B1"].view(np.float16), B2=L["B2"].view(np.float16))
    y16 = ref.Layer(L16).forward(L["x"])
    assert np.isnan(y16).any() or np.abs(np.nan_to_num(y16) - y).max() > 1e-3
