"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle, element by element on
the same seeded inputs: all routes and every output row of the five workloads and of the small, ragged
and degenerate cases (a few very large extra shapes on sampled rows)."""
import numpy as np
import pytest

from oracle import ref
from paper_2510_02345_b200 import inputs
from parity import check_routes, check_y, compare

pytestmark = pytest.mark.gpu

_cache = {}


def layer_for(name, seed=0):
    key = (name, seed)
    if key not in _cache:
        _cache.clear()                      # keep at most one large layer on the host
        _cache[key] = inputs.make_layer(inputs.CONFIGS[name], seed)
    return _cache[key]


def run_gpu(L, x_np, T_max=None, options=None):
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    m = ClusteredMoELayer(L, T_max=T_max if T_max is not None else max(1, x_np.shape[0]), options=options)
    x = torch.from_numpy(x_np).cuda()
    cid, eid, gates = m.route(x)
    y = m.forward(x)
    torch.cuda.synchronize()
    assert m.status() == 0
    out = dict(cid=cid.cpu().numpy(), eid=eid.cpu().numpy(), gates=gates.cpu().numpy(),
               y=y.float().cpu().numpy(), module=m)
    return out


def full_check(L, x_np, sample=None, seed=0, label=None, options=None, T_max=None):
    s = L["shape"]
    o = ref.Layer(L)
    got = run_gpu(L, x_np, T_max=T_max, options=options)
    T = x_np.shape[0]
    idx = None
    if sample is not None and sample < T:
        idx = np.sort(np.random.default_rng(seed).choice(T, sample, replace=False)).astype(np.int32)
    err, tol, ties = compare(L, o, x_np, got["cid"], got["eid"], got["gates"], got["y"], idx=idx, label=label)
    print(f"{s.name}: T={T} near-ties {ties} checked {T if idx is None else idx.size} rows, max err {err:.3e} (tol {tol:.3e})")
    return got


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_tiny_full(seed):
    L = layer_for("tiny", seed)
    full_check(L, L["x"])


def test_bert_full():
    L = layer_for("bert")
    full_check(L, L["x"])


@pytest.mark.parametrize("name", ["gpt2m", "skew"])
def test_large_full(name):
    L = layer_for(name)
    got = full_check(L, L["x"])
    if name == "skew":
        share = np.bincount(got["cid"], minlength=8) / L["x"].shape[0]
        assert abs(share[0] - 0.429) < 0.02 and share[-1] < 0.06


def test_decode_full():
    L = layer_for("decode")
    full_check(L, L["x"])


@pytest.mark.parametrize("T", [1, 2, 127, 129, 257, 300])
def test_ragged_token_counts(T):
    s = inputs.small_shape(T=T, d=64, d_ff=160, E=8, G=2, r=4, k=2)
    L = inputs.make_layer(s, 3)
    full_check(L, L["x"])


@pytest.mark.parametrize("kw", [
    dict(E=8, G=2, r=0, k=2),      # no residual: dense FFN per cluster
    dict(E=5, G=5, r=4, k=1),      # one expert per cluster: plain top-1 MoE
    dict(E=8, G=2, r=8, k=4),      # k == K
    dict(E=8, G=1, r=16, k=2),     # a single cluster
    dict(E=16, G=2, r=32, k=3),    # K = 8, odd k, largest rank
    dict(E=32, G=2, r=4, k=8),     # K = 16: C(16,8) > 64 -> sub-key is the lowest expert
], ids=["r0", "K1", "k_eq_K", "G1", "k3_r32", "k8"])
def test_shape_variants(kw):
    s = inputs.small_shape(T=200, d=96, d_ff=224, **kw)
    L = inputs.make_layer(s, 4)
    full_check(L, L["x"])


def test_empty_cluster_and_labels():
    s = inputs.small_shape(T=150, d=64, d_ff=96, E=9, G=3, r=4, k=2)
    L = inputs.make_layer(s, 6)
    L["b_c"] = np.array([0.0, -50.0, 0.0], np.float32)        # cluster 1 never wins
    L["b_e"] = np.zeros((3, 3), np.float32)
    label = (np.arange(9, dtype=np.int32) * 7 + 100)
    L["expert_global_id"] = label
    got = full_check(L, L["x"], label=label)
    assert not np.any(got["cid"] == 1)


def test_zero_tokens_and_reuse():
    import torch
    s = inputs.small_shape(T=64, d=64, d_ff=96, E=8, G=2, r=4, k=2)
    L = inputs.make_layer(s, 8)
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    m = ClusteredMoELayer(L, T_max=64)
    empty = torch.empty((0, 64), dtype=torch.float16, device="cuda")
    assert m.forward(empty).shape == (0, 64)
    o = ref.Layer(L)
    # the same handle, different batch sizes back to back
    for T in (64, 5, 33):
        x_np = inputs.make_tokens(s, T, seed=T)
        x = torch.from_numpy(x_np).cuda()
        cid, eid, gates = m.route(x)
        y = m.forward(x)
        torch.cuda.synchronize()
        compare(L, o, x_np, cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), y.float().cpu().numpy())
    assert m.status() == 0


def test_runtime_errors():
    import torch
    from paper_2510_02345_b200 import binding
    s = inputs.small_shape(T=16, d=64, d_ff=96, E=8, G=2, r=4, k=2)
    L = inputs.make_layer(s, 9)
    m = binding.ClusteredMoELayer(L, T_max=16)
    x = torch.zeros((32, 64), dtype=torch.float16, device="cuda")
    with pytest.raises(binding.CmoeError) as ei:
        m.forward(x)
    assert ei.value.code == -4
    rc = binding.lib().cmoe_forward(m.handle, x.data_ptr() + 2, 8, x.data_ptr(), 0)   # misaligned x
    assert rc == -1


def test_permutation_equivariance_on_gpu():
    import torch
    L = layer_for("tiny")
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    m = ClusteredMoELayer(L)
    x = torch.from_numpy(L["x"]).cuda()
    perm = torch.randperm(x.shape[0], generator=torch.Generator().manual_seed(0)).cuda()
    y = m.forward(x).float()
    yp = m.forward(x[perm].contiguous()).float()
    torch.cuda.synchronize()
    # rows move with their tokens (summation order of the rank-r partials may differ slightly)
    assert torch.allclose(yp, y[perm], atol=2e-3, rtol=1e-3)


# ---- batches large enough for the tiled router kernel (T >= 1024), on odd router shapes ---------------
@pytest.mark.parametrize("kw", [
    dict(T=1100, d=96, d_ff=64, E=36, G=12, r=0, k=2),      # more than eight clusters, K = 3
    dict(T=1500, d=160, d_ff=64, E=10, G=2, r=0, k=3),      # K = 5: a ragged group of expert rows
    dict(T=1027, d=1056, d_ff=32, E=8, G=8, r=0, k=1),      # d not a multiple of 256, one expert per cluster
    dict(T=2048, d=2304, d_ff=32, E=64, G=2, r=0, k=8),     # prototypes staged in several chunks, K = 32
    dict(T=1024, d=4096, d_ff=32, E=4, G=2, r=0, k=2),      # two clusters, rows of 16 KB: staged in two pieces
], ids=["G12", "K5", "d1056", "d2304_K32", "G2_d4096"])
def test_router_tile_kernel_shapes(kw):
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    s = inputs.small_shape(**kw)
    L = inputs.make_layer(s, 17)
    rng = np.random.default_rng(1)
    L["b_c"] = (rng.standard_normal(s.G) * 0.2).astype(np.float32)
    L["b_e"] = (rng.standard_normal((s.G, s.K)) * 0.2).astype(np.float32)
    m = ClusteredMoELayer(L, options=dict(router_fp32=1))      # the CUDA-core kernels, also for these large batches
    x = torch.from_numpy(L["x"]).cuda()
    cid, eid, gates = m.route(x)
    torch.cuda.synchronize()
    check_routes(s, ref.Layer(L).route(L["x"]), cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), layer=L, x=L["x"])


@pytest.mark.parametrize("kw", [
    dict(T=1100, d=128, d_ff=64, E=36, G=12, r=0, k=2),     # 48 router rows -> 96 MMA columns
    dict(T=1500, d=256, d_ff=64, E=10, G=2, r=0, k=3),      # K = 5
    dict(T=1027, d=1024, d_ff=32, E=8, G=8, r=0, k=1),      # ragged last tile of 128 tokens
    dict(T=1300, d=256, d_ff=64, E=128, G=16, r=0, k=2),    # 144 router rows: two MMAs of 144 columns per step
    dict(T=1100, d=384, d_ff=64, E=144, G=16, r=0, k=3),    # 160 router rows, K = 9: the widest router the ring has room for
], ids=["G12", "K5", "ragged", "rows144", "rows160"])
def test_router_tensor_core_shapes(kw):
    """Large batches are routed on the tensor cores from split fp16 router matrices: same routes as the
    oracle outside the near-tie band, gates to 1e-5."""
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    s = inputs.small_shape(**kw)
    L = inputs.make_layer(s, 18)
    rng = np.random.default_rng(2)
    L["b_c"] = (rng.standard_normal(s.G) * 0.2).astype(np.float32)
    L["b_e"] = (rng.standard_normal((s.G, s.K)) * 0.2).astype(np.float32)
    m = ClusteredMoELayer(L)
    x = torch.from_numpy(L["x"]).cuda()
    cid, eid, gates = m.route(x)
    torch.cuda.synchronize()
    assert m.status() == 0
    check_routes(s, ref.Layer(L).route(L["x"]), cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), layer=L, x=L["x"])


def test_route_does_not_depend_on_the_batch():
    """With the fp32 CUDA-core router kernels (the router_fp32 option keeps large batches off the tensor-core
    router) a token's route is bit-identical whether it arrives in a large batch (tiled kernel) or in a
    small one (per-token kernel): both sum every dot product in the same order."""
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    L = layer_for("bert")
    m = ClusteredMoELayer(L, options=dict(router_fp32=1))
    x = torch.from_numpy(L["x"]).cuda()
    big = [t.clone() for t in m.route(x)]
    small = m.route(x[1000:1300].contiguous())
    torch.cuda.synchronize()
    for b, s_ in zip(big, small):
        assert torch.equal(b[1000:1300], s_)


# ---- shapes that take the tensor-core path (d, d_ff multiples of 128, T_max > 128) ----------------
@pytest.mark.parametrize("T", [129, 200, 640, 1111])
def test_tensor_path_ragged(T):
    s = inputs.small_shape(T=T, d=128, d_ff=256, E=8, G=2, r=16, k=2)
    L = inputs.make_layer(s, 12)
    got = full_check(L, L["x"])
    assert got["module"].info.path == 1


@pytest.mark.parametrize("kw", [
    dict(d=128, d_ff=384, E=8, G=2, r=0, k=2),
    dict(d=256, d_ff=128, E=6, G=3, r=8, k=1),
    dict(d=384, d_ff=256, E=16, G=2, r=32, k=2),     # K = 8, down tile 128 wide
    dict(d=256, d_ff=512, E=4, G=4, r=4, k=1),       # one expert per cluster
    dict(d=512, d_ff=256, E=12, G=3, r=16, k=2),     # down tile 256 wide
], ids=["r0", "r8k1", "K8r32", "K1r4", "bn256"])
def test_tensor_path_variants(kw):
    s = inputs.small_shape(T=700, **kw)
    L = inputs.make_layer(s, 13)
    # K r > 64: kept on the path with the rank-r terms in its epilogue (clusters not split into parts)
    whole = s.E // s.G * s.r > 64
    got = full_check(L, L["x"], options=dict(force_path=3) if whole else None)
    assert got["module"].info.path == 1
    if whole:
        assert got["module"].info.T_pad_max < 2 * 700


def test_tensor_path_empty_cluster():
    s = inputs.small_shape(T=400, d=128, d_ff=256, E=12, G=3, r=16, k=2)
    L = inputs.make_layer(s, 14)
    L["b_c"] = np.array([0.0, -50.0, 0.0], np.float32)
    got = full_check(L, L["x"])
    assert got["module"].info.path == 1 and not np.any(got["cid"] == 1)


# The up kernel has two tile widths: 256 columns (one accumulator updated in place for the second
# expert) where d_ff allows, else 128 columns (two accumulators).  The up_tile option keeps the narrow one.
@pytest.mark.parametrize("kw", [
    dict(d=128, d_ff=768, E=8, G=2, r=16, k=2),      # three N tiles: a unit of three
    dict(d=256, d_ff=1024, E=8, G=2, r=16, k=2),     # several units per row tile
    dict(d=128, d_ff=512, E=8, G=2, r=0, k=2),       # no residuals
    dict(d=128, d_ff=512, E=8, G=2, r=8, k=1),       # one kept expert: no second pass
    dict(d=128, d_ff=256, E=16, G=2, r=8, k=2),      # K = 8; one N tile per row tile: S rows written directly
    dict(d=128, d_ff=256, E=8, G=2, r=4, k=2),       # direct rows, r = 4
    dict(d=128, d_ff=256, E=4, G=2, r=32, k=2),      # direct rows, r = 32 (K = 2)
    dict(d=128, d_ff=256, E=8, G=2, r=16, k=1),      # direct rows, one kept expert
], ids=["nt3", "units", "r0", "k1", "K8r8", "direct_r4", "direct_r32", "direct_k1"])
@pytest.mark.parametrize("tile", ["256", "128"])
def test_up_kernel_tile_widths(kw, tile):
    s = inputs.small_shape(T=1500, **kw)
    L = inputs.make_layer(s, 21)
    got = full_check(L, L["x"], options=dict(up_tile=int(tile)))
    assert got["module"].info.path == 1


def test_bert_with_the_narrow_up_kernel():
    L = layer_for("bert")
    full_check(L, L["x"], options=dict(up_tile=128))


@pytest.mark.parametrize("T,kw", [
    (129, dict(d=128, d_ff=256, E=8, G=2, r=16, k=2)),        # ragged: most rows of the last tiles are padding
    (1111, dict(d=256, d_ff=256, E=6, G=3, r=8, k=1)),
    (1500, dict(d=384, d_ff=512, E=16, G=2, r=4, k=2)),       # K = 8, r = 4
], ids=["ragged", "k1", "K8r4"])
def test_rows_gathered_by_the_projection_kernel(T, kw):
    # option row_gather: the kernel of t = x U1 reads x by TMA row gather and writes the permuted copy itself
    s = inputs.small_shape(T=T, **kw)
    L = inputs.make_layer(s, 31)
    got = full_check(L, L["x"], options=dict(row_gather=1))
    assert got["module"].info.path == 1


def test_bert_with_gathered_rows():
    L = layer_for("bert")
    full_check(L, L["x"], options=dict(row_gather=1))


# ---- shapes that take the weight-streaming path (T_max <= 128, d and d_ff multiples of 128) ---------
@pytest.mark.parametrize("kw", [
    dict(T=1, d=128, d_ff=128, E=8, G=2, r=4, k=2),
    dict(T=5, d=256, d_ff=384, E=8, G=2, r=16, k=2),
    dict(T=64, d=128, d_ff=256, E=16, G=2, r=32, k=3),      # K = 8, odd k, largest rank
    dict(T=100, d=256, d_ff=128, E=4, G=1, r=8, k=2),       # one cluster: two token segments (64 + 36)
    dict(T=128, d=384, d_ff=640, E=6, G=3, r=0, k=2),       # no residual, ragged K split
    dict(T=77, d=128, d_ff=256, E=5, G=5, r=4, k=1),        # one expert per cluster
], ids=["T1", "T5", "K8k3r32", "G1_two_segments", "r0", "K1"])
def test_stream_path_variants(kw):
    s = inputs.small_shape(**kw)
    L = inputs.make_layer(s, 21)
    got = full_check(L, L["x"])
    assert got["module"].info.path == 2


def test_stream_path_empty_cluster_and_reuse():
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    s = inputs.small_shape(T=90, d=128, d_ff=256, E=12, G=3, r=16, k=2)
    L = inputs.make_layer(s, 22)
    L["b_c"] = np.array([0.0, -50.0, 0.0], np.float32)
    got = full_check(L, L["x"])
    assert got["module"].info.path == 2 and not np.any(got["cid"] == 1)
    m = ClusteredMoELayer(L, T_max=128)
    o = ref.Layer(L)
    for T in (128, 3, 40):                                  # the same handle, different batch sizes
        x_np = inputs.make_tokens(s, T, seed=T)
        x = torch.from_numpy(x_np).cuda()
        cid, eid, gates = m.route(x)
        y = m.forward(x)
        torch.cuda.synchronize()
        compare(L, o, x_np, cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), y.float().cpu().numpy())
    assert m.status() == 0


@pytest.mark.parametrize("name", ["bert", "decode"])
def test_forward_is_repeatable(name):
    """Twenty forwards of the same batch on one handle agree with the first one up to the summation order of the
    fp32 atomics (rank-r partial sums, K ranges): hand-overs between the kernels' roles that lost an update or read
    a buffer early would show up as a run that differs."""
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    L = layer_for(name)
    m = ClusteredMoELayer(L)
    x = torch.from_numpy(L["x"]).cuda()
    first = m.forward(x).float().clone()
    scale = float(first.abs().max())
    for _ in range(20):
        y = m.forward(x).float()
        assert float((y - first).abs().max()) <= 2e-3 * scale
    torch.cuda.synchronize()
    assert m.status() == 0


# ---- host-buffer entry point: chunked copies overlapped with the kernels ---------------------------------
@pytest.mark.parametrize("T", [700, 5000, 9000])
def test_forward_host_equals_forward(T):
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    s = inputs.small_shape(T=T, d=128, d_ff=256, E=8, G=2, r=16, k=2)
    L = inputs.make_layer(s, 31)
    m = ClusteredMoELayer(L)
    xh = torch.from_numpy(L["x"]).pin_memory()
    y_dev = m.forward(xh.cuda())
    yh = torch.empty_like(xh).pin_memory()
    m.forward_host(xh, yh)
    torch.cuda.synchronize()
    assert m.status() == 0
    a, b = y_dev.float().cpu().numpy(), yh.float().numpy()
    # the same kernels on chunks of the batch: equal up to the order of the fp32 atomics (and, for a last
    # chunk below 1024 tokens, the fp32 router instead of the split-fp16 one on near-ties)
    bad = np.abs(a - b) > 2e-3 * np.abs(a).max() + 1e-3
    assert bad.any(axis=1).mean() <= 0.002
    # and against the oracle
    # and against the oracle (rows of tokens whose near-tie a chunk's router may have settled the other way are left out)
    o = ref.Layer(L)
    r = o.route(L["x"])
    cid, eid, gates = m.route(xh.cuda())
    decided, _, _ = check_routes(s, r, cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), layer=L, x=L["x"])
    idx = np.arange(0, T, 7, dtype=np.int32)
    idx = idx[decided[idx]]
    check_y(b[idx], o.forward(L["x"], idx))
    m.close()


def test_forward_host_small_batch_on_the_streaming_path():
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    s = inputs.small_shape(T=48, d=256, d_ff=512, E=8, G=2, r=8, k=2)
    L = inputs.make_layer(s, 32)
    m = ClusteredMoELayer(L)
    assert m.info.path == 2
    xh = torch.from_numpy(L["x"]).pin_memory()
    yh = m.forward_host(xh)
    y_dev = m.forward(xh.cuda())
    torch.cuda.synchronize()
    assert m.status() == 0
    assert np.abs(yh.float().numpy() - y_dev.float().cpu().numpy()).max() <= 2e-3 * np.abs(y_dev.float().cpu().numpy()).max() + 1e-3
    m.close()


def test_headline_shape_at_another_batch_size():
    """The headline shape with a batch that does not fill whole-row work units evenly (partial units, fp32
    reductions into s and the expansion kernel instead of the direct rows)."""
    s = inputs.small_shape(T=20000, d=1024, d_ff=4096, E=32, G=8, r=16, k=2)
    L = inputs.make_layer(s, 5)
    got = full_check(L, L["x"])
    assert got["module"].info.path == 1


# ---- layers in which the rank-r residual terms dominate (Eq. 7) ---------------------------------------------
# In the workloads the residual moves h and y by a few percent, so a partial mistake in it (a neighbouring
# scale group, one factor's scale, a wrong block of the expanded rank index) could hide inside the tolerance.
# Here the bases are zero, or a quarter of their size beside factors twelve times larger, on every path that
# evaluates the residual.
_RESID_CASES = [
    # generic CUDA-core path (d, d_ff not multiples of 128)
    ("generic_r4_k2", dict(T=200, d=96, d_ff=224, E=8, G=2, r=4, k=2), None),
    ("generic_r32_k3", dict(T=200, d=96, d_ff=224, E=16, G=2, r=32, k=3), None),
    # first tensor-core path: K * r > 64, rank-r terms in the epilogue
    ("tc1_K8_r32", dict(T=700, d=384, d_ff=256, E=16, G=2, r=32, k=2), dict(force_path=3)),
    ("tc1_K8_r16_k1", dict(T=700, d=256, d_ff=384, E=16, G=2, r=16, k=1), dict(force_path=3)),
    # the same shapes as halves / quarters of the clusters on the pair path
    ("parts_K8_r32", dict(T=700, d=384, d_ff=256, E=16, G=2, r=32, k=2), None),
    ("parts_K8_r16_k1", dict(T=700, d=256, d_ff=384, E=16, G=2, r=16, k=1), None),
    # pair path, 256-column up tiles: several units per row tile, whole-row units (direct rows), both k
    ("pair_wide_units", dict(T=1500, d=256, d_ff=1024, E=8, G=2, r=16, k=2), None),
    ("pair_wide_direct_r4", dict(T=1500, d=128, d_ff=256, E=8, G=2, r=4, k=2), None),
    ("pair_wide_direct_r8_K8", dict(T=1500, d=128, d_ff=256, E=16, G=2, r=8, k=2), None),
    ("pair_wide_direct_r32", dict(T=1500, d=128, d_ff=256, E=4, G=2, r=32, k=2), None),
    ("pair_wide_k1", dict(T=1500, d=128, d_ff=512, E=8, G=2, r=8, k=1), None),
    # pair path, 128-column up tiles
    ("pair_narrow_r16", dict(T=1500, d=128, d_ff=768, E=8, G=2, r=16, k=2), dict(up_tile=128)),
    ("pair_narrow_dff384", dict(T=700, d=256, d_ff=384, E=8, G=2, r=8, k=2), None),
    # weight-streaming path
    ("stream_r4", dict(T=64, d=128, d_ff=256, E=8, G=2, r=4, k=2), None),
    ("stream_r16_k1", dict(T=100, d=256, d_ff=128, E=4, G=1, r=16, k=1), None),
    ("stream_r32_k3", dict(T=64, d=128, d_ff=256, E=16, G=2, r=32, k=3), None),
]


@pytest.mark.parametrize("mode", ["zero_bases", "large_factors"])
@pytest.mark.parametrize("name,kw,options", _RESID_CASES, ids=[c[0] for c in _RESID_CASES])
def test_residual_dominated_layers(name, kw, options, mode):
    s = inputs.small_shape(**kw)
    if mode == "zero_bases":
        L = inputs.make_layer(s, 61, base_scale=0.0, factor_std=0.2)
    else:
        L = inputs.make_layer(s, 62, base_scale=0.25, factor_std=0.25)
    # the residual really dominates: U V is several times B
    o = ref.Layer(L)
    W = o.weight(0, 1).astype(np.float64)
    Bpart = L["B1"][0].astype(np.float64)
    assert (W - Bpart).std() > 2.0 * Bpart.std()
    full_check(L, L["x"], options=options)


# ---- canaries around the arena and the outputs; scratch not assumed to start at zero ----------------------
@pytest.mark.parametrize("kw", [
    dict(d=96, d_ff=224, E=8, G=2, r=4, k=2),          # generic path
    dict(d=384, d_ff=256, E=16, G=2, r=32, k=2),       # first tensor-core path
    dict(d=256, d_ff=256, E=16, G=2, r=16, k=2),       # pair path, clusters as halves (virtual tokens)
    dict(d=128, d_ff=256, E=8, G=2, r=16, k=2),        # pair path, wide tiles
    dict(d=256, d_ff=384, E=8, G=2, r=8, k=2),         # pair path, narrow tiles
], ids=["generic", "tc1", "pair_halves", "pair_wide", "pair_narrow"])
@pytest.mark.parametrize("T", [1, 127, 129, 257, 1500])
def test_nothing_is_written_outside_the_arena_or_y(kw, T):
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    s = inputs.small_shape(T=1500, **kw)
    L = inputs.make_layer(s, 71)
    # arena pre-filled with 0xFF (NaN as fp16 / fp32, -1 as int32): nothing may rely on zeroed scratch
    whole = s.E // s.G * s.r > 64          # first tensor-core path: the clusters are not split into parts
    m = ClusteredMoELayer(L, T_max=1500, guard_bytes=1 << 16, fill_byte=0xFF, options=dict(force_path=3) if whole else None)
    x_np = inputs.make_tokens(s, T, seed=T)
    band = 4096
    buf = torch.full((T * s.d + 2 * band,), float("nan"), dtype=torch.float16, device="cuda")
    y = buf[band:band + T * s.d].view(T, s.d)
    x = torch.from_numpy(x_np).cuda()
    cid, eid, gates = m.route(x)
    m.forward(x, out=y)
    torch.cuda.synchronize()
    assert m.status() == 0
    assert m.guards_intact(), "bytes around the arena were overwritten"
    assert bool(torch.isnan(buf[:band]).all()) and bool(torch.isnan(buf[band + T * s.d:]).all()), "bytes around y were overwritten"
    assert bool(torch.isfinite(y).all())
    compare(L, ref.Layer(L), x_np, cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), y.float().cpu().numpy())
    m.close()


@pytest.mark.parametrize("T", [1, 17, 64, 128])
def test_nothing_is_written_outside_the_arena_or_y_streaming(T):
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    s = inputs.small_shape(T=128, d=256, d_ff=384, E=8, G=2, r=16, k=2)
    L = inputs.make_layer(s, 72)
    m = ClusteredMoELayer(L, T_max=128, guard_bytes=1 << 16, fill_byte=0xFF)
    assert m.info.path == 2
    x_np = inputs.make_tokens(s, T, seed=T)
    band = 4096
    buf = torch.full((T * s.d + 2 * band,), float("nan"), dtype=torch.float16, device="cuda")
    y = buf[band:band + T * s.d].view(T, s.d)
    x = torch.from_numpy(x_np).cuda()
    cid, eid, gates = m.route(x)
    m.forward(x, out=y)
    torch.cuda.synchronize()
    assert m.status() == 0 and m.guards_intact()
    assert bool(torch.isnan(buf[:band]).all()) and bool(torch.isnan(buf[band + T * s.d:]).all())
    compare(L, ref.Layer(L), x_np, cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), y.float().cpu().numpy())
    m.close()


# ---- the bounded waits' error path ---------------------------------------------------------------------------
def test_wait_timeout_is_reported_once_and_the_handle_stays_usable():
    """A wait that runs into its cycle limit (a barrier nothing arrives on, a limit of about a millisecond) sets the
    status word and the kernel returns normally: cmoe_status says CMOE_ERR_TIMEOUT once, then CMOE_OK, and the next
    forward on the same handle is right."""
    import torch
    from paper_2510_02345_b200 import binding
    L = layer_for("tiny")
    m = binding.ClusteredMoELayer(L)
    x = torch.from_numpy(L["x"]).cuda()
    m.forward(x)
    assert m.status() == 0
    binding.cmoe_selftest_wait_timeout(m.handle, 2_000_000, torch.cuda.current_stream().cuda_stream)
    assert m.status() == -6
    assert m.status() == 0
    cid, eid, gates = m.route(x)
    y = m.forward(x)
    torch.cuda.synchronize()
    assert m.status() == 0
    compare(L, ref.Layer(L), L["x"], cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), y.float().cpu().numpy())
    with pytest.raises(binding.CmoeError):
        binding.cmoe_selftest_wait_timeout(m.handle, 0, 0)
    m.close()


# ---- routing by-products (Eq. 5, load CoV) -------------------------------------------------------------------
@pytest.mark.parametrize("name", ["tiny", "bert", "skew", "decode"])
def test_expert_stats_match_the_oracle(name):
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    L = layer_for(name)
    s = L["shape"]
    m = ClusteredMoELayer(L)
    x = torch.from_numpy(L["x"]).cuda()
    mu0 = np.random.default_rng(5).standard_normal((s.E, s.d)).astype(np.float32)
    mu = torch.from_numpy(mu0.copy()).cuda()
    loads, xbar, cov = m.expert_stats(x, mu=mu, beta=0.05)
    torch.cuda.synchronize()
    o = ref.Layer(L)
    mu_ref = mu0.copy()
    loads_ref, xbar_ref, cov_ref = o.expert_stats(L["x"], mu=mu_ref, beta=0.05)
    r = o.route(L["x"])
    cid, eid, gates = m.route(x)
    decided, ties, _ = check_routes(s, r, cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy(), layer=L, x=L["x"])
    n_band = int((~decided).sum())
    got = loads.cpu().numpy()
    assert got.sum() == s.k * s.T
    # integer counts: equal, up to the tokens inside the near-tie band (each may move one unit between two experts per slot)
    assert np.abs(got - loads_ref).sum() <= 2 * s.k * n_band
    if n_band == 0:
        assert np.array_equal(got, loads_ref)
        assert np.allclose(xbar.cpu().numpy(), xbar_ref, atol=2e-5, rtol=1e-5)
        assert np.allclose(mu.cpu().numpy(), mu_ref, atol=2e-5, rtol=1e-5)
        assert abs(float(cov) - cov_ref) < 1e-6
    else:
        bound = 4.0 * n_band / max(1, loads_ref.min())          # a few banded tokens move a mean by at most this much
        assert np.abs(xbar.cpu().numpy() - xbar_ref).max() <= 8.0 * bound + 2e-5
        assert abs(float(cov) - cov_ref) < 1e-3
    m.close()


def test_expert_stats_empty_batch_and_untouched_centroids():
    import torch
    from paper_2510_02345_b200.binding import ClusteredMoELayer
    s = inputs.small_shape(T=150, d=64, d_ff=96, E=9, G=3, r=4, k=2)
    L = inputs.make_layer(s, 6)
    L["b_c"] = np.array([0.0, -50.0, 0.0], np.float32)        # cluster 1 never wins: its experts get no tokens
    m = ClusteredMoELayer(L)
    x = torch.from_numpy(L["x"]).cuda()
    mu0 = torch.ones((s.E, s.d), dtype=torch.float32, device="cuda")
    mu = mu0.clone()
    loads, xbar, cov = m.expert_stats(x, mu=mu, beta=0.5)
    torch.cuda.synchronize()
    assert int(loads[3:6].sum()) == 0 and bool((mu[3:6] == 1).all()) and not bool(xbar[3:6].any())
    assert int(loads.sum()) == s.k * s.T
    loads0, xbar0, cov0 = m.expert_stats(x[:0], mu=mu, beta=0.5)
    torch.cuda.synchronize()
    assert int(loads0.sum()) == 0 and not bool(xbar0.any()) and float(cov0) == 0.0
    m.close()


# ---- variants of the same path: bfloat16 bases, and the headline shape at other ranks / k / expert counts ------
@pytest.mark.parametrize("kw", [
    dict(T=200, d=96, d_ff=224, E=8, G=2, r=4, k=2),          # generic path
    dict(T=1500, d=256, d_ff=1024, E=8, G=2, r=16, k=2),      # pair path
    dict(T=64, d=256, d_ff=384, E=8, G=2, r=8, k=2),          # weight-streaming path
], ids=["generic", "pair", "stream"])
def test_bf16_bases(kw):
    s = inputs.small_shape(**kw)
    L = inputs.make_layer(s, 81, base_dtype="bf16")
    full_check(L, L["x"])


@pytest.mark.parametrize("kw", [
    dict(r=4, k=2, E=32, G=8),
    dict(r=8, k=1, E=32, G=8),
    dict(r=32, k=2, E=16, G=8),       # K = 2: the widest rank the pair path takes
    dict(r=16, k=2, E=64, G=16),      # K = 4 with sixteen clusters
    dict(r=8, k=2, E=64, G=8),        # K = 8
], ids=["r4", "r8_k1", "r32_K2", "G16", "K8_r8"])
def test_headline_shape_variants(kw):
    """T = 16384, d = 1024, d_ff = 4096 with other ranks, k and expert counts, all on the pair path; every row."""
    s = inputs.small_shape(T=16384, d=1024, d_ff=4096, **kw)
    L = inputs.make_layer(s, 7)
    got = full_check(L, L["x"])
    assert got["module"].info.path == 1


_wide_layer = {}


def _wide_clusters_layer():
    """d = 2048, d_ff = 8192, K = 8, r = 32 (K r = 256; 537 MB of bases): large enough for the pieces to win."""
    if not _wide_layer:
        s = inputs.small_shape(T=256, d=2048, d_ff=8192, E=64, G=8, r=32, k=2)
        _wide_layer["L"] = inputs.make_layer(s, 27)
    return _wide_layer["L"]


@pytest.mark.parametrize("T,T_max", [(129, 129), (200, 256), (256, 256), (128, 256), (50, 200)])
def test_wide_clusters_on_few_tokens_stream_in_pieces(T, T_max):
    """K r > 64 with 128 < T_max <= 384 on a layer with enough weights: the call's tokens go through the weight-streaming
    kernels in consecutive pieces of 128 tokens (splitting the clusters would run 4 G row tiles that are mostly padding).
    Every row against the oracle; routes and expert loads of the whole call."""
    import torch
    L = _wide_clusters_layer()
    s = L["shape"]
    x = L["x"][:T]
    got = full_check(L, x, T_max=T_max)
    m = got["module"]
    assert m.info.path == 2 and m.info.T_pad_max < 2 * 128 + 8 * 16
    loads, _, _ = m.expert_stats(torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    want = np.bincount(ref.Layer(L).route(x)["expert_slot"].reshape(-1), minlength=s.E)
    assert int(loads.sum()) == s.k * T and np.abs(loads.cpu().numpy() - want).sum() <= 8


@pytest.mark.parametrize("T,kw", [
    (385, dict(d=2048, d_ff=8192, E=64, G=8, r=32, k=2)),     # past the limit of the pieces
    (300, dict(d=256, d_ff=512, E=16, G=2, r=32, k=2)),       # a small layer: the quarters are estimated faster
], ids=["T385", "small_layer"])
def test_wide_clusters_beyond_the_streamed_pieces(T, kw):
    """Where the pieces would not pay (more than 384 tokens, or a layer with few weights) the clusters run as
    quarters on the pair path; sampled rows."""
    if kw["d"] == 2048:
        L = dict(_wide_clusters_layer())
        s = inputs.small_shape(T=T, **kw)
        L["shape"] = s
        L["x"] = inputs.make_tokens(s, T, seed=5)
    else:
        L = inputs.make_layer(inputs.small_shape(T=T, **kw), 27)
    got = full_check(L, L["x"], sample=128)
    assert got["module"].info.path == 1 and got["module"].info.T_pad_max >= 4 * T


def test_decode_shaped_layer_on_a_large_batch():
    """The decode-shaped layer (K = 8, r = 32: K r = 256) on a prefill-sized batch: quarters of two experts on the pair
    path; sampled rows."""
    s = inputs.small_shape(T=2048, d=4096, d_ff=14336, E=64, G=8, r=32, k=2)
    L = inputs.make_layer(s, 9)
    got = full_check(L, L["x"], sample=256)
    assert got["module"].info.path == 1


@pytest.mark.parametrize("T,kw", [
    (1027, dict(d=128, d_ff=256, E=8, G=2, r=16, k=2)),        # ragged last router tile
    (4096, dict(d=768, d_ff=3072, E=16, G=4, r=16, k=2)),      # the bert shape
    (3000, dict(d=256, d_ff=512, E=12, G=3, r=8, k=1)),        # one kept expert; an empty cluster (bias below)
    (2500, dict(d=256, d_ff=256, E=16, G=2, r=16, k=2)),       # expert halves: virtual tokens share their token's row
], ids=["ragged", "bert", "empty_cluster", "halves"])
def test_rows_moved_by_the_scatter_blocks(T, kw):
    """cmoe_options.move_in_scatter: the blocks that place the tokens of a router tile also move their rows (one
    launch less).  Every row against the oracle."""
    s = inputs.small_shape(T=T, **kw)
    L = inputs.make_layer(s, 23)
    if s.G == 3:
        L["b_c"] = np.array([0.0, -50.0, 0.0], np.float32)
    plain = run_gpu(L, L["x"])["module"].info.launches_forward
    got = full_check(L, L["x"], options=dict(move_in_scatter=1))
    assert got["module"].info.path == 1
    assert got["module"].info.launches_forward == plain - 1


def test_many_experts_beyond_the_pair_path():
    """E = 128 in G = 16 clusters with r = 16 (K r = 128 > 64, the expanded rank index of the pair path holds 64): the
    clusters are handled as two halves of four experts on the pair path; sampled rows."""
    s = inputs.small_shape(T=4096, d=1024, d_ff=4096, E=128, G=16, r=16, k=2)
    L = inputs.make_layer(s, 8)
    got = full_check(L, L["x"], sample=512)
    assert got["module"].info.path == 1


@pytest.mark.parametrize("T,kw", [
    (700, dict(d=256, d_ff=256, E=16, G=2, r=16, k=2)),        # K = 8, r = 16: halves of four experts
    (1500, dict(d=128, d_ff=512, E=8, G=2, r=32, k=2)),        # K = 4, r = 32: halves of two experts, both kept or one each
    (1111, dict(d=256, d_ff=256, E=32, G=2, r=8, k=1)),        # K = 16, r = 8, one kept expert: one half has none
    (129, dict(d=128, d_ff=256, E=24, G=3, r=16, k=2)),        # ragged, mostly padding rows
    (2048, dict(d=256, d_ff=512, E=32, G=4, r=16, k=3)),       # k = 3 of K = 8: generic fallback of the pair path? (k <= 2 only)
    (1200, dict(d=128, d_ff=256, E=16, G=2, r=32, k=2)),       # K = 8, r = 32: quarters of two experts
    (900, dict(d=256, d_ff=512, E=32, G=2, r=16, k=2)),        # K = 16, r = 16: quarters of four experts
    (1300, dict(d=128, d_ff=512, E=24, G=3, r=32, k=1)),       # K = 8, r = 32, one kept expert: three quarters have none
    (131, dict(d=128, d_ff=256, E=16, G=2, r=32, k=2)),        # quarters, ragged, mostly padding rows
], ids=["K8r16", "K4r32", "K16r8k1", "ragged", "k3", "K8r32", "K16r16", "K8r32k1", "quarters_ragged"])
def test_expert_halves(T, kw):
    """K r > 64: every cluster as two (else four) virtual clusters of K / 2 (K / 4) experts sharing its base, as many
    virtual tokens per token (its kept experts of that part, the other slots at gate zero; no row for a part without
    any), outputs summed.  Every row against the oracle."""
    s = inputs.small_shape(T=T, **kw)
    L = inputs.make_layer(s, 17)
    got = full_check(L, L["x"])
    if kw["k"] <= 2:
        assert got["module"].info.path == 1
        assert got["module"].info.T_pad_max >= 2 * T            # two virtual tokens per token


def test_expert_halves_report_the_tokens_own_routes_and_loads():
    """cmoe_route and cmoe_expert_stats of a layer that works on expert halves: the token's k experts among all K
    of its cluster (full_check compares them with the oracle), every token counted k times."""
    import torch
    s = inputs.small_shape(T=900, d=128, d_ff=256, E=16, G=2, r=16, k=2)
    L = inputs.make_layer(s, 18)
    got = full_check(L, L["x"])
    assert got["eid"].shape == (s.T, s.k) and got["eid"].max() >= s.E // 2
    m = got["module"]
    loads, _, _ = m.expert_stats(torch.from_numpy(L["x"]).cuda())
    torch.cuda.synchronize()
    want = np.bincount(ref.Layer(L).route(L["x"])["expert_slot"].reshape(-1), minlength=s.E)
    assert int(loads.sum()) == s.k * s.T
    assert np.abs(loads.cpu().numpy() - want).sum() <= 16          # near-tie tokens only


# ---- zero residual blocks (Sec. 3.4: blocks pruned by the cosine gate) are found at create time and skipped ----
def _prune(L, which, experts, via):
    """Zero one factor of the residual block `which` (1: up, 2: down) of the listed experts: `via` = "U" or "V",
    by its codes ("q") or by its scales ("s")."""
    s = L["shape"]
    fac, how = via[0], via[1]
    name = f"{fac}{which}{how}"
    a = L[name].copy()
    per = a.size // s.E
    for e in experts:
        a[e * per:(e + 1) * per] = 0
    L[name] = a


@pytest.mark.parametrize("kw", [
    dict(T=1500, d=256, d_ff=1024, E=8, G=2, r=16, k=2),      # pair path, 256-column up tiles
    dict(T=1500, d=128, d_ff=768, E=8, G=2, r=16, k=2),       # pair path, whole-row units
    dict(T=700, d=256, d_ff=384, E=16, G=2, r=8, k=2),        # pair path, 128-column up tiles, two experts per step
    dict(T=64, d=256, d_ff=384, E=8, G=2, r=8, k=2),          # weight-streaming path
    dict(T=200, d=96, d_ff=224, E=8, G=2, r=4, k=2),          # generic path
], ids=["pair_wide", "pair_direct", "pair_narrow_r8", "stream", "generic"])
def test_zero_residual_blocks_are_skipped_and_change_nothing(kw):
    s = inputs.small_shape(**kw)
    L = inputs.make_layer(s, 91, base_scale=0.25, factor_std=0.25)      # residual-dominated: a wrongly skipped block shows
    _prune(L, 1, [0, 1], "Vq")          # up blocks of experts 0, 1: all codes of V1 zero
    _prune(L, 1, [2], "Us")             # up block of expert 2: all scales of U1 zero
    _prune(L, 2, [1, 3], "Uq")          # down blocks of experts 1, 3
    _prune(L, 2, list(range(s.K, 2 * s.K)), "Vs")      # every down block of cluster 1
    got = full_check(L, L["x"])
    assert got["module"].info.pruned_blocks == 3 + 2 + s.K
