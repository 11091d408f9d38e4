"""cmoe_route_static, the routing call for callers that cannot allocate device memory (a plugin in
a host application with a frozen memory pool, a dispatcher that runs before any layer handle
exists): it must give what cmoe_route gives, call after call, although all its calls share
one fixed device array that still holds the previous call's router.  It always routes with the fp32
CUDA-core kernels: below 1024 tokens that is the very kernel cmoe_route uses (identical outputs);
from 1024 tokens on cmoe_route takes the tensor-core router, so there the static call is checked
against the CPU oracle, like every other router.

Collected last on purpose: a run that stops at the first failure has then already run everything
else."""
import numpy as np
import pytest

from paper_2510_02345_b200 import inputs

pytestmark = pytest.mark.gpu


def route_both_ways(L, x_np):
    import torch
    from paper_2510_02345_b200 import binding
    s = L["shape"]
    m = binding.ClusteredMoELayer(L, T_max=max(1, x_np.shape[0]))
    x = torch.from_numpy(x_np).cuda()
    want = [t.cpu().numpy() for t in m.route(x)]
    dev = {n: (None if L.get(n) is None else torch.from_numpy(np.ascontiguousarray(L[n], np.float32)).cuda())
           for n in ("C", "R", "b_c", "b_e")}
    T = x.shape[0]
    cid = torch.full((T,), -7, dtype=torch.int32, device="cuda")
    eid = torch.full((T, s.k), -7, dtype=torch.int32, device="cuda")
    gates = torch.full((T, s.k), -7.0, dtype=torch.float32, device="cuda")
    ptr = lambda t: None if t is None else t.data_ptr()
    binding.cmoe_route_static(s.d, s.E, s.G, s.k, ptr(dev["C"]), ptr(dev["R"]), ptr(dev["b_c"]), ptr(dev["b_e"]),
                              x.data_ptr(), T, cid.data_ptr(), eid.data_ptr(), gates.data_ptr(),
                              torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    got = [cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy()]
    m.close()
    return want, got


def test_static_route_matches_route_on_consecutive_calls():
    # call 1: biased router; call 2: a different, smaller router without biases (stale biases and
    # stale rows of the first call are still in the array); call 3: the first one again.
    L1 = inputs.make_layer(inputs.small_shape(T=300, d=128, d_ff=64, E=12, G=3, r=0, k=2), 21)
    rng = np.random.default_rng(0)
    L1["b_c"] = (rng.standard_normal(3) * 0.3).astype(np.float32)
    L1["b_e"] = (rng.standard_normal((3, 4)) * 0.3).astype(np.float32)
    L2 = inputs.make_layer(inputs.small_shape(T=77, d=64, d_ff=64, E=8, G=2, r=0, k=3), 22)
    for L in (L1, L2, L1):
        want, got = route_both_ways(L, L["x"])
        assert np.array_equal(got[0], want[0])
        assert np.array_equal(got[1], want[1])
        assert np.allclose(got[2], want[2], atol=1e-5, rtol=0)     # the parity tests' gate tolerance


def _route_static(L, x_np):
    import torch
    from paper_2510_02345_b200 import binding
    s = L["shape"]
    x = torch.from_numpy(x_np).cuda()
    dev = {n: (None if L.get(n) is None else torch.from_numpy(np.ascontiguousarray(L[n], np.float32)).cuda())
           for n in ("C", "R", "b_c", "b_e")}
    T = x.shape[0]
    cid = torch.full((T,), -7, dtype=torch.int32, device="cuda")
    eid = torch.full((T, s.k), -7, dtype=torch.int32, device="cuda")
    gates = torch.full((T, s.k), -7.0, dtype=torch.float32, device="cuda")
    ptr = lambda t: None if t is None else t.data_ptr()
    binding.cmoe_route_static(s.d, s.E, s.G, s.k, ptr(dev["C"]), ptr(dev["R"]), ptr(dev["b_c"]), ptr(dev["b_e"]),
                              x.data_ptr(), T, cid.data_ptr(), eid.data_ptr(), gates.data_ptr(),
                              torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    return cid.cpu().numpy(), eid.cpu().numpy(), gates.cpu().numpy()


@pytest.mark.parametrize("kw", [
    dict(T=1500, d=256, d_ff=64, E=12, G=3, r=0, k=2),
    dict(T=1024, d=4096, d_ff=64, E=4, G=2, r=0, k=2),      # two clusters, wide rows: the prototypes are staged in pieces
    dict(T=2100, d=1056, d_ff=32, E=36, G=12, r=0, k=3),    # more than eight clusters
], ids=["G3", "G2_d4096", "G12"])
def test_static_route_large_batches_against_the_oracle(kw):
    """Batches of 1024 tokens and more take the tiled fp32 kernel, reading the router from the fixed array: routes
    bit-exact against the oracle outside the 1e-4 band, valid inside it, gates to 1e-5; twice in a row."""
    from oracle import ref
    from parity import check_routes
    L = inputs.make_layer(inputs.small_shape(**kw), 23)
    rng = np.random.default_rng(3)
    s = L["shape"]
    L["b_c"] = (rng.standard_normal(s.G) * 0.2).astype(np.float32)
    L["b_e"] = (rng.standard_normal((s.G, s.K)) * 0.2).astype(np.float32)
    r = ref.Layer(L).route(L["x"])
    for _ in range(2):
        cid, eid, gates = _route_static(L, L["x"])
        check_routes(s, r, cid, eid, gates, layer=L, x=L["x"])


def test_static_route_rejects_what_does_not_fit():
    from paper_2510_02345_b200 import binding
    L = binding.lib()
    # (G+E)*d*4 bytes = 72*8192*4 > 2 MiB: refused before any launch, pointers never touched
    assert L.cmoe_route_static(8192, 64, 8, 2, None, None, None, None, None, 4, None, None, None, None) == -3
    assert L.cmoe_route_static(100, 8, 2, 2, None, None, None, None, None, 4, None, None, None, None) == -2
    assert L.cmoe_route_static(64, 8, 2, 2, None, None, None, None, None, 0, None, None, None, None) == 0
    assert L.cmoe_route_static(64, 8, 2, 2, None, None, None, None, None, 4, None, None, None, None) == -1
