"""GPU parity of cmoe_expert_similarity (Eq. 2-4) against its numpy oracle.

S_param's dot products run on the tensor cores with the fp32 weights cut to tf32 (10 mantissa bits, truncation): each
product carries a relative error below 2^-9, of random sign around a common bias that the normalisation by the norms
(computed the same way) cancels, so over n >= 10^4 terms the cosine is off by far less than 1e-3: the tolerance is
2e-4 absolute on S_param and S, 2e-6 on S_task (fp32 CUDA-core dot products)."""
import numpy as np
import pytest

from oracle import similarity_ref as ref
from paper_2510_02345_b200 import inputs

pytestmark = pytest.mark.gpu

TOL_PARAM, TOL_TASK = 2e-4, 2e-6


def _run(W, mu, alpha):
    import torch
    from paper_2510_02345_b200 import binding
    out = binding.expert_similarity(None if W is None else torch.from_numpy(W).cuda(),
                                    None if mu is None else torch.from_numpy(mu).cuda(), alpha)
    torch.cuda.synchronize()
    assert int(out["status"].item()) == 0
    return {k: v.cpu().numpy() for k, v in out.items() if k != "status"}


@pytest.mark.parametrize("E,n,d", [(32, 1024 * 64, 1024), (8, 32 * 37, 64), (128, 32 * 1001, 256), (20, 4096, 48),
                                   (1, 64, 8), (17, 32 * 3, 5), (64, 768 * 768, 768)],
                         ids=["E32", "E8_short", "E128_ragged", "E20", "E1", "E17_tiny", "E64_larger_than_L2"])
def test_similarity_against_the_oracle(E, n, d):
    rng = np.random.default_rng(E * 1000 + d)
    # correlated experts: groups of four around a common matrix, as the clustering would see them
    groups = rng.standard_normal(((E + 3) // 4, n), dtype=np.float32)
    W = rng.standard_normal((E, n), dtype=np.float32)
    W *= np.float32(0.5)
    W += groups[np.arange(E) // 4]
    mu = (rng.standard_normal((E, d)) + 0.3).astype(np.float32)
    got = _run(W, mu, 0.7)
    want = ref.fused_similarity(W, mu, 0.7)
    assert np.abs(got["S_param"] - want["S_param"]).max() <= TOL_PARAM
    assert np.abs(got["S_task"] - want["S_task"]).max() <= TOL_TASK
    assert np.abs(got["S"] - want["S"]).max() <= TOL_PARAM
    assert np.array_equal(np.diag(got["S_param"]), np.ones(E, np.float32))
    # the structure the clustering relies on survives tf32: same group > other groups
    if E >= 8:
        assert got["S_param"][0, 1] > 0.5 and abs(got["S_param"][0, 4]) < 0.2


def test_dense_experts_of_the_generator_and_a_zero_expert():
    W = inputs.make_dense_experts(E=16, G=4, d_in=256, d_out=512, seed=3)
    W = np.ascontiguousarray(W, dtype=np.float32)
    W[5] = 0.0                                           # an expert of norm zero: similarity 0, diagonal 1
    got = _run(W.reshape(16, -1), None, 1.0)
    want = ref.cosine_matrix(W)
    assert set(got) == {"S_param"}
    assert np.abs(got["S_param"] - want).max() <= TOL_PARAM
    assert np.all(got["S_param"][5, np.arange(16) != 5] == 0.0) and got["S_param"][5, 5] == 1.0


def test_task_similarity_alone_and_argument_checks():
    import torch
    from paper_2510_02345_b200 import binding
    rng = np.random.default_rng(9)
    mu = rng.standard_normal((12, 100)).astype(np.float32)
    got = _run(None, mu, 0.3)
    assert set(got) == {"S_task"}
    assert np.abs(got["S_task"] - ref.cosine_matrix(mu)).max() <= TOL_TASK
    q = binding.cmoe_similarity_desc()
    q.E, q.alpha = 4, 0.5
    assert binding.lib().cmoe_expert_similarity(binding.C.byref(q), None) == -1     # neither W nor mu
    Wt = torch.zeros((4, 48), dtype=torch.float32, device="cuda")
    St = torch.zeros((4, 4), dtype=torch.float32, device="cuda")
    q.W, q.n, q.S_param = Wt.data_ptr(), 48, St.data_ptr()
    assert binding.lib().cmoe_expert_similarity(binding.C.byref(q), None) == -1     # n % 32 != 0
    q.n, q.alpha = 32, 1.5
    assert binding.lib().cmoe_expert_similarity(binding.C.byref(q), None) == -1     # alpha outside [0, 1]
    q.alpha, q.E = 0.5, 129
    assert binding.lib().cmoe_expert_similarity(binding.C.byref(q), None) == -1     # E > 128
