"""Pins of the similarity oracle (Eq. 2-4) against what the mathematics fixes and an independent library routine."""
import numpy as np
import pytest

from oracle import similarity_ref as ref


def test_hand_worked_angles():
    # 60 degrees, 90 degrees, 180 degrees and a scaled copy, written out by hand
    V = np.array([[1.0, 0.0, 0.0],
                  [1.0, np.sqrt(3.0), 0.0],      # 60 degrees from row 0
                  [0.0, 0.0, 2.0],               # orthogonal to both
                  [-3.0, 0.0, 0.0],              # opposite to row 0
                  [5.0, 0.0, 0.0]])              # row 0 scaled
    S = ref.cosine_matrix(V)
    want = np.array([[1.0, 0.5, 0.0, -1.0, 1.0],
                     [0.5, 1.0, 0.0, -0.5, 0.5],
                     [0.0, 0.0, 1.0, 0.0, 0.0],
                     [-1.0, -0.5, 0.0, 1.0, -1.0],
                     [1.0, 0.5, 0.0, -1.0, 1.0]])
    np.testing.assert_allclose(S, want, atol=1e-12)


def test_against_sklearn():
    from sklearn.metrics.pairwise import cosine_similarity
    rng = np.random.default_rng(0)
    V = rng.standard_normal((12, 257))
    np.testing.assert_allclose(ref.cosine_matrix(V), cosine_similarity(V), atol=1e-12)
    # matrices are flattened expert by expert (Eq. 2: "flattening its weight matrix")
    W = rng.standard_normal((6, 9, 11))
    np.testing.assert_allclose(ref.cosine_matrix(W), cosine_similarity(W.reshape(6, -1)), atol=1e-12)


def test_invariants():
    rng = np.random.default_rng(1)
    base = rng.standard_normal((4, 300))
    V = np.concatenate([base + 0.3 * rng.standard_normal((4, 300)) for _ in range(3)])     # correlated groups
    S = ref.cosine_matrix(V)
    np.testing.assert_allclose(S, S.T, atol=1e-15)
    np.testing.assert_allclose(np.diag(S), 1.0, atol=1e-12)
    assert np.abs(S).max() <= 1.0 + 1e-12
    assert np.linalg.eigvalsh(S).min() > -1e-10                      # a Gram matrix of unit vectors
    # invariant under positive rescaling of any expert, sign flips flip the row and the column
    scale = rng.uniform(0.1, 10.0, size=12)
    np.testing.assert_allclose(ref.cosine_matrix(V * scale[:, None]), S, atol=1e-12)
    flip = np.ones(12); flip[3] = -1.0
    np.testing.assert_allclose(ref.cosine_matrix(V * flip[:, None]), S * np.outer(flip, flip), atol=1e-12)
    # members of one group are closer to each other than to the other groups
    same = S[0, 4], S[0, 8]
    other = np.abs(S[0, [1, 2, 3, 5, 6, 7]])
    assert min(same) > other.max()


def test_zero_vector_reading():
    V = np.array([[1.0, 2.0], [0.0, 0.0], [2.0, 4.0]])
    S = ref.cosine_matrix(V)
    np.testing.assert_allclose(S, [[1, 0, 1], [0, 1, 0], [1, 0, 1]], atol=1e-12)


def test_fused_score_eq4():
    rng = np.random.default_rng(2)
    W = rng.standard_normal((5, 40))
    mu = rng.standard_normal((5, 7))
    r1 = ref.fused_similarity(W, mu, 1.0)
    r0 = ref.fused_similarity(W, mu, 0.0)
    np.testing.assert_allclose(r1["S"], r1["S_param"], atol=1e-15)
    np.testing.assert_allclose(r0["S"], r0["S_task"], atol=1e-15)
    r7 = ref.fused_similarity(W, mu, 0.7)
    np.testing.assert_allclose(r7["S"], 0.7 * r1["S_param"] + 0.3 * r0["S_task"], atol=1e-15)
    # hand-worked: S_param = 0.5, S_task = -1 at alpha = 0.7 gives 0.35 - 0.3 = 0.05
    W2 = np.array([[1.0, 0.0], [1.0, np.sqrt(3.0)]])
    mu2 = np.array([[2.0], [-1.0]])
    assert ref.fused_similarity(W2, mu2, 0.7)["S"][0, 1] == pytest.approx(0.05, abs=1e-12)
    with pytest.raises(AssertionError):
        ref.fused_similarity(W, mu, 1.5)


# ---- planted mistakes: each must make one of the pins above fail ------------------------------------------------
_MUTANTS = {
    "norm_without_root": ("norm = np.sqrt((V * V).sum(axis=1))", "norm = (V * V).sum(axis=1)"),
    "one_norm_only": ("/ (norm[i] * norm[j])", "/ (norm[i] * norm[i])"),
    "alpha_swapped": ("S=alpha * S_param + (1.0 - alpha) * S_task", "S=(1.0 - alpha) * S_param + alpha * S_task"),
    "task_from_weights": ("S_task = cosine_matrix(mu)", "S_task = cosine_matrix(W)"),
    "matrices_not_flattened": ("V = np.asarray(V, dtype=np.float64).reshape(V.shape[0], -1)", "V = np.asarray(V, dtype=np.float64)[:, 0] if np.ndim(V) == 3 else np.asarray(V, dtype=np.float64)"),
    "zero_vector_gives_one": ("out[i, j] = 1.0 if i == j else 0.0", "out[i, j] = 1.0"),
}


@pytest.mark.parametrize("name", sorted(_MUTANTS))
def test_planted_mistakes_are_caught(name, monkeypatch):
    import inspect
    import types
    src = inspect.getsource(ref)
    old, new = _MUTANTS[name]
    assert src.count(old) == 1
    mutant = types.ModuleType("similarity_mutant")
    exec(compile(src.replace(old, new), "similarity_mutant", "exec"), mutant.__dict__)
    monkeypatch.setattr(ref, "cosine_matrix", mutant.cosine_matrix)
    monkeypatch.setattr(ref, "fused_similarity", mutant.fused_similarity)
    caught = 0
    for pin in (test_hand_worked_angles, test_against_sklearn, test_invariants, test_zero_vector_reading, test_fused_score_eq4):
        try:
            pin()
        except (AssertionError, ValueError, IndexError):
            caught += 1
    assert caught >= 1, f"no pin notices the planted mistake {name}"
