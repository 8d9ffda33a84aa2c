"""Pins for the oracle's retrieval scoring: closed-form cosines, invariances, the selection rule."""
import math

import numpy as np

import oracle


def test_cosines_of_known_angles():
    ang = np.deg2rad([0.0, 30.0, 60.0, 90.0, 120.0, 180.0])
    E = np.stack([np.cos(ang), np.sin(ang), np.zeros_like(ang), np.zeros_like(ang)], axis=1)[None] * 3.0
    q = np.array([[2.0, 0.0, 0.0, 0.0]])
    scores, chosen = oracle.retrieval_select(E, q, k=10, threshold=0.3)
    np.testing.assert_allclose(scores[0], np.cos(ang), atol=1e-7)
    assert chosen == [[0, 1, 2]]                       # cos 60 = 0.5 passes, cos 90 = 0 does not


def test_scale_invariance_and_zero_vectors():
    rng = np.random.default_rng(1)
    E = rng.normal(size=(1, 6, 8)).astype(np.float32)
    q = rng.normal(size=(1, 8)).astype(np.float32)
    s1, c1 = oracle.retrieval_select(E, q, k=6, threshold=-1.0)
    s2, c2 = oracle.retrieval_select(E * np.array([1, 2, 4, 8, 16, 32], np.float32)[None, :, None], q * 4, k=6, threshold=-1.0)
    np.testing.assert_allclose(s1, s2, atol=1e-12)
    assert c1 == c2 and sorted(c1[0]) == list(range(6))
    E[0, 3] = 0
    s3, c3 = oracle.retrieval_select(E, q, k=6, threshold=0.0)
    assert s3[0, 3] == 0.0


def test_selection_rule_threshold_topk_ties_and_lengths():
    # scores by construction: e_i = (s_i, sqrt(1 - s_i^2)) against q = (1, 0)
    s = [0.9, 0.31, 0.3, 0.2999, 0.9, 0.5, 0.7]
    E = np.array([[x, math.sqrt(1 - x * x)] for x in s])[None]
    q = np.array([[1.0, 0.0]])
    scores, chosen = oracle.retrieval_select(E, q, k=4, threshold=0.3)
    np.testing.assert_allclose(scores[0], s, atol=1e-7)
    assert chosen == [[0, 4, 6, 5]]                    # ties: lower index first; cut at k
    _, chosen = oracle.retrieval_select(E, q, k=10, threshold=0.3)
    assert chosen[0][:4] == [0, 4, 6, 5] and set(chosen[0][4:]) <= {1, 2} and 3 not in chosen[0]
    _, chosen = oracle.retrieval_select(E, q, k=10, threshold=0.3, n_chunks=[2])
    assert chosen == [[0, 1]]                          # chunks past the request's count do not exist
    _, chosen = oracle.retrieval_select(E, q, k=3, threshold=0.95)
    assert chosen == [[]]


def test_matches_a_library_matmul_on_random_vectors():
    rng = np.random.default_rng(2)
    E = rng.normal(size=(3, 40, 32)).astype(np.float32)
    q = rng.normal(size=(3, 32)).astype(np.float32)
    scores, chosen = oracle.retrieval_select(E, q, k=5, threshold=0.1)
    En = E.astype(np.float64) / np.linalg.norm(E.astype(np.float64), axis=-1, keepdims=True)
    qn = q.astype(np.float64) / np.linalg.norm(q.astype(np.float64), axis=-1, keepdims=True)
    ref = np.einsum("bnd,bd->bn", En, qn)
    np.testing.assert_allclose(scores, ref, atol=1e-12)
    for b in range(3):
        order = np.argsort(-ref[b], kind="stable")
        assert chosen[b] == [int(i) for i in order if ref[b, i] >= 0.1][:5]
