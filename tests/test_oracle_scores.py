"""Pins for oracle/scores.py: a full sort and a library softmax, plus the special rows."""
import numpy as np
import scipy.special

from oracle.scores import scores_from_logits


def test_against_full_sort_and_library_softmax():
    rng = np.random.default_rng(1)
    z = rng.normal(size=(50, 97)) * 4
    yhat, pmax, delta = scores_from_logits(z)
    srt = np.sort(z, axis=1)
    assert np.array_equal(yhat, np.argsort(-z, axis=1, kind="stable")[:, 0])
    np.testing.assert_allclose(delta, srt[:, -1] - srt[:, -2], rtol=0, atol=1e-12)
    np.testing.assert_allclose(pmax, scipy.special.softmax(z, axis=1).max(axis=1), rtol=1e-12)


def test_excluded_column_takes_no_part():
    rng = np.random.default_rng(2)
    z = rng.normal(size=(20, 33))
    z[:, 32] = 50.0                        # the excluded id would win everywhere
    yhat, pmax, delta = scores_from_logits(z, exclude_id=32)
    y2, p2, d2 = scores_from_logits(z[:, :32])
    assert np.array_equal(yhat, y2)
    np.testing.assert_allclose(pmax, p2, rtol=1e-12)
    np.testing.assert_allclose(delta, d2, atol=1e-12)


def test_special_rows():
    V = 64
    z = np.zeros((1, V)); z[0, 17] = 60.0
    yhat, pmax, delta = scores_from_logits(z)
    assert yhat[0] == 17 and abs(pmax[0] - 1.0) < 1e-12 and delta[0] == 60.0
    z = np.full((1, V), 3.25)
    yhat, pmax, delta = scores_from_logits(z)
    assert yhat[0] == 0 and delta[0] == 0.0 and abs(pmax[0] - 1.0 / V) < 1e-15
    yhat, pmax, delta = scores_from_logits(z, exclude_id=0)
    assert yhat[0] == 1 and delta[0] == 0.0 and abs(pmax[0] - 1.0 / (V - 1)) < 1e-15
    z = np.array([[1.0, 5.0, 5.0, 2.0]])   # exact tie: lowest id, zero margin
    yhat, pmax, delta = scores_from_logits(z)
    assert yhat[0] == 1 and delta[0] == 0.0
