"""Oracle: per-position prediction and stability scores from a row of logits (Sec. 3.2, Eq. 1;
Algorithm 1, the score step).  TEST INFRASTRUCTURE, not a product path.

  yhat  = argmax_v z_v            (ties -> lowest id; the paper is silent)
  delta = z_(1) - z_(2)           (Eq. 1: difference of the two largest LOGITS; z_(2) is the
                                   largest value among v != yhat, so an exact tie gives 0)
  p_max = 1 / sum_v exp(z_v - z_(1))   (softmax probability of yhat, the score the benchmark
                                        configurations threshold)
With exclude_id >= 0 that column (the MASK token) takes no part in any of the three, so a
committed token is never MASK (reading; the paper is silent).

Pins: a full sort and a library softmax on random rows; one-hot-dominant and all-equal rows.
"""
import numpy as np


def scores_from_logits(z, exclude_id=-1):
    """z: [M, V] float64 -> (yhat int32 [M], p_max float64 [M], delta float64 [M])."""
    z = np.array(z, dtype=np.float64, copy=True)
    if z.ndim == 1:
        z = z[None, :]
    M, V = z.shape
    if exclude_id >= 0:
        z[:, exclude_id] = -np.inf
    yhat = np.argmax(z, axis=1)                       # first occurrence = lowest id
    z1 = z[np.arange(M), yhat]
    rest = z.copy()
    rest[np.arange(M), yhat] = -np.inf
    z2 = rest.max(axis=1)
    delta = z1 - z2
    p_max = 1.0 / np.exp(z - z1[:, None]).sum(axis=1)
    return yhat.astype(np.int32), p_max, delta
