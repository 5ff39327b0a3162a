"""Float64 oracle of the paper's JS functional-disagreement metric (test infrastructure only).

App. D.2: for every token position u, p_m(u) = softmax(logits of worker m), pbar(u) = softmax(
logits of the parameter-averaged model);
    JS(p, q)  = 1/2 KL(p || (p+q)/2) + 1/2 KL(q || (p+q)/2)
    d_JS      = sqrt(JS / ln 2)                       (normalised JS distance, in [0, 1])
    CD_JS     = mean over workers m and positions u of d_JS(p_m(u), pbar(u)).
The paper computes it in float64 in the log domain and only on the 100 tokens with the highest
probability under the averaged model, recomputed at every measurement.  It does not say what
happens to the truncated tails; the reading taken here is that both distributions are
restricted to those tokens and renormalised over them (so they stay distributions and
d_JS stays in [0, 1]).  Ties at the cut are broken towards the lower token index.
"""
from __future__ import annotations

import numpy as np


def top_tokens(avg_logits_row: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest logits of one row (= highest softmax probability), ties to the
    lower index, returned in ascending index order."""
    v = np.asarray(avg_logits_row, dtype=np.float64)
    order = np.lexsort((np.arange(v.size), -v))      # by value descending, then index ascending
    return np.sort(order[:k])


def _log_softmax(z: np.ndarray) -> np.ndarray:
    z = np.asarray(z, dtype=np.float64)
    m = z.max()
    return z - (m + np.log(np.exp(z - m).sum()))


def js_distance(logits_p: np.ndarray, logits_q: np.ndarray) -> float:
    """Normalised JS distance of softmax(logits_p) and softmax(logits_q), log domain, float64."""
    lp, lq = _log_softmax(logits_p), _log_softmax(logits_q)
    lm = np.logaddexp(lp, lq) + np.log(0.5)          # log of the mixture (p + q) / 2
    js = 0.5 * np.sum(np.exp(lp) * (lp - lm)) + 0.5 * np.sum(np.exp(lq) * (lq - lm))
    return float(np.sqrt(max(js, 0.0) / np.log(2.0)))


def cd_js(worker_logits: np.ndarray, avg_logits: np.ndarray, k: int = 100):
    """worker_logits [K, U, V], avg_logits [U, V] -> (top indices [U, k], d_js [K, U], CD_JS)."""
    wl = np.asarray(worker_logits)
    al = np.asarray(avg_logits)
    K, U, V = wl.shape
    k = min(k, V)
    idx = np.empty((U, k), dtype=np.int64)
    d = np.empty((K, U), dtype=np.float64)
    for u in range(U):
        idx[u] = top_tokens(al[u], k)
        a = al[u, idx[u]].astype(np.float64)
        for m in range(K):
            d[m, u] = js_distance(wl[m, u, idx[u]].astype(np.float64), a)
    return idx, d, float(d.mean())
