"""CPU oracle for the augmented BalanceKV of Section 4.3 -- test infrastructure only.

The paper says only that a small set of tokens whose key embeddings are strongly anti-correlated
with the rest is preserved deterministically and that the standard procedure runs on the remaining
tokens; it gives neither the measure of anti-correlation nor a threshold.  Reading taken here:
token j of an appended block is preserved when the cosine between its key and the block's mean key
is at most tau (a zero key or a zero mean counts as cosine 0), decided in double; tau is a parameter.
Preserved tokens keep weight 1 and never enter a SoftmaxBalance call; the others form an ordinary
BalanceKV stream (Algorithm 3 over Algorithm 2) in their own order.
"""
import numpy as np

from .binding import OracleParams, OracleStream, merged_estimate


def anticorrelated(K, tau) -> np.ndarray:
    """Boolean mask over the rows of K [n, d]: <k_j, kbar> <= tau ||k_j|| ||kbar||, kbar the mean row."""
    K = np.asarray(K, np.float64)
    mean = K.sum(axis=0) / K.shape[0]
    dots = K @ mean
    scale = np.sqrt((K * K).sum(axis=1) * float(mean @ mean))
    return np.where(scale > 0.0, dots <= tau * scale, 0.0 <= tau)       # a zero key or mean: cosine 0


class PreservingOracle:
    """One (sequence, KV head): preserved tokens (weight 1) beside a BalanceKV stream of the rest.
    The rest draws its coins with the layer coordinate layer0 + 1 (the slot it lives in)."""

    def __init__(self, d, t, T, tau, layer0=0, head=0, max_tokens=None, seed=0, c_override=0.0, W=0):
        self.d, self.tau = d, float(tau)
        self.rest = OracleStream(OracleParams(d=d, t=t, T=T, W=W, layer=layer0 + 1, head=head, max_tokens=max_tokens,
                                              seed=seed, c_override=c_override))
        self.kept_K, self.kept_V, self.kept_pos, self.rest_pos = [], [], [], []
        self.n = 0

    def append(self, K, V):
        K = np.asarray(K, np.float64).reshape(-1, self.d)
        V = np.asarray(V, np.float64).reshape(-1, self.d)
        m = anticorrelated(K, self.tau)
        pos = self.n + np.arange(K.shape[0])
        self.n += K.shape[0]
        self.kept_K.extend(K[m]); self.kept_V.extend(V[m]); self.kept_pos.extend(pos[m])
        if (~m).any():
            self.rest.append(K[~m], V[~m])
            self.rest_pos.extend(pos[~m])
        return m

    def force_eta(self, level, ordinal, eta):
        self.rest.force_eta(level, ordinal, eta)

    def compress(self):
        return self.rest.compress()

    def views(self):
        """[(K, V, w, stream positions)] of the preserved set and of the compressed rest."""
        n_k = len(self.kept_pos)
        keep = (np.asarray(self.kept_K, np.float64).reshape(n_k, self.d), np.asarray(self.kept_V, np.float64).reshape(n_k, self.d),
                np.ones(n_k), np.asarray(self.kept_pos, np.int64))
        Kr, Vr, w, idx = self.rest.view()
        return [keep, (Kr, Vr, w, np.asarray(self.rest_pos, np.int64)[idx])]

    def estimate(self, q):
        """Theorem 3.3's estimator over the union of both sets (numerator and denominator alike)."""
        v = self.views()
        return merged_estimate(v, v, q)
