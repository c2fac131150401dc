"""CPU oracle for the value-norm buckets of BalanceKV (Algorithm 1) -- test infrastructure only.

Algorithm 1 sends token j to the MergeAndReduce instance MR-Numerator_i of the bucket i with
2^i >= ||v_j||_2 >= 2^(i-1), keeps the running maximum v_max of the value norms, erases every
instance whose bucket lies at or below a threshold proportional to v_max, and forms the
numerator of its output ratio from the union of the surviving instances' level sets.

Readings taken here (the text leaves them open):
  * a norm that is an exact power of two satisfies the printed condition for two indices;
    the smaller one is taken, i.e. bucket i holds 2^(i-1) < ||v|| <= 2^i;
  * a zero value has no bucket and contributes nothing to the numerator: it is dropped;
  * the erase threshold is printed as eps/(2n) e^{-r^2/sqrt d} v_max in Algorithm 1 and used as
    eps/sqrt(n) v_max in the proof of Theorem 1.1; both have the form rho * v_max, so rho is a
    parameter (`erase_ratio`) and the rule is "erase bucket i when 2^i <= rho * v_max";
  * instances exist for the `n_buckets` indices i_top, i_top-1, ..., i_top-n_buckets+1 only
    (Algorithm 1 keeps O(log n) of them): a token above i_top is an error, a token below the
    lowest index is treated like a token of an erased bucket.
Bucket i's instance draws its coins with the layer coordinate layer0 + (i_top - i).
"""
import math

import numpy as np

from .binding import OracleParams, OracleStream, merged_estimate

NO_BUCKET = -(1 << 30)


def value_bucket(v) -> int:
    """The index i with 2^(i-1) < ||v||_2 <= 2^i (Algorithm 1, the bucketing step), decided on the
    squared norm in double: the smallest i with 4^i >= ||v||^2.  NO_BUCKET for v = 0."""
    ns = float(np.dot(np.asarray(v, np.float64), np.asarray(v, np.float64)))
    if ns == 0.0:
        return NO_BUCKET
    i = math.ceil(0.5 * math.log2(ns))
    while 4.0 ** i < ns:          # log2 rounding at the boundaries
        i += 1
    while 4.0 ** (i - 1) >= ns:
        i -= 1
    return i


class BucketedOracle:
    """Algorithm 1's numerator side for one (sequence, KV head): one MergeAndReduce instance per
    value-norm bucket, erasure of the small-norm buckets, union of the survivors."""

    def __init__(self, d, t, T, i_top, n_buckets, erase_ratio=0.0, layer0=0, head=0, max_tokens=None,
                 seed=0, c_override=0.0, W=0):
        self.d, self.i_top, self.n_buckets, self.rho = d, i_top, n_buckets, float(erase_ratio)
        self._mk = lambda b: OracleStream(OracleParams(d=d, t=t, T=T, W=W, layer=layer0 + b, head=head,
                                                       max_tokens=max_tokens, seed=seed, c_override=c_override))
        self.inst = {}                    # slot b -> OracleStream
        self.route = {}                   # slot b -> stream positions of the tokens it received
        self.erased = []                  # stream positions dropped (erased bucket, below range, zero value)
        self.vmax2 = 0.0
        self.n = 0

    def _is_erased(self, i) -> bool:
        # 2^i <= rho * v_max, compared on squares
        return self.rho > 0.0 and 4.0 ** i <= self.rho * self.rho * self.vmax2

    def append(self, K, V):
        K = np.asarray(K, np.float64).reshape(-1, self.d)
        V = np.asarray(V, np.float64).reshape(-1, self.d)
        for k, v in zip(K, V):
            j = self.n
            self.n += 1
            i = value_bucket(v)
            if i != NO_BUCKET and i > self.i_top:
                raise ValueError("value norm above the highest bucket")
            b = self.i_top - i
            if i != NO_BUCKET and b < self.n_buckets:
                if b not in self.inst:
                    self.inst[b], self.route[b] = self._mk(b), []
                self.inst[b].append(k[None, :], v[None, :])
                self.route[b].append(j)
            else:
                self.erased.append(j)
            self.vmax2 = max(self.vmax2, float(np.dot(v, v)))
            for bb in [bb for bb in self.inst if self._is_erased(self.i_top - bb)]:
                self.erased.extend(self.route[bb])
                del self.inst[bb], self.route[bb]

    def force_eta(self, b, level, ordinal, eta):
        self.inst[b].force_eta(level, ordinal, eta)

    def compress(self):
        return sum(s.compress() for s in self.inst.values())

    def views(self):
        """(K, V, w, stream positions) of every surviving bucket, highest norms first."""
        out = []
        for b in sorted(self.inst):
            Kb, Vb, w, idx = self.inst[b].view()
            out.append((Kb, Vb, w, np.asarray(self.route[b], np.int64)[idx]))
        return out

    def estimate(self, q, denominator_views):
        """Algorithm 1's output ratio: union of the buckets' sets above, `denominator_views` below."""
        return merged_estimate(self.views(), denominator_views, q)
