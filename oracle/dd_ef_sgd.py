"""DD-EF-SGD (Algorithm 1 of the paper) as a plain CPU program — TEST INFRASTRUCTURE ONLY.

The method approximates nothing on this path: Top-k is an exact selection and the rest is
element-wise arithmetic, so the oracle is the definition written out, one worker and one
statement of Algorithm 1 at a time.

    worker i :  a      = e_i + gamma * g_i                (argument of C_delta)
                Delta_i = C_delta(a)  -- the k largest-|a| entries, zero elsewhere
                e_i    = a - Delta_i
    server   :  x      = x - (1/n) * sum_i Delta_{t-tau}^i

Readings taken where the paper is silent (each is also listed in the design notes):
  * "largest" is by |a|, compared through the IEEE-754 bit pattern with the sign cleared;
    among equal magnitudes the lower index wins;
  * k = ceil(delta * d), clamped to [1, d] (the Top-k contraction lemma needs k/d >= delta);
  * Top-k is global over the flat length-d vector; the per-layer variant (`layer_offsets`)
    keeps k(delta, d_l) entries in each range [offset_l, offset_{l+1}) instead;
  * iterations are numbered from 0 and update t applies the aggregate of step t - tau iff
    t - tau >= 0 (the paper's "g_{t-tau} = e_{t-tau} = 0 if t - tau <= 0" boundary);
  * when tau changes between steps the server drains its cache exactly once, oldest first:
    at update t every cached aggregate with step id <= t - tau is applied;
  * state is fp32; each of the two arithmetic statements is one fused multiply-add; the
    n messages are summed in fp32 in worker order 0..n-1, starting from +0.
A float64 shadow of the parameters is kept beside the fp32 ones for tolerance checks.
"""
import ctypes
import math

import numpy as np

from . import _native

ABS_MASK = np.uint32(0x7FFFFFFF)


def k_from_delta(delta, d):
    """Number of kept entries for compression ratio delta (Top-k lemma: k/d >= delta)."""
    if not (0.0 < delta <= 1.0):
        raise ValueError("delta must lie in (0, 1]")
    prod = float(delta) * float(d)
    near = round(prod)
    # delta*d that is an integer up to double rounding (0.1 * 1e8) keeps that integer
    if abs(prod - near) <= 1e-6:
        k = int(near)
    else:
        k = int(math.ceil(prod))
    return max(1, min(int(d), k))


def magnitude_key(a):
    """Unsigned 31-bit key whose order is the order of |a| (+0 and -0 both map to 0)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a.view(np.uint32) & ABS_MASK


def accumulate(alpha, g, e):
    """a = e + alpha*g element-wise, one fused multiply-add per element (Algorithm 1).

    g is float32, or uint16 holding bfloat16 bit patterns (widened exactly)."""
    e = np.ascontiguousarray(e, dtype=np.float32)
    is_bf16 = g.dtype == np.uint16
    g = np.ascontiguousarray(g, dtype=np.uint16 if is_bf16 else np.float32)
    assert g.shape == e.shape and e.ndim == 1
    a = np.empty_like(e)
    _native.lib().orc_accumulate(ctypes.c_float(alpha), g.ctypes.data, int(is_bf16),
                                 e.ctypes.data, a.ctypes.data, e.size)
    return a


def topk_select(a, k):
    """Indices (ascending) of the k largest-|a| entries; equal magnitudes -> lower index.

    Definition by full sort: order all d positions by (key descending, index ascending) and
    keep the first k."""
    d = a.size
    assert 1 <= k <= d < 2 ** 32
    key = magnitude_key(a).astype(np.uint64)
    idx = np.arange(d, dtype=np.uint64)
    # one 64-bit word per position; larger word == earlier in the order
    word = (key << np.uint64(32)) | (np.uint64(0xFFFFFFFF) - idx)
    word.sort()
    top = word[d - k:]
    sel = (np.uint64(0xFFFFFFFF) - (top & np.uint64(0xFFFFFFFF))).astype(np.uint32)
    sel.sort()
    return sel


def topk_select_per_layer(a, layer_offsets, delta):
    """Per-layer variant of C_delta: the k(delta, d_l) largest-|a| entries of every range
    [layer_offsets[l], layer_offsets[l+1]), same tie rule inside a range.  Indices ascending."""
    parts = []
    for lo, hi in zip(layer_offsets[:-1], layer_offsets[1:]):
        lo, hi = int(lo), int(hi)
        parts.append(topk_select(a[lo:hi], k_from_delta(delta, hi - lo)).astype(np.uint64) + lo)
    return np.concatenate(parts).astype(np.uint32)


def compress(a, k, sel=None):
    """C_delta(a) as (indices ascending, values) and the residual a - C_delta(a).  `sel`
    overrides the Top-k choice (Random-k passes its own index set)."""
    if sel is None:
        sel = topk_select(a, k)
    vals = a[sel].copy()
    resid = a.copy()
    resid[sel] = np.float32(0.0)
    return sel, vals, resid


def aggregate(msgs, d):
    """S = sum_i Delta^i, fp32 in worker order from +0, plus a float64 shadow sum."""
    S = np.zeros(d, dtype=np.float32)
    S64 = np.zeros(d, dtype=np.float64)
    for sel, vals in msgs:           # worker order 0..n-1; indices are unique per worker
        S[sel] = S[sel] + vals
        S64[sel] = S64[sel] + vals.astype(np.float64)
    return S, S64


def apply_update(x, S, scale):
    """x <- x - scale*S, one fused multiply-add per element (Algorithm 1, server update)."""
    _native.lib().orc_apply(ctypes.c_float(-np.float32(scale)), S.ctypes.data,
                            x.ctypes.data, x.size)


class DDEFSGD:
    """State and one-iteration driver of Algorithm 1 for n workers simulated in one process.

    lr_in_compress=True is the paper's form (a = e + gamma*g, update scale 1/n);
    False moves the stepsize to the server (a = e + g, update scale gamma/n)."""

    def __init__(self, d, n, delta, tau, lr, x0=None, lr_in_compress=True, compressor="topk",
                 seed=0, layer_offsets=None):
        self.d, self.n = int(d), int(n)
        self.layer_offsets = None if layer_offsets is None else [int(v) for v in layer_offsets]
        if self.layer_offsets is not None:
            assert compressor == "topk" and self.layer_offsets[0] == 0
            assert self.layer_offsets[-1] == self.d
        self.lr = np.float32(lr)
        self.lr_in_compress = bool(lr_in_compress)
        assert compressor in ("topk", "randk")
        self.compressor, self.seed = compressor, int(seed)
        self.delta, self.tau = float(delta), int(tau)
        self.k = self._k_of(delta)
        self.x = (np.zeros(d, np.float32) if x0 is None
                  else np.array(x0, dtype=np.float32, copy=True))
        self.x64 = self.x.astype(np.float64)
        self.e = np.zeros((n, d), dtype=np.float32)      # e_0^i = 0
        self.cache = []                                   # server cache: (step, S, S64), FIFO
        self.t = 0

    def _k_of(self, delta):
        """Entries per message: k(delta, d), or the sum of the layers' k(delta, d_l)."""
        if self.layer_offsets is None:
            return k_from_delta(delta, self.d)
        return sum(k_from_delta(delta, hi - lo)
                   for lo, hi in zip(self.layer_offsets[:-1], self.layer_offsets[1:]))

    def set_policy(self, delta, tau):
        """New (delta, tau) from the next iteration on (Algorithm 2's broadcast)."""
        self.delta, self.tau = float(delta), int(tau)
        self.k = self._k_of(delta)

    def set_lr(self, lr):
        self.lr = np.float32(lr)

    def step(self, g):
        """One iteration t of Algorithm 1.  g: [n, d] float32 or uint16 (bfloat16 bits).

        Returns a dict with this step's messages, aggregate and the step ids applied."""
        n, d = self.n, self.d
        assert g.shape == (n, d)
        alpha = self.lr if self.lr_in_compress else np.float32(1.0)
        beta = np.float32(1.0) if self.lr_in_compress else self.lr
        msgs = []
        for i in range(n):                                # worker side
            a = accumulate(alpha, g[i], self.e[i])
            chosen = None
            if self.compressor == "randk":
                from . import random_k
                chosen = random_k.randk_select(d, self.k, self.seed, self.t, i)
            elif self.layer_offsets is not None:
                chosen = topk_select_per_layer(a, self.layer_offsets, self.delta)
            sel, vals, resid = compress(a, self.k, chosen)
            self.e[i] = resid
            msgs.append((sel, vals))
        S, S64 = aggregate(msgs, d)                       # server receives step t
        self.cache.append((self.t, S, S64))
        scale = np.float32(beta / np.float32(n))
        applied = []
        while self.cache and self.cache[0][0] <= self.t - self.tau:
            s, Ss, Ss64 = self.cache.pop(0)
            apply_update(self.x, Ss, scale)
            self.x64 -= float(scale) * Ss64
            applied.append(s)
        self.t += 1
        return {"msgs": msgs, "S": S, "S64": S64, "applied": applied, "k": self.k}

    def in_flight(self):
        """Aggregates still in the server cache (sent but not yet applied)."""
        return [(s, S) for (s, S, _) in self.cache]
