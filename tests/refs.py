"""Independent reference computations used to pin the CPU oracle.

Nothing here is derived from the oracle's code: ``brute_force`` is the
definition of a CTC labelling probability (sum over all alignments that
collapse to the labelling), ``PyPrefixSearch`` is a second, separately
written dictionary-of-tuples prefix beam search, ``greedy`` is best-path
decoding.
"""
from __future__ import annotations

import itertools
import math

import numpy as np


def collapse(path, blank):
    out, prev = [], None
    for c in path:
        if c != prev and c != blank:
            out.append(int(c))
        prev = c
    return tuple(out)


def brute_force(lp: np.ndarray, blank: int, keep: np.ndarray | None = None,
                best_alignment: bool = False) -> dict:
    """log P(labelling) for every labelling, by enumerating all V**T alignments.

    ``keep`` [T,V] (bool) restricts each frame to its surviving tokens.
    Probabilities are summed in float64 with math.fsum.  ``best_alignment``: the
    log-probability of the labelling's single most probable alignment instead of their sum.
    """
    T, V = lp.shape
    terms: dict = {}
    p = np.exp(lp.astype(np.float64))
    for path in itertools.product(range(V), repeat=T):
        if keep is not None and not all(keep[t, c] for t, c in enumerate(path)):
            continue
        w = 1.0
        for t, c in enumerate(path):
            w *= p[t, c]
        terms.setdefault(collapse(path, blank), []).append(w)
    total = max if best_alignment else math.fsum
    return {k: (math.log(s) if (s := total(v)) > 0 else -math.inf) for k, v in terms.items()}


def greedy(lp: np.ndarray, blank: int):
    return collapse(lp.argmax(axis=1).tolist(), blank)


def _lse(a, b):
    if a == -math.inf:
        return b
    if b == -math.inf:
        return a
    m = max(a, b)
    return m + math.log1p(math.exp(min(a, b) - m))


class PyPrefixSearch:
    """Dictionary-keyed CTC prefix beam search, optional per-frame survivor sets."""

    def __init__(self, blank: int, K: int, beam_threshold: float = 0.0, merge_max: bool = False):
        self.blank, self.K, self.beam_threshold = blank, K, beam_threshold
        self._mix = max if merge_max else _lse
        self.beam = {(): (0.0, -math.inf)}
        self.revivals = 0          # prefixes that re-entered the beam after leaving it
        self._ever = {()}
        self._prev = {()}

    def step(self, lp_row, survivors):
        nxt: dict = {}

        def add(key, which, val):
            pb, pnb = nxt.get(key, (-math.inf, -math.inf))
            nxt[key] = (self._mix(pb, val), pnb) if which == 0 else (pb, self._mix(pnb, val))

        for seq, (pb, pnb) in self.beam.items():
            tot = self._mix(pb, pnb)
            for c in survivors:
                v = float(lp_row[c])
                if c == self.blank:
                    add(seq, 0, tot + v)
                elif seq and c == seq[-1]:
                    add(seq, 1, pnb + v)
                    add(seq + (c,), 1, pb + v)
                else:
                    add(seq + (c,), 1, tot + v)
        mix = self._mix
        items = [(k, v) for k, v in nxt.items() if mix(*v) > -math.inf]
        items.sort(key=lambda kv: (-mix(*kv[1]), len(kv[0]), kv[0]))
        items = items[: self.K]
        if self.beam_threshold > 0 and items:
            floor = mix(*items[0][1]) - self.beam_threshold
            items = [kv for kv in items if mix(*kv[1]) >= floor]
        self.beam = dict(items)
        now = set(self.beam)
        self.revivals += len([s for s in now if s in self._ever and s not in self._prev])
        self._ever |= now
        self._prev = now

    def results(self):
        out = [(k, self._mix(*v)) for k, v in self.beam.items()]
        out.sort(key=lambda kv: (-kv[1], len(kv[0]), kv[0]))
        return out


def top_n_tokens(row: np.ndarray, n: int):
    """The n most probable tokens of a frame; at a tie the lower id comes first."""
    return [int(c) for c in np.argsort(-row.astype(np.float64), kind="stable")[:n]]


def py_decode(lp: np.ndarray, blank: int, K: int, log_r: np.float32 | None, top_n: int = 0,
              beam_threshold: float = 0.0, merge_max: bool = False):
    """Decode one utterance [T,V]; ``log_r`` None means no survivor test at all.

    ``top_n`` > 0: only the top_n most probable tokens of a frame are candidates for the
    survivor test.  ``beam_threshold`` > 0: kept prefixes score at least best - beam_threshold."""
    T, V = lp.shape
    s = PyPrefixSearch(blank, K, beam_threshold, merge_max)
    for t in range(T):
        cand = top_n_tokens(lp[t], top_n) if top_n > 0 else range(V)
        if log_r is None:
            surv = sorted(cand)
        else:
            thr = np.float32(lp[t].max()) + np.float32(log_r)
            surv = sorted(c for c in cand if lp[t, c] >= thr)
        s.step(lp[t], surv)
    return s


def ctc_forward_logprob(lp: np.ndarray, seq, blank: int, keep: np.ndarray | None = None) -> float:
    """log P(seq | lp) by the textbook CTC forward (alpha) recursion in float64.

    ``lp`` [T,V] log-probabilities; ``keep`` [T,V] (bool) restricts every frame to its surviving
    tokens (the others get probability 0).  This is the sum over ALL alignments of ``seq``, so it
    is an upper bound of what any beam search can assign to ``seq`` on the same frames."""
    lp = np.asarray(lp, dtype=np.float64)
    if keep is not None:
        lp = np.where(keep, lp, -np.inf)
    T = lp.shape[0]
    ext = [blank]
    for c in seq:
        ext += [int(c), blank]
    ext = np.asarray(ext, dtype=np.int64)
    S = len(ext)
    # a state may be entered from two states back iff it is a label that differs from the
    # label two states back (blanks and repeated labels may not be skipped over)
    skip = np.zeros(S, dtype=bool)
    skip[2:] = (ext[2:] != blank) & (ext[2:] != ext[:-2])
    alpha = np.full(S, -np.inf)
    if T == 0:
        return 0.0 if S == 1 else -np.inf
    if S == 1:  # the empty labelling: blank at every frame
        return float(lp[:, blank].sum())
    alpha[0] = lp[0, blank]
    if S > 1:
        alpha[1] = lp[0, ext[1]]
    with np.errstate(invalid="ignore", divide="ignore"):
        for t in range(1, T):
            a1 = np.concatenate(([-np.inf], alpha[:-1]))
            a2 = np.where(skip, np.concatenate(([-np.inf, -np.inf], alpha[:-2])), -np.inf)
            m = np.maximum(alpha, np.maximum(a1, a2))
            tot = np.where(np.isfinite(m),
                           m + np.log(np.exp(alpha - m) + np.exp(a1 - m) + np.exp(a2 - m)), -np.inf)
            alpha = tot + lp[t, ext]
        last = np.logaddexp(alpha[-1], alpha[-2])
    return float(last)
