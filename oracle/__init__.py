"""ctypes front end of the CPU oracle (``fltop_oracle.cpp``).  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may use
this package.  It shares no code with the CUDA library and never imports it.

Pins (see ``tests/test_oracle_*.py``): brute-force enumeration of all
alignments on tiny inputs (with and without pruning), the closed-form total
mass, the CTC forward recursion for single labellings, greedy decoding at K=1,
chunked == one-shot, padding invariance, monotonicity of the survivor set in R.
Finite-K selection on general inputs has no pin beyond its definition and a
second, separately written Python implementation: "parity unpinned" at
near-ties of the K-th score.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fltop_oracle.cpp")
_LIB = os.path.join(_HERE, "libfltop_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fused multiply-add, see the source header)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-fPIC",
                               "-shared", "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        c = ctypes
        lib.oracle_log_r.restype = c.c_float
        lib.oracle_log_r.argtypes = [c.c_float]
        lib.oracle_prune.restype = None
        lib.oracle_prune.argtypes = [c.c_void_p, c.c_int64, c.c_int, c.c_float, c.c_void_p,
                                     c.c_void_p]
        lib.oracle_stream_create.restype = c.c_void_p
        lib.oracle_stream_create.argtypes = [c.c_int, c.c_int, c.c_int, c.c_float]
        lib.oracle_stream_destroy.restype = None
        lib.oracle_stream_destroy.argtypes = [c.c_void_p]
        lib.oracle_stream_reset.restype = None
        lib.oracle_stream_reset.argtypes = [c.c_void_p]
        lib.oracle_stream_feed.restype = None
        lib.oracle_stream_feed.argtypes = [c.c_void_p, c.c_void_p, c.c_int64, c.c_void_p,
                                           c.c_void_p]
        lib.oracle_stream_results.restype = c.c_int
        lib.oracle_stream_results.argtypes = [c.c_void_p] + [c.c_void_p] * 5 + [c.c_int]
        lib.oracle_stream_options.restype = None
        lib.oracle_stream_options.argtypes = [c.c_void_p, c.c_int, c.c_double]
        lib.oracle_prune_topn.restype = None
        lib.oracle_prune_topn.argtypes = [c.c_void_p, c.c_int64, c.c_int, c.c_float, c.c_int,
                                          c.c_void_p, c.c_void_p]
        lib.oracle_decode_opt.restype = None
        lib.oracle_decode_opt.argtypes = [c.c_void_p, c.c_int64, c.c_int64, c.c_void_p, c.c_int,
                                          c.c_int, c.c_int, c.c_int, c.c_int, c.c_float, c.c_int,
                                          c.c_double, c.c_int, c.c_void_p, c.c_void_p, c.c_void_p,
                                          c.c_void_p, c.c_void_p, c.c_void_p, c.c_int]
        lib.oracle_stream_merge_max.restype = None
        lib.oracle_stream_merge_max.argtypes = [c.c_void_p, c.c_int]
        lib.oracle_decode.restype = None
        lib.oracle_decode.argtypes = [c.c_void_p, c.c_int64, c.c_int64, c.c_void_p, c.c_int,
                                      c.c_int, c.c_int, c.c_int, c.c_int, c.c_float, c.c_int,
                                      c.c_void_p, c.c_void_p, c.c_void_p, c.c_void_p,
                                      c.c_void_p, c.c_void_p]
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def log_r(r: float) -> np.float32:
    return np.float32(_load().oracle_log_r(float(np.float32(r))))


def prune(lp: np.ndarray, r: float, top_n: int = 0):
    """Survivor mask [.., V] (bool) and count [..] of every frame of ``lp`` [.., V].

    ``top_n`` > 0 keeps at most the top_n most probable tokens of a frame (N of Algorithm 1)."""
    lp = np.ascontiguousarray(lp, dtype=np.float32)
    V = lp.shape[-1]
    n = lp.size // V if V else 0
    keep = np.zeros(lp.shape, dtype=np.uint8)
    counts = np.zeros(lp.shape[:-1], dtype=np.int32)
    _load().oracle_prune_topn(_ptr(lp), n, V, float(np.float32(r)), int(top_n), _ptr(keep),
                              _ptr(counts))
    return keep.astype(bool), counts


class DecodeResult:
    """tokens [B,K,L] int32, lens [B,K] int32, scores [B,K] float64, nhyp [B]."""

    def __init__(self, tokens, lens, scores, nhyp, keep=None, counts=None):
        self.tokens, self.lens, self.scores, self.nhyp = tokens, lens, scores, nhyp
        self.keep, self.counts = keep, counts

    def hyps(self, b: int):
        """[(token tuple, score)] of utterance b, best first."""
        return [(tuple(int(x) for x in self.tokens[b, k, : self.lens[b, k]]),
                 float(self.scores[b, k])) for k in range(int(self.nhyp[b]))]


def decode(lp: np.ndarray, lengths, blank: int, K: int, r: float, max_len: int | None = None,
           want_masks: bool = False, top_n: int = 0, beam_threshold: float = 0.0,
           merge_max: bool = False) -> DecodeResult:
    """Frame-pruned CTC prefix beam search of a padded batch ``lp`` [B,T,V].

    ``top_n`` and ``beam_threshold`` are N and beam_threshold of Algorithm 1 (0 = off).
    ``merge_max``: masses are combined by max instead of log-sum (Algorithm 1's literal
    score' = score + logit: a prefix scores as its best single alignment)."""
    lp = np.ascontiguousarray(lp, dtype=np.float32)
    B, T, V = lp.shape
    lengths = np.ascontiguousarray(lengths, dtype=np.int32)
    L = max(1, T if max_len is None else max_len)
    tokens = np.zeros((B, K, L), dtype=np.int32)
    lens = np.zeros((B, K), dtype=np.int32)
    scores = np.full((B, K), -np.inf, dtype=np.float64)
    nhyp = np.zeros(B, dtype=np.int32)
    keep = np.zeros((B, T, V), dtype=np.uint8) if want_masks else None
    counts = np.zeros((B, T), dtype=np.int32) if want_masks else None
    _load().oracle_decode_opt(_ptr(lp), T * V, V, _ptr(lengths), B, T, V, blank, K,
                              float(np.float32(r)), int(top_n), float(beam_threshold), L,
                              _ptr(tokens), _ptr(lens), _ptr(scores), _ptr(nhyp), _ptr(keep),
                              _ptr(counts), int(bool(merge_max)))
    return DecodeResult(tokens, lens, scores, nhyp,
                        None if keep is None else keep.astype(bool), counts)


class Stream:
    """One utterance decoded incrementally; state persists between ``feed`` calls."""

    def __init__(self, V: int, blank: int, K: int, r: float, top_n: int = 0,
                 beam_threshold: float = 0.0, merge_max: bool = False):
        self.V, self.K = V, K
        self._h = _load().oracle_stream_create(V, blank, K, float(np.float32(r)))
        _load().oracle_stream_options(self._h, int(top_n), float(beam_threshold))
        _load().oracle_stream_merge_max(self._h, int(bool(merge_max)))

    def feed(self, lp: np.ndarray):
        lp = np.ascontiguousarray(lp, dtype=np.float32).reshape(-1, self.V)
        _load().oracle_stream_feed(self._h, _ptr(lp), lp.shape[0], None, None)

    def reset(self):
        _load().oracle_stream_reset(self._h)

    def results(self, max_len: int = 4096, with_parts: bool = False):
        tokens = np.zeros((self.K, max_len), dtype=np.int32)
        lens = np.zeros(self.K, dtype=np.int32)
        scores = np.zeros(self.K, dtype=np.float64)
        pb = np.zeros(self.K, dtype=np.float64)
        pnb = np.zeros(self.K, dtype=np.float64)
        n = _load().oracle_stream_results(self._h, _ptr(tokens), _ptr(lens), _ptr(scores),
                                          _ptr(pb), _ptr(pnb), max_len)
        out = [(tuple(int(x) for x in tokens[k, : lens[k]]), float(scores[k])) for k in range(n)]
        if with_parts:
            return out, pb[:n], pnb[:n]
        return out

    def close(self):
        if self._h:
            _load().oracle_stream_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
