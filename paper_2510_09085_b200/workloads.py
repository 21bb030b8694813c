"""Seeded synthetic emission generators (inputs only, none of the decoder's arithmetic).

The paper decodes wav2vec2-large emissions on LibriSpeech with a 32-symbol
character vocabulary (Section 4) and observes that nearly all probability mass
sits on one to four tokens per frame (Section 4.1).  Neither the audio nor the
encoder is available, so these generators produce frame-level log-probability
matrices of the same shape and "peakiness": every frame has one dominant token,
most frames are easy (one large logit), a minority are hard (a few competitors
close to the dominant token).

Everything is drawn from ``numpy.random.Generator(PCG64(seed))``; logits and the
log-softmax are computed in float64 and rounded once to float32.  The same
arrays are handed to the CPU oracle and to the CUDA library.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass(frozen=True)
class EmissionRecipe:
    """Parameters of the peaky-frame generator."""

    vocab_size: int = 32
    blank_id: int = 0
    p_blank: float = 0.65      # probability that the dominant token is blank
    p_repeat: float = 0.2      # a non-blank dominant repeats the previous char
    hard_fraction: float = 0.10
    boost_easy: float = 8.0    # added to the dominant logit on easy frames
    boost_hard: float = 4.0    # added to the dominant logit on hard frames
    boost_comp: float = 3.5    # added to each competitor on hard frames
    comp_min: int = 1
    comp_max: int = 2
    comp_zipf: float = 0.0     # 0 = uniform competitors, else Zipf exponent


@dataclass(frozen=True)
class Workload:
    """A named decoding job: emissions plus decoder parameters."""

    name: str
    emissions: np.ndarray       # [B, Tmax, V] float32 log-probs, padding = 0.0
    lengths: np.ndarray         # [B] int32
    blank_id: int
    beam_width: int
    thresholds: tuple           # the r values this workload is decoded at
    chunk_frames: int = 0       # > 0 for streaming workloads
    meta: dict = field(default_factory=dict)


CHAR_RECIPE = EmissionRecipe()
SUBWORD_RECIPE = EmissionRecipe(
    vocab_size=1024, hard_fraction=0.15, boost_easy=9.0, boost_hard=5.0,
    boost_comp=4.5, comp_min=2, comp_max=5, comp_zipf=1.1)


def _dominant_tokens(rng: np.random.Generator, T: int, rc: EmissionRecipe) -> np.ndarray:
    """Per-frame dominant token ids following the blank / repeat / fresh recipe."""
    V, blank = rc.vocab_size, rc.blank_id
    u_blank = rng.random(T)
    u_rep = rng.random(T)
    nonblank_ids = np.array([c for c in range(V) if c != blank], dtype=np.int64)
    fresh_char = nonblank_ids[rng.integers(0, V - 1, size=T)]
    is_blank = u_blank < rc.p_blank
    wants_repeat = (~is_blank) & (u_rep < rc.p_repeat)
    is_fresh = (~is_blank) & (~wants_repeat)
    # a repeat copies the most recent non-blank dominant; chains of repeats end
    # at a fresh draw, so forward-fill the index of the last fresh frame.
    idx = np.where(is_fresh, np.arange(T), -1)
    last_fresh = np.maximum.accumulate(idx)
    # a would-be repeat with nothing before it becomes a fresh draw
    orphan = wants_repeat & (last_fresh < 0)
    dom = np.full(T, blank, dtype=np.int64)
    dom[is_fresh] = fresh_char[is_fresh]
    dom[orphan] = fresh_char[orphan]
    if orphan.any():
        idx = np.where(is_fresh | orphan, np.arange(T), -1)
        last_fresh = np.maximum.accumulate(idx)
    rep = wants_repeat & ~orphan
    dom[rep] = fresh_char[last_fresh[rep]]
    return dom


def _zipf_pmf(V: int, a: float) -> np.ndarray:
    w = 1.0 / np.power(np.arange(1, V + 1, dtype=np.float64), a)
    return w / w.sum()


def make_utterance(rng: np.random.Generator, T: int, rc: EmissionRecipe) -> np.ndarray:
    """One utterance of log-softmax emissions, [T, V] float32."""
    V = rc.vocab_size
    logits = rng.standard_normal((T, V))
    if T == 0:
        return logits.astype(np.float32)
    dom = _dominant_tokens(rng, T, rc)
    hard = rng.random(T) < rc.hard_fraction
    rows = np.arange(T)
    logits[rows, dom] += np.where(hard, rc.boost_hard, rc.boost_easy)
    n_comp = rng.integers(rc.comp_min, rc.comp_max + 1, size=T)
    pmf = _zipf_pmf(V, rc.comp_zipf) if rc.comp_zipf > 0 else None
    for t in np.nonzero(hard)[0]:
        chosen: list[int] = []
        while len(chosen) < int(n_comp[t]):
            c = int(rng.choice(V, p=pmf)) if pmf is not None else int(rng.integers(0, V))
            if c != int(dom[t]) and c not in chosen:
                chosen.append(c)
        logits[t, chosen] += rc.boost_comp
    m = logits.max(axis=1, keepdims=True)
    lse = m + np.log(np.exp(logits - m).sum(axis=1, keepdims=True))
    return (logits - lse).astype(np.float32)


def make_batch(seed: int, lengths, rc: EmissionRecipe) -> tuple[np.ndarray, np.ndarray]:
    """Padded batch [B, max(lengths), V]; frames past an utterance's length are 0."""
    lengths = np.asarray(lengths, dtype=np.int32)
    rng = np.random.default_rng(np.random.PCG64(seed))
    B = len(lengths)
    Tmax = int(lengths.max()) if B else 0
    out = np.zeros((B, Tmax, rc.vocab_size), dtype=np.float32)
    for b in range(B):
        out[b, : lengths[b]] = make_utterance(rng, int(lengths[b]), rc)
    return out, lengths


def _uniform_lengths(seed: int, B: int, lo: int, hi: int) -> np.ndarray:
    rng = np.random.default_rng(np.random.PCG64(seed + 7919))
    return rng.integers(lo, hi + 1, size=B).astype(np.int32)


def workload_pr1(seed: int = 0) -> Workload:
    """Single 200-frame character utterance, K=8, r in {0.01, 0}."""
    em, ln = make_batch(seed, [200], CHAR_RECIPE)
    return Workload("pr1_T200_V32_K8", em, ln, 0, 8, (0.01, 0.0))


def workload_wav2vec2(seed: int = 1, batch: int = 64, beam_width: int = 50,
                      thresholds=(1e-3, 0.0)) -> Workload:
    """Character-CTC batch: T uniform in [250, 1750] (5-35 s at 50 frames/s)."""
    ln = _uniform_lengths(seed, batch, 250, 1750)
    em, ln = make_batch(seed, ln, CHAR_RECIPE)
    return Workload(f"wav2vec2_B{batch}_V32_K{beam_width}", em, ln, 0, beam_width,
                    tuple(thresholds))


SWEEP_BEAMS = (10, 50, 100, 500)
SWEEP_THRESHOLDS = (0.0, 1e-4, 1e-3, 1e-2, 0.1)


def workload_subword(seed: int = 2, batch: int = 256, beam_width: int = 32,
                     thresholds=(1e-3, 0.0)) -> Workload:
    """Subword-CTC batch: V=1024, T uniform in [100, 800] (25 frames/s)."""
    ln = _uniform_lengths(seed, batch, 100, 800)
    em, ln = make_batch(seed, ln, SUBWORD_RECIPE)
    return Workload(f"subword_B{batch}_V1024_K{beam_width}", em, ln, 0, beam_width,
                    tuple(thresholds))


def workload_streaming(seed: int = 3, streams: int = 1024, chunks: int = 100,
                       chunk_frames: int = 16, beam_width: int = 16) -> Workload:
    """Concurrent character streams delivered in fixed-size chunks, r=1e-2."""
    T = chunks * chunk_frames
    em, ln = make_batch(seed, [T] * streams, CHAR_RECIPE)
    return Workload(f"stream_S{streams}_C{chunk_frames}_K{beam_width}", em, ln, 0,
                    beam_width, (1e-2,), chunk_frames=chunk_frames,
                    meta={"chunks": chunks})


def make_small(seed: int, B: int, T_lo: int, T_hi: int, V: int, hard_fraction: float = 0.3,
               boost_easy: float = 3.0) -> tuple[np.ndarray, np.ndarray]:
    """Small, deliberately less peaky batches for element-by-element parity tests."""
    rc = EmissionRecipe(vocab_size=V, hard_fraction=hard_fraction, boost_easy=boost_easy,
                        boost_hard=2.0, boost_comp=1.5, comp_min=1,
                        comp_max=max(1, min(3, V - 2)))
    ln = _uniform_lengths(seed, B, T_lo, T_hi)
    return make_batch(seed, ln, rc)
