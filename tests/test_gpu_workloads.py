"""Full-size workloads in the benchmark's launch configuration against the oracle: the
wav2vec2-shaped batch (every utterance), every cell of the beam / threshold sweep, the subword
batch and the per-frame survivor masks of the kernels that prune inside."""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import check_hyps, masks_from_entries, masks_from_words
from tests.test_gpu_parity import _binding, _dev, gpu_decode

pytestmark = pytest.mark.gpu
THREADS = max(1, min(16, len(os.sched_getaffinity(0))))


def _oracle_each(wl, K, r, sample):
    """The oracle on every sampled utterance, utterances in parallel host threads (the C++
    oracle runs outside the interpreter lock)."""
    def one(b):
        n = int(wl.lengths[b])
        return oracle.decode(wl.emissions[b: b + 1, :n], wl.lengths[b: b + 1], wl.blank_id, K, r,
                             want_masks=True)
    with ThreadPoolExecutor(max_workers=THREADS) as ex:
        return list(ex.map(one, sample))


def _compare_sampled(wl, K, r, sample, frac=0.25, d=None):
    own = d is None
    if own:
        d = gpu_decode(wl.emissions, wl.lengths, wl.blank_id, K, r)
    assert (d.status.cpu().numpy() == 0).all()
    unmatched = 0
    for b, res in zip(sample, _oracle_each(wl, K, r, sample)):
        n = int(wl.lengths[b])
        unmatched += check_hyps(d.hyps(b), res.hyps(0), K, max_unmatched_frac=frac,
                                where=f"{wl.name} utt {b} K={K} r={r}", lp=wl.emissions[b, :n],
                                keep=res.keep[0, :n], blank=wl.blank_id)
    # every utterance: scores sorted, lengths consistent, nothing out of range
    lens = d.lens.cpu().numpy()
    nh = d.nhyp.cpu().numpy()
    assert (nh >= 1).all() and (nh <= K).all()
    assert (lens.max(axis=1) <= wl.lengths).all()
    if own:
        d.close()
    return unmatched


@pytest.fixture(scope="module")
def wav2vec2():
    return W.workload_wav2vec2()


def test_wav2vec2_batch_pruned(wav2vec2):
    # the benchmark's own case, B=64, K=50, r=1e-3: every utterance against the oracle, and
    # not one hypothesis that the oracle's beam does not hold
    assert _compare_sampled(wav2vec2, 50, 1e-3, list(range(64)), frac=0.0) == 0


def test_wav2vec2_batch_unpruned(wav2vec2):
    # the benchmark's second leg, r = 0: every utterance
    n = _compare_sampled(wav2vec2, 50, 0.0, list(range(64)), frac=0.0)
    print(f"wav2vec2 r=0: {n} unmatched hypotheses of {64 * 50}")
    assert n == 0


def test_wav2vec2_survivors_bit_exact(wav2vec2):
    wl = wav2vec2
    B, T, V = wl.emissions.shape
    for r in (1e-3, 1e-4, 0.1):
        d = _binding().Decoder(V, 0, 2, r, B, T)
        counts, entries = d.prune(_dev(wl.emissions), _dev(wl.lengths))
        torch.cuda.synchronize()
        counts, entries = counts.cpu().numpy(), entries.cpu().numpy()
        for b in (0, 17, 63):
            n = wl.lengths[b]
            okeep, ocnt = oracle.prune(wl.emissions[b, :n], r)
            assert (counts[b, :n] == ocnt).all() and (counts[b, n:] == 0).all()
            keep, _ = masks_from_entries(counts[b: b + 1], entries[b: b + 1], V)
            assert (keep[0, :n] == okeep).all()
        d.close()


def _masks_of_decode(wl, K, r, streaming_chunk=0, warp_mode=1):
    """Per-frame survivor masks written by the decode kernel itself (instrumented launch)."""
    bd = _binding()
    B, T, V = wl.emissions.shape
    words = torch.from_numpy(np.full((B, T), 0xdeadbeef, dtype=np.uint32).view(np.int32)).cuda()
    x, ln = _dev(wl.emissions), _dev(wl.lengths)
    if not streaming_chunk:
        d = bd.Decoder(V, wl.blank_id, K, r, B, T)
        d.set_test_hook(bd.FLTOP_HOOK_SURVIVOR_MASKS, words)
        d.decode(x, ln)
        torch.cuda.synchronize()
        d.close()
        return words.cpu().numpy().view(np.uint32)
    C = streaming_chunk
    d = bd.Decoder(V, wl.blank_id, K, r, B, T, max_chunk_frames=C)
    d.set_warp_decode(warp_mode)
    full = _dev(np.full(B, C, dtype=np.int32))
    chunk_words = torch.zeros((B, C), dtype=torch.int32, device="cuda")
    d.set_test_hook(bd.FLTOP_HOOK_SURVIVOR_MASKS, chunk_words)
    out = np.zeros((B, T), dtype=np.uint32)
    for i in range(T // C):
        flags = _dev(np.full(B, 1 if i == 0 else 0, dtype=np.uint8))
        d.stream_step(x[:, i * C: (i + 1) * C].contiguous(), full, flags, readback=False)
        torch.cuda.synchronize()
        out[:, i * C: (i + 1) * C] = chunk_words.cpu().numpy().view(np.uint32)
    assert (d.status.cpu().numpy() == 0).all()
    d.close()
    return out


def test_survivor_masks_inside_the_decode_kernels_bit_exact(wav2vec2):
    # the benchmarked path prunes inside the decode kernel: its per-frame survivor sets, not
    # only those of the separate prune kernel, are compared with the oracle bit for bit
    pr1 = W.workload_pr1()
    for r in pr1.thresholds:
        got = _masks_of_decode(pr1, pr1.beam_width, r)
        okeep, _ = oracle.prune(pr1.emissions[0], r)
        assert (masks_from_words(got[0], 32) == okeep).all()
    for r in (1e-3, 0.0):
        got = _masks_of_decode(wav2vec2, 50, r)
        for b in range(64):
            n = int(wav2vec2.lengths[b])
            okeep, _ = oracle.prune(wav2vec2.emissions[b, :n], r)
            assert (masks_from_words(got[b, :n], 32) == okeep).all(), f"utt {b} r={r}"
            assert (got[b, n:] == np.uint32(0xdeadbeef)).all()
    # serving shape: 1024 streams in 16-frame chunks, with the block-per-stream kernel the
    # library picks at this size and with the warp-per-stream kernel
    st = W.workload_streaming(streams=1024, chunks=6)
    for warp_mode in (1, 2):
        got = _masks_of_decode(st, st.beam_width, st.thresholds[0], st.chunk_frames, warp_mode)
        for b in range(0, 1024, 37):
            okeep, _ = oracle.prune(st.emissions[b], st.thresholds[0])
            assert (masks_from_words(got[b], 32) == okeep).all(), f"stream {b} mode {warp_mode}"


@pytest.mark.parametrize("K", W.SWEEP_BEAMS)
@pytest.mark.parametrize("r", W.SWEEP_THRESHOLDS)
def test_sweep_cells(wav2vec2, K, r):
    # every cell of the beam / threshold sweep: all 64 utterances; for the widest beams, where
    # the oracle is slow, the shorter half.  Not one hypothesis outside the oracle's beam.
    order = np.argsort(wav2vec2.lengths)
    sample = [int(order[i]) for i in range(32 if K >= 500 else 64)]
    n = _compare_sampled(wav2vec2, K, r, sample, frac=0.0)
    print(f"sweep K={K} r={r}: {n} unmatched hypotheses of {len(sample) * K}")
    assert n == 0


def test_subword_batch():
    wl = W.workload_subword()
    order = np.argsort(wl.lengths)
    d = gpu_decode(wl.emissions, wl.lengths, wl.blank_id, 32, 1e-3)
    sample = [int(order[i]) for i in range(0, 256, 2)]  # every other utterance by length
    n = _compare_sampled(wl, 32, 1e-3, sample, frac=0.0, d=d)
    print(f"subword r=1e-3: {n} unmatched hypotheses of {len(sample) * 32}")
    assert n == 0
    d.close()
    _compare_sampled(wl, 32, 0.0, [int(order[i]) for i in (0, 3, 9, 20, 35, 50, 70, 90)])
    # survivors bit exact on the same input
    B, T, V = wl.emissions.shape
    d = _binding().Decoder(V, 0, 2, 1e-3, B, T)
    counts, entries = d.prune(_dev(wl.emissions), _dev(wl.lengths))
    torch.cuda.synchronize()
    for b in (3, 200):
        n = wl.lengths[b]
        okeep, ocnt = oracle.prune(wl.emissions[b, :n], 1e-3)
        c = counts[b].cpu().numpy()
        assert (c[:n] == ocnt).all() and (c[n:] == 0).all()
        keep, _ = masks_from_entries(c[None], entries[b: b + 1].cpu().numpy(), V)
        assert (keep[0, :n] == okeep).all()
    d.close()
