"""Full-size workloads in the benchmark's launch configuration vs the oracle on samples."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import check_hyps, masks_from_entries
from tests.test_gpu_parity import _binding, _dev, gpu_decode

pytestmark = pytest.mark.gpu


def _compare_sampled(wl, K, r, sample, frac=0.25):
    d = gpu_decode(wl.emissions, wl.lengths, wl.blank_id, K, r)
    assert (d.status.cpu().numpy() == 0).all()
    res = oracle.decode(wl.emissions[sample], wl.lengths[sample], wl.blank_id, K, r)
    swaps = 0
    for i, b in enumerate(sample):
        swaps += check_hyps(d.hyps(b), res.hyps(i), K, max_unmatched_frac=frac,
                            where=f"{wl.name} utt {b} K={K} r={r}")
    # every utterance: scores sorted, lengths consistent, nothing out of range
    lens = d.lens.cpu().numpy()
    nh = d.nhyp.cpu().numpy()
    assert (nh >= 1).all() and (nh <= K).all()
    assert (lens.max(axis=1) <= wl.lengths).all()
    d.close()
    return swaps


@pytest.fixture(scope="module")
def wav2vec2():
    return W.workload_wav2vec2()


def test_wav2vec2_batch_pruned(wav2vec2):
    # B=64, K=50, r=1e-3: every utterance against the oracle
    _compare_sampled(wav2vec2, 50, 1e-3, list(range(64)))


def test_wav2vec2_batch_unpruned_sampled(wav2vec2):
    order = np.argsort(wav2vec2.lengths)
    sample = [int(order[0]), int(order[20]), int(order[40]), int(order[-1])]
    _compare_sampled(wav2vec2, 50, 0.0, sample)


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


@pytest.mark.parametrize("K,r,n_sample", [(10, 0.0, 3), (10, 0.1, 6), (100, 1e-2, 3),
                                          (100, 1e-4, 2), (500, 1e-3, 1), (500, 0.0, 1)])
def test_sweep_cells_sampled(wav2vec2, K, r, n_sample):
    order = np.argsort(wav2vec2.lengths)
    sample = [int(x) for x in order[:n_sample]]       # the shortest utterances keep the oracle fast
    _compare_sampled(wav2vec2, K, r, sample)


def test_subword_batch_sampled():
    wl = W.workload_subword()
    order = np.argsort(wl.lengths)
    _compare_sampled(wl, 32, 1e-3, [int(order[0]), int(order[1]), int(order[128])])
    _compare_sampled(wl, 32, 0.0, [int(order[0])])
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
