"""Pruning inside the decode kernel (vocabularies of at most 32 tokens) against the separate
prune kernel and against the oracle: where the frames are pruned must not change a bit."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import check_hyps
from tests.test_gpu_parity import _binding, _dev

pytestmark = pytest.mark.gpu


def _decode(em_dev, ln, V, K, r, fusion, top_n=0, theta=0.0):
    # (the general block kernel on both sides: the bit-for-bit comparisons below are about
    # where the frames are pruned, not about which decode kernel runs; the row kernel, which
    # serves these shapes by default, has its own tests)
    B, T = em_dev.shape[:2]
    bd = _binding()
    d = bd.Decoder(V, 0, K, r, max(B, 1), max(T, 1), top_n=top_n, beam_threshold=theta)
    d.set_test_hook(bd.FLTOP_HOOK_ROW_KERNEL, None, 0)
    d.set_fusion(fusion)
    before = d.launch_count
    d.decode(em_dev, _dev(np.asarray(ln, dtype=np.int32)))
    torch.cuda.synchronize()
    return d, d.launch_count - before


def _same_stats(a, b):
    # (probe counts of the fingerprint table depend on the order entries went in)
    sa, sb = a.last_call_stats(), b.last_call_stats()
    for key in ("frames", "survivors", "trie_nodes_created", "live_hypotheses_sum",
                "max_node_ids_used"):
        assert sa[key] == sb[key], key


def _same_outputs(a, b, B):
    assert torch.equal(a.nhyp[:B], b.nhyp[:B])
    assert torch.equal(a.status[:B], b.status[:B])
    for u in range(B):
        n = int(a.nhyp[u])
        assert torch.equal(a.lens[u, :n], b.lens[u, :n])
        assert torch.equal(a.scores[u, :n], b.scores[u, :n])          # bit for bit
        # (hypotheses whose scores tie exactly come in no particular order)
        assert sorted(a.hyps(u)) == sorted(b.hyps(u))
    _same_stats(a, b)


@pytest.mark.parametrize("V,K,r,top_n", [(32, 50, 1e-3, 0), (32, 50, 0.0, 0), (32, 20, 7e-3, 4),
                                         (32, 8, 0.0, 4), (32, 16, 0.5, 1), (20, 30, 1e-2, 0),
                                         (5, 12, 0.05, 2), (2, 4, 0.0, 0), (32, 300, 1e-3, 0),
                                         (32, 100, 0.0, 31)])
def test_fused_pruning_changes_nothing(V, K, r, top_n):
    B = 9
    em, ln = W.make_small(900 + V + K, B, 60, 60, V)
    T = em.shape[1]
    ln[:8] = [0, 1, 2, 3, 4, T, 17, 40]  # every length the three-frame pipeline starts up on
    em[:, :, :] = np.where(np.arange(T)[None, :, None] < ln[:, None, None], em, np.nan)
    x = _dev(em)
    fused, n_fused = _decode(x, ln, V, K, r, 1, top_n)
    apart, n_apart = _decode(x, ln, V, K, r, 0, top_n)
    assert n_fused == 1 and n_apart == (3 if 0 < top_n < V else 2)
    assert (fused.status[:B] == 0).all()
    _same_outputs(fused, apart, B)
    res = oracle.decode(np.nan_to_num(em, nan=0.0), ln, 0, K, r, top_n=top_n)
    for b in range(B):
        check_hyps(fused.hyps(b), res.hyps(b), K, where=f"fused utt {b}")
    fused.close()
    apart.close()


def test_fused_pruning_on_strided_rows():
    # rows taken out of a wider tensor: row pitch 40 floats, first token at an odd offset
    B, T, V, K = 4, 33, 32, 24
    wide = np.full((B, T, 40), np.nan, dtype=np.float32)
    em, ln = W.make_small(78, B, T, T, V)
    wide[:, :, 3:35] = em
    x = _dev(wide)[:, :, 3:35]
    assert x.stride(1) == 40 and x.stride(2) == 1
    for r, n in [(1e-3, 0), (0.0, 3), (0.2, 2)]:
        fused, _ = _decode(x, ln, V, K, r, 1, n)
        apart, _ = _decode(x, ln, V, K, r, 0, n)
        _same_outputs(fused, apart, B)
        res = oracle.decode(em, ln, 0, K, r, top_n=n)
        for b in range(B):
            check_hyps(fused.hyps(b), res.hyps(b), K, where=f"strided utt {b} r={r} n={n}")
        fused.close()
        apart.close()


@pytest.mark.parametrize("n", [1, 2, 3])
def test_fused_top_n_breaks_ties_like_the_prune_kernel(n):
    # equal log-probabilities at the N-th place: the lower token id stays.  The beam is wide
    # enough to hold every prefix, so the set of hypotheses is unique whatever order equal
    # scores come out in.
    B, T, V, K = 3, 6, 32, 1024
    em, ln = W.make_small(83, B, T, T, V)
    em[:, :, 5] = em[:, :, 9]
    em[:, :, 30] = em[:, :, 9]
    em[:, 1::2, :] = np.float32(np.log(1.0 / V))        # whole frames tied
    x = _dev(em)
    fused, _ = _decode(x, ln, V, K, 0.0, 1, n)
    apart, _ = _decode(x, ln, V, K, 0.0, 0, n)
    _same_stats(fused, apart)
    res = oracle.decode(em, ln, 0, K, 0.0, top_n=n)
    for b in range(B):
        f, a, o = dict(fused.hyps(b)), dict(apart.hyps(b)), dict(res.hyps(b))
        assert f == a and set(f) == set(o) and len(f) < K
        for seq, sc in f.items():
            assert abs(sc - o[seq]) <= 1e-3
    fused.close()
    apart.close()


def test_fused_pruning_with_impossible_tokens():
    # log-probability -inf: kept by R = 0 (nothing is below the threshold), dropped otherwise
    em, ln = W.make_small(79, 3, 25, 25, 32)
    em[:, :, 7:19] = -np.inf
    em[1, 4, :] = -np.inf                 # a frame in which nothing is possible
    x = _dev(em)
    for r in (0.0, 1e-3):
        fused, _ = _decode(x, ln, 32, 10, r, 1)
        apart, _ = _decode(x, ln, 32, 10, r, 0)
        _same_outputs(fused, apart, 3)
        fused.close()
        apart.close()


@pytest.mark.parametrize("C", [1, 2, 3, 5, 16])
def test_fused_streaming_equals_one_shot(C):
    V, K, r = 32, 16, 1e-2
    B = 6
    em, ln = W.make_small(80 + C, B, 5, 70, V)
    T = em.shape[1]
    x = _dev(em)
    one, _ = _decode(x, ln, V, K, r, 0, top_n=4)
    outs = []
    for fusion in (1, 0):
        d = _binding().Decoder(V, 0, K, r, B, T, max_chunk_frames=C, top_n=4)
        d.set_test_hook(_binding().FLTOP_HOOK_ROW_KERNEL, None, 0)
        d.set_fusion(fusion)
        n_chunks = (T + C - 1) // C
        for i in range(n_chunks):
            t0 = i * C
            chunk = torch.zeros((B, C, V), dtype=torch.float32, device="cuda")
            w = min(C, T - t0)
            chunk[:, :w] = x[:, t0: t0 + w]
            clen = np.clip(ln - t0, 0, C).astype(np.int32)
            flags = np.full(B, (1 if i == 0 else 0) | (2 if i == n_chunks - 1 else 0),
                            dtype=np.uint8)
            d.stream_step(chunk, _dev(clen), _dev(flags))
        torch.cuda.synchronize()
        outs.append(d)
    for d in outs:
        assert torch.equal(one.nhyp[:B], d.nhyp[:B])
        assert torch.equal(one.scores[:B], d.scores[:B])
        for b in range(B):
            assert one.hyps(b) == d.hyps(b)
        d.close()
    one.close()


@pytest.mark.parametrize("V,K,r", [(48, 8, 1e-2), (64, 50, 1e-3), (300, 4, 0.05), (1024, 32, 1e-3),
                                   (1024, 32, 0.0), (1024, 100, 1e-3), (256, 300, 1e-2)])
def test_fused_pruning_of_wide_rows_changes_nothing(V, K, r):
    # vocabularies of 33 to 1024 tokens: the decode block walks its own rows (float32, rows on
    # 16-byte boundaries, no top-N stage); bit for bit what the separate prune kernel gives
    B = 6
    em, ln = W.make_small(8100 + V + K, B, 40, 40, V)
    T = em.shape[1]
    ln[:5] = [0, 1, 2, 3, T]
    em[:, :, :] = np.where(np.arange(T)[None, :, None] < ln[:, None, None], em, np.nan)
    x = _dev(em)
    fused, n_fused = _decode(x, ln, V, K, r, 1)
    apart, n_apart = _decode(x, ln, V, K, r, 0)
    assert n_fused == 1 and n_apart == 2
    assert (fused.status[:B] == 0).all()
    _same_outputs(fused, apart, B)
    clean = np.nan_to_num(em, nan=0.0)
    res = oracle.decode(clean, ln, 0, K, r, want_masks=True)
    for b in range(B):
        check_hyps(fused.hyps(b), res.hyps(b), K, where=f"V={V} utt {b}", lp=clean[b, : ln[b]],
                   keep=res.keep[b, : ln[b]], max_unmatched_frac=0.25 if K >= 100 else 0.0)
    assert fused.beam_state_bytes < apart.beam_state_bytes      # no survivor lists
    fused.close()
    apart.close()


def test_rows_that_cannot_be_pruned_inside_take_the_separate_kernel():
    # a vocabulary that is not a multiple of four, rows off the 16-byte grid, a top-N stage on a
    # wide vocabulary, more than 1024 tokens: two (or three) launches, same results as ever
    em, ln = W.make_small(81, 2, 20, 20, 50)
    d, launches = _decode(_dev(em), ln, 50, 8, 1e-2, 1)
    assert launches == 2
    res = oracle.decode(em, ln, 0, 8, 1e-2)
    for b in range(2):
        check_hyps(d.hyps(b), res.hyps(b), 8, where=f"V=50 utt {b}")
    d.close()
    em, ln = W.make_small(82, 2, 20, 20, 64)
    wide = torch.zeros((2, 20, 70), device="cuda")
    wide[:, :, 3:67] = _dev(em)
    d, launches = _decode(wide[:, :, 3:67], ln, 64, 8, 1e-2, 1)
    assert launches == 2
    d.close()
    d, launches = _decode(_dev(em), ln, 64, 8, 1e-2, 1, top_n=4)
    assert launches == 3
    res = oracle.decode(em, ln, 0, 8, 1e-2, top_n=4)
    for b in range(2):
        check_hyps(d.hyps(b), res.hyps(b), 8, where=f"V=64 top-4 utt {b}")
    d.close()
    em, ln = W.make_small(83, 2, 12, 12, 2048)
    d, launches = _decode(_dev(em), ln, 2048, 8, 1e-3, 1)
    assert launches == 2
    d.close()


def test_fusion_mode_is_validated():
    b = _binding()
    d = b.Decoder(32, 0, 4, 0.0, 1, 4)
    with pytest.raises(b.FltopError):
        d.set_fusion(2)
    assert b.lib().fltop_set_fusion(None, 1) == b.FLTOP_ERR_INVALID_ARG
    d.close()
