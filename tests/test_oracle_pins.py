"""Pins of the CPU oracle against things other than itself (no GPU needed)."""
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.refs import brute_force, greedy, py_decode

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "ctc_two_frame.txt")


def _rand_logp(seed, T, V, sharp=1.5):
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((T, V)) * sharp
    x = x - np.log(np.exp(x).sum(1, keepdims=True))
    return x.astype(np.float32)


def _oracle_hyps(lp, blank, K, r):
    res = oracle.decode(lp[None], [lp.shape[0]], blank, K, r, want_masks=True)
    return dict(res.hyps(0)), res


# ---------------------------------------------------------------- golden file
def _read_golden():
    frames, cases, cur = [], {}, None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        w = line.split()
        if w[0] == "frame":
            frames.append([float(x) for x in w[1:]])
        elif w[0] == "case":
            cur = cases.setdefault(float(w[1].split("=")[1]), {"hyps": {}, "surv": []})
        elif w[0] == "survivors":
            cur["surv"].append([int(x) for x in w[1:]])
        elif w[0] == "hyp":
            cur["hyps"][tuple(int(x) for x in w[2:])] = float(w[1])
    return np.log(np.array(frames)).astype(np.float32), cases


def test_hand_worked_example():
    lp, cases = _read_golden()
    for r, case in cases.items():
        got, res = _oracle_hyps(lp, 0, 16, r)
        assert set(got) == set(case["hyps"])
        for seq, p in case["hyps"].items():
            assert got[seq] == pytest.approx(math.log(p), abs=1e-6)
        if case["surv"]:
            assert res.keep[0].astype(int).tolist() == case["surv"]


# ---------------------------------------------------------------- brute force
@pytest.mark.parametrize("seed,T,V,blank", [(0, 4, 3, 0), (1, 5, 3, 2), (2, 6, 3, 1),
                                            (3, 5, 4, 0), (4, 6, 4, 3), (5, 1, 2, 0)])
def test_unpruned_scores_equal_exact_sums(seed, T, V, blank):
    lp = _rand_logp(seed, T, V)
    exact = brute_force(lp, blank)
    got, _ = _oracle_hyps(lp, blank, 10000, 0.0)
    assert set(got) == set(exact)
    for seq, v in exact.items():
        assert got[seq] == pytest.approx(v, abs=1e-9)


@pytest.mark.parametrize("seed,T,V,blank,r", [(10, 5, 4, 0, 0.3), (11, 6, 4, 0, 0.5),
                                              (12, 6, 3, 1, 0.2), (13, 6, 4, 2, 0.7),
                                              (14, 5, 4, 0, 1.0), (15, 6, 4, 0, 0.05)])
def test_pruned_scores_equal_sums_over_surviving_alignments(seed, T, V, blank, r):
    lp = _rand_logp(seed, T, V, sharp=1.0)
    got, res = _oracle_hyps(lp, blank, 10000, r)
    keep = res.keep[0]
    # the mask itself, from the definition, in float32
    lr = np.float32(math.log(np.float32(r)))
    for t in range(T):
        thr = np.float32(lp[t].max() + lr)
        assert keep[t].tolist() == [bool(lp[t, c] >= thr) for c in range(V)]
    # this seed set must exercise "blank pruned" and "last token pruned"
    exact = {k: v for k, v in brute_force(lp, blank, keep).items() if v > -math.inf}
    assert set(got) == set(exact)
    for seq, v in exact.items():
        assert got[seq] == pytest.approx(v, abs=1e-9)


def test_pruned_cases_cover_blank_and_repeat_pruning():
    hit_blank = hit_nonblank = False
    for seed, T, V, blank, r in [(10, 5, 4, 0, 0.3), (11, 6, 4, 0, 0.5), (12, 6, 3, 1, 0.2),
                                 (13, 6, 4, 2, 0.7), (15, 6, 4, 0, 0.05)]:
        keep, _ = oracle.prune(_rand_logp(seed, T, V, sharp=1.0), r)
        hit_blank |= bool((~keep[:, blank]).any())
        hit_nonblank |= bool((~np.delete(keep, blank, axis=1)).any())
    assert hit_blank and hit_nonblank


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("r", [0.0, 0.05, 0.4])
def test_total_mass_closed_form(r):
    # with an unbounded beam the hypotheses partition the surviving alignments:
    # log sum_h P(h) = sum_t log sum_{c in S_t} p[t,c]   (= 0 for r = 0)
    lp = _rand_logp(21, 11, 4, sharp=1.0)
    got, res = _oracle_hyps(lp, 0, 200000, r)
    p = np.exp(lp.astype(np.float64))
    expect = float(np.log((p * res.keep[0]).sum(1)).sum())
    total = math.log(math.fsum(math.exp(v) for v in got.values()))
    assert total == pytest.approx(expect, abs=1e-9)
    if r == 0.0:
        assert expect == pytest.approx(0.0, abs=1e-5)


def _ctc_logprob(lp, seq, blank):
    """log P(seq | x) by the CTC forward recursion (torch's ctc_loss, float64)."""
    x = torch.from_numpy(lp.astype(np.float64))[:, None, :]
    tgt = torch.tensor([list(seq)], dtype=torch.long).reshape(1, -1)
    loss = torch.nn.functional.ctc_loss(
        x, tgt, torch.tensor([lp.shape[0]]), torch.tensor([len(seq)]), blank=blank,
        reduction="sum", zero_infinity=False)
    return -float(loss)


def test_scores_equal_ctc_forward_recursion_with_unbounded_beam():
    lp = _rand_logp(31, 12, 4, sharp=1.0)
    got, _ = _oracle_hyps(lp, 0, 500000, 0.0)
    seqs = sorted(got, key=lambda s: -got[s])[:40] + [s for s in got if len(s) == 6][:20]
    for seq in seqs:
        if len(seq) == 0:
            continue
        assert got[seq] == pytest.approx(_ctc_logprob(lp, seq, 0), abs=1e-8)


def test_finite_beam_scores_are_lower_bounds_and_tight_on_peaky_input():
    wl = W.workload_pr1()
    lp = wl.emissions[0]
    for r in wl.thresholds:
        got, _ = _oracle_hyps(lp, 0, wl.beam_width, r)
        best = max(got, key=got.get)
        for seq, v in got.items():
            exact = _ctc_logprob(lp, seq, 0)
            assert v <= exact + 1e-9
        # mass lost to evicted lagging prefixes and pruned tokens stays small
        assert got[best] == pytest.approx(_ctc_logprob(lp, best, 0), abs=0.15)


# ---------------------------------------------------------------- special cases
def test_beam_one_equals_greedy_on_easy_frames():
    rc = W.EmissionRecipe(hard_fraction=0.0)
    em, ln = W.make_batch(5, [300, 120, 64], rc)
    res = oracle.decode(em, ln, 0, 1, 0.0)
    for b in range(3):
        assert res.hyps(b)[0][0] == greedy(em[b, : ln[b]], 0)


def test_threshold_zero_equals_search_without_survivor_test():
    em, ln = W.make_small(7, 3, 20, 40, 6)
    res = oracle.decode(em, ln, 0, 12, 0.0, want_masks=True)
    for b in range(3):
        assert res.keep[b, : ln[b]].all()
        ref = py_decode(em[b, : ln[b]], 0, 12, None).results()
        got = res.hyps(b)
        assert [s for s, _ in got] == [s for s, _ in ref]
        np.testing.assert_allclose([v for _, v in got], [v for _, v in ref], atol=1e-9)


@pytest.mark.parametrize("K,r", [(4, 0.05), (8, 0.2), (3, 0.0), (16, 0.01)])
def test_matches_second_implementation_with_finite_beam(K, r):
    em, ln = W.make_small(9, 4, 30, 60, 5)
    res = oracle.decode(em, ln, 0, K, r)
    revivals = 0
    for b in range(4):
        ref = py_decode(em[b, : ln[b]], 0, K, oracle.log_r(r))
        revivals += ref.revivals
        got, want = res.hyps(b), ref.results()
        assert [s for s, _ in got] == [s for s, _ in want]
        np.testing.assert_allclose([v for _, v in got], [v for _, v in want], atol=1e-9)
    if K <= 4:
        assert revivals > 0   # prefixes leave and re-enter the beam in these cases


def test_survivor_set_properties():
    wl = W.workload_pr1()
    lp = wl.emissions[0]
    prev = None
    for r in [0.0, 1e-4, 1e-3, 1e-2, 0.1, 0.5, 1.0]:
        keep, counts = oracle.prune(lp, r)
        assert (counts == keep.sum(1)).all()
        assert keep[np.arange(lp.shape[0]), lp.argmax(1)].all()      # arg-max always survives
        if r == 0.0:
            assert keep.all()
        if prev is not None:
            assert (prev | ~keep).all()                               # S(r1) >= S(r2), r1 < r2
        prev = keep
    assert oracle.prune(lp, 1.0)[1].min() >= 1
    assert oracle.log_r(0.0) == -np.inf
    assert oracle.log_r(1e-3) == np.float32(math.log(float(np.float32(1e-3))))


def test_chunked_equals_one_shot():
    em, ln = W.make_small(11, 1, 90, 90, 6)
    lp = em[0]
    whole = oracle.decode(em, ln, 0, 6, 0.02).hyps(0)
    for cuts in ([16] * 6, [1, 2, 3, 50, 34], [90]):
        s = oracle.Stream(6, 0, 6, 0.02)
        t = 0
        for c in cuts:
            s.feed(lp[t: t + c])
            t += c
        assert t >= 90
        assert s.results() == whole
        s.reset()
        s.feed(lp)
        assert s.results() == whole
        s.close()


def test_padding_is_never_read():
    em, ln = W.make_small(13, 3, 10, 30, 5)
    a = oracle.decode(em, ln, 0, 5, 0.01)
    em2 = em.copy()
    for b in range(3):
        em2[b, ln[b]:] = np.nan
    b_ = oracle.decode(em2, ln, 0, 5, 0.01)
    assert (a.tokens == b_.tokens).all() and (a.lens == b_.lens).all()
    assert np.array_equal(a.scores, b_.scores)


def test_empty_and_invalid_lengths():
    em, _ = W.make_small(17, 3, 8, 8, 4)
    res = oracle.decode(em, [0, 8, 99], 0, 3, 0.0)
    assert res.nhyp.tolist()[0] == 1 and res.hyps(0) == [((), 0.0)]
    assert res.nhyp[2] == 0
    assert (res.lens[0] == 0).all() and res.scores[0, 1] == -np.inf


# ---------------------------------------------------------------- N and beam_threshold of Algorithm 1
@pytest.mark.parametrize("V,n", [(8, 1), (8, 3), (32, 4), (32, 32), (100, 7)])
def test_top_n_keeps_the_n_most_probable_tokens(V, n):
    # stage 1 of Algorithm 1 against numpy's stable sort: with R = 0 the survivors are exactly
    # the n largest entries of the row (ties: lower id), with R > 0 their intersection with
    # the uncapped survivor set
    lp = _rand_logp(40 + V, 30, V)
    lp[3, :] = lp[3, 0]                      # a row of exact ties: ids 0 .. n-1 must win
    lp[4, 2] = lp[4, 5] = lp[4].max() + 1.0  # a tie for first place
    keep, cnt = oracle.prune(lp, 0.0, top_n=n)
    for t in range(lp.shape[0]):
        want = np.zeros(V, dtype=bool)
        want[np.argsort(-lp[t].astype(np.float64), kind="stable")[:n]] = True
        assert (keep[t] == want).all() and cnt[t] == min(n, V)
    keep_r, _ = oracle.prune(lp, 0.05)
    keep_rn, cnt_rn = oracle.prune(lp, 0.05, top_n=n)
    keep_n, _ = oracle.prune(lp, 0.0, top_n=n)
    assert (keep_rn == (keep_r & keep_n)).all()
    assert (cnt_rn <= n).all() and keep_rn[np.arange(30), lp.argmax(1)].all()
    # n >= V and n = 0 change nothing
    assert (oracle.prune(lp, 0.05, top_n=V)[0] == keep_r).all()
    assert (oracle.prune(lp, 0.05, top_n=0)[0] == keep_r).all()


@pytest.mark.parametrize("seed,T,V,n,r", [(0, 5, 4, 2, 0.0), (1, 6, 3, 1, 0.0), (2, 5, 4, 3, 0.2)])
def test_top_n_inside_the_search_is_brute_force_over_the_kept_tokens(seed, T, V, n, r):
    lp = _rand_logp(seed + 70, T, V)
    keep = np.zeros((T, V), dtype=bool)
    for t in range(T):
        keep[t, np.argsort(-lp[t].astype(np.float64), kind="stable")[:n]] = True
        if r > 0:
            keep[t] &= lp[t] >= np.float32(lp[t].max()) + oracle.log_r(r)
    exact = {k: v for k, v in brute_force(lp, 0, keep).items() if v > -math.inf}
    res = oracle.decode(lp[None], [T], 0, 4096, r, top_n=n, want_masks=True)
    assert (res.keep[0] == keep).all()
    got = dict(res.hyps(0))
    assert set(got) == set(exact)
    for k, v in exact.items():
        assert got[k] == pytest.approx(v, abs=1e-9)


def test_top_n_one_is_greedy_whatever_the_beam():
    lp = _rand_logp(5, 60, 12)
    for K in (1, 5):
        res = oracle.decode(lp[None], [60], 0, K, 0.0, top_n=1)
        assert res.hyps(0)[0][0] == greedy(lp, 0)
        assert res.nhyp[0] == 1          # one token per frame: one prefix


@pytest.mark.parametrize("K,theta,r,n", [(6, 2.0, 0.0, 0), (10, 0.5, 0.05, 0), (8, 4.0, 0.01, 3),
                                         (4, 1e-9, 0.0, 0)])
def test_beam_threshold_and_top_n_match_the_second_implementation(K, theta, r, n):
    for seed in range(4):
        lp = _rand_logp(200 + seed, 40, 6, sharp=1.0)
        ref = py_decode(lp, 0, K, None if r == 0 else oracle.log_r(r), top_n=n,
                        beam_threshold=theta).results()
        got = oracle.decode(lp[None], [40], 0, K, r, top_n=n, beam_threshold=theta).hyps(0)
        assert [s for s, _ in got] == [s for s, _ in ref]
        np.testing.assert_allclose([v for _, v in got], [v for _, v in ref], atol=1e-9)


def test_beam_threshold_invariants():
    lp = _rand_logp(9, 80, 8, sharp=3.0)
    base = oracle.decode(lp[None], [80], 0, 12, 0.01).hyps(0)
    # off, and a threshold nothing can reach, change nothing
    assert oracle.decode(lp[None], [80], 0, 12, 0.01, beam_threshold=0.0).hyps(0) == base
    assert oracle.decode(lp[None], [80], 0, 12, 0.01, beam_threshold=1e9).hyps(0) == base
    for theta in (8.0, 3.0, 1.0, 0.2, 0.01):
        h = oracle.decode(lp[None], [80], 0, 12, 0.01, beam_threshold=theta).hyps(0)
        assert all(s >= h[0][1] - theta for _, s in h) and 1 <= len(h) <= 12
    # a vanishing threshold leaves the single best prefix of every frame: the K = 1 search
    one = oracle.decode(lp[None], [80], 0, 12, 0.01, beam_threshold=1e-12).hyps(0)
    assert len(one) == 1 and one == oracle.decode(lp[None], [80], 0, 1, 0.01).hyps(0)


def test_streaming_with_options_equals_one_shot():
    lp = _rand_logp(31, 50, 10, sharp=1.0)
    full = oracle.decode(lp[None], [50], 0, 6, 0.02, top_n=4, beam_threshold=3.0).hyps(0)
    st = oracle.Stream(10, 0, 6, 0.02, top_n=4, beam_threshold=3.0)
    for a, b in [(0, 7), (7, 8), (8, 33), (33, 50)]:
        st.feed(lp[a:b])
    assert st.results() == full


# ---------------------------------------------------------------- merge by max (best alignment)
@pytest.mark.parametrize("seed,T,V,blank,r", [(40, 4, 3, 0, 0.0), (41, 6, 3, 1, 0.0),
                                              (42, 6, 4, 2, 0.0), (43, 6, 4, 0, 0.3),
                                              (44, 5, 4, 3, 0.6)])
def test_merge_max_scores_equal_the_best_alignment_of_each_labelling(seed, T, V, blank, r):
    lp = _rand_logp(seed, T, V, sharp=1.0)
    res = oracle.decode(lp[None], [T], blank, 10000, r, want_masks=True, merge_max=True)
    got = dict(res.hyps(0))
    exact = {k: v for k, v in brute_force(lp, blank, res.keep[0], best_alignment=True).items()
             if v > -math.inf}
    assert set(got) == set(exact)
    for seq, v in exact.items():
        assert got[seq] == pytest.approx(v, abs=1e-9)
    # the sum over alignments can only be larger, and is for a labelling with several of them
    summed = dict(oracle.decode(lp[None], [T], blank, 10000, r).hyps(0))
    assert all(summed[s] >= got[s] - 1e-12 for s in got)
    assert any(summed[s] > got[s] + 1e-6 for s in got)


@pytest.mark.parametrize("K", [1, 3, 50])
def test_merge_max_best_hypothesis_is_the_best_path_whatever_the_beam(K):
    # under max the best partial alignment is the best-scoring prefix at every frame, so it is
    # never cut: top-1 = collapse of the frame-wise argmax, score = sum of the row maxima
    lp = _rand_logp(45, 60, 7, sharp=2.0)
    top = oracle.decode(lp[None], [60], 0, K, 0.0, merge_max=True).hyps(0)[0]
    assert top[0] == greedy(lp, 0)
    assert top[1] == pytest.approx(float(lp.astype(np.float64).max(axis=1).sum()), abs=1e-9)


@pytest.mark.parametrize("K,r,n,theta", [(4, 0.05, 0, 0.0), (8, 0.0, 0, 0.0), (6, 0.01, 3, 4.0)])
def test_merge_max_matches_the_second_implementation(K, r, n, theta):
    em, ln = W.make_small(46, 3, 30, 50, 6)
    res = oracle.decode(em, ln, 0, K, r, top_n=n, beam_threshold=theta, merge_max=True)
    for b in range(3):
        ref = py_decode(em[b, : ln[b]], 0, K, oracle.log_r(r), top_n=n, beam_threshold=theta,
                        merge_max=True)
        got, want = res.hyps(b), ref.results()
        assert [s for s, _ in got] == [s for s, _ in want]
        np.testing.assert_allclose([v for _, v in got], [v for _, v in want], atol=1e-9)


def test_merge_max_streaming_equals_one_shot():
    lp = _rand_logp(47, 40, 8, sharp=1.0)
    full = oracle.decode(lp[None], [40], 0, 5, 0.02, merge_max=True).hyps(0)
    st = oracle.Stream(8, 0, 5, 0.02, merge_max=True)
    for a, b in [(0, 1), (1, 19), (19, 40)]:
        st.feed(lp[a:b])
    assert st.results() == full
