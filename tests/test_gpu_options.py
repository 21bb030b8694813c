"""N (top-N stage) and beam_threshold of Algorithm 1 on the CUDA path vs the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import TOL, check_hyps, masks_from_entries
from tests.test_gpu_parity import _binding, _dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("V,r,n", [(32, 0.0, 4), (32, 1e-3, 4), (32, 0.0, 1), (32, 0.0, 31),
                                   (1024, 1e-3, 4), (1024, 0.0, 40), (1024, 0.0, 700),
                                   (260, 1e-2, 16), (5, 0.0, 2), (48, 0.0, 48), (48, 0.0, 100)])
def test_top_n_survivors_bit_exact(V, r, n):
    B, T = 4, 29
    em, ln = W.make_small(500 + V + n, B, T, T, V)
    em[0, 3, :] = em[0, 3, 0]                      # exact ties: the lowest ids must stay
    em[1, 5, 1:4] = em[1, 5].max() + 0.5           # a three-way tie for first place
    d = _binding().Decoder(V, 0, 2, r, B, T, top_n=n)
    counts, entries = d.prune(_dev(em), _dev(ln))
    torch.cuda.synchronize()
    keep, vals = masks_from_entries(counts.cpu().numpy(), entries.cpu().numpy(), V)
    for b in range(B):
        okeep, ocnt = oracle.prune(em[b], r, top_n=n)
        assert (counts[b].cpu().numpy() == ocnt).all()
        assert (keep[b] == okeep).all()
        assert np.array_equal(vals[b][okeep], em[b][okeep])
    d.close()


def _compare(em, ln, K, r, top_n=0, theta=0.0, frac=0.0, merge_max=False):
    """Every utterance against the oracle.  With a beam threshold the two sides may differ on
    hypotheses within the tolerance of the threshold, so the beams are compared there as sets."""
    B, T, V = em.shape
    d = _binding().Decoder(V, 0, K, r, B, T, top_n=top_n, beam_threshold=theta,
                           merge_max=merge_max)
    d.decode(_dev(em), _dev(ln))
    torch.cuda.synchronize()
    assert (d.status.cpu().numpy()[:B] == 0).all()
    st = d.last_call_stats()
    res = oracle.decode(em, ln, 0, K, r, top_n=top_n, beam_threshold=theta, merge_max=merge_max,
                        want_masks=True)
    res.mean_live = st["live_hypotheses_sum"] / max(1, st["frames"])
    for b in range(B):
        g, o = d.hyps(b), res.hyps(b)
        if theta <= 0:
            check_hyps(g, o, K, max_unmatched_frac=frac, where=f"utt {b}", lp=em[b, : ln[b]],
                       keep=res.keep[b, : ln[b]])
            continue
        gm, om = dict(g), dict(o)
        assert g[0][0] == o[0][0] or abs(o[0][1] - o[1][1]) < TOL
        floor = o[0][1] - theta
        assert all(s >= g[0][1] - theta - TOL for _, s in g) and len(g) <= K
        for seq, sc in o:
            if seq in gm:
                assert abs(gm[seq] - sc) <= TOL
            else:
                assert sc <= floor + TOL or (len(o) == K and sc <= o[-1][1] + TOL), (b, sc, floor)
        for seq, sc in g:
            assert seq in om or sc <= floor + TOL or (len(o) == K and sc <= o[-1][1] + TOL), (b, sc, floor)
    d.close()
    return res


@pytest.mark.parametrize("V,K,r,n", [(32, 8, 0.01, 4), (32, 50, 1e-3, 4), (32, 20, 0.0, 2),
                                     (8, 6, 0.0, 1), (1024, 16, 1e-3, 8), (40, 12, 0.007, 4)])
def test_decode_with_top_n_matches_oracle(V, K, r, n):
    em, ln = W.make_small(900 + V + K, 5, 30, 110, V)
    _compare(em, ln, K, r, top_n=n)


@pytest.mark.parametrize("V,K,r,theta", [(32, 16, 0.01, 5.0), (32, 50, 1e-3, 25.0), (8, 12, 0.0, 1.0),
                                         (32, 50, 1e-3, 2.0), (6, 8, 0.05, 0.3), (32, 8, 0.0, 1e9)])
def test_decode_with_beam_threshold_matches_oracle(V, K, r, theta):
    em, ln = W.make_small(1200 + V + K, 5, 30, 110, V)
    res = _compare(em, ln, K, r, theta=theta)
    if theta == 0.3:
        assert (res.nhyp < K).any()        # the threshold really shortens some beams


def test_beam_threshold_shortens_the_beam_on_peaky_frames():
    # prefixes held per frame (the paper's "beams") against the second implementation
    from tests.refs import PyPrefixSearch
    wl = W.workload_pr1()
    lp = wl.emissions[0]
    for theta in (0.0, 3.0, 1.0):
        got = _compare(wl.emissions, wl.lengths, 8, 0.01, theta=theta).mean_live
        ref, held = PyPrefixSearch(0, 8, theta), 0
        for t in range(lp.shape[0]):
            thr = np.float32(lp[t].max()) + oracle.log_r(0.01)
            ref.step(lp[t], [c for c in range(32) if lp[t, c] >= thr])
            held += len(ref.beam)
        assert abs(got - held / lp.shape[0]) < 0.02, (theta, got, held / lp.shape[0])
        assert theta == 0.0 or got < 7.0


def test_paper_operating_point_on_the_wav2vec2_shape():
    # N = 4, R = 0.007, beam_threshold = 25 (Sections 4.2 and 4.3), beam 50, sampled utterances
    wl = W.workload_wav2vec2(batch=16)
    sample = [int(i) for i in np.argsort(wl.lengths)[:6]]
    _compare(wl.emissions[sample], wl.lengths[sample], 50, 0.007, top_n=4, theta=25.0)


def test_streaming_with_options_equals_one_shot():
    V, K, r, C = 32, 12, 0.01, 9
    em, ln = W.make_small(66, 4, 40, 100, V)
    B, T, _ = em.shape
    one = _binding().Decoder(V, 0, K, r, B, T, top_n=3, beam_threshold=2.0)
    one.decode(_dev(em), _dev(ln))
    st = _binding().Decoder(V, 0, K, r, B, T, max_chunk_frames=C, top_n=3, beam_threshold=2.0)
    x = _dev(em)
    n_chunks = (T + C - 1) // C
    for i in range(n_chunks):
        t0 = i * C
        chunk = torch.zeros((B, C, V), dtype=torch.float32, device="cuda")
        w = min(C, T - t0)
        chunk[:, :w] = x[:, t0: t0 + w]
        clen = np.clip(ln - t0, 0, C).astype(np.int32)
        flags = np.full(B, (1 if i == 0 else 0) | (2 if i == n_chunks - 1 else 0), dtype=np.uint8)
        st.stream_step(chunk, _dev(clen), _dev(flags))
    torch.cuda.synchronize()
    assert torch.equal(one.nhyp[:B], st.nhyp[:B]) and torch.equal(one.scores[:B], st.scores[:B])
    for b in range(B):
        assert one.hyps(b) == st.hyps(b)


# ------------------------------------------------------------------ merge by max
@pytest.mark.parametrize("V,K,r,n,theta", [(32, 50, 1e-3, 0, 0.0), (32, 20, 0.0, 0, 0.0),
                                           (32, 8, 0.01, 4, 0.0), (1024, 16, 1e-3, 0, 0.0),
                                           (32, 300, 1e-3, 0, 0.0), (12, 10, 0.02, 3, 6.0)])
def test_decode_with_merge_max_matches_oracle(V, K, r, n, theta):
    em, ln = W.make_small(1500 + V + K, 5, 30, 110, V)
    _compare(em, ln, K, r, top_n=n, theta=theta, merge_max=True)


def test_merge_max_best_hypothesis_is_the_best_path():
    # closed form: under max the best prefix is the collapse of the frame-wise argmax and its
    # score the sum of the row maxima, at any beam width
    em, ln = W.make_small(1600, 6, 40, 160, 32)
    for K in (1, 7, 50):
        d = _binding().Decoder(32, 0, K, 0.0, 6, em.shape[1], merge_max=True)
        d.decode(_dev(em), _dev(ln))
        torch.cuda.synchronize()
        for b in range(6):
            row = em[b, : ln[b]]
            seq, sc = d.hyps(b)[0]
            path, prev = [], None
            for c in row.argmax(axis=1):
                if c != prev and c != 0:
                    path.append(int(c))
                prev = c
            assert list(seq) == path
            assert abs(sc - float(row.astype(np.float64).max(axis=1).sum())) <= TOL
        d.close()


def test_merge_max_streaming_equals_one_shot():
    em, ln = W.make_small(1700, 4, 20, 90, 32)
    T = em.shape[1]
    one = _binding().Decoder(32, 0, 12, 1e-2, 4, T, merge_max=True)
    one.decode(_dev(em), _dev(ln))
    st = _binding().Decoder(32, 0, 12, 1e-2, 4, T, max_chunk_frames=8, merge_max=True)
    x = _dev(em)
    n_chunks = (T + 7) // 8
    for i in range(n_chunks):
        chunk = torch.zeros((4, 8, 32), dtype=torch.float32, device="cuda")
        w = min(8, T - 8 * i)
        chunk[:, :w] = x[:, 8 * i: 8 * i + w]
        clen = np.clip(ln - 8 * i, 0, 8).astype(np.int32)
        flags = np.full(4, (1 if i == 0 else 0) | (2 if i == n_chunks - 1 else 0), dtype=np.uint8)
        st.stream_step(chunk, _dev(clen), _dev(flags))
    torch.cuda.synchronize()
    for b in range(4):
        assert one.hyps(b) == st.hyps(b)
    one.close()
    st.close()
