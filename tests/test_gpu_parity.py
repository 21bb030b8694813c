"""CUDA library vs CPU oracle, element by element, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import TOL, check_hyps, masks_from_entries

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2510_09085_b200 import binding
    return binding


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def gpu_decode(em, ln, blank, K, r, max_out_len=None):
    B, T, V = em.shape
    d = _binding().Decoder(V, blank, K, r, max(B, 1), max(T, 1), max_out_len=max_out_len)
    d.decode(_dev(em), _dev(np.asarray(ln, dtype=np.int32)))
    torch.cuda.synchronize()
    return d


def compare_batch(em, ln, blank, K, r, utterances=None, max_unmatched_frac=0.0):
    d = gpu_decode(em, ln, blank, K, r)
    status = d.status.cpu().numpy()
    sel = range(len(ln)) if utterances is None else utterances
    assert (status[: len(ln)] == 0).all(), status
    res = oracle.decode(em[list(sel)], np.asarray(ln)[list(sel)], blank, K, r, want_masks=True)
    swaps = 0
    for i, b in enumerate(sel):
        n = int(ln[b])
        swaps += check_hyps(d.hyps(b), res.hyps(i), K, max_unmatched_frac=max_unmatched_frac,
                            where=f"utt {b} K={K} r={r}", lp=em[b, :n], keep=res.keep[i, :n],
                            blank=blank)
    d.close()
    return swaps


# ------------------------------------------------------------------ prune: bit exact
@pytest.mark.parametrize("V,r", [(32, 1e-3), (32, 0.0), (32, 1.0), (1024, 1e-3), (1024, 0.0),
                                 (5, 0.05), (48, 0.01), (100, 0.2), (2, 0.5), (260, 1e-2),
                                 (2048, 1e-3), (4100, 1e-3)])
def test_prune_masks_bit_exact(V, r):
    B, T = 5, 37
    em, ln = W.make_small(100 + V, B, 0, T, V)
    T = em.shape[1]
    ln[0] = T
    em[:, :, :] = np.where(np.arange(T)[None, :, None] < ln[:, None, None], em, np.nan)
    d = _binding().Decoder(V, 0, 2, r, B, max(T, 1))
    counts, entries = d.prune(_dev(em), _dev(ln))
    torch.cuda.synchronize()
    keep, vals = masks_from_entries(counts.cpu().numpy(), entries.cpu().numpy(), V)
    for b in range(B):
        n = ln[b]
        okeep, ocnt = oracle.prune(em[b, :n], r)
        assert (counts[b, :n].cpu().numpy() == ocnt).all()
        assert (counts[b, n:].cpu().numpy() == 0).all()
        assert (keep[b, :n] == okeep).all()
        assert np.array_equal(vals[b, :n][okeep], em[b, :n][okeep])
    d.close()


def test_prune_strided_and_unaligned_rows():
    V = 32
    em, ln = W.make_small(3, 4, 20, 50, V)
    B, T, _ = em.shape
    wide = torch.zeros((B, T, V + 5), dtype=torch.float32, device="cuda")
    view = wide[:, :, 3: 3 + V]                     # rows neither packed nor 16-byte aligned
    view.copy_(_dev(em))
    d = _binding().Decoder(V, 0, 4, 0.01, B, T)
    counts, entries = d.prune(view, _dev(ln))
    d.decode(view, _dev(ln))
    torch.cuda.synchronize()
    keep, _ = masks_from_entries(counts.cpu().numpy(), entries.cpu().numpy(), V)
    res = oracle.decode(em, ln, 0, 4, 0.01, want_masks=True)
    for b in range(B):
        assert (keep[b, : ln[b]] == res.keep[b, : ln[b]]).all()
        check_hyps(d.hyps(b), res.hyps(b), 4, where=f"strided utt {b}")
    d.close()


# ------------------------------------------------------------------ decode: small cases
@pytest.mark.parametrize("V,K,r", [(5, 3, 0.05), (5, 4, 0.0), (5, 8, 0.2), (8, 16, 0.01),
                                   (32, 8, 0.01), (32, 50, 1e-3), (32, 50, 0.0), (3, 2, 0.0),
                                   (2, 4, 0.0), (64, 5, 1e-4), (6, 1, 0.0), (6, 200, 0.0),
                                   (40, 33, 0.3), (12, 600, 0.0)])
def test_decode_small_matches_oracle(V, K, r):
    em, ln = W.make_small(1000 + 7 * V + K, 6, 30, 140, V)
    compare_batch(em, ln, 0, K, r)


def test_decode_nonzero_blank_and_sharp_inputs():
    rc = W.EmissionRecipe(vocab_size=16, blank_id=9, hard_fraction=0.25, boost_easy=5.0,
                          boost_hard=3.0, boost_comp=2.5)
    em, ln = W.make_batch(21, [80, 3, 1, 200, 64], rc)
    for K, r in [(6, 0.02), (6, 0.0), (40, 0.3)]:
        compare_batch(em, ln, 9, K, r)


def test_prefixes_that_leave_and_reenter_the_beam():
    # small beams on flat inputs: prefixes are evicted and derived again later, so
    # one trie node per token sequence is required for the merge to stay exact
    from tests.refs import py_decode
    em, ln = W.make_small(9, 4, 30, 60, 5)
    revivals = sum(py_decode(em[b, : ln[b]], 0, 4, oracle.log_r(0.05)).revivals for b in range(4))
    assert revivals > 0
    compare_batch(em, ln, 0, 4, 0.05)
    compare_batch(em, ln, 0, 3, 0.0)


def test_pr1_reference_config():
    wl = W.workload_pr1()
    for r in wl.thresholds:
        compare_batch(wl.emissions, wl.lengths, wl.blank_id, wl.beam_width, r)


# ------------------------------------------------------------------ edge cases
def test_empty_ragged_and_invalid_lengths():
    V, K = 8, 5
    em, _ = W.make_small(5, 5, 40, 40, V)
    ln = np.array([0, 40, 1, 41, -3], dtype=np.int32)
    d = gpu_decode(em, ln, 0, K, 0.01)
    st = d.status.cpu().numpy()
    assert st[:5].tolist() == [0, 0, 0, 1, 1]
    assert d.hyps(0) == [((), 0.0)]
    assert d.nhyp[3] == 0 and d.nhyp[4] == 0
    assert (d.lens[3] == 0).all() and torch.isinf(d.scores[3]).all()
    res = oracle.decode(em[1:3], ln[1:3], 0, K, 0.01)
    check_hyps(d.hyps(1), res.hyps(0), K)
    check_hyps(d.hyps(2), res.hyps(1), K)
    n = int(d.nhyp[2])
    assert (d.lens[2, n:] == 0).all() and torch.isinf(d.scores[2, n:]).all()
    d.close()


def test_padding_is_never_read():
    em, ln = W.make_small(13, 4, 10, 60, 6)
    a = gpu_decode(em, ln, 0, 5, 0.01)
    em2 = em.copy()
    for b in range(4):
        em2[b, ln[b]:] = np.nan
    b_ = gpu_decode(em2, ln, 0, 5, 0.01)
    assert torch.equal(a.lens, b_.lens) and torch.equal(a.scores, b_.scores)
    for b in range(4):
        assert a.hyps(b) == b_.hyps(b)


def test_truncated_output_reports_true_length():
    em, ln = W.make_small(17, 2, 100, 100, 6)
    full = gpu_decode(em, ln, 0, 4, 0.0)
    cut = gpu_decode(em, ln, 0, 4, 0.0, max_out_len=3)
    assert torch.equal(full.lens, cut.lens)
    assert (cut.status[:2].cpu().numpy() & 4).all()
    for b in range(2):
        for k in range(int(full.nhyp[b])):
            assert torch.equal(full.tokens[b, k, :3], cut.tokens[b, k, :3]) or full.lens[b, k] < 3


def test_run_to_run_determinism():
    wl = W.workload_wav2vec2(batch=8)
    a = gpu_decode(wl.emissions, wl.lengths, 0, 50, 1e-3)
    b = gpu_decode(wl.emissions, wl.lengths, 0, 50, 1e-3)
    assert torch.equal(a.scores, b.scores) and torch.equal(a.lens, b.lens)
    assert torch.equal(a.nhyp, b.nhyp)
    for u in range(8):
        assert a.hyps(u) == b.hyps(u)


def test_host_side_argument_errors():
    bd = _binding()
    cfg = bd.make_config(32, 0, 8, 0.01, 4, 100)
    code, h = bd.fltop_create(cfg)
    assert code == bd.FLTOP_OK
    x = torch.zeros((4, 100, 32), device="cuda")
    ln = torch.zeros(4, dtype=torch.int32, device="cuda")
    tok = torch.zeros((4, 8, 100), dtype=torch.int32, device="cuda")
    le = torch.zeros((4, 8), dtype=torch.int32, device="cuda")
    sc = torch.zeros((4, 8), device="cuda")
    nh = torch.zeros(4, dtype=torch.int32, device="cuda")
    ok = (h, x, 3200, 32, ln, 4, 100, tok, le, sc, nh)
    assert bd.fltop_decode(*ok) == bd.FLTOP_OK
    assert bd.fltop_decode(h, x, 3200, 32, ln, 5, 100, tok, le, sc, nh) == bd.FLTOP_ERR_CAPACITY
    assert bd.fltop_decode(h, x, 3200, 32, ln, 4, 101, tok, le, sc, nh) == bd.FLTOP_ERR_CAPACITY
    assert bd.fltop_decode(h, None, 3200, 32, ln, 4, 100, tok, le, sc, nh) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.fltop_decode(h, x, 3200, 31, ln, 4, 100, tok, le, sc, nh) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.fltop_decode(h, x, 3200, 32, ln, 4, 100, tok, le, None, nh) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.fltop_decode(h, x, 3200, 32, ln, 0, 100, tok, le, sc, nh) == bd.FLTOP_OK
    assert bd.fltop_stream_step(h, x, ln, None, 4, 16, tok, le, sc, nh) == bd.FLTOP_ERR_STATE
    torch.cuda.synchronize()
    assert bd.fltop_destroy(h) == bd.FLTOP_OK
    # caller-provided workspace
    need = bd.fltop_workspace_size(cfg)
    ws = torch.empty(need + 256, dtype=torch.uint8, device="cuda")
    base = (ws.data_ptr() + 255) // 256 * 256
    small = bd.make_config(32, 0, 8, 0.01, 4, 100, workspace=base, workspace_bytes=need - 1)
    assert bd.fltop_create(small)[0] == bd.FLTOP_ERR_OOM
    own = bd.make_config(32, 0, 8, 0.01, 4, 100, workspace=base, workspace_bytes=need)
    code, h2 = bd.fltop_create(own)
    assert code == bd.FLTOP_OK
    assert bd.fltop_decode(h2, x, 3200, 32, ln, 4, 100, tok, le, sc, nh) == bd.FLTOP_OK
    torch.cuda.synchronize()
    assert bd.fltop_destroy(h2) == bd.FLTOP_OK


# ------------------------------------------------------------------ crowded cut / ties
def test_many_near_equal_scores_take_the_exact_select_path():
    # nearly flat rows: the candidates of a frame fall into very few score-histogram
    # bins, so the cut bin holds far more members than the pairwise ranking handles
    rng = np.random.default_rng(5)
    B, T, V = 3, 14, 16
    x = rng.standard_normal((B, T, V)) * 0.02
    em = (x - np.log(np.exp(x).sum(-1, keepdims=True))).astype(np.float32)
    ln = np.array([T, T - 3, 5], dtype=np.int32)
    for K, r in [(8, 0.0), (20, 0.5), (100, 0.0)]:
        d = gpu_decode(em, ln, 0, K, r)
        res = oracle.decode(em, ln, 0, K, r, want_masks=True)
        for b in range(B):
            check_hyps(d.hyps(b), res.hyps(b), K, max_unmatched_frac=0.3,
                       where=f"flat utt {b} K={K}", lp=em[b, : ln[b]], keep=res.keep[b, : ln[b]])
        d.close()


@pytest.mark.parametrize("spread", [0.02, 0.001])
def test_wide_beam_with_a_crowded_cut_bin(spread):
    # wide beams split a crowded cut bin a second time; at the larger spread the finer bins
    # separate the candidates, at the smaller one even those stay crowded and the exact
    # selection has to finish the job
    rng = np.random.default_rng(6)
    B, T, V = 2, 12, 16
    x = rng.standard_normal((B, T, V)) * spread
    em = (x - np.log(np.exp(x).sum(-1, keepdims=True))).astype(np.float32)
    ln = np.array([T, T - 2], dtype=np.int32)
    for K in (300, 700):
        d = gpu_decode(em, ln, 0, K, 0.0)
        res = oracle.decode(em, ln, 0, K, 0.0)
        for b in range(B):
            check_hyps(d.hyps(b), res.hyps(b), K, max_unmatched_frac=0.3,
                       where=f"flat wide utt {b} K={K} spread={spread}", lp=em[b, : ln[b]])
        d.close()


def test_exact_ties_keep_a_valid_beam():
    # constant rows: every extension of a prefix ties exactly.  Which of the tied
    # candidates survive is not unique; every kept hypothesis must carry its exact
    # score and no dropped hypothesis may beat a kept one.
    T, V, K = 5, 4, 6
    em = np.full((1, T, V), np.log(1.0 / V), dtype=np.float32)
    ln = np.array([T], dtype=np.int32)
    full = dict(oracle.decode(em, ln, 0, 100000, 0.0).hyps(0))      # every labelling, exact
    d = gpu_decode(em, ln, 0, K, 0.0)
    ref = oracle.decode(em, ln, 0, K, 0.0).hyps(0)
    got = d.hyps(0)
    assert len(got) == K and len(set(s for s, _ in got)) == K
    # finite-beam scores are lower bounds of the exact ones and the score lists agree
    for seq, sc in got:
        assert sc <= full[seq] + TOL
    np.testing.assert_allclose(sorted(s for _, s in got), sorted(s for _, s in ref), atol=TOL)
    d.close()


# ------------------------------------------------------------------ launch shape / large V
def test_results_do_not_depend_on_the_block_size():
    # threads per utterance block is a tuning knob: every setting must give the same beam
    em, ln = W.make_small(31, 4, 40, 120, 32)
    ref = None
    for nt in (96, 128, 256, 512, 1024):
        B, T, V = em.shape
        d = _binding().Decoder(V, 0, 20, 1e-2, B, T)
        d.set_block_threads(nt)
        d.decode(_dev(em), _dev(ln))
        torch.cuda.synchronize()
        assert (d.status.cpu().numpy()[:B] == 0).all()
        got = [d.hyps(b) for b in range(B)]
        if ref is None:
            ref = got
        else:
            assert got == ref, f"block of {nt} threads changed the result"
        d.close()


def _embed_in_large_vocabulary(em5, V, ids):
    """A 5-token emission matrix spread over a V-token vocabulary (the other tokens get a
    negligible but non-zero probability), renormalised in float64."""
    B, T, _ = em5.shape
    p = np.full((B, T, V), 1e-13, dtype=np.float64)
    p[:, :, ids] = np.exp(em5.astype(np.float64))
    p /= p.sum(-1, keepdims=True)
    return np.log(p).astype(np.float32)


def test_large_vocabulary_prefixes_leave_and_reenter():
    # token ids far above 64 with a tiny beam on flat rows: prefixes are evicted and derived
    # again, and every re-entry must merge with its descendants still in the beam
    from tests.refs import py_decode
    em5, ln = W.make_small(9, 4, 30, 60, 5)
    em = _embed_in_large_vocabulary(em5, 300, [0, 7, 70, 150, 299])
    revivals = sum(py_decode(em[b, : ln[b]], 0, 4, oracle.log_r(0.05)).revivals for b in range(4))
    assert revivals > 0
    compare_batch(em, ln, 0, 4, 0.05)
    compare_batch(em, ln, 0, 3, 0.0)


@pytest.mark.parametrize("V,K,r", [(32, 1024, 0.0), (32, 1500, 1e-3), (4096, 4, 1e-3), (2048, 16, 0.0)])
def test_largest_shapes_fit_and_match(V, K, r):
    # beam widths and vocabularies near what one SM's shared memory holds (generic layout,
    # radix fallback for the wide beams), on short utterances so that the oracle stays quick
    em, ln = W.make_small(4000 + V + K, 2, 6, 14, V)
    compare_batch(em, ln, 0, K, r, max_unmatched_frac=0.25)


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16])
@pytest.mark.parametrize("V", [256, 640, 1024])
def test_prune_through_the_shared_memory_ring_bit_exact(V, dtype):
    # the staged variant of the prune kernel (rows fetched by asynchronous bulk copies into a
    # ring in shared memory, bounded waits): same survivors, bit for bit, and no wait ran out
    bd = _binding()
    if dtype == torch.float16 and V == 256:
        pytest.skip("rows below 1 KB are not staged")
    B, T = 7, 41
    em, ln = W.make_small(300 + V, B, 0, T, V)
    T = em.shape[1]
    ln[0], ln[1] = T, 0
    x = torch.from_numpy(em).to(dtype).cuda()
    wide = x.float().cpu().numpy()
    d = bd.Decoder(V, 0, 2, 1e-2, B, max(T, 1), emission_dtype=dtype)
    d.set_test_hook(bd.FLTOP_HOOK_PRUNE_STAGING, None, 1)
    counts, entries = d.prune(x, _dev(ln))
    d.set_fusion(0)
    d.decode(x, _dev(ln))
    torch.cuda.synchronize()
    keep, vals = masks_from_entries(counts.cpu().numpy(), entries.cpu().numpy(), V)
    for b in range(B):
        n = ln[b]
        okeep, ocnt = oracle.prune(wide[b, :n], 1e-2)
        assert (counts[b, :n].cpu().numpy() == ocnt).all() and (counts[b, n:].cpu().numpy() == 0).all()
        assert (keep[b, :n] == okeep).all()
        assert np.array_equal(vals[b, :n][okeep], wide[b, :n][okeep])
    assert d.last_call_stats()["prune_copy_timeouts"] == 0
    d.close()
