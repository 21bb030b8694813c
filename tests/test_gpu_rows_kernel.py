"""The row kernel (character vocabularies, beams of at most 64, frames pruned inside) against
the oracle, against the general block kernel, and with its instrumented launches: per-frame
survivor masks bit for bit, the bounded probe walks of the fingerprint table."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import check_hyps, masks_from_words
from tests.refs import ctc_forward_logprob
from tests.test_gpu_parity import _binding, _dev

pytestmark = pytest.mark.gpu


def _decoder(V, K, r, B, T, rows=True, **kw):
    bd = _binding()
    d = bd.Decoder(V, 0, K, r, max(B, 1), max(T, 1), **kw)
    d.set_test_hook(bd.FLTOP_HOOK_ROW_KERNEL, None, 1 if rows else 0)
    return d


def _same_hyps(a, b, where, tol=1e-4):
    assert [seq for seq, _ in a] == [seq for seq, _ in b], where
    assert np.allclose([sc for _, sc in a], [sc for _, sc in b], rtol=0, atol=tol), where


def _run(em, ln, K, r, rows=True, nt=0, **kw):
    B, T, V = em.shape
    d = _decoder(V, K, r, B, T, rows, **kw)
    if nt:
        d.set_block_threads(nt)
    d.decode(_dev(em), _dev(np.asarray(ln, dtype=np.int32)))
    torch.cuda.synchronize()
    return d


@pytest.mark.parametrize("V,K,r,top_n", [(32, 50, 1e-3, 0), (32, 50, 0.0, 0), (32, 64, 1e-2, 0),
                                         (32, 8, 0.01, 0), (32, 33, 0.3, 0), (32, 20, 7e-3, 4),
                                         (32, 16, 0.5, 1), (5, 12, 0.05, 2), (2, 4, 0.0, 0),
                                         (17, 1, 0.0, 0), (3, 64, 0.0, 0), (31, 40, 1e-4, 0),
                                         (32, 65, 1e-3, 0), (32, 100, 0.0, 0), (32, 128, 1e-2, 0),
                                         (32, 97, 7e-3, 4), (6, 128, 0.0, 0)])
def test_row_kernel_matches_oracle_and_block_kernel(V, K, r, top_n):
    B = 9
    em, ln = W.make_small(7300 + V + K, B, 70, 70, V)
    T = em.shape[1]
    ln[:8] = [0, 1, 2, 3, 4, T, 17, 40]   # every length the row prefetch starts up on
    em[:, :, :] = np.where(np.arange(T)[None, :, None] < ln[:, None, None], em, np.nan)
    rows = _run(em, ln, K, r, True, top_n=top_n)
    block = _run(em, ln, K, r, False, top_n=top_n)
    assert (rows.status[:B] == 0).all() and (block.status[:B] == 0).all()
    clean = np.nan_to_num(em, nan=0.0)
    res = oracle.decode(clean, ln, 0, K, r, top_n=top_n, want_masks=True)
    for b in range(B):
        check_hyps(rows.hyps(b), res.hyps(b), K, where=f"rows utt {b}", lp=clean[b, : ln[b]],
                   keep=res.keep[b, : ln[b]])
        # the two kernels evaluate the same formulas in the same precision; they move the zero
        # of their relative scores at different frames, so the last bits may differ
        _same_hyps(rows.hyps(b), block.hyps(b), f"utt {b}")
    sr, sb = rows.last_call_stats(), block.last_call_stats()
    for key in ("frames", "survivors", "trie_nodes_created", "live_hypotheses_sum",
                "max_node_ids_used"):
        assert sr[key] == sb[key], key
    rows.close()
    block.close()


@pytest.mark.parametrize("nt", [96, 128, 160, 256, 384, 512, 1024])
def test_row_kernel_result_does_not_depend_on_the_block_size(nt):
    em, ln = W.make_small(7401, 4, 40, 120, 32)
    ref = _run(em, ln, 50, 1e-2)
    got = _run(em, ln, 50, 1e-2, nt=nt)
    assert (got.status[:4] == 0).all()
    for b in range(4):
        assert got.hyps(b) == ref.hyps(b), f"block of {nt} threads changed the result"
    ref.close()
    got.close()


@pytest.mark.parametrize("kernel", ["rows", "block", "warp"])
@pytest.mark.parametrize("r,top_n", [(1e-2, 0), (0.0, 0), (7e-3, 4), (1.0, 0)])
def test_survivor_masks_of_the_fused_kernels_bit_exact(kernel, r, top_n):
    # every kernel that prunes the frames itself writes, in its instrumented launch, the
    # survivor set of each frame: Algorithm 1's top-N stage and conditional break, bit for bit
    bd = _binding()
    V, K, B = 32, 16, 7
    em, ln = W.make_small(7500, B, 5, 90, V)
    T = em.shape[1]
    d = _decoder(V, K, r, B, T, rows=(kernel == "rows"), top_n=top_n)
    d.set_warp_decode(2 if kernel == "warp" else 0)
    words = torch.from_numpy(np.full((B, T), 0xdeadbeef, dtype=np.uint32).view(np.int32)).cuda()
    d.set_test_hook(bd.FLTOP_HOOK_SURVIVOR_MASKS, words)
    d.decode(_dev(em), _dev(ln))
    torch.cuda.synchronize()
    got = words.cpu().numpy().view(np.uint32)
    for b in range(B):
        n = int(ln[b])
        okeep, _ = oracle.prune(em[b, :n], r, top_n=top_n)
        assert (masks_from_words(got[b, :n], V) == okeep).all(), f"{kernel} utt {b}"
        assert (got[b, n:] == np.uint32(0xdeadbeef)).all()      # frames past the length: untouched
    d.close()


def test_full_fingerprint_table_is_reported_not_spun_on():
    # a table with fewer slots than beam entries: inserts find no free slot, their bounded
    # probe walks run out, and the utterance is flagged; every output stays in bounds
    bd = _binding()
    em, ln = W.make_small(7600, 3, 30, 50, 32)
    B, T, V = em.shape
    for rows in (True, False):
        d = _decoder(V, 24, 1e-2, B, T, rows)
        d.set_test_hook(bd.FLTOP_HOOK_TABLE_SLOTS, None, 8)
        d.decode(_dev(em), _dev(ln))
        torch.cuda.synchronize()
        st = d.status.cpu().numpy()[:B]
        assert (st & bd.FLTOP_ST_INTERNAL).all(), st
        nh = d.nhyp.cpu().numpy()[:B]
        assert (nh >= 1).all() and (nh <= 24).all()
        assert (d.lens.cpu().numpy()[:B] <= T).all()
        d.set_test_hook(bd.FLTOP_HOOK_TABLE_SLOTS, None, 0)   # back to the full table
        d.decode(_dev(em), _dev(ln))
        torch.cuda.synchronize()
        assert (d.status.cpu().numpy()[:B] == 0).all()
        d.close()
    d = _decoder(V, 24, 1e-2, B, T)
    with pytest.raises(bd.FltopError):
        d.set_test_hook(bd.FLTOP_HOOK_TABLE_SLOTS, None, 12)    # not a power of two
    with pytest.raises(bd.FltopError):
        d.set_test_hook(99, None, 0)
    d.close()


def test_row_kernel_near_equal_scores_and_exact_ties():
    # nearly flat rows crowd the cut bin beyond what the pairwise ranking takes (the exact
    # bit-by-bit selection runs); constant rows tie exactly
    rng = np.random.default_rng(12)
    B, T, V = 3, 12, 16
    for spread in (0.02, 0.001):
        x = rng.standard_normal((B, T, V)) * spread
        em = (x - np.log(np.exp(x).sum(-1, keepdims=True))).astype(np.float32)
        ln = np.array([T, T - 3, 5], dtype=np.int32)
        for K, r in [(8, 0.0), (20, 0.5), (64, 0.0)]:
            d = _run(em, ln, K, r)
            res = oracle.decode(em, ln, 0, K, r, want_masks=True)
            for b in range(B):
                check_hyps(d.hyps(b), res.hyps(b), K, max_unmatched_frac=0.3,
                           where=f"flat utt {b} K={K}", lp=em[b, : ln[b]],
                           keep=res.keep[b, : ln[b]])
            d.close()
    # constant rows over the whole vocabulary: hundreds of candidates tie exactly, which no
    # binning can separate - the bit-by-bit selection has to run
    em = np.full((1, 4, 32), np.log(1.0 / 32), dtype=np.float32)
    ln = np.array([4], dtype=np.int32)
    d = _run(em, ln, 50, 0.0)
    assert d.last_call_stats()["exact_select_frames"] > 0 and int(d.status[0]) == 0
    ref = oracle.decode(em, ln, 0, 50, 0.0).hyps(0)
    got = d.hyps(0)
    assert len(got) == 50 and len(set(s for s, _ in got)) == 50
    for seq, sc in got:
        assert sc <= ctc_forward_logprob(em[0], seq, 0) + 1e-3
    np.testing.assert_allclose(sorted(s for _, s in got), sorted(s for _, s in ref), atol=1e-3)
    d.close()
    Tt, Vt, Kt = 5, 4, 6
    em = np.full((1, Tt, Vt), np.log(1.0 / Vt), dtype=np.float32)
    ln = np.array([Tt], dtype=np.int32)
    full = dict(oracle.decode(em, ln, 0, 100000, 0.0).hyps(0))      # every labelling, exact
    d = _run(em, ln, Kt, 0.0)
    ref = oracle.decode(em, ln, 0, Kt, 0.0).hyps(0)
    got = d.hyps(0)
    assert len(got) == Kt and len(set(s for s, _ in got)) == Kt
    for seq, sc in got:
        assert sc <= full[seq] + 1e-3
    np.testing.assert_allclose(sorted(s for _, s in got), sorted(s for _, s in ref), atol=1e-3)
    d.close()


def test_row_kernel_more_utterances_than_sms():
    # blocks share SMs (smaller blocks, the 64-register instantiation), beams of exactly 64
    # with one surviving token per frame
    B, V, K = 160, 32, 64
    em, ln = W.make_small(7700, B, 6, 30, V)
    d = _run(em, ln, K, 0.0, top_n=1)
    assert (d.status[:B] == 0).all()
    sample = [0, 1, 77, 159]
    res = oracle.decode(em[sample], ln[sample], 0, K, 0.0, top_n=1)
    for i, b in enumerate(sample):
        check_hyps(d.hyps(b), res.hyps(i), K, where=f"utt {b}")
    d.close()


@pytest.mark.parametrize("C,K", [(1, 40), (3, 40), (16, 40), (5, 100)])
def test_row_kernel_streaming_equals_one_shot(C, K):
    V, r, B = 32, 1e-2, 6
    em, ln = W.make_small(7800 + C, B, 5, 70, V)
    T = em.shape[1]
    x = _dev(em)
    one = _run(em, ln, K, r)
    d = _decoder(V, K, r, B, T, max_chunk_frames=C)
    n_chunks = (T + C - 1) // C
    for i in range(n_chunks):
        t0 = i * C
        chunk = torch.zeros((B, C, V), dtype=torch.float32, device="cuda")
        w = min(C, T - t0)
        chunk[:, :w] = x[:, t0: t0 + w]
        clen = np.clip(ln - t0, 0, C).astype(np.int32)
        flags = np.full(B, (1 if i == 0 else 0) | (2 if i == n_chunks - 1 else 0), dtype=np.uint8)
        d.stream_step(chunk, _dev(clen), _dev(flags))
    torch.cuda.synchronize()
    assert torch.equal(one.nhyp[:B], d.nhyp[:B])
    for b in range(B):
        # (a run of blank-only frames is cut at a chunk boundary: last bits may differ)
        _same_hyps(one.hyps(b), d.hyps(b), f"stream {b}")
    one.close()
    d.close()


def test_block_kernel_with_fewer_stay_lanes_than_beam_entries():
    # small blocks asked for by hand leave the general kernel fewer stay lanes than the beam
    # has entries; every stay candidate must still be placed
    em, ln = W.make_small(7900, 3, 40, 90, 32)
    for K in (50, 100, 200):
        res = oracle.decode(em, ln, 0, K, 1e-2, want_masks=True)
        for nt in (96, 128, 160, 192):
            d = _run(em, ln, K, 1e-2, rows=False, nt=nt)
            assert (d.status[:3] == 0).all()
            for b in range(3):
                check_hyps(d.hyps(b), res.hyps(b), K, where=f"K={K} nt={nt} utt {b}",
                           lp=em[b, : ln[b]], keep=res.keep[b, : ln[b]])
            d.close()
    # the library's own sizing when blocks share SMs and one token survives a frame
    B, K = 200, 64
    em, ln = W.make_small(7901, B, 6, 24, 32)
    d = _run(em, ln, K, 0.0, rows=False, top_n=1)
    sample = [0, 99, 199]
    res = oracle.decode(em[sample], ln[sample], 0, K, 0.0, top_n=1)
    for i, b in enumerate(sample):
        check_hyps(d.hyps(b), res.hyps(i), K, where=f"utt {b}")
    d.close()


def test_trie_capacity_knob_and_lazy_survivor_lists():
    # max_trie_nodes: a capacity below the worst case holds less memory and changes nothing as
    # long as it suffices; one that runs out is reported per utterance, never written past
    bd = _binding()
    wl = W.workload_wav2vec2(batch=8)
    B, T, V = wl.emissions.shape
    K, r = 50, 1e-3
    full = _run(wl.emissions, wl.lengths, K, r)
    used = full.last_call_stats()["max_node_ids_used"]
    assert used < 0.5 * K * T
    half = _run(wl.emissions, wl.lengths, K, r, max_trie_nodes=K * T // 2)
    assert half.beam_state_bytes < 0.55 * full.beam_state_bytes
    assert (half.status[:B] == 0).all()
    for b in range(B):
        assert half.hyps(b) == full.hyps(b)
    short = _run(wl.emissions, wl.lengths, K, r, max_trie_nodes=used // 2)
    st = short.status.cpu().numpy()[:B]
    assert (st & bd.FLTOP_ST_ARENA_FULL).any() and not (st & ~bd.FLTOP_ST_ARENA_FULL).any()
    assert (short.lens.cpu().numpy()[:B] <= T).all()
    # survivor lists exist only once a call takes the separate prune kernel
    before = half.beam_state_bytes
    half.set_fusion(0)
    half.decode(_dev(wl.emissions), _dev(wl.lengths))
    torch.cuda.synchronize()
    assert half.beam_state_bytes >= before + B * T * V * 8
    for b in range(B):
        _same_hyps(half.hyps(b), full.hyps(b), f"utt {b}")
    for d in (full, half, short):
        d.close()
