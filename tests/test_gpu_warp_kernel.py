"""The warp-per-utterance decode kernel (narrow beams over narrow vocabularies), forced on:
against the oracle, against the block kernel, in batch and streaming form, on the degenerate
inputs, and on a stream count where the library picks it by itself."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import check_hyps
from tests.test_gpu_parity import _binding, _dev

pytestmark = pytest.mark.gpu


def _decoder(V, K, r, B, T, warp, **kw):
    d = _binding().Decoder(V, 0, K, r, max(B, 1), max(T, 1), **kw)
    d.set_warp_decode(2 if warp else 0)
    return d


def _run(em_dev, ln, V, K, r, warp, **kw):
    B, T = em_dev.shape[:2]
    d = _decoder(V, K, r, B, T, warp, **kw)
    d.decode(em_dev, _dev(np.asarray(ln, dtype=np.int32)))
    torch.cuda.synchronize()
    return d


@pytest.mark.parametrize("V,K,r,n", [(32, 10, 1e-3, 0), (32, 32, 1e-3, 0), (32, 16, 0.0, 0),
                                     (32, 8, 0.01, 4), (32, 1, 0.0, 0), (20, 12, 0.05, 0),
                                     (5, 7, 0.0, 2), (2, 3, 0.0, 0), (32, 32, 0.0, 31)])
def test_warp_kernel_matches_oracle_and_block_kernel(V, K, r, n):
    B = 11
    em, ln = W.make_small(7000 + V + K, B, 90, 90, V)
    T = em.shape[1]
    ln[:6] = [0, 1, 2, 3, T, 47]
    x = _dev(em)
    res = oracle.decode(em, ln, 0, K, r, top_n=n)
    w = _run(x, ln, V, K, r, True, top_n=n)
    k = _run(x, ln, V, K, r, False, top_n=n)
    assert (w.status[:B] == 0).all() and w.launch_count == 1
    assert torch.equal(w.nhyp[:B], k.nhyp[:B])
    # the same formulas in the same precision; the kernels move the zero of their relative
    # scores at different frames, so a score may differ in its last bit
    assert torch.allclose(w.scores[:B], k.scores[:B], rtol=0, atol=1e-4)
    sw, sk = w.last_call_stats(), k.last_call_stats()
    for key in ("frames", "survivors", "trie_nodes_created", "live_hypotheses_sum",
                "max_node_ids_used"):
        assert sw[key] == sk[key], key
    for b in range(B):
        check_hyps(w.hyps(b), res.hyps(b), K, where=f"warp kernel utt {b}")
    w.close()
    k.close()


@pytest.mark.parametrize("spread,K", [(0.02, 8), (0.02, 20), (0.001, 32)])
def test_warp_kernel_on_near_equal_scores(spread, K):
    # nearly flat rows crowd the cut bin (more than 64 members: the bit-by-bit search for the
    # K-th key takes over)
    rng = np.random.default_rng(11)
    B, T, V = 3, 10, 16
    x = rng.standard_normal((B, T, V)) * spread
    em = (x - np.log(np.exp(x).sum(-1, keepdims=True))).astype(np.float32)
    ln = np.array([T, T - 3, 5], dtype=np.int32)
    w = _run(_dev(em), ln, V, K, 0.0, True)
    res = oracle.decode(em, ln, 0, K, 0.0)
    for b in range(B):
        check_hyps(w.hyps(b), res.hyps(b), K, max_unmatched_frac=0.3, where=f"flat utt {b} K={K}",
                   lp=em[b, : ln[b]])
    w.close()


def test_warp_kernel_on_exact_ties():
    # constant rows: every extension of a prefix ties exactly.  Which of the tied candidates a
    # frame keeps is not unique; the kept hypotheses must be distinct, K of them, best first,
    # and none may score above the exact probability of its labelling
    T, V, K = 5, 4, 6
    em = np.full((1, T, V), np.log(1.0 / V), dtype=np.float32)
    full = dict(oracle.decode(em, [T], 0, 100000, 0.0).hyps(0))
    w = _run(_dev(em), [T], V, K, 0.0, True)
    got = w.hyps(0)
    assert len(got) == K and len(set(s for s, _ in got)) == K
    assert all(got[i][1] >= got[i + 1][1] for i in range(K - 1))
    for seq, sc in got:
        assert sc <= full[seq] + 1e-3
    w.close()


@pytest.mark.parametrize("dtype", [torch.float32, torch.float16, torch.bfloat16])
@pytest.mark.parametrize("C", [1, 5, 16])
def test_warp_kernel_streaming_equals_one_shot(dtype, C):
    V, K, r, B = 32, 16, 1e-2, 7
    em, ln = W.make_small(7100 + C, B, 5, 70, V)
    T = em.shape[1]
    x = torch.from_numpy(em).to(dtype).cuda()
    wide = x.float().cpu().numpy()
    res = oracle.decode(wide, ln, 0, K, r, top_n=4, want_masks=True)
    d = _decoder(V, K, r, B, T, True, top_n=4, max_chunk_frames=C, emission_dtype=dtype)
    n_chunks = (T + C - 1) // C
    for i in range(n_chunks):
        chunk = torch.zeros((B, C, V), dtype=dtype, device="cuda")
        w = min(C, T - i * C)
        chunk[:, :w] = x[:, i * C: i * C + w]
        clen = np.clip(ln - i * C, 0, C).astype(np.int32)
        flags = np.full(B, (1 if i == 0 else 0) | (2 if i == n_chunks - 1 else 0), dtype=np.uint8)
        d.stream_step(chunk, _dev(clen), _dev(flags))
    torch.cuda.synchronize()
    loose = 0.3 if dtype == torch.bfloat16 else 0.0       # coarse values tie at the cut
    for b in range(B):
        check_hyps(d.hyps(b), res.hyps(b), K, max_unmatched_frac=loose, where=f"stream {b}",
                   lp=wide[b, : ln[b]], keep=res.keep[b, : ln[b]])
    d.close()


def test_warp_kernel_degenerate_inputs():
    V, K = 8, 4
    em, _ = W.make_small(7200, 4, 64, 64, V)
    ln = np.array([64, -3, 999, 0], dtype=np.int32)
    w = _run(_dev(em), ln, V, K, 0.0, True)
    st = w.status[:4].cpu().numpy()
    assert st[1] == 1 and st[2] == 1 and st[0] == 0 and st[3] == 0
    assert w.nhyp[:4].tolist() == [K, 0, 0, 1]
    assert w.hyps(3) == [((), 0.0)]
    w.close()
    # rows in which nothing is possible: the beam dies and says so
    em[0, 5, :] = -np.inf
    w = _run(_dev(em), np.array([64, 64, 64, 64], dtype=np.int32), V, K, 0.0, True)
    assert int(w.status[0]) & 8 and int(w.nhyp[0]) == 0
    w.close()
    # a stream fed past the frames its trie arena was sized for reports it and stays in bounds
    d = _decoder(V, K, 0.0, 2, 8, True, max_chunk_frames=8)
    x = _dev(em[2:4])
    full = _dev(np.full(2, 8, dtype=np.int32))
    for i in range(8):
        flags = _dev(np.full(2, 2 | (i == 0), dtype=np.uint8))
        d.stream_step(x[:, 8 * i: 8 * i + 8].contiguous(), full, flags)
    torch.cuda.synchronize()
    assert (d.status[:2].cpu().numpy() & 2).all()
    d.close()


def test_many_streams_take_the_warp_kernel_by_themselves():
    # 2048 streams on one GPU are more than eight per SM: same results as the block kernel
    S, C, V, K, r = 2048, 8, 32, 16, 1e-2
    wl = W.workload_streaming(streams=S, chunks=3, chunk_frames=C, beam_width=K)
    x = _dev(wl.emissions)
    outs = []
    for mode in (1, 0):
        d = _binding().Decoder(V, 0, K, r, S, 3 * C, max_chunk_frames=C)
        d.set_warp_decode(mode)
        full = _dev(np.full(S, C, dtype=np.int32))
        for i in range(3):
            flags = _dev(np.full(S, (1 if i == 0 else 0) | (2 if i == 2 else 0), dtype=np.uint8))
            d.stream_step(x[:, i * C:(i + 1) * C].contiguous(), full, flags)
        torch.cuda.synchronize()
        assert int((d.status != 0).sum()) == 0
        outs.append(d)
    assert torch.equal(outs[0].nhyp, outs[1].nhyp)
    assert torch.allclose(outs[0].scores, outs[1].scores, rtol=0, atol=1e-4)
    sample = [0, 777, 2047]
    res = oracle.decode(wl.emissions[sample], wl.lengths[sample], 0, K, r)
    for i, b in enumerate(sample):
        check_hyps(outs[0].hyps(b), res.hyps(i), K, where=f"stream {b}")
    for d in outs:
        d.close()


def test_warp_decode_mode_is_validated():
    b = _binding()
    d = b.Decoder(32, 0, 4, 0.0, 1, 4)
    with pytest.raises(b.FltopError):
        d.set_warp_decode(3)
    assert b.lib().fltop_set_warp_decode(None, 1) == b.FLTOP_ERR_INVALID_ARG
    d.close()
