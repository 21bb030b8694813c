"""fltop_decode_host (host buffers in, host buffers out, transfers pipelined by the library)
against fltop_decode on device buffers: same bits, whatever the grouping and the order."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import check_hyps
from tests.test_gpu_parity import _binding, _dev

pytestmark = pytest.mark.gpu


def _both(em, ln, V, K, r, pin=True, **kw):
    B, T = em.shape[:2]
    d = _binding().Decoder(V, 0, K, r, max(B, 1), max(T, 1), **kw)
    d.enable_host_io(pin=pin)
    d.decode(_dev(em), _dev(np.asarray(ln, dtype=np.int32)))
    torch.cuda.synchronize()
    host_em = torch.from_numpy(np.ascontiguousarray(em))
    host_ln = torch.from_numpy(np.asarray(ln, dtype=np.int32))
    if pin:
        host_em, host_ln = host_em.pin_memory(), host_ln.pin_memory()
    d.h_tokens.fill_(-7)
    d.decode_host(host_em, host_ln)
    return d


def _check_same(d, B):
    """Host-call outputs against the device-call outputs of the same Decoder.  Scores, counts and
    status must be the same bits; tokens and lengths too, except between hypotheses whose scores
    tie exactly (their order, and which of them makes the cut, is not unique)."""
    assert torch.equal(d.nhyp[:B].cpu(), d.h_nhyp[:B])
    assert torch.equal(d.status[:B].cpu(), d.h_status[:B])
    assert torch.equal(d.scores[:B].cpu(), d.h_scores[:B])
    tok, lens, sc = d.tokens[:B].cpu(), d.lens[:B].cpu(), d.scores[:B].cpu()
    L = tok.shape[2]
    for b in range(B):
        n = int(d.h_nhyp[b])
        for k in range(n):
            tied = (k > 0 and sc[b, k] == sc[b, k - 1]) or (k + 1 < n and sc[b, k] == sc[b, k + 1]) \
                or k == n - 1
            if tied:
                continue
            assert int(lens[b, k]) == int(d.h_lens[b, k])
            ln = min(int(lens[b, k]), L)
            assert torch.equal(tok[b, k, :ln], d.h_tokens[b, k, :ln])
        assert (d.h_lens[b, n:] == 0).all()
        # nothing is written where no hypothesis is
        assert (d.h_tokens[b, n:] == -7).all()


@pytest.mark.parametrize("B,V,K,r,kw", [
    (1, 32, 8, 1e-3, {}), (7, 32, 20, 0.0, {}), (8, 32, 50, 1e-3, {}), (9, 32, 50, 1e-2, {}),
    (40, 32, 12, 1e-3, dict(top_n=4, beam_threshold=25.0)), (21, 48, 16, 1e-2, {}),
    (150, 32, 6, 1e-2, {}),          # more than 16 groups of 8: groups grow
    (10, 32, 300, 1e-3, {}),
])
def test_host_buffers_give_the_same_bits(B, V, K, r, kw):
    em, ln = W.make_small(4000 + B + V, B, 0, 70, V)
    if B >= 7:
        ln[2] = 0
    d = _both(em, ln, V, K, r, **kw)
    assert (d.h_status[:B] == 0).all()
    _check_same(d, B)
    sel = list(range(0, B, max(1, B // 5)))
    res = oracle.decode(em[sel], ln[sel], 0, K, r, top_n=kw.get("top_n", 0),
                        beam_threshold=kw.get("beam_threshold", 0.0))
    for i, b in enumerate(sel):
        check_hyps(d.host_hyps(b), res.hyps(i), K, where=f"host utt {b}")
    h2d, d2h = d.host_io_bytes()
    assert h2d == 4 * B + 4 * V * int(ln.sum())          # only the valid frames cross the bus
    assert d2h < 4 * B * (2 * K + 2) + 4 * K * int(ln.sum()) + 1
    d.close()


def test_host_buffers_pageable_strided_and_bad_lengths():
    B, T, V, K = 11, 40, 32, 10
    em, ln = W.make_small(4100, B, T, T, V)
    ln[:] = np.arange(B) * 3 + 5
    ln[4], ln[7] = -2, T + 9                      # flagged by the kernel, nothing copied for them
    d = _both(em, ln, V, K, 1e-3, pin=False)
    st = d.h_status[:B].numpy()
    assert st[4] == 1 and st[7] == 1 and (np.delete(st, [4, 7]) == 0).all()
    _check_same(d, B)
    # rows taken out of a wider host tensor
    wide = torch.full((B, T, 40), float("nan")).pin_memory()
    wide[:, :, 5:37] = torch.from_numpy(em)
    d.h_tokens.fill_(-7)
    d.decode_host(wide[:, :, 5:37], torch.from_numpy(ln))
    _check_same(d, B)
    d.close()


def test_host_calls_are_refused_where_they_cannot_work():
    b = _binding()
    d = b.Decoder(32, 0, 4, 0.0, 2, 8)
    x = torch.zeros((2, 8, 32)).pin_memory()
    ln = torch.full((2,), 8, dtype=torch.int32)
    out = [torch.zeros(n, dtype=t) for n, t in ((2 * 4 * 8, torch.int32), (8, torch.int32),
                                                (8, torch.float32), (2, torch.int32))]
    ptr = lambda t: b._p(t)
    args = (ptr(x), 8 * 32, 32, ptr(ln), 2, 8, ptr(out[0]), ptr(out[1]), ptr(out[2]), ptr(out[3]),
            None, None)
    assert b.lib().fltop_decode_host(d.h, *args) == b.FLTOP_ERR_STATE      # not enabled
    d.enable_host_io()
    d.enable_host_io()                                                      # a no-op
    assert b.lib().fltop_decode_host(d.h, *args) == b.FLTOP_OK
    big = (ptr(x), 8 * 32, 32, ptr(ln), 3, 8) + args[6:]
    assert b.lib().fltop_decode_host(d.h, *big) == b.FLTOP_ERR_CAPACITY
    nul = (None,) + args[1:]
    assert b.lib().fltop_decode_host(d.h, *nul) == b.FLTOP_ERR_INVALID_ARG
    d.close()
    s = b.Decoder(32, 0, 4, 0.0, 2, 8, max_chunk_frames=4)
    with pytest.raises(b.FltopError):
        s.enable_host_io()
    s.close()


def test_host_buffers_on_the_benchmark_batch():
    # the full wav2vec2-shaped batch (B=64, K=50, r=1e-3) as bench.py's end-to-end leg runs it
    wl = W.workload_wav2vec2()
    B = wl.emissions.shape[0]
    d = _both(wl.emissions, wl.lengths, 32, 50, 1e-3)
    assert (d.h_status[:B] == 0).all()
    _check_same(d, B)
    h2d, d2h = d.host_io_bytes()
    assert h2d == 4 * B + 4 * 32 * int(wl.lengths.sum())
    assert d2h < 0.3 * d.tokens.numel() * 4          # far less than the padded token tensor
    d.close()
