"""Emissions stored as fp16 / bf16: they are widened exactly on load, so every result must be
the one the oracle gives on the widened float32 values."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import check_hyps, masks_from_entries
from tests.test_gpu_parity import _binding, _dev

pytestmark = pytest.mark.gpu

HALF = [torch.float16, torch.bfloat16]


def _narrow(em, dtype):
    """(device tensor of `dtype`, the same values as float32 numpy)."""
    x = torch.from_numpy(np.ascontiguousarray(em)).to(dtype)
    return x.cuda(), x.float().numpy()


@pytest.mark.parametrize("dtype", HALF)
@pytest.mark.parametrize("V,r,n", [(32, 1e-3, 0), (32, 0.0, 0), (1024, 1e-3, 0), (48, 0.01, 4),
                                   (30, 0.05, 0), (5, 0.05, 2), (2052, 1e-3, 0)])
def test_prune_of_half_precision_rows_is_bit_exact(dtype, V, r, n):
    B, T = 4, 29
    em, ln = W.make_small(5000 + V, B, 0, T, V)
    T = em.shape[1]
    ln[0] = T
    x, wide = _narrow(em, dtype)
    d = _binding().Decoder(V, 0, 2, r, B, max(T, 1), top_n=n, emission_dtype=dtype)
    counts, entries = d.prune(x, _dev(ln))
    torch.cuda.synchronize()
    keep, vals = masks_from_entries(counts.cpu().numpy(), entries.cpu().numpy(), V)
    for b in range(B):
        k = ln[b]
        okeep, ocnt = oracle.prune(wide[b, :k], r, n)
        assert np.array_equal(counts.cpu().numpy()[b, :k], ocnt)
        assert np.array_equal(keep[b, :k], okeep)
        assert np.array_equal(vals[b, :k][okeep], wide[b, :k][okeep])     # widened exactly
        assert (counts.cpu().numpy()[b, k:] == 0).all()
    d.close()


def test_prune_of_rows_at_odd_offsets():
    # a view that starts one element into the buffer: no vector load is possible
    B, T, V = 3, 17, 32
    em, ln = W.make_small(5100, B, T, T, V)
    for dtype in HALF:
        flat = torch.zeros(B * T * V + 1, dtype=dtype, device="cuda")
        x, wide = _narrow(em, dtype)
        flat[1:] = x.reshape(-1)
        view = flat[1:].view(B, T, V)
        d = _binding().Decoder(V, 0, 4, 1e-2, B, T, emission_dtype=dtype)
        counts, _ = d.prune(view, _dev(ln))
        ref = np.stack([oracle.prune(wide[b], 1e-2)[1] for b in range(B)])
        assert np.array_equal(counts.cpu().numpy(), ref)
        d.decode(view, _dev(ln))                      # pruning falls back to the separate kernel
        torch.cuda.synchronize()
        res = oracle.decode(wide, ln, 0, 4, 1e-2)
        for b in range(B):
            check_hyps(d.hyps(b), res.hyps(b), 4, where=f"odd offset {dtype} utt {b}")
        d.close()


@pytest.mark.parametrize("dtype", HALF)
@pytest.mark.parametrize("V,K,r,kw", [(32, 50, 1e-3, {}), (32, 12, 0.0, dict(top_n=4)),
                                      (1024, 16, 1e-3, {}), (20, 8, 0.02, dict(merge_max=True)),
                                      (31, 8, 0.02, {})])
def test_decode_of_half_precision_rows_matches_oracle(dtype, V, K, r, kw):
    B = 5
    em, ln = W.make_small(5200 + V + K, B, 80, 80, V)
    T = em.shape[1]
    ln[:] = [0, 1, T, 37, 64]
    x, wide = _narrow(em, dtype)
    res = oracle.decode(wide, ln, 0, K, r, want_masks=True, **kw)
    outs = []
    for fusion in (1, 0):
        d = _binding().Decoder(V, 0, K, r, B, max(T, 1), emission_dtype=dtype, **kw)
        d.set_fusion(fusion)
        before = d.launch_count
        d.decode(x, _dev(ln))
        torch.cuda.synchronize()
        fused = V <= 32 and V % 2 == 0 and fusion == 1
        assert (d.launch_count - before == 1) == fused
        assert (d.status[:B] == 0).all()
        # sums of coarse bf16 values tie exactly all the time once only the best alignment
        # counts; which of the tied prefixes a frame keeps at its cut is then not unique, and
        # neither are their descendants (the best hypothesis is: it is never at the cut)
        loose = 0.5 if (dtype == torch.bfloat16 and kw.get("merge_max")) else 0.0
        for b in range(B):
            check_hyps(d.hyps(b), res.hyps(b), K, max_unmatched_frac=loose,
                       where=f"{dtype} V={V} fusion={fusion} utt {b}", lp=wide[b, : ln[b]],
                       keep=res.keep[b, : ln[b]], cascade=0.5)
        outs.append(d)
    # (coarse bf16 values tie often: which of two equal-scoring hypotheses comes first, or
    # makes the cut, is not unique - the scores are)
    if not kw.get("merge_max"):
        assert torch.allclose(outs[0].scores[:B], outs[1].scores[:B], rtol=0, atol=1e-4)
    for d in outs:
        d.close()


def test_half_precision_through_host_buffers_and_streams():
    B, V, K, r = 6, 32, 10, 1e-2
    em, ln = W.make_small(5300, B, 10, 60, V)
    T = em.shape[1]
    for dtype in HALF:
        x, wide = _narrow(em, dtype)
        res = oracle.decode(wide, ln, 0, K, r)
        d = _binding().Decoder(V, 0, K, r, B, T, emission_dtype=dtype)
        d.enable_host_io()
        d.decode_host(x.cpu().pin_memory(), torch.from_numpy(ln))
        for b in range(B):
            check_hyps(d.host_hyps(b), res.hyps(b), K, where=f"host {dtype} utt {b}")
        assert d.host_io_bytes()[0] == 4 * B + 2 * V * int(ln.sum())
        d.close()
        s = _binding().Decoder(V, 0, K, r, B, T, max_chunk_frames=7, emission_dtype=dtype)
        n_chunks = (T + 6) // 7
        for i in range(n_chunks):
            chunk = torch.zeros((B, 7, V), dtype=dtype, device="cuda")
            w = min(7, T - 7 * i)
            chunk[:, :w] = x[:, 7 * i: 7 * i + w]
            clen = np.clip(ln - 7 * i, 0, 7).astype(np.int32)
            flags = np.full(B, (1 if i == 0 else 0) | (2 if i == n_chunks - 1 else 0),
                            dtype=np.uint8)
            s.stream_step(chunk, _dev(clen), _dev(flags))
        torch.cuda.synchronize()
        for b in range(B):
            check_hyps(s.hyps(b), res.hyps(b), K, where=f"stream {dtype} utt {b}")
        s.close()
