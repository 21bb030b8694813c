"""Chunked decoding through fltop_stream_step vs one-shot decoding and the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import check_hyps
from tests.test_gpu_parity import _binding, _dev, gpu_decode

pytestmark = pytest.mark.gpu


def _stream_all(em, ln, blank, K, r, C, max_frames=None):
    """Feed a padded batch chunk by chunk; returns the Decoder after the last chunk."""
    B, T, V = em.shape
    d = _binding().Decoder(V, blank, K, r, B, max_frames or max(T, 1), max_chunk_frames=C)
    x = _dev(em)
    n_chunks = (T + C - 1) // C
    for i in range(n_chunks):
        t0 = i * C
        chunk = torch.zeros((B, C, V), dtype=torch.float32, device="cuda")
        w = min(C, T - t0)
        chunk[:, :w] = x[:, t0: t0 + w]
        clen = np.clip(np.asarray(ln) - t0, 0, C).astype(np.int32)
        flags = np.full(B, (1 if i == 0 else 0) | (2 if i == n_chunks - 1 else 0), dtype=np.uint8)
        d.stream_step(chunk, _dev(clen), _dev(flags))
    torch.cuda.synchronize()
    return d


@pytest.mark.parametrize("V,K,r,C", [(6, 4, 0.05, 7), (32, 16, 1e-2, 16), (32, 8, 0.0, 1),
                                     (12, 40, 1e-3, 50)])
def test_chunked_equals_one_shot(V, K, r, C):
    em, ln = W.make_small(300 + V, 5, 20, 130, V)
    one = gpu_decode(em, ln, 0, K, r)
    st = _stream_all(em, ln, 0, K, r, C)
    assert torch.equal(one.nhyp[:5], st.nhyp[:5])
    assert torch.equal(one.scores[:5], st.scores[:5])
    for b in range(5):
        assert one.hyps(b) == st.hyps(b)
    res = oracle.decode(em, ln, 0, K, r)
    for b in range(5):
        check_hyps(st.hyps(b), res.hyps(b), K, where=f"stream {b}")


def test_reset_idle_streams_and_midway_readback():
    V, K, r, C = 8, 6, 0.02, 10
    em, _ = W.make_small(77, 3, 60, 60, V)
    d = _binding().Decoder(V, 0, K, r, 3, 200, max_chunk_frames=C)
    x = _dev(em)
    ref = [oracle.Stream(V, 0, K, r) for _ in range(3)]
    for i in range(6):
        chunk = x[:, i * C: (i + 1) * C].contiguous()
        # stream 1 idles on odd chunks; stream 2 is reset before chunk 3
        clen = np.array([C, 0 if i % 2 else C, C - 3], dtype=np.int32)
        flags = np.array([2 | (i == 0), 2 | (i == 0), 2 | (i == 0 or i == 3)], dtype=np.uint8)
        d.stream_step(chunk, _dev(clen), _dev(flags))
        torch.cuda.synchronize()
        for s in range(3):
            if flags[s] & 1:
                ref[s].reset()
            ref[s].feed(em[s, i * C: i * C + clen[s]])
            check_hyps(d.hyps(s), ref[s].results(), K, where=f"chunk {i} stream {s}")
    assert (d.status.cpu().numpy() == 0).all()


def test_stream_without_readback_then_emit():
    V, K, r, C = 32, 16, 1e-2, 16
    em, ln = W.make_small(5, 4, 64, 64, V)
    d = _binding().Decoder(V, 0, K, r, 4, 64, max_chunk_frames=C)
    x = _dev(em)
    full = _dev(np.full(4, C, dtype=np.int32))
    for i in range(4):
        flags = _dev(np.full(4, 1 if i == 0 else 0, dtype=np.uint8))
        d.stream_step(x[:, i * C: (i + 1) * C].contiguous(), full, flags, readback=False)
    zero = _dev(np.zeros(4, dtype=np.int32))
    d.stream_step(x[:, :C].contiguous(), zero, None)      # no frames, default flags: emit
    torch.cuda.synchronize()
    res = oracle.decode(em, ln, 0, K, r)
    for b in range(4):
        check_hyps(d.hyps(b), res.hyps(b), K)


def test_arena_exhaustion_is_reported_not_faulted():
    # feeding more frames than the handle was sized for must set the status bit and
    # stay in bounds (the trie arena holds K * max_frames + 1 nodes per stream)
    V, K, C = 8, 4, 8
    em, _ = W.make_small(91, 2, 64, 64, V)
    d = _binding().Decoder(V, 0, K, 0.0, 2, 8, max_chunk_frames=C)
    x = _dev(em)
    full = _dev(np.full(2, C, dtype=np.int32))
    for i in range(8):
        flags = _dev(np.full(2, 2 | (i == 0), dtype=np.uint8))
        d.stream_step(x[:, i * C: (i + 1) * C].contiguous(), full, flags)
    torch.cuda.synchronize()
    assert (d.status.cpu().numpy() & 2).all()


def test_serving_workload_sampled():
    wl = W.workload_streaming(streams=1024, chunks=100)
    S, T, V = wl.emissions.shape
    C, K, r = wl.chunk_frames, wl.beam_width, wl.thresholds[0]
    d = _binding().Decoder(V, 0, K, r, S, T, max_chunk_frames=C)
    x = _dev(wl.emissions)
    full = _dev(np.full(S, C, dtype=np.int32))
    n = T // C
    for i in range(n):
        flags = _dev(np.full(S, (1 if i == 0 else 0) | (2 if i == n - 1 else 0), dtype=np.uint8))
        d.stream_step(x[:, i * C: (i + 1) * C].contiguous(), full, flags, readback=(i == n - 1))
    torch.cuda.synchronize()
    assert (d.status.cpu().numpy() == 0).all()
    sample = [0, 1, 511, 1023]
    res = oracle.decode(wl.emissions[sample], wl.lengths[sample], 0, K, r, want_masks=True)
    for i, s in enumerate(sample):
        check_hyps(d.hyps(s), res.hyps(i), K, max_unmatched_frac=0.25, where=f"stream {s}",
                   lp=wl.emissions[s], keep=res.keep[i])
