"""Nothing is written outside what a call was given: the handle's scratch lives in a
caller-provided workspace with guard bands on both sides, every output array sits between
guard bands too, and after decoding (every decode kernel, pruning inside and apart, batch and
streaming, a trie arena that runs out) the bands still hold their pattern."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import check_hyps
from tests.test_gpu_parity import _binding, _dev

pytestmark = pytest.mark.gpu
GUARD = 4096  # bytes on each side
PATTERN = 0xA5


class Guarded:
    """A device array of `count` elements with GUARD bytes of pattern before and after."""

    def __init__(self, count, dtype):
        self.nbytes = count * torch.empty(0, dtype=dtype).element_size()
        pad = (-self.nbytes) % 256
        self.raw = torch.full((GUARD + self.nbytes + pad + GUARD,), PATTERN, dtype=torch.uint8,
                              device="cuda")
        self.view = self.raw[GUARD: GUARD + self.nbytes].view(dtype)
        self.pad = pad

    def intact(self):
        head = self.raw[:GUARD]
        tail = self.raw[GUARD + self.nbytes:]
        return bool((head == PATTERN).all()) and bool((tail == PATTERN).all())


def _guarded_handle(bd, V, K, r, B, T, **kw):
    cfg = bd.make_config(V, 0, K, r, B, T, **kw)
    need = bd.fltop_workspace_size(cfg)
    assert need > 0
    ws = Guarded(need + 256, torch.uint8)
    base = (ws.view.data_ptr() + 255) // 256 * 256
    cfg = bd.make_config(V, 0, K, r, B, T, workspace=base, workspace_bytes=need, **kw)
    code, h = bd.fltop_create(cfg)
    assert code == bd.FLTOP_OK
    return h, ws, cfg.max_out_len


CASES = [
    # V, K, r, B, T, what
    (32, 50, 1e-3, 5, 90, "rows"),
    (32, 100, 0.0, 3, 60, "rows"),
    (32, 50, 1e-3, 5, 90, "block"),
    (32, 16, 1e-2, 40, 50, "warp"),
    (32, 300, 1e-3, 2, 50, "block"),
    (200, 20, 1e-3, 4, 60, "block"),     # rows of 200 tokens pruned inside the block
    (200, 20, 1e-3, 4, 60, "apart"),     # ... and by the separate kernel
    (2048, 6, 1e-2, 2, 30, "block"),     # survivor lists inside the workspace
]


@pytest.mark.parametrize("V,K,r,B,T,what", CASES)
def test_batch_decode_stays_inside_its_buffers(V, K, r, B, T, what):
    bd = _binding()
    em, ln = W.make_small(9100 + V + K, B, 5, T, V)
    T = em.shape[1]
    h, ws, L = _guarded_handle(bd, V, K, r, B, T)
    if what == "block":
        assert bd.lib().fltop_set_test_hook(h, bd.FLTOP_HOOK_ROW_KERNEL, None, 0, 0) == bd.FLTOP_OK
        assert bd.lib().fltop_set_warp_decode(h, 0) == bd.FLTOP_OK
    elif what == "warp":
        assert bd.lib().fltop_set_warp_decode(h, 2) == bd.FLTOP_OK
    elif what == "apart":
        assert bd.lib().fltop_set_fusion(h, 0) == bd.FLTOP_OK
    x = Guarded(em.size, torch.float32)
    x.view.copy_(torch.from_numpy(em).reshape(-1))
    lens_in = _dev(ln)
    tok, le = Guarded(B * K * L, torch.int32), Guarded(B * K, torch.int32)
    sc, nh, st = Guarded(B * K, torch.float32), Guarded(B, torch.int32), Guarded(B, torch.int32)
    for _ in range(2):
        code = bd.fltop_decode(h, x.view, T * V, V, lens_in, B, T, tok.view, le.view, sc.view,
                               nh.view, st.view)
        assert code == bd.FLTOP_OK
    torch.cuda.synchronize()
    for g in (ws, x, tok, le, sc, nh, st):
        assert g.intact()
    assert (st.view.cpu().numpy() == 0).all()
    # and what was written inside is right
    res = oracle.decode(em, ln, 0, K, r, want_masks=True)
    lens = le.view.cpu().numpy().reshape(B, K)
    scores = sc.view.cpu().numpy().reshape(B, K)
    tokens = tok.view.cpu().numpy().reshape(B, K, L)
    nhyp = nh.view.cpu().numpy()
    for b in range(B):
        got = [(tuple(tokens[b, k, : lens[b, k]].tolist()), float(scores[b, k])) for k in range(nhyp[b])]
        check_hyps(got, res.hyps(b), K, where=f"utt {b}", lp=em[b, : ln[b]], keep=res.keep[b, : ln[b]])
    assert bd.fltop_destroy(h) == bd.FLTOP_OK


@pytest.mark.parametrize("K,warp_mode", [(40, 0), (16, 2)])
def test_streaming_stays_inside_its_buffers(K, warp_mode):
    # stream states live in the workspace too; chunks of 7 frames, the last one ragged
    bd = _binding()
    V, r, S, C = 32, 1e-2, 6, 7
    em, ln = W.make_small(9300 + K, S, 10, 45, V)
    T = em.shape[1]
    h, ws, L = _guarded_handle(bd, V, K, r, S, T, max_chunk_frames=C)
    assert bd.lib().fltop_set_warp_decode(h, warp_mode) == bd.FLTOP_OK
    tok, le = Guarded(S * K * L, torch.int32), Guarded(S * K, torch.int32)
    sc, nh, st = Guarded(S * K, torch.float32), Guarded(S, torch.int32), Guarded(S, torch.int32)
    n_chunks = (T + C - 1) // C
    keep_alive = []
    for i in range(n_chunks):
        t0 = i * C
        chunk = Guarded(S * C * V, torch.float32)
        part = np.zeros((S, C, V), dtype=np.float32)
        w = min(C, T - t0)
        part[:, :w] = em[:, t0: t0 + w]
        chunk.view.copy_(torch.from_numpy(part).reshape(-1))
        clen = _dev(np.clip(ln - t0, 0, C).astype(np.int32))
        flags = _dev(np.full(S, (1 if i == 0 else 0) | (2 if i == n_chunks - 1 else 0), dtype=np.uint8))
        code = bd.fltop_stream_step(h, chunk.view, clen, flags, S, C, tok.view, le.view, sc.view,
                                    nh.view, st.view)
        assert code == bd.FLTOP_OK
        keep_alive.append((chunk, clen, flags))
    torch.cuda.synchronize()
    for g in [ws, tok, le, sc, nh, st] + [k[0] for k in keep_alive]:
        assert g.intact()
    assert (st.view.cpu().numpy() == 0).all()
    res = oracle.decode(em, ln, 0, K, r, want_masks=True)
    lens = le.view.cpu().numpy().reshape(S, K)
    scores = sc.view.cpu().numpy().reshape(S, K)
    tokens = tok.view.cpu().numpy().reshape(S, K, L)
    nhyp = nh.view.cpu().numpy()
    for b in range(S):
        got = [(tuple(tokens[b, k, : lens[b, k]].tolist()), float(scores[b, k])) for k in range(nhyp[b])]
        check_hyps(got, res.hyps(b), K, where=f"stream {b}", lp=em[b, : ln[b]], keep=res.keep[b, : ln[b]])
    assert bd.fltop_destroy(h) == bd.FLTOP_OK


@pytest.mark.parametrize("what", ["rows", "block", "warp"])
def test_a_trie_arena_that_runs_out_is_not_written_past(what):
    # max_trie_nodes far below what the utterances need: they are flagged FLTOP_ST_ARENA_FULL,
    # and neither the neighbouring arenas' guard nor the outputs' are touched
    bd = _binding()
    V, K, r, B, T = 32, 16, 0.0, 4, 80
    em, ln = W.make_small(9400, B, 60, T, V)
    T = em.shape[1]
    h, ws, L = _guarded_handle(bd, V, K, r, B, T, max_trie_nodes=2 * K + 4)
    if what == "block":
        assert bd.lib().fltop_set_test_hook(h, bd.FLTOP_HOOK_ROW_KERNEL, None, 0, 0) == bd.FLTOP_OK
        assert bd.lib().fltop_set_warp_decode(h, 0) == bd.FLTOP_OK
    elif what == "warp":
        assert bd.lib().fltop_set_warp_decode(h, 2) == bd.FLTOP_OK
    else:
        assert bd.lib().fltop_set_warp_decode(h, 0) == bd.FLTOP_OK
    x, lens_in = _dev(em), _dev(ln)
    tok, le = Guarded(B * K * L, torch.int32), Guarded(B * K, torch.int32)
    sc, nh, st = Guarded(B * K, torch.float32), Guarded(B, torch.int32), Guarded(B, torch.int32)
    assert bd.fltop_decode(h, x, T * V, V, lens_in, B, T, tok.view, le.view, sc.view, nh.view,
                           st.view) == bd.FLTOP_OK
    torch.cuda.synchronize()
    for g in (ws, tok, le, sc, nh, st):
        assert g.intact()
    status = st.view.cpu().numpy()
    assert ((status & 2) != 0).all(), status   # FLTOP_ST_ARENA_FULL on every utterance
    lens = le.view.cpu().numpy()
    assert (lens >= 0).all() and (lens <= T).all()
    assert bd.fltop_destroy(h) == bd.FLTOP_OK
