"""fltop_decode_static - the entry point for callers that cannot allocate device memory
where they decode (real-time threads, plug-ins inside a fixed memory pool).  It must give
what fltop_decode gives, call after call, although every call reuses the same fixed scratch
array inside the library, and it must leave the amount of free device memory alone.  This
file sorts last on purpose: a run that stops at the first failure has then already run every
other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2510_09085_b200 import workloads as W
from tests.parity import check_hyps

pytestmark = pytest.mark.gpu


def _static_call(bd, x, n, V, K, r, B, T):
    tok = torch.full((B, K, T), -7, dtype=torch.int32, device="cuda")
    lens = torch.full((B, K), -7, dtype=torch.int32, device="cuda")
    sc = torch.full((B, K), 7.0, dtype=torch.float32, device="cuda")
    nh = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    st = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    code = bd.fltop_decode_static(V, 0, K, r, x, x.stride(0), x.stride(1), n, B, T, T, tok, lens,
                                  sc, nh, st)
    assert code == bd.FLTOP_OK
    torch.cuda.synchronize()
    return tok, lens, sc, nh, st


def _both(bd, em, ln, K, r):
    B, T, V = em.shape
    x = torch.from_numpy(em).cuda()
    n = torch.from_numpy(np.asarray(ln, dtype=np.int32)).cuda()
    ref = bd.Decoder(V, 0, K, r, B, T)
    # the same kernels on both sides (the static call always takes the separate prune kernel
    # and the general decode kernel)
    ref.set_fusion(0)
    ref.decode(x, n)
    tok, lens, sc, nh, st = _static_call(bd, x, n, V, K, r, B, T)
    assert torch.equal(nh, ref.nhyp[:B]) and torch.equal(lens, ref.lens[:B])
    assert (st == 0).all() and (ref.status[:B] == 0).all()
    # same kernels, same inputs: the tolerance of the parity tests (1e-3 nats) is far from needed
    assert torch.allclose(sc, ref.scores[:B], atol=1e-3, rtol=0)
    for b in range(B):
        for k in range(int(nh[b])):
            L = int(lens[b, k])
            assert torch.equal(tok[b, k, :L], ref.tokens[b, k, :L])
    # ... and against the CPU oracle, like every other entry point
    res = oracle.decode(em, ln, 0, K, r)
    for b in range(B):
        m = int(nh[b])
        got = [(tuple(tok[b, k, : int(lens[b, k])].tolist()), float(sc[b, k])) for k in range(m)]
        check_hyps(got, res.hyps(b), K, where=f"static utt {b}")
    ref.close()


def test_static_scratch_decode_matches_handle_decode_twice_in_a_row():
    from paper_2510_09085_b200 import binding as bd
    # first call: a larger problem that dirties most of the fixed scratch
    em1, ln1 = W.make_small(41, 8, 100, 400, 32)
    _both(bd, em1, ln1, 16, 1e-2)
    # second call, straight after, smaller and different: stale contents must not leak in
    em2, ln2 = W.make_small(42, 3, 20, 90, 12)
    _both(bd, em2, ln2, 5, 0.0)
    # and the first problem again
    _both(bd, em1, ln1, 16, 1e-2)


def test_static_scratch_decode_leaves_free_device_memory_alone():
    # cudaMemGetInfo sees every allocation on the device, the library's own included (torch's
    # counters see only torch's).  After a warm-up call (the first call on a device sets the
    # library up), further calls must not move the free-memory figure.
    from paper_2510_09085_b200 import binding as bd
    em, ln = W.make_small(43, 4, 50, 120, 32)
    B, T, V = em.shape
    x = torch.from_numpy(em).cuda()
    n = torch.from_numpy(ln).cuda()
    _static_call(bd, x, n, V, 8, 1e-2, B, T)                 # warm-up
    outs = [torch.empty((B, 8, T), dtype=torch.int32, device="cuda"),
            torch.empty((B, 8), dtype=torch.int32, device="cuda"),
            torch.empty((B, 8), dtype=torch.float32, device="cuda"),
            torch.empty((B,), dtype=torch.int32, device="cuda"),
            torch.empty((B,), dtype=torch.int32, device="cuda")]
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(3):
        code = bd.fltop_decode_static(V, 0, 8, 1e-2, x, x.stride(0), x.stride(1), n, B, T, T, *outs)
        assert code == bd.FLTOP_OK
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free_before


def test_static_scratch_rejects_problems_beyond_its_capacity():
    from paper_2510_09085_b200 import binding as bd
    x = torch.zeros((2, 8, 128), device="cuda")
    ln = torch.zeros(2, dtype=torch.int32, device="cuda")
    out = [torch.zeros((2, 4, 8), dtype=torch.int32, device="cuda"),
           torch.zeros((2, 4), dtype=torch.int32, device="cuda"),
           torch.zeros((2, 4), device="cuda"), torch.zeros(2, dtype=torch.int32, device="cuda")]
    # vocabulary above the limit
    assert bd.fltop_decode_static(128, 0, 4, 0.0, x, 1024, 128, ln, 2, 8, 8, *out) == \
        bd.FLTOP_ERR_CAPACITY
    # too many frames / too many trie nodes
    assert bd.fltop_decode_static(32, 0, 4, 0.0, x, 0, 32, ln, 2, 4096, 8, *out) == \
        bd.FLTOP_ERR_CAPACITY
    assert bd.fltop_decode_static(32, 0, 2000, 0.0, x, 0, 32, ln, 2, 100, 8, *out) == \
        bd.FLTOP_ERR_CAPACITY
    assert bd.fltop_decode_static(32, 40, 4, 0.0, x, 256, 32, ln, 2, 8, 8, *out) == \
        bd.FLTOP_ERR_INVALID_ARG
