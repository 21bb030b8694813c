"""The C-ABI library without a GPU: it loads, exports what the header declares, and
rejects bad arguments on the host before touching CUDA."""
import ctypes
import os
import re

import pytest

from paper_2510_09085_b200 import build as lib_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bd():
    lib_build.build()
    from paper_2510_09085_b200 import binding
    binding.lib()
    return binding


def test_library_exports_every_declared_symbol(bd):
    header = open(os.path.join(ROOT, "include", "fltop.h")).read()
    declared = set(re.findall(r"\b(fltop_[a-z_]+)\s*\(", header))
    assert declared == set(bd.EXPORTS)
    raw = ctypes.CDLL(bd.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name


def test_config_struct_matches_header(bd):
    header = open(os.path.join(ROOT, "include", "fltop.h")).read()
    body = header[header.index("typedef struct {"): header.index("} fltop_config;")]
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = re.findall(r"\b(\w+);", body)
    assert fields == [f[0] for f in bd.fltop_config._fields_]


@pytest.mark.parametrize("kw", [
    dict(vocab_size=1), dict(vocab_size=9000), dict(blank_id=-1), dict(blank_id=32),
    dict(beam_width=0), dict(beam_width=5000), dict(threshold_r=-0.1), dict(threshold_r=1.5),
    dict(threshold_r=float("nan")), dict(max_batch=0), dict(max_frames=0), dict(max_out_len=0),
    dict(top_n=-1), dict(max_trie_nodes=-1), dict(beam_threshold=float("nan")), dict(merge_max=2), dict(emission_dtype=3), dict(emission_dtype=-1), dict(device=-1), dict(max_chunk_frames=-1),
    dict(max_chunk_frames=101), dict(workspace=8, workspace_bytes=1 << 40),
    dict(beam_width=2048, vocab_size=8192),     # needs more shared memory than one SM has
])
def test_invalid_config_is_rejected_on_the_host(bd, kw):
    base = dict(vocab_size=32, blank_id=0, beam_width=8, threshold_r=0.01, max_batch=4,
                max_frames=100)
    base.update(kw)
    cfg = bd.make_config(**base)
    assert bd.fltop_workspace_size(cfg) == 0
    code, h = bd.fltop_create(cfg)
    assert code == bd.FLTOP_ERR_INVALID_ARG and not h.value


def test_optional_knobs_of_algorithm_1_are_accepted(bd):
    for kw in (dict(top_n=4), dict(beam_threshold=25.0), dict(top_n=100, beam_threshold=-1.0),
               dict(merge_max=1), dict(emission_dtype=1), dict(emission_dtype=2)):
        cfg = bd.make_config(32, 0, 8, 0.01, 4, 100, **kw)
        assert bd.fltop_workspace_size(cfg) > 0


def test_null_arguments(bd):
    assert bd.lib().fltop_create(None, None) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.fltop_create(None)[0] == bd.FLTOP_ERR_INVALID_ARG
    assert bd.lib().fltop_destroy(None) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.lib().fltop_decode(None, None, 0, 0, None, 0, 0, None, None, None, None, None,
                                 None) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.lib().fltop_stream_step(None, None, None, None, 0, 0, None, None, None, None, None,
                                      None) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.lib().fltop_prune(None, None, 0, 0, None, 0, 0, None, None, None) == \
        bd.FLTOP_ERR_INVALID_ARG
    assert bd.lib().fltop_set_profiling(None, 1) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.lib().fltop_enable_host_io(None) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.lib().fltop_decode_host(None, None, 0, 0, None, 0, 0, None, None, None, None, None,
                                      None) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.lib().fltop_last_host_io_bytes(None, None) == bd.FLTOP_ERR_INVALID_ARG
    assert bd.lib().fltop_launch_count(None) == 0


def test_workspace_size_accounts_for_every_region(bd):
    # a character vocabulary is pruned inside the decode kernel: no survivor lists in the
    # workspace, only the trie arenas (8-byte nodes) and the per-utterance statistics
    cfg = bd.make_config(32, 0, 50, 1e-3, 64, 1750)
    need = bd.fltop_workspace_size(cfg)
    expect = 64 * (50 * 1750 + 2) * 8
    assert expect <= need <= expect + 2 * 256 + 64 * 32
    # a smaller trie capacity shrinks it; it is never taken below what two frames can create
    small = bd.make_config(32, 0, 50, 1e-3, 64, 1750, max_trie_nodes=40000)
    assert 64 * 40000 * 8 <= bd.fltop_workspace_size(small) <= 64 * 40000 * 8 + 2 * 256 + 64 * 32
    tiny = bd.make_config(32, 0, 50, 1e-3, 64, 1750, max_trie_nodes=1)
    assert bd.fltop_workspace_size(tiny) >= 64 * (2 * 50 + 4) * 8
    huge = bd.make_config(32, 0, 50, 1e-3, 64, 1750, max_trie_nodes=2 ** 31 - 1)
    assert bd.fltop_workspace_size(huge) == need
    # vocabularies above 1024 always take the separate prune kernel: counts and survivor
    # lists are inside
    frames = 8 * 100
    wide = bd.make_config(2048, 0, 8, 1e-3, 8, 100)
    expect = frames * 4 + frames * 2048 * 8 + 8 * (8 * 100 + 2) * 8
    assert expect <= bd.fltop_workspace_size(wide) <= expect + 4 * 256 + 8 * 32
    scfg = bd.make_config(32, 0, 16, 1e-2, 1024, 1600, max_chunk_frames=16)
    sneed = bd.fltop_workspace_size(scfg)
    assert sneed < 1024 * (16 * 1600 + 2) * 8 + 1024 * 4 * 200 + 64 * 1024
    too_small = bd.make_config(32, 0, 50, 1e-3, 64, 1750, workspace=256, workspace_bytes=1024)
    assert bd.fltop_create(too_small)[0] == bd.FLTOP_ERR_OOM


def test_status_strings(bd):
    assert bd.status_string(0) == "ok"
    assert "capacity" in bd.status_string(bd.FLTOP_ERR_CAPACITY)
    assert bd.status_string(99) == "unknown status"


def test_create_without_a_gpu_reports_cuda_error(bd):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    code, h = bd.fltop_create(bd.make_config(32, 0, 8, 0.01, 4, 100))
    assert code == bd.FLTOP_ERR_CUDA and not h.value
