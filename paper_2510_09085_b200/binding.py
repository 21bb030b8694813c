"""ctypes binding of the C-ABI library (``include/fltop.h``): argument marshalling only.

Every decoding step runs in the CUDA kernels of ``libfltop.so``.  There is no
CPU fallback: loading fails with an ImportError if the library has not been
built, and every call raises ``FltopError`` on a non-zero return code.
torch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libfltop.so")

FLTOP_OK, FLTOP_ERR_INVALID_ARG, FLTOP_ERR_CUDA, FLTOP_ERR_OOM, FLTOP_ERR_CAPACITY, \
    FLTOP_ERR_STATE = range(6)
FLTOP_ST_BAD_LENGTH, FLTOP_ST_ARENA_FULL, FLTOP_ST_TRUNCATED, FLTOP_ST_EMPTY_BEAM, \
    FLTOP_ST_INTERNAL = 1, 2, 4, 8, 16

EXPORTS = ("fltop_workspace_size", "fltop_create", "fltop_decode", "fltop_stream_step",
           "fltop_destroy", "fltop_prune", "fltop_status_string", "fltop_last_cuda_error",
           "fltop_beam_state_bytes", "fltop_launch_count", "fltop_last_call_stats", "fltop_set_profiling",
           "fltop_last_kernel_ms", "fltop_decode_static", "fltop_set_block_threads",
           "fltop_set_fusion", "fltop_enable_host_io", "fltop_decode_host",
           "fltop_last_host_io_bytes", "fltop_set_warp_decode", "fltop_set_test_hook")


class fltop_config(C.Structure):
    _fields_ = [("vocab_size", C.c_int32), ("blank_id", C.c_int32), ("beam_width", C.c_int32),
                ("threshold_r", C.c_float), ("max_batch", C.c_int32), ("max_frames", C.c_int32),
                ("max_chunk_frames", C.c_int32), ("max_out_len", C.c_int32),
                ("top_n", C.c_int32), ("beam_threshold", C.c_float), ("merge_max", C.c_int32),
                ("emission_dtype", C.c_int32), ("max_trie_nodes", C.c_int32),
                ("device", C.c_int32),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t)]


FLTOP_EMISSION_F32, FLTOP_EMISSION_F16, FLTOP_EMISSION_BF16 = 0, 1, 2
FLTOP_HOOK_SURVIVOR_MASKS, FLTOP_HOOK_PHASE_CLOCKS, FLTOP_HOOK_TABLE_SLOTS, \
    FLTOP_HOOK_ROW_KERNEL, FLTOP_HOOK_PRUNE_STAGING = 1, 2, 3, 4, 5
EMISSION_CODES = {torch.float32: FLTOP_EMISSION_F32, torch.float16: FLTOP_EMISSION_F16,
                  torch.bfloat16: FLTOP_EMISSION_BF16}


class FltopError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {status_string(code)} ({code})")


_lib = None


def lib():
    """The loaded library; raises ImportError if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2510_09085_b200.build` "
                "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
        L.fltop_workspace_size.restype = C.c_size_t
        L.fltop_workspace_size.argtypes = [C.POINTER(fltop_config)]
        L.fltop_create.restype = C.c_int
        L.fltop_create.argtypes = [C.POINTER(fltop_config), C.POINTER(vp)]
        L.fltop_decode.restype = C.c_int
        L.fltop_decode.argtypes = [vp, vp, i64, i64, vp, i32, i32, vp, vp, vp, vp, vp, vp]
        L.fltop_stream_step.restype = C.c_int
        L.fltop_stream_step.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, vp]
        L.fltop_destroy.restype = C.c_int
        L.fltop_destroy.argtypes = [vp]
        L.fltop_prune.restype = C.c_int
        L.fltop_prune.argtypes = [vp, vp, i64, i64, vp, i32, i32, vp, vp, vp]
        L.fltop_status_string.restype = C.c_char_p
        L.fltop_status_string.argtypes = [C.c_int]
        L.fltop_last_cuda_error.restype = C.c_int
        L.fltop_last_cuda_error.argtypes = [vp]
        L.fltop_beam_state_bytes.restype = C.c_size_t
        L.fltop_beam_state_bytes.argtypes = [vp]
        L.fltop_launch_count.restype = C.c_int64
        L.fltop_launch_count.argtypes = [vp]
        L.fltop_last_call_stats.restype = C.c_int
        L.fltop_last_call_stats.argtypes = [vp, C.POINTER(C.c_int64)]
        L.fltop_set_profiling.restype = C.c_int
        L.fltop_set_profiling.argtypes = [vp, C.c_int]
        L.fltop_last_kernel_ms.restype = C.c_int
        L.fltop_last_kernel_ms.argtypes = [vp, C.POINTER(C.c_float)]
        L.fltop_set_block_threads.restype = C.c_int
        L.fltop_set_block_threads.argtypes = [vp, i32]
        L.fltop_set_fusion.restype = C.c_int
        L.fltop_set_fusion.argtypes = [vp, C.c_int]
        L.fltop_set_warp_decode.restype = C.c_int
        L.fltop_set_warp_decode.argtypes = [vp, C.c_int]
        L.fltop_enable_host_io.restype = C.c_int
        L.fltop_enable_host_io.argtypes = [vp]
        L.fltop_decode_host.restype = C.c_int
        L.fltop_decode_host.argtypes = [vp, vp, i64, i64, vp, i32, i32, vp, vp, vp, vp, vp, vp]
        L.fltop_last_host_io_bytes.restype = C.c_int
        L.fltop_last_host_io_bytes.argtypes = [vp, C.POINTER(C.c_int64)]
        L.fltop_set_test_hook.restype = C.c_int
        L.fltop_set_test_hook.argtypes = [vp, C.c_int, vp, i64, i64]
        L.fltop_decode_static.restype = C.c_int
        L.fltop_decode_static.argtypes = [i32, i32, i32, C.c_float, vp, i64, i64, vp, i32, i32,
                                          i32, vp, vp, vp, vp, vp, vp]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().fltop_status_string(int(code)).decode()


def make_config(vocab_size, blank_id, beam_width, threshold_r, max_batch, max_frames,
                max_chunk_frames=0, max_out_len=None, device=0, workspace=0, workspace_bytes=0,
                top_n=0, beam_threshold=0.0, merge_max=0, emission_dtype=0,
                max_trie_nodes=0) -> fltop_config:
    return fltop_config(vocab_size, blank_id, beam_width, threshold_r, max_batch, max_frames,
                        max_chunk_frames, max_frames if max_out_len is None else max_out_len,
                        top_n, beam_threshold, int(merge_max), int(emission_dtype),
                        int(max_trie_nodes), device,
                        workspace or None,
                        workspace_bytes)


def fltop_workspace_size(cfg: fltop_config) -> int:
    return int(lib().fltop_workspace_size(C.byref(cfg)))


def fltop_create(cfg: fltop_config):
    """Returns (code, handle) exactly as the C call does."""
    h = C.c_void_p()
    code = lib().fltop_create(C.byref(cfg) if cfg is not None else None, C.byref(h))
    return code, h


def _p(t):
    if t is None:
        return None
    if isinstance(t, int):
        return C.c_void_p(t)
    return C.c_void_p(t.data_ptr())


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def fltop_decode(h, logp, stride_b, stride_t, lengths, B, T, tokens, lens, scores, nhyp,
                 status=None, stream=None) -> int:
    return lib().fltop_decode(h, _p(logp), stride_b, stride_t, _p(lengths), B, T, _p(tokens),
                              _p(lens), _p(scores), _p(nhyp), _p(status), _stream_ptr(stream))


def fltop_stream_step(h, chunk, chunk_lens, flags, S, Cf, tokens, lens, scores, nhyp,
                      status=None, stream=None) -> int:
    return lib().fltop_stream_step(h, _p(chunk), _p(chunk_lens), _p(flags), S, Cf, _p(tokens),
                                   _p(lens), _p(scores), _p(nhyp), _p(status),
                                   _stream_ptr(stream))


def fltop_prune(h, logp, stride_b, stride_t, lengths, B, T, counts, entries, stream=None) -> int:
    return lib().fltop_prune(h, _p(logp), stride_b, stride_t, _p(lengths), B, T, _p(counts),
                             _p(entries), _stream_ptr(stream))


def fltop_decode_static(vocab_size, blank_id, beam_width, threshold_r, logp, stride_b, stride_t,
                        lengths, B, T, max_out_len, tokens, lens, scores, nhyp, status=None,
                        stream=None) -> int:
    """Allocation-free batch decode on the current device (fixed scratch inside the library)."""
    return lib().fltop_decode_static(vocab_size, blank_id, beam_width, threshold_r, _p(logp),
                                     stride_b, stride_t, _p(lengths), B, T, max_out_len,
                                     _p(tokens), _p(lens), _p(scores), _p(nhyp), _p(status),
                                     _stream_ptr(stream))


def fltop_destroy(h) -> int:
    return lib().fltop_destroy(h)


class Decoder:
    """Owns one handle plus the output tensors; thin convenience over the C calls."""

    def __init__(self, vocab_size, blank_id, beam_width, threshold_r, max_batch, max_frames,
                 max_chunk_frames=0, max_out_len=None, device=0, top_n=0, beam_threshold=0.0,
                 merge_max=False, emission_dtype=torch.float32, max_trie_nodes=0):
        self.cfg = make_config(vocab_size, blank_id, beam_width, threshold_r, max_batch,
                               max_frames, max_chunk_frames, max_out_len, device, top_n=top_n,
                               beam_threshold=beam_threshold, merge_max=int(bool(merge_max)),
                               emission_dtype=EMISSION_CODES[emission_dtype],
                               max_trie_nodes=max_trie_nodes)
        self.emission_dtype = emission_dtype
        code, self.h = fltop_create(self.cfg)
        if code != FLTOP_OK:
            self.h = None
            raise FltopError(code, "fltop_create")
        self.device = torch.device("cuda", device)
        K, L = beam_width, self.cfg.max_out_len
        self.tokens = torch.zeros((max_batch, K, L), dtype=torch.int32, device=self.device)
        self.lens = torch.zeros((max_batch, K), dtype=torch.int32, device=self.device)
        self.scores = torch.zeros((max_batch, K), dtype=torch.float32, device=self.device)
        self.nhyp = torch.zeros((max_batch,), dtype=torch.int32, device=self.device)
        self.status = torch.zeros((max_batch,), dtype=torch.int32, device=self.device)

    # --- batch ---------------------------------------------------------------------
    def decode(self, logp: torch.Tensor, lengths: torch.Tensor, stream=None):
        """logp [B,T,V] CUDA of the handle's emission dtype (last dim contiguous), lengths [B]
        int32 CUDA."""
        assert logp.is_cuda and logp.dtype == self.emission_dtype and logp.stride(2) == 1
        assert lengths.is_cuda and lengths.dtype == torch.int32 and lengths.is_contiguous()
        B, T, _ = logp.shape
        code = fltop_decode(self.h, logp, logp.stride(0), logp.stride(1), lengths, B, T,
                            self.tokens, self.lens, self.scores, self.nhyp, self.status, stream)
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_decode")
        return self

    # --- batch, host buffers -------------------------------------------------------
    def enable_host_io(self, pin: bool = True):
        """Allocates the library's staging and the host output tensors (pinned unless pin=False)."""
        code = lib().fltop_enable_host_io(self.h)
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_enable_host_io")
        mk = (lambda t: t.pin_memory()) if pin else (lambda t: t)
        self.h_tokens = mk(torch.zeros(self.tokens.shape, dtype=torch.int32))
        self.h_lens = mk(torch.zeros(self.lens.shape, dtype=torch.int32))
        self.h_scores = mk(torch.zeros(self.scores.shape, dtype=torch.float32))
        self.h_nhyp = mk(torch.zeros(self.nhyp.shape, dtype=torch.int32))
        self.h_status = mk(torch.zeros(self.status.shape, dtype=torch.int32))

    def decode_host(self, logp: torch.Tensor, lengths: torch.Tensor, stream=None):
        """logp [B,T,V] float32 and lengths [B] int32 in HOST memory; the results are in the
        host tensors h_tokens / h_lens / h_scores / h_nhyp / h_status when this returns."""
        assert not logp.is_cuda and logp.dtype == self.emission_dtype and logp.stride(2) == 1
        assert not lengths.is_cuda and lengths.dtype == torch.int32 and lengths.is_contiguous()
        B, T, _ = logp.shape
        code = lib().fltop_decode_host(self.h, _p(logp), logp.stride(0), logp.stride(1),
                                       _p(lengths), B, T, _p(self.h_tokens), _p(self.h_lens),
                                       _p(self.h_scores), _p(self.h_nhyp), _p(self.h_status),
                                       _stream_ptr(stream))
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_decode_host")
        return self

    def host_io_bytes(self):
        """(host-to-device, device-to-host) bytes of the most recent decode_host."""
        out = (C.c_int64 * 2)()
        code = lib().fltop_last_host_io_bytes(self.h, out)
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_last_host_io_bytes")
        return int(out[0]), int(out[1])

    def host_hyps(self, b: int):
        """[(token tuple, score)] of utterance b from the host outputs of decode_host."""
        n = int(self.h_nhyp[b])
        lens = self.h_lens[b, :n].tolist()
        sc = self.h_scores[b, :n].tolist()
        return [(tuple(self.h_tokens[b, k, : lens[k]].tolist()), sc[k]) for k in range(n)]

    # --- streaming -----------------------------------------------------------------
    def stream_step(self, chunk: torch.Tensor, chunk_lens: torch.Tensor, flags=None,
                    readback=True, stream=None):
        assert chunk.is_cuda and chunk.dtype == self.emission_dtype and chunk.is_contiguous()
        S, Cf, _ = chunk.shape
        outs = (self.tokens, self.lens, self.scores, self.nhyp) if readback else (None,) * 4
        code = fltop_stream_step(self.h, chunk, chunk_lens, flags, S, Cf, *outs, self.status,
                                 stream)
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_stream_step")
        return self

    def prune(self, logp: torch.Tensor, lengths: torch.Tensor, stream=None):
        """Survivor counts [B,T] and entries [B,T,V,2] (int32 token, float32 bits)."""
        B, T, V = logp.shape
        counts = torch.zeros((B, T), dtype=torch.int32, device=logp.device)
        entries = torch.zeros((B, T, V, 2), dtype=torch.int32, device=logp.device)
        code = fltop_prune(self.h, logp, logp.stride(0), logp.stride(1), lengths, B, T, counts,
                           entries, stream)
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_prune")
        return counts, entries

    # --- results -------------------------------------------------------------------
    def hyps(self, b: int):
        """[(token tuple, score)] of utterance / stream b, best first (synchronises)."""
        n = int(self.nhyp[b])
        lens = self.lens[b, :n].tolist()
        toks = self.tokens[b, :n].cpu()
        sc = self.scores[b, :n].tolist()
        return [(tuple(toks[k, : lens[k]].tolist()), sc[k]) for k in range(n)]

    def set_profiling(self, on: bool):
        code = lib().fltop_set_profiling(self.h, int(on))
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_set_profiling")

    def set_block_threads(self, threads: int):
        code = lib().fltop_set_block_threads(self.h, int(threads))
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_set_block_threads")

    def set_fusion(self, mode: int):
        code = lib().fltop_set_fusion(self.h, int(mode))
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_set_fusion")

    def set_warp_decode(self, mode: int):
        code = lib().fltop_set_warp_decode(self.h, int(mode))
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_set_warp_decode")

    def last_kernel_ms(self):
        ms = (C.c_float * 2)()
        code = lib().fltop_last_kernel_ms(self.h, ms)
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_last_kernel_ms")
        return float(ms[0]), float(ms[1])

    def set_test_hook(self, hook: int, buffer=None, a: int = 0, b: int = 0):
        """fltop_set_test_hook; `buffer` is a CUDA tensor (kept alive by the caller) or None."""
        code = lib().fltop_set_test_hook(self.h, int(hook), _p(buffer), int(a), int(b))
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_set_test_hook")

    def last_call_stats(self) -> dict:
        out = (C.c_int64 * 8)()
        code = lib().fltop_last_call_stats(self.h, out)
        if code != FLTOP_OK:
            raise FltopError(code, "fltop_last_call_stats")
        return {"frames": out[0], "survivors": out[1], "trie_nodes_created": out[2],
                "live_hypotheses_sum": out[3], "max_node_ids_used": out[4],
                "tag_clashes": out[5], "exact_select_frames": out[6],
                "prune_copy_timeouts": out[7]}

    @property
    def beam_state_bytes(self) -> int:
        return int(lib().fltop_beam_state_bytes(self.h))

    @property
    def launch_count(self) -> int:
        return int(lib().fltop_launch_count(self.h))

    def close(self):
        if getattr(self, "h", None):
            fltop_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
