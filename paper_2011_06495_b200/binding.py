"""Thin Python binding of the C-ABI library (argument marshalling only).

Every step of the method runs in the CUDA kernels of libmvsparse.so; this module only
turns torch tensors into raw pointers, allocates the caller-owned workspace and checks
status codes.  There is no CPU fallback: if the library has not been built, importing
`load()` raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmvsparse.so")
LIB_DEBUG_PATH = os.path.join(_HERE, "libmvsparse_debug.so")     # the checked build, see MvContext.debug_status

MV_OK = 0
MV_ERR_INVALID_ARG = -1
MV_ERR_WORKSPACE = -2
MV_ERR_CUDA = -3
MV_ERR_TOO_LARGE = -4
MV_ERR_TIMEOUT = -5
MV_SELECT_STATIC_MAX_D = 1 << 24
MV_MODE_AUTO = 0
MV_MODE_GENERAL = 1
MV_MODE_TRACK = 2
MV_DBG_CAND_OVERFLOW, MV_DBG_WINDOW_OVERFLOW, MV_DBG_FALLBACK, MV_DBG_LIST_OVERFLOW = 1, 2, 4, 8
MV_DBG_PICK_RANGE, MV_DBG_LIST_RANGE, MV_DBG_OUT_RANGE, MV_DBG_GATHER_RANGE, MV_DBG_INTERNAL = 16, 32, 64, 128, 256

_lib = None
_lib_debug = None


class MvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


def load() -> ctypes.CDLL:
    """Loads libmvsparse.so (built in-tree by paper_2011_06495_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        _lib = _open(LIB_PATH, "python -m paper_2011_06495_b200.build")
    return _lib


def load_debug() -> ctypes.CDLL:
    """Loads the checked build libmvsparse_debug.so (same ABI; its kernels report clamped or refused
    indices through mv_debug_status); raises if absent."""
    global _lib_debug
    if _lib_debug is None:
        _lib_debug = _open(LIB_DEBUG_PATH, "python -m paper_2011_06495_b200.build --debug")
    return _lib_debug


def _open(path: str, how: str) -> ctypes.CDLL:
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `{how}` (there is no CPU fallback)")
    lib = ctypes.CDLL(path)
    c_vp, c_i, c_i64, c_sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
    lib.mv_workspace_bytes.restype = c_sz
    lib.mv_workspace_bytes.argtypes = [c_i, c_i64, c_i64]
    lib.mv_create.restype = c_i
    lib.mv_create.argtypes = [ctypes.POINTER(c_vp), c_vp, c_vp, c_sz]
    lib.mv_destroy.restype = c_i
    lib.mv_destroy.argtypes = [c_vp]
    lib.mv_set_mode.restype = c_i
    lib.mv_set_mode.argtypes = [c_vp, c_i]
    lib.mv_sparse_step.restype = c_i
    lib.mv_sparse_step.argtypes = [c_vp, c_vp, c_vp, c_i, c_i64, c_i64, c_vp, c_vp]
    lib.mv_vote.restype = c_i
    lib.mv_vote.argtypes = [c_vp, c_vp, c_vp, c_i, c_i64, c_i64, c_vp, c_vp, c_vp, c_vp]
    lib.mv_select.restype = c_i
    lib.mv_select.argtypes = [c_vp, c_vp, c_i, c_i64, c_i64, c_vp, c_vp]
    lib.mv_ad_step.restype = c_i
    lib.mv_ad_step.argtypes = [c_vp, c_vp, c_vp, c_vp, c_i, c_i64, c_i64, c_i64, c_vp, c_vp, c_vp, c_vp, c_vp]
    lib.mv_topk_union_step.restype = c_i
    lib.mv_topk_union_step.argtypes = [c_vp, c_vp, c_vp, c_i, c_i64, c_i64, c_vp, c_vp, c_i64, c_vp]
    lib.mv_select_static.restype = c_i
    lib.mv_select_static.argtypes = [c_vp, c_vp, c_i, c_i64, c_i64, c_vp, c_vp]
    lib.mv_aggregate.restype = c_i
    lib.mv_aggregate.argtypes = [c_vp, c_vp, c_i, c_i64, c_i64, c_vp, c_vp]
    lib.mv_sparse_step_host.restype = c_i
    lib.mv_sparse_step_host.argtypes = [c_vp, c_vp, c_i, c_i64, c_i64, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp]
    lib.mv_read_diag.restype = c_i
    lib.mv_read_diag.argtypes = [c_vp, c_i, c_vp]
    lib.mv_set_kernel_timing.restype = c_i
    lib.mv_set_kernel_timing.argtypes = [c_vp, c_i]
    lib.mv_read_kernel_timing.restype = c_i
    lib.mv_read_kernel_timing.argtypes = [c_vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(c_i)]
    lib.mv_set_phase_timing.restype = c_i
    lib.mv_set_phase_timing.argtypes = [c_vp, c_i]
    lib.mv_read_phase_times.restype = c_i
    lib.mv_read_phase_times.argtypes = [c_vp, ctypes.POINTER(ctypes.c_float), c_i, ctypes.POINTER(c_i)]
    lib.mv_last_launches.restype = c_i
    lib.mv_last_launches.argtypes = [c_vp]
    lib.mv_status_string.restype = ctypes.c_char_p
    lib.mv_status_string.argtypes = [c_i]
    c_u64 = ctypes.c_uint64
    lib.mv_select_rs.restype = c_i
    lib.mv_select_rs.argtypes = [c_vp, c_vp, c_i, c_i64, c_i64, c_u64, c_u64, c_vp, c_vp]
    lib.mv_rs_step.restype = c_i
    lib.mv_rs_step.argtypes = [c_vp, c_vp, c_vp, c_i, c_i64, c_i64, c_u64, c_u64, c_vp, c_vp]
    lib.mv_aggregate_partial.restype = c_i
    lib.mv_aggregate_partial.argtypes = [c_vp, c_vp, c_i, c_i64, c_i64, c_vp, c_vp]
    lib.mv_finish_mean.restype = c_i
    lib.mv_finish_mean.argtypes = [c_vp, c_vp, c_i64, c_i, c_vp]
    # wire formats (include/mv_wire.h)
    lib.mv_pos_offset_bits.restype = c_i
    lib.mv_pos_offset_bits.argtypes = [c_i64]
    lib.mv_pos_stream_bits.restype = c_i64
    lib.mv_pos_stream_bits.argtypes = [c_i64, c_i64, c_i64]
    lib.mv_pos_decode_workspace_bytes.restype = c_sz
    lib.mv_pos_decode_workspace_bytes.argtypes = [c_i64, c_i64]
    lib.mv_pos_encode.restype = c_i
    lib.mv_pos_encode.argtypes = [c_vp, c_vp, c_i64, c_i64, c_i64, c_vp]
    lib.mv_pos_decode.restype = c_i
    lib.mv_pos_decode.argtypes = [c_vp, c_vp, c_i64, c_i64, c_i64, c_vp, c_i64, c_vp, c_vp, c_sz]
    lib.mv_quant_stream_words.restype = c_i64
    lib.mv_quant_stream_words.argtypes = [c_i64, c_i]
    lib.mv_quant_workspace_bytes.restype = c_sz
    lib.mv_quant_workspace_bytes.argtypes = [c_i]
    lib.mv_quantize.restype = c_i
    lib.mv_quantize.argtypes = [c_vp, c_vp, c_i64, c_i, c_vp, c_vp, c_vp, c_sz]
    lib.mv_dequantize.restype = c_i
    lib.mv_dequantize.argtypes = [c_vp, c_vp, c_i64, c_i, c_vp]
    lib.mv_set_tail_kernel.restype = c_i
    lib.mv_set_tail_kernel.argtypes = [c_vp, c_i]
    lib.mv_fallback_count.restype = c_i
    lib.mv_fallback_count.argtypes = [c_vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.mv_debug_status.restype = c_i
    lib.mv_debug_status.argtypes = [c_vp, ctypes.POINTER(c_i)]
    lib.mv_debug_build.restype = c_i
    lib.mv_debug_build.argtypes = []
    return lib


def status_string(status: int) -> str:
    return load().mv_status_string(int(status)).decode()


def workspace_bytes(N: int, d: int, K: int) -> int:
    return int(load().mv_workspace_bytes(int(N), int(d), int(K)))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _check(status: int, where: str):
    if status != MV_OK:
        raise MvError(status, where)


def mv_select_static(votes, N: int, K: int, out_idx, mask_bits=None, stream: Optional[torch.cuda.Stream] = None):
    """mv_select without a context or a workspace (scratch is an array built into the library);
    for callers that may not allocate device memory.  d is limited to MV_SELECT_STATIC_MAX_D."""
    st = stream if stream is not None else torch.cuda.current_stream(votes.device)
    _check(load().mv_select_static(ctypes.c_void_p(st.cuda_stream), _ptr(votes), int(N), votes.numel(), int(K),
                                   _ptr(out_idx), _ptr(mask_bits)), "mv_select_static")


def _stream_ptr(t: torch.Tensor, stream: Optional[torch.cuda.Stream]):
    st = stream if stream is not None else torch.cuda.current_stream(t.device)
    return ctypes.c_void_p(st.cuda_stream)


def pos_offset_bits(B: int) -> int:
    return int(load().mv_pos_offset_bits(int(B)))


def pos_stream_bits(d: int, B: int, K: int) -> int:
    return int(load().mv_pos_stream_bits(int(d), int(B), int(K)))


def pos_decode_workspace_bytes(nbits: int, B: int) -> int:
    return int(load().mv_pos_decode_workspace_bytes(int(nbits), int(B)))


def quant_stream_words(K: int, q: int) -> int:
    return int(load().mv_quant_stream_words(int(K), int(q)))


def quant_workspace_bytes(q: int) -> int:
    return int(load().mv_quant_workspace_bytes(int(q)))


def mv_pos_encode(idx, d: int, B: int, words, stream: Optional[torch.cuda.Stream] = None):
    """Position stream of an ascending int32 index list into `words` (uint32/int32, caller-sized)."""
    _check(load().mv_pos_encode(_stream_ptr(words, stream), _ptr(idx), idx.numel(), int(d), int(B), _ptr(words)),
           "mv_pos_encode")


def mv_pos_decode(words, nbits: int, d: int, B: int, idx, result, workspace, stream: Optional[torch.cuda.Stream] = None):
    _check(load().mv_pos_decode(_stream_ptr(words, stream), _ptr(words), int(nbits), int(d), int(B), _ptr(idx),
                                idx.numel(), _ptr(result), _ptr(workspace), workspace.numel() * workspace.element_size()),
           "mv_pos_decode")


def mv_quantize(v, q: int, words, workspace, value_range=None, stream: Optional[torch.cuda.Stream] = None):
    _check(load().mv_quantize(_stream_ptr(words, stream), _ptr(v), v.numel(), int(q), _ptr(words), _ptr(value_range),
                              _ptr(workspace), workspace.numel() * workspace.element_size()), "mv_quantize")


def mv_dequantize(words, K: int, q: int, out, stream: Optional[torch.cuda.Stream] = None):
    _check(load().mv_dequantize(_stream_ptr(words, stream), _ptr(words), int(K), int(q), _ptr(out)), "mv_dequantize")


class MvContext:
    """A context bound to the current CUDA stream and to a workspace tensor it keeps alive."""

    def __init__(self, N: int, d: int, K: int, device="cuda", stream: Optional[torch.cuda.Stream] = None,
                 mode: int = MV_MODE_AUTO, debug: bool = False):
        self.lib = load_debug() if debug else load()
        self.N, self.d, self.K = int(N), int(d), int(K)
        nbytes = workspace_bytes(N, d, K)
        if nbytes == 0:
            raise MvError(MV_ERR_INVALID_ARG, "mv_workspace_bytes")
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.workspace.device)
        handle = ctypes.c_void_p()
        _check(self.lib.mv_create(ctypes.byref(handle), ctypes.c_void_p(self.stream.cuda_stream),
                                  _ptr(self.workspace), nbytes), "mv_create")
        self.handle = handle
        self.set_mode(mode)

    def close(self):
        if getattr(self, "handle", None):
            self.lib.mv_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_tail_kernel(self, enable: int):
        """Whole steps as two kernels (streaming pass + one persistent tail kernel): 0 never, 1 where it pays
        (the default), 2 wherever it can run."""
        _check(self.lib.mv_set_tail_kernel(self.handle, int(enable)), "mv_set_tail_kernel")

    def set_mode(self, mode: int):
        _check(self.lib.mv_set_mode(self.handle, int(mode)), "mv_set_mode")

    # the calls below mirror include/mv_sparse.h one to one
    def mv_sparse_step(self, grads, err, out_idx, out_val, K: Optional[int] = None):
        N, d = grads.shape
        _check(self.lib.mv_sparse_step(self.handle, _ptr(grads), _ptr(err), N, d, K or self.K,
                                       _ptr(out_idx), _ptr(out_val)), "mv_sparse_step")

    def mv_vote(self, grads, err, worker_idx=None, worker_bits=None, votes=None, thresh=None, K: Optional[int] = None):
        N, d = grads.shape
        _check(self.lib.mv_vote(self.handle, _ptr(grads), _ptr(err), N, d, K or self.K, _ptr(worker_idx),
                                _ptr(worker_bits), _ptr(votes), _ptr(thresh)), "mv_vote")

    def mv_select(self, votes, N: int, out_idx, mask_bits=None, K: Optional[int] = None):
        _check(self.lib.mv_select(self.handle, _ptr(votes), N, votes.numel(), K or self.K, _ptr(out_idx),
                                  _ptr(mask_bits)), "mv_select")

    def mv_aggregate(self, acc, idx, out_val):
        N, d = acc.shape
        _check(self.lib.mv_aggregate(self.handle, _ptr(acc), N, d, idx.numel(), _ptr(idx), _ptr(out_val)),
               "mv_aggregate")

    def mv_ad_step(self, grads, err, prev_bits, K_ad: int, out_idx, out_val, add_bits=None, drop_bits=None,
                   msum=None, K: Optional[int] = None):
        N, d = grads.shape
        _check(self.lib.mv_ad_step(self.handle, _ptr(grads), _ptr(err), _ptr(prev_bits), N, d, K or self.K, int(K_ad),
                                   _ptr(out_idx), _ptr(out_val), _ptr(add_bits), _ptr(drop_bits), _ptr(msum)),
               "mv_ad_step")

    def mv_topk_union_step(self, grads, err, out_idx, out_val, count, K: Optional[int] = None):
        """SSGD-top-K: out_idx / out_val [capacity >= min(d, N K)], count: int32 [1] on the device."""
        N, d = grads.shape
        _check(self.lib.mv_topk_union_step(self.handle, _ptr(grads), _ptr(err), N, d, K or self.K, _ptr(out_idx),
                                           _ptr(out_val), out_idx.numel(), _ptr(count)), "mv_topk_union_step")

    def mv_select_rs(self, votes, N: int, seed: int, draw: int, out_idx, mask_bits=None, K: Optional[int] = None):
        _check(self.lib.mv_select_rs(self.handle, _ptr(votes), int(N), votes.numel(), int(K or self.K), int(seed), int(draw),
                                     _ptr(out_idx), _ptr(mask_bits)), "mv_select_rs")

    def mv_rs_step(self, grads, err, seed: int, draw: int, out_idx, out_val, K: Optional[int] = None):
        N, d = grads.shape
        _check(self.lib.mv_rs_step(self.handle, _ptr(grads), _ptr(err), int(N), int(d), int(K or self.K), int(seed), int(draw),
                                   _ptr(out_idx), _ptr(out_val)), "mv_rs_step")

    def mv_aggregate_partial(self, acc, idx, out_sum):
        N, d = acc.shape
        _check(self.lib.mv_aggregate_partial(self.handle, _ptr(acc), N, d, idx.numel(), _ptr(idx), _ptr(out_sum)),
               "mv_aggregate_partial")

    def mv_finish_mean(self, total, N_total: int, out_val):
        _check(self.lib.mv_finish_mean(ctypes.c_void_p(self.stream.cuda_stream), _ptr(total), total.numel(), int(N_total),
                                       _ptr(out_val)), "mv_finish_mean")

    def mv_sparse_step_host(self, h_grads, h_out_idx, h_out_val, d_grads, d_err, d_out_idx, d_out_val,
                            K: Optional[int] = None):
        N, d = h_grads.shape
        _check(self.lib.mv_sparse_step_host(self.handle, _ptr(h_grads), N, d, K or self.K, _ptr(h_out_idx),
                                            _ptr(h_out_val), _ptr(d_grads), _ptr(d_err), _ptr(d_out_idx),
                                            _ptr(d_out_val)), "mv_sparse_step_host")

    def read_diag(self, N: Optional[int] = None) -> torch.Tensor:
        N = N or self.N
        out = torch.zeros((N, 4), dtype=torch.int64)
        buf = (ctypes.c_uint32 * (4 * N))()
        _check(self.lib.mv_read_diag(self.handle, N, buf), "mv_read_diag")
        out.copy_(torch.tensor(list(buf), dtype=torch.int64).view(N, 4))
        return out

    def set_kernel_timing(self, every: int):
        """0: off; n >= 1: time the streaming pass on every n-th step."""
        _check(self.lib.mv_set_kernel_timing(self.handle, int(every)), "mv_set_kernel_timing")

    def read_kernel_timing(self):
        """(total milliseconds, launches covered) of the streaming pass since the last read."""
        ms, cnt = ctypes.c_float(), ctypes.c_int()
        _check(self.lib.mv_read_kernel_timing(self.handle, ctypes.byref(ms), ctypes.byref(cnt)),
               "mv_read_kernel_timing")
        return float(ms.value), int(cnt.value)

    def set_phase_timing(self, enable: int):
        """0: off; 1: an event after every launch; 100 + i: only the start and the end of launch i."""
        _check(self.lib.mv_set_phase_timing(self.handle, int(enable)), "mv_set_phase_timing")

    def read_phase_times(self):
        """Milliseconds per kernel launch of the last call, in launch order."""
        buf = (ctypes.c_float * 47)()
        cnt = ctypes.c_int()
        _check(self.lib.mv_read_phase_times(self.handle, buf, 47, ctypes.byref(cnt)), "mv_read_phase_times")
        return [float(buf[i]) for i in range(cnt.value)]

    def last_launches(self) -> int:
        return int(self.lib.mv_last_launches(self.handle))

    def fallback_count(self) -> int:
        """Worker selections that took the full-row route since the context's first call."""
        total = ctypes.c_uint32()
        _check(self.lib.mv_fallback_count(self.handle, ctypes.byref(total)), "mv_fallback_count")
        return int(total.value)

    def debug_status(self) -> int:
        """MV_DBG_* bits collected by a checked build since the last read (always 0 in a normal build)."""
        word = ctypes.c_int()
        _check(self.lib.mv_debug_status(self.handle, ctypes.byref(word)), "mv_debug_status")
        return int(word.value)
