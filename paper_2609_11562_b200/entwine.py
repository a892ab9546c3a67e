"""ctypes binding over the C-ABI library (include/entwine.h).

Argument marshalling only: every step of the path runs in the CUDA library.  Importing this
module fails loudly if libentwine.so has not been built (there is no fallback).
Device-buffer arguments are torch CUDA tensors (bf16, contiguous) or raw integer addresses;
`stream` is a torch.cuda.Stream, a raw handle or None (the current torch stream).
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libentwine.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2609_11562_b200.build` "
        "(or __graft_entry__.build()); this package has no CPU fallback")
_lib = ctypes.CDLL(LIB_PATH)

ORDER_ROW_MAJOR, ORDER_INTERLEAVED, ORDER_M_MAJOR = 0, 1, 2
OK, ERR_INVALID, ERR_RESOURCES, ERR_CUDA, ERR_TIMEOUT, ERR_INTERNAL = 0, -1, -2, -3, -4, -5
ERR_TOO_LARGE = -6
OPT_RANK, OPT_BLOCK_N, OPT_WAIT_BUDGET_NS, OPT_TAIL_HELP = 1, 2, 3, 4
OPT_WITHHOLD_PEER, OPT_NUM_SMS, OPT_POISON_PARTIAL, OPT_PAIR_CTAS, OPT_COLOCATE = 5, 6, 7, 8, 9
OPT_PREFETCH, OPT_STAGES, OPT_L2_HINTS, OPT_LISTS, OPT_RELEASE_GROUP = 10, 11, 12, 13, 14
OPT_KBLOCKS_PER_STAGE, OPT_LDA, OPT_LDB, OPT_REG_CONSUMER, OPT_SPLIT_LAST_WAVE, OPT_B_LAYOUT = 15, 16, 17, 18, 19, 20
OPT_CONSUMER_TMA = 21
B_LAYOUT_NK, B_LAYOUT_KN = 0, 1
RELEASE_PARTITION, RELEASE_WHOLE = -1, -2
(EXPORT_COUNTS, EXPORT_ORDER, EXPORT_TILES, EXPORT_FLAG_SEQ, EXPORT_LIST_OFFS, EXPORT_TASKS,
 EXPORT_PEER_OFFS) = range(7)

# every symbol include/entwine.h declares
SYMBOLS = ("entwine_plan", "entwine_set_option", "entwine_gemm_rs", "entwine_gemm_rs_host",
           "entwine_gemm_only", "entwine_comm_only", "entwine_read_partial", "entwine_plan_export",
           "entwine_last_status", "entwine_destroy", "entwine_strerror", "entwine_gemm_rs_static",
           "entwine_gemm_rs_norm", "entwine_heap_bytes", "entwine_gemm_rs_pull",
           "entwine_gemm_rs_host_begin", "entwine_gemm_rs_host_wait", "entwine_last_sm_clock",
           "entwine_plan_workspace_bytes", "entwine_plan_set_workspace")

_vp, _i64, _int = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int
_lib.entwine_plan.argtypes = [ctypes.POINTER(_vp), _i64, _i64, _i64, _int, _int, _int]
_lib.entwine_set_option.argtypes = [_vp, _int, _i64]
_lib.entwine_gemm_rs_norm.argtypes = [_vp, _vp, _vp, _vp, _vp, _vp, ctypes.c_float, _vp, _vp, _vp, _vp]
_lib.entwine_gemm_rs.argtypes = [_vp] * 7
_lib.entwine_heap_bytes.argtypes = [_vp, ctypes.POINTER(_i64), ctypes.POINTER(_i64)]
_lib.entwine_gemm_rs_pull.argtypes = [_vp, _vp, _vp, _vp, _i64, ctypes.c_uint32, _int, _vp, _vp]
_lib.entwine_gemm_rs_host.argtypes = [_vp] * 6
_lib.entwine_gemm_rs_host_begin.argtypes = [_vp] * 6
_lib.entwine_gemm_rs_host_wait.argtypes = [_vp]
_lib.entwine_gemm_only.argtypes = [_vp] * 4
_lib.entwine_comm_only.argtypes = [_vp, _vp, _vp, _vp, _vp, _int, _vp]
_lib.entwine_read_partial.argtypes = [_vp, _vp, _vp]
_lib.entwine_plan_export.argtypes = [_vp, _int, _vp, ctypes.POINTER(ctypes.c_size_t)]
_lib.entwine_last_status.argtypes = [_vp, ctypes.POINTER(_i64)]
_lib.entwine_last_sm_clock.argtypes = [_vp, ctypes.POINTER(_i64)]
_lib.entwine_plan_workspace_bytes.argtypes = [_vp, ctypes.POINTER(ctypes.c_size_t)]
_lib.entwine_plan_set_workspace.argtypes = [_vp, _vp, ctypes.c_size_t]
_lib.entwine_destroy.argtypes = [_vp]
_lib.entwine_gemm_rs_static.argtypes = [_vp] * 7 + [ctypes.POINTER(_i64)]
_lib.entwine_strerror.argtypes = [_int]
_lib.entwine_strerror.restype = ctypes.c_char_p
for _name in SYMBOLS:
    if _name != "entwine_strerror":
        getattr(_lib, _name).restype = _int


class EntwineError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} ({code})")


def strerror(code: int) -> str:
    return _lib.entwine_strerror(code).decode()


def _check(code: int, what: str):
    if code != OK:
        raise EntwineError(code, what)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(s):
    if s is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(s, int):
        return s
    return s.cuda_stream


_EXPORT_DTYPE = {EXPORT_COUNTS: np.int64, EXPORT_ORDER: np.int32, EXPORT_TILES: np.int32,
                 EXPORT_FLAG_SEQ: np.int32, EXPORT_LIST_OFFS: np.int32, EXPORT_TASKS: np.int64,
                 EXPORT_PEER_OFFS: np.int64}


class Plan:
    """entwine_plan / entwine_destroy as a Python object; methods mirror the C entry points."""

    def __init__(self, M, N, K_local, W, tile_order=ORDER_INTERLEAVED, n_comm_sms=0, **options):
        self._h = _vp()
        _check(_lib.entwine_plan(ctypes.byref(self._h), M, N, K_local, W, tile_order, n_comm_sms),
               "entwine_plan")
        self.M, self.N, self.K, self.W = M, N, K_local, W
        self.tile_order, self.n_comm_sms = tile_order, n_comm_sms
        self.rank = 0
        keys = {"rank": OPT_RANK, "block_n": OPT_BLOCK_N, "wait_budget_ns": OPT_WAIT_BUDGET_NS,
                "tail_help": OPT_TAIL_HELP, "num_sms": OPT_NUM_SMS, "poison_partial": OPT_POISON_PARTIAL,
                "pair_ctas": OPT_PAIR_CTAS, "colocate": OPT_COLOCATE, "prefetch": OPT_PREFETCH, "stages": OPT_STAGES, "l2_hints": OPT_L2_HINTS, "lists": OPT_LISTS, "release_group": OPT_RELEASE_GROUP,
                "kblocks_per_stage": OPT_KBLOCKS_PER_STAGE, "reg_consumer": OPT_REG_CONSUMER, "split_last_wave": OPT_SPLIT_LAST_WAVE, "b_layout": OPT_B_LAYOUT, "consumer_tma": OPT_CONSUMER_TMA, "lda": OPT_LDA, "ldb": OPT_LDB}
        # num_sms first: it bounds the others
        for name in sorted(options, key=lambda n: {"num_sms": 0, "b_layout": 1}.get(n, 2)):
            self.set_option(keys[name], options[name])

    def set_option(self, key, value):
        _check(_lib.entwine_set_option(self._h, key, int(value)), f"entwine_set_option({key})")
        if key == OPT_RANK:
            self.rank = int(value)

    def gemm_rs(self, A, B, peer_partials, out_shard, send_bufs, stream=None):
        _check(_lib.entwine_gemm_rs(self._h, _ptr(A), _ptr(B), _ptr(peer_partials), _ptr(out_shard),
                                    _ptr(send_bufs), _stream(stream)), "entwine_gemm_rs")

    def gemm_rs_norm(self, A, B, peer_partials, residual, weight, eps, hidden_out, norm_out, send_bufs,
                     stream=None):
        _check(_lib.entwine_gemm_rs_norm(self._h, _ptr(A), _ptr(B), _ptr(peer_partials), _ptr(residual),
                                         _ptr(weight), float(eps), _ptr(hidden_out), _ptr(norm_out),
                                         _ptr(send_bufs), _stream(stream)), "entwine_gemm_rs_norm")

    def heap_bytes(self):
        """(least bytes of one rank's heap segment, offset of its flag array)."""
        seg, off = _i64(0), _i64(0)
        _check(_lib.entwine_heap_bytes(self._h, ctypes.byref(seg), ctypes.byref(off)), "entwine_heap_bytes")
        return seg.value, off.value

    def gemm_rs_pull(self, A, B, heap, heap_stride, epoch, out_shard, produce_only=False, stream=None):
        _check(_lib.entwine_gemm_rs_pull(self._h, _ptr(A), _ptr(B), _ptr(heap), int(heap_stride), int(epoch),
                                         1 if produce_only else 0, _ptr(out_shard), _stream(stream)),
               "entwine_gemm_rs_pull")

    def gemm_rs_host(self, A, B, peer_partials, out_shard, send_bufs):
        """Host tensors (CPU, bf16, contiguous; pinned for speed)."""
        _check(_lib.entwine_gemm_rs_host(self._h, _ptr(A), _ptr(B), _ptr(peer_partials),
                                         _ptr(out_shard), _ptr(send_bufs)), "entwine_gemm_rs_host")

    def gemm_rs_host_begin(self, A, B, peer_partials, out_shard, send_bufs):
        """Enqueue one host-buffer call (at most two outstanding); pair with gemm_rs_host_wait."""
        _check(_lib.entwine_gemm_rs_host_begin(self._h, _ptr(A), _ptr(B), _ptr(peer_partials),
                                               _ptr(out_shard), _ptr(send_bufs)), "entwine_gemm_rs_host_begin")

    def gemm_rs_host_wait(self):
        _check(_lib.entwine_gemm_rs_host_wait(self._h), "entwine_gemm_rs_host_wait")

    def gemm_rs_static(self, A, B, peer_partials, out_shard, send_bufs, stream=None, want_status=True):
        """The fused call on the library's fixed scratch array: for callers that must not
        allocate device memory (see include/entwine.h).  Problems above the array's limits raise
        EntwineError(ERR_TOO_LARGE).  With want_status the call synchronises the stream and
        returns the status dict; overlapping calls on one device race."""
        out = (_i64 * 8)() if want_status else None
        code = _lib.entwine_gemm_rs_static(self._h, _ptr(A), _ptr(B), _ptr(peer_partials), _ptr(out_shard),
                                           _ptr(send_bufs), _stream(stream), out)
        _check(code, "entwine_gemm_rs_static")
        if not want_status:
            return None
        names = ("code", "cta", "where", "flags_published", "tiles_reduced", "tiles_pushed",
                 "t_gemm_ns", "t_end_ns")
        return {k: int(v) for k, v in zip(names, out)}

    def gemm_only(self, A, B, stream=None):
        _check(_lib.entwine_gemm_only(self._h, _ptr(A), _ptr(B), _stream(stream)), "entwine_gemm_only")

    def comm_only(self, partial, peer_partials, out_shard, send_bufs, n_ctas=0, stream=None):
        _check(_lib.entwine_comm_only(self._h, _ptr(partial), _ptr(peer_partials), _ptr(out_shard),
                                      _ptr(send_bufs), n_ctas, _stream(stream)), "entwine_comm_only")

    def read_partial(self, dst, stream=None):
        _check(_lib.entwine_read_partial(self._h, _ptr(dst), _stream(stream)), "entwine_read_partial")

    def export(self, what) -> np.ndarray:
        n = ctypes.c_size_t(0)
        _check(_lib.entwine_plan_export(self._h, what, None, ctypes.byref(n)), "entwine_plan_export")
        buf = np.zeros(n.value // np.dtype(_EXPORT_DTYPE[what]).itemsize, _EXPORT_DTYPE[what])
        cap = ctypes.c_size_t(buf.nbytes)
        _check(_lib.entwine_plan_export(self._h, what, buf.ctypes.data_as(_vp), ctypes.byref(cap)),
               "entwine_plan_export")
        return buf

    def counts(self) -> dict:
        c = self.export(EXPORT_COUNTS)
        names = ("P_blk", "Q", "cpb", "x", "n_tasks", "n_reduce", "n_push", "flags_published",
                 "peer_flags_prepublished", "min_flag_reads", "bytes_peer_read", "bytes_own_read",
                 "bytes_push_write", "bytes_out_write", "n_gemm_ctas", "n_comm_ctas")
        return {k: int(v) for k, v in zip(names, c)}

    def last_status(self, check=True) -> dict:
        out = (_i64 * 8)()
        code = _lib.entwine_last_status(self._h, out)
        names = ("code", "cta", "where", "flags_published", "tiles_reduced", "tiles_pushed",
                 "t_gemm_ns", "t_end_ns")
        st = {k: int(v) for k, v in zip(names, out)}
        if check and code != OK:
            raise EntwineError(code, f"device status {st}")
        return st

    def workspace_bytes(self) -> int:
        n = ctypes.c_size_t(0)
        _check(_lib.entwine_plan_workspace_bytes(self._h, ctypes.byref(n)), "entwine_plan_workspace_bytes")
        return int(n.value)

    def set_workspace(self, buf, nbytes=None):
        """buf: a CUDA tensor (kept alive by this object) or a raw device address with nbytes."""
        if buf is None:
            _check(_lib.entwine_plan_set_workspace(self._h, None, 0), "entwine_plan_set_workspace")
            self._ws = None
            return
        n = nbytes if nbytes is not None else buf.numel() * buf.element_size()
        _check(_lib.entwine_plan_set_workspace(self._h, _ptr(buf), n), "entwine_plan_set_workspace")
        self._ws = buf

    def last_sm_clock_mhz(self) -> float:
        """SM clock of the launch that the last last_status() call reported (0.0 if unknown)."""
        out = (_i64 * 2)()
        _check(_lib.entwine_last_sm_clock(self._h, out), "entwine_last_sm_clock")
        return out[0] / out[1] * 1e3 if out[1] > 0 else 0.0

    def destroy(self):
        if self._h:
            _lib.entwine_destroy(self._h)
            self._h = _vp()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
