"""Thin ctypes binding of libtessera.so: argument marshalling only.

Every step of the path runs inside the library's kernels.  torch appears here
only as the owner of device memory and of the current stream.  Importing this
module fails loudly when the library has not been built; there is no fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libtessera.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        "libtessera.so is missing: build it with `python -m paper_2609_32999_b200.build` "
        "(nvcc, sm_100a).  This package has no CPU or eager fallback.")
_lib = ctypes.CDLL(LIB_PATH)

OK = 0
INVALID_ARG, UNSORTED_POSITIONS, UNIT_OVERLAP, UNCOVERED_POSITION = -1, -2, -3, -4
PAGE_OUT_OF_RANGE, OUT_OF_PAGES, UNSUPPORTED_SHAPE, CUDA_ERROR, DEVICE_TIMEOUT = -5, -6, -7, -8, -9
PLAN_HOST_ONLY = 1
FUSE_ROPE = 1

_I32P = ctypes.POINTER(ctypes.c_int32)


class ModelCfg(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("rope_theta", ctypes.c_double), ("inv_freq", ctypes.POINTER(ctypes.c_double)),
                ("rope_pairing", ctypes.c_int32), ("sm_scale", ctypes.c_float)]


class ComposeDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("seq_len", _I32P), ("unit_off", _I32P), ("unit_len", _I32P),
                ("unit_cached_pos", _I32P), ("unit_cached_stride", _I32P), ("unit_target_pos", _I32P),
                ("unit_page_off", _I32P), ("unit_pages", _I32P), ("recompute_off", _I32P),
                ("recompute_pos", _I32P), ("free_pages", _I32P), ("n_free", ctypes.c_int32),
                ("unit_src_offset", _I32P), ("num_source_pages", ctypes.c_int32), ("unit_target_stride", _I32P),
                ("unit_retain_page_off", _I32P), ("unit_retain_pages", _I32P), ("retain_pool_pages", ctypes.c_int32)]


class PlanInfo(ctypes.Structure):
    _fields_ = [("total_tokens", ctypes.c_int64), ("n_q", ctypes.c_int64), ("cached_tokens", ctypes.c_int64),
                ("qk_pairs", ctypes.c_int64), ("gather_bytes", ctypes.c_int64), ("attn_flops", ctypes.c_int64),
                ("n_rope_rows", ctypes.c_int32), ("n_gather_items", ctypes.c_int32),
                ("n_attn_items", ctypes.c_int32), ("attn_kernel", ctypes.c_int32),
                ("retained_tokens", ctypes.c_int64), ("attn_mma_pairs", ctypes.c_int64)]


EXPORTS = ["tessera_plan_create", "tessera_plan_destroy", "tessera_plan_block_table", "tessera_plan_get_info",
           "tessera_plan_status", "tessera_kv_compose", "tessera_kv_compose_from", "tessera_kv_compose_from_fp8", "tessera_kv_retain_fp8", "tessera_rope_shift", "tessera_rope_fresh", "tessera_extend_write", "tessera_partial_prefill_attn", "tessera_kv_compose_k8", "tessera_partial_prefill_attn_k8",
           "tessera_composed_prefill_host", "tessera_composed_prefill_host_tier", "tessera_rope_shift_static", "tessera_selftest_bounded_wait", "tessera_last_error",
           "tessera_launch_count"]

_vp = ctypes.c_void_p
_lib.tessera_plan_create.argtypes = [ctypes.POINTER(ModelCfg), ctypes.POINTER(ComposeDesc), ctypes.c_int32,
                                     ctypes.c_uint32, ctypes.POINTER(_vp), _vp]
_lib.tessera_plan_destroy.argtypes = [_vp]
_lib.tessera_plan_block_table.argtypes = [_vp, ctypes.POINTER(_I32P), ctypes.POINTER(_I32P), ctypes.POINTER(_I32P)]
_lib.tessera_plan_get_info.argtypes = [_vp, ctypes.POINTER(PlanInfo)]
_lib.tessera_plan_status.argtypes = [_vp, _I32P, _vp]
_lib.tessera_kv_compose.argtypes = [_vp, _vp, _vp, ctypes.c_uint32, _vp]
_lib.tessera_kv_compose_from.argtypes = [_vp, _vp, _vp, _vp, _vp, ctypes.c_uint32, _vp]
_lib.tessera_kv_compose_from_fp8.argtypes = [_vp, _vp, _vp, ctypes.c_float, ctypes.c_float, _vp, _vp, ctypes.c_uint32, _vp]
_lib.tessera_kv_retain_fp8.argtypes = [_vp, _vp, _vp, _vp, _vp, ctypes.c_float, ctypes.c_float, ctypes.c_uint32, _vp]
_lib.tessera_rope_shift.argtypes = [_vp, _vp, _vp]
_lib.tessera_rope_fresh.argtypes = [_vp, _vp, _vp, _vp]
_lib.tessera_extend_write.argtypes = [_vp] * 9
_lib.tessera_partial_prefill_attn.argtypes = [_vp] * 9
_lib.tessera_kv_compose_k8.argtypes = [_vp, _vp, _vp, _vp, _vp, ctypes.c_float, ctypes.c_uint32, _vp]
_lib.tessera_partial_prefill_attn_k8.argtypes = [_vp, _vp, ctypes.c_float, _vp, _vp, ctypes.c_float, _vp, _vp, _vp, _vp, _vp]
_lib.tessera_composed_prefill_host.argtypes = [_vp] * 9
_lib.tessera_composed_prefill_host_tier.argtypes = [_vp, _vp, _vp, ctypes.c_int32, ctypes.c_float, ctypes.c_float,
                                                    _vp, _vp, _vp, _vp, _vp, _vp, _vp, ctypes.c_int32, _vp]
_lib.tessera_rope_shift_static.argtypes = [ctypes.POINTER(ModelCfg), _vp, ctypes.c_int64, _vp, _vp, ctypes.c_int32,
                                           _I32P, ctypes.c_int32, _vp]
_lib.tessera_selftest_bounded_wait.argtypes = [ctypes.c_int64, _I32P, ctypes.POINTER(ctypes.c_int64), _vp]
_lib.tessera_last_error.argtypes = [ctypes.c_char_p, ctypes.c_int32]
_lib.tessera_launch_count.argtypes = []
_lib.tessera_launch_count.restype = ctypes.c_int64
for _n in EXPORTS[:-1]:
    getattr(_lib, _n).restype = ctypes.c_int32


class TesseraError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__("tessera status %d: %s" % (status, text))
        self.status = status


def last_error() -> str:
    buf = ctypes.create_string_buffer(512)
    _lib.tessera_last_error(buf, 512)
    return buf.value.decode("utf-8", "replace")


def _check(st: int) -> None:
    if st != OK:
        raise TesseraError(st, last_error())


def launch_count() -> int:
    return int(_lib.tessera_launch_count())


def _arr(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(_I32P)


def _dev(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    if isinstance(stream, int):
        return stream or None
    return stream.cuda_stream or None


class Plan:
    """tessera_plan_create / tessera_plan_destroy with host arrays taken from a Workload-like
    object (anything with the descriptor's field names and a `.shape` model description)."""

    def __init__(self, w, host_only: bool = False, stream=None, inv_freq=None):
        sh = w.shape
        self._keep = [_arr(getattr(w, f)) for f in
                      ("seq_len", "unit_off", "unit_len", "unit_cached_pos", "unit_cached_stride",
                       "unit_target_pos", "unit_page_off", "unit_pages", "recompute_off", "recompute_pos",
                       "free_pages")]
        a = self._keep
        self._inv = None if inv_freq is None else np.ascontiguousarray(inv_freq, dtype=np.float64)
        cfg = ModelCfg(sh.num_q_heads, sh.num_kv_heads, sh.head_dim, sh.page_size, float(sh.rope_theta),
                       None if self._inv is None else self._inv.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                       int(sh.rope_pairing), float(sh.sm_scale))
        opt = [None if getattr(w, f, None) is None else _arr(getattr(w, f))
               for f in ("unit_src_offset", "unit_target_stride", "unit_retain_page_off", "unit_retain_pages")]
        op = [None if x is None else _ptr(x) for x in opt]
        desc = ComposeDesc(len(a[0]), *[_ptr(x) for x in a[:11]], len(a[10]), op[0],
                           int(getattr(w, "num_source_pages", 0) or 0), op[1], op[2], op[3],
                           int(getattr(w, "retain_pool_pages", 0) or 0))
        self._opt = opt
        self._h = _vp()
        self.host_only = host_only
        st = _lib.tessera_plan_create(ctypes.byref(cfg), ctypes.byref(desc), int(w.num_pool_pages),
                                      PLAN_HOST_ONLY if host_only else 0, ctypes.byref(self._h),
                                      None if host_only else _stream(stream))
        _check(st)
        self.batch = len(a[0])
        self.info = PlanInfo()
        _check(_lib.tessera_plan_get_info(self._h, ctypes.byref(self.info)))
        # share of the tensor-core (row, key) products that is not an algorithmic (query row, key) pair
        pairs = self.info.qk_pairs * sh.num_q_heads
        self.masked_mma_fraction = 1.0 - pairs / self.info.attn_mma_pairs if self.info.attn_mma_pairs else 0.0

    def block_table(self):
        """(page_off, pages, src_slot) as numpy copies of the plan's host tables."""
        po, pg, ss = _I32P(), _I32P(), _I32P()
        _check(_lib.tessera_plan_block_table(self._h, ctypes.byref(po), ctypes.byref(pg), ctypes.byref(ss)))
        page_off = np.ctypeslib.as_array(po, shape=(self.batch + 1,)).copy()
        n_pages, n_tok = int(page_off[-1]), int(self.info.total_tokens)
        pages = np.ctypeslib.as_array(pg, shape=(n_pages,)).copy() if n_pages else np.zeros(0, np.int32)
        src = np.ctypeslib.as_array(ss, shape=(n_tok,)).copy() if n_tok else np.zeros(0, np.int32)
        return page_off, pages, src

    def status(self, stream=None) -> int:
        detail = ctypes.c_int32(0)
        st = _lib.tessera_plan_status(self._h, ctypes.byref(detail), _stream(stream))
        if st not in (OK, DEVICE_TIMEOUT):
            _check(st)
        return int(detail.value)

    def kv_compose(self, k_pool, v_pool, fuse_rope: bool = True, stream=None) -> None:
        _check(_lib.tessera_kv_compose(self._h, _dev(k_pool), _dev(v_pool), FUSE_ROPE if fuse_rope else 0,
                                       _stream(stream)))

    def kv_compose_from(self, k_src, v_src, k_pool, v_pool, fuse_rope: bool = True, stream=None) -> None:
        """Sources in a separate pool (pinned host tensors or device tensors), destinations in the pools."""
        _check(_lib.tessera_kv_compose_from(self._h, _dev(k_src), _dev(v_src), _dev(k_pool), _dev(v_pool),
                                            FUSE_ROPE if fuse_rope else 0, _stream(stream)))

    def kv_compose_from_fp8(self, k_src8, v_src8, k_scale: float, v_scale: float, k_pool, v_pool,
                            fuse_rope: bool = True, stream=None) -> None:
        """Sources are e4m3 codes (uint8 or float8_e4m3fn tensors) standing for code * scale."""
        _check(_lib.tessera_kv_compose_from_fp8(self._h, _dev(k_src8), _dev(v_src8), k_scale, v_scale, _dev(k_pool),
                                                _dev(v_pool), FUSE_ROPE if fuse_rope else 0, _stream(stream)))

    def kv_retain_fp8(self, k_src, v_src, k_dst8, v_dst8, k_scale: float, v_scale: float, fuse_rope: bool = True,
                      stream=None) -> None:
        """16-bit source pools -> e4m3 destination pools (the plan's destination pages index the 8-bit pools)."""
        _check(_lib.tessera_kv_retain_fp8(self._h, _dev(k_src), _dev(v_src), _dev(k_dst8), _dev(v_dst8), k_scale, v_scale,
                                          FUSE_ROPE if fuse_rope else 0, _stream(stream)))

    def rope_shift(self, k_pool, stream=None) -> None:
        _check(_lib.tessera_rope_shift(self._h, _dev(k_pool), _stream(stream)))

    def rope_fresh(self, q, k_new, stream=None) -> None:
        """Rotate fresh q / k_new rows in place for their target positions (either may be None)."""
        _check(_lib.tessera_rope_fresh(self._h, _dev(q), _dev(k_new), _stream(stream)))

    def extend_write(self, k_pool, v_pool, q, k_new_raw, v_new, k_cache=None, v_cache=None, stream=None) -> None:
        """Fused write side of the extend pass: rotate q in place, write rotated K / V rows to their slots
        and the raw rows of captured units to k_cache / v_cache (attention then runs with k_new = v_new = None)."""
        _check(_lib.tessera_extend_write(self._h, _dev(k_pool), _dev(v_pool), _dev(q), _dev(k_new_raw), _dev(v_new),
                                         _dev(k_cache), _dev(v_cache), _stream(stream)))

    def partial_prefill_attn(self, k_pool, v_pool, q, k_new, v_new, out, lse=None, stream=None) -> None:
        _check(_lib.tessera_partial_prefill_attn(self._h, _dev(k_pool), _dev(v_pool), _dev(q), _dev(k_new),
                                                 _dev(v_new), _dev(out), _dev(lse), _stream(stream)))

    def kv_compose_k8(self, k_src, v_src, k_pool8, v_pool, k_scale: float, fuse_rope: bool = True, stream=None) -> None:
        """16-bit source pools -> keys as e4m3 codes in k_pool8 (rotated on the way), values into the 16-bit v_pool."""
        _check(_lib.tessera_kv_compose_k8(self._h, _dev(k_src), _dev(v_src), _dev(k_pool8), _dev(v_pool), float(k_scale),
                                          FUSE_ROPE if fuse_rope else 0, _stream(stream)))

    def partial_prefill_attn_k8(self, k_pool8, k_scale: float, v_pool, q, q_scale: float, k_new, v_new, out, lse=None,
                                stream=None) -> None:
        """Attention over 8-bit (e4m3) key pages: q is quantised by the call, k_pool8 holds codes."""
        _check(_lib.tessera_partial_prefill_attn_k8(self._h, _dev(k_pool8), float(k_scale), _dev(v_pool), _dev(q),
                                                    float(q_scale), _dev(k_new), _dev(v_new), _dev(out), _dev(lse),
                                                    _stream(stream)))

    def composed_prefill_host(self, k_pool, v_pool, q_host, k_new_host, v_new_host, out_host, lse_host=None,
                              stream=None) -> None:
        _check(_lib.tessera_composed_prefill_host(self._h, _dev(k_pool), _dev(v_pool), _dev(q_host),
                                                  _dev(k_new_host), _dev(v_new_host), _dev(out_host),
                                                  _dev(lse_host), _stream(stream)))

    def composed_prefill_host_tier(self, k_src_host, v_src_host, k_pool, v_pool, q, k_new, v_new, out, lse=None,
                                   src_format: int = 0, k_scale: float = 1.0, v_scale: float = 1.0,
                                   reader_blocks: int = 0, stream=None) -> None:
        """Cached units in pinned host pools (bf16, or e4m3 codes with src_format=1), pulled over the link
        chunk by chunk by a small reader launch while attention of the chunks already there runs."""
        _check(_lib.tessera_composed_prefill_host_tier(self._h, _dev(k_src_host), _dev(v_src_host), int(src_format),
                                                       float(k_scale), float(v_scale), _dev(k_pool), _dev(v_pool),
                                                       _dev(q), _dev(k_new), _dev(v_new), _dev(out), _dev(lse),
                                                       int(reader_blocks), _stream(stream)))

    def destroy(self) -> None:
        if self._h:
            _check(_lib.tessera_plan_destroy(self._h))
            self._h = _vp()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


def selftest_bounded_wait(max_cycles: int, stream=None):
    """tessera_selftest_bounded_wait: returns (status, code, [cycles first wait, cycles second wait, success mask])."""
    code = ctypes.c_int32(0)
    cyc = (ctypes.c_int64 * 3)()
    st = _lib.tessera_selftest_bounded_wait(int(max_cycles), ctypes.byref(code), cyc, _stream(stream))
    return int(st), int(code.value), [int(x) for x in cyc]


STATIC_MAX_SHIFTS = 512


def rope_shift_static(shape, k_pool, slots, slot_shift, shifts, stream=None, inv_freq=None,
                      num_pool_slots: Optional[int] = None) -> None:
    """tessera_rope_shift_static: rotate the listed pool slots in place without any device
    allocation.  `slots` / `slot_shift` are int32 device tensors, `shifts` a host int32 sequence;
    `num_pool_slots` (default: every row of k_pool) bounds the slot ids the kernel accepts."""
    inv = None if inv_freq is None else np.ascontiguousarray(inv_freq, dtype=np.float64)
    cfg = ModelCfg(shape.num_q_heads, shape.num_kv_heads, shape.head_dim, shape.page_size, float(shape.rope_theta),
                   None if inv is None else inv.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                   int(shape.rope_pairing), float(shape.sm_scale))
    sh = _arr(shifts)
    if num_pool_slots is None:
        num_pool_slots = int(k_pool.shape[0]) * int(k_pool.shape[1])
    _check(_lib.tessera_rope_shift_static(ctypes.byref(cfg), _dev(k_pool), int(num_pool_slots), _dev(slots),
                                          _dev(slot_shift), int(slots.numel()), _ptr(sh), len(sh), _stream(stream)))


def plan_create_status(w, host_only: bool = True) -> int:
    """Status code of tessera_plan_create for `w` (the plan, if any, is destroyed at once)."""
    try:
        Plan(w, host_only=host_only).destroy()
        return OK
    except TesseraError as e:
        return e.status
