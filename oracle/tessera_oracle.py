"""ctypes front end of the fp64 CPU oracle (tessera_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the
bench's CPU-baseline leg.  It never imports the CUDA package and the CUDA
package never imports it.  Tensors cross as raw bf16 bit patterns (uint16).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "tessera_oracle.c")
_LIB = os.path.join(_HERE, "libtessera_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math: summation order is the written one)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_placement.restype = ctypes.c_int
        _lib.oracle_assemble.restype = ctypes.c_int
        _lib.oracle_assemble_ex.restype = ctypes.c_int
        _lib.oracle_e4m3_decode.restype = None
        _lib.oracle_e4m3_encode.restype = None
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_rope_rotate.restype = None
        _lib.oracle_attention_rows.restype = None
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _opt(w, name):
    v = getattr(w, name, None)
    return None if v is None else _i32(v)


def bits(t) -> np.ndarray:
    """bf16 torch tensor (any device) -> contiguous uint16 numpy array of its bits."""
    import torch
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def placement(w):
    """Block table and per-position sources of a workload.  Returns
    (status, page_off[batch+1], pages, src_slot[sum T], fresh_idx[sum T])."""
    batch = w.batch
    B = w.shape.page_size
    n_pages = int(sum(-(-int(t) // B) for t in w.seq_len))
    page_off = np.zeros(batch + 1, np.int32)
    pages = np.full(max(n_pages, 1), -1, np.int32)
    total = int(w.seq_len.sum())
    src_slot = np.full(max(total, 1), -7, np.int32)
    fresh = np.full(max(total, 1), -7, np.int32)
    st = lib().oracle_placement(
        ctypes.c_int(batch), _p(_i32(w.seq_len)), _p(_i32(w.unit_off)), _p(_i32(w.unit_len)),
        _p(_i32(w.unit_target_pos)), _p(_i32(w.unit_page_off)), _p(_i32(w.unit_pages)),
        _p(_i32(w.recompute_off)), _p(_i32(w.recompute_pos)), _p(_i32(w.free_pages)),
        ctypes.c_int(len(w.free_pages)), ctypes.c_int(B), _p(_opt(w, "unit_src_offset")),
        _p(page_off), _p(pages), _p(src_slot), _p(fresh))
    return st, page_off, pages[:n_pages], src_slot[:total], fresh[:total]


def rope_rotate(x: np.ndarray, delta: float, theta: float, inv_freq: Optional[np.ndarray] = None,
                pairing: int = 0) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty_like(x)
    if inv_freq is not None:
        inv_freq = np.ascontiguousarray(inv_freq, dtype=np.float64)
    lib().oracle_rope_rotate(_p(x), _p(out), ctypes.c_int(x.shape[-1]), ctypes.c_double(delta),
                             ctypes.c_double(theta), _p(inv_freq), ctypes.c_int(pairing))
    return out


class Assembled:
    """Assembled KV of one request: k (fp64, unrounded), v_bits, and for rows that
    are bit copies (recomputed rows, delta == 0) k_bits with k_exact set."""
    def __init__(self, T, H_kv, D):
        self.k = np.zeros((T, H_kv, D), np.float64)
        self.v_bits = np.zeros((T, H_kv, D), np.uint16)
        self.k_bits = np.zeros((T, H_kv, D), np.uint16)
        self.k_exact = np.zeros(T, np.uint8)
        self.delta = np.zeros(T, np.int32)


def e4m3_decode(codes: np.ndarray) -> np.ndarray:
    """uint8 e4m3 codes -> float64 values (NaN for the NaN code)."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    out = np.empty(codes.shape, np.float64)
    lib().oracle_e4m3_decode(_p(codes), _p(out), ctypes.c_long(codes.size))
    return out


def f64_to_bf16_bits(values: np.ndarray) -> np.ndarray:
    """float64 values -> bf16 bit patterns, one round-to-nearest-even of the exact value."""
    values = np.ascontiguousarray(values, dtype=np.float64)
    out = np.empty(values.shape, np.uint16)
    fn = lib().oracle_f64_to_bf16_rne
    fn.restype = ctypes.c_uint16
    fn.argtypes = [ctypes.c_double]
    flat, o = values.ravel(), out.ravel()
    for i in range(flat.size):
        o[i] = fn(float(flat[i]))
    return out


def e4m3_encode(values: np.ndarray) -> np.ndarray:
    """float32 values -> uint8 e4m3 codes: nearest, ties to even, saturating at +-448."""
    values = np.ascontiguousarray(values, dtype=np.float32)
    out = np.empty(values.shape, np.uint8)
    lib().oracle_e4m3_encode(_p(values), _p(out), ctypes.c_long(values.size))
    return out


def assemble(w, r: int, k_pool_bits, v_pool_bits, k_new_bits, v_new_bits,
             inv_freq: Optional[np.ndarray] = None, src_fmt: int = 0, k_scale: float = 1.0,
             v_scale: float = 1.0, fresh_k_raw: bool = False) -> Assembled:
    """src_fmt 0: 16-bit source pools given as bf16 bits; 1: 8-bit (e4m3 codes, uint8) source pools,
    a code standing for code * scale.  fresh_k_raw: k_new holds un-rotated keys, which the request sees
    rotated for their positions."""
    sh = w.shape
    T = int(w.seq_len[r])
    a = Assembled(T, sh.num_kv_heads, sh.head_dim)
    if inv_freq is not None:
        inv_freq = np.ascontiguousarray(inv_freq, dtype=np.float64)
    st = lib().oracle_assemble_ex(
        ctypes.c_int(r), _p(_i32(w.seq_len)), _p(_i32(w.unit_off)), _p(_i32(w.unit_len)),
        _p(_i32(w.unit_cached_pos)), _p(_i32(w.unit_cached_stride)), _p(_i32(w.unit_target_pos)),
        _p(_i32(w.unit_page_off)), _p(_i32(w.unit_pages)), _p(_i32(w.recompute_off)),
        _p(_i32(w.recompute_pos)), ctypes.c_int(sh.page_size), ctypes.c_int(sh.num_kv_heads),
        ctypes.c_int(sh.head_dim), ctypes.c_double(sh.rope_theta), _p(inv_freq),
        ctypes.c_int(sh.rope_pairing),
        _p(k_pool_bits), _p(v_pool_bits), _p(k_new_bits), _p(v_new_bits),
        _p(_opt(w, "unit_src_offset")), _p(_opt(w, "unit_target_stride")),
        ctypes.c_int(src_fmt), ctypes.c_float(k_scale), ctypes.c_float(v_scale), ctypes.c_int(int(fresh_k_raw)),
        _p(a.k), _p(a.v_bits), _p(a.k_bits), _p(a.k_exact), _p(a.delta))
    if st != 0:
        raise ValueError("oracle_assemble: request %d has positions nobody supplies" % r)
    return a


def attention_rows(w, k_asm: np.ndarray, v_bits: np.ndarray, q_bits: np.ndarray,
                   row_q: Sequence[int], row_h: Sequence[int], row_pos: Sequence[int],
                   scale: Optional[float] = None):
    """O [n_rows, D] (fp64) and LSE [n_rows] for the listed (query token, head) rows
    of ONE request whose assembled K (fp64) / V (bits) are given.  q_bits: bf16 bits (uint16), or the
    queries themselves as float64 (values that are not bf16 numbers)."""
    sh = w.shape
    if scale is None:
        scale = sh.sm_scale if sh.sm_scale else 1.0 / np.sqrt(sh.head_dim)
    row_q, row_h, row_pos = _i32(row_q), _i32(row_h), _i32(row_pos)
    n = len(row_q)
    out = np.zeros((n, sh.head_dim), np.float64)
    lse = np.zeros(n, np.float64)
    k_asm = np.ascontiguousarray(k_asm, dtype=np.float64)
    v_bits = np.ascontiguousarray(v_bits, dtype=np.uint16)
    if q_bits.dtype == np.float64:
        fn, q_arg = lib().oracle_attention_rows_qf64, np.ascontiguousarray(q_bits)
        fn.restype = None
    else:
        fn, q_arg = lib().oracle_attention_rows, q_bits
    fn(ctypes.c_int(k_asm.shape[0]), ctypes.c_int(sh.num_q_heads), ctypes.c_int(sh.num_kv_heads),
       ctypes.c_int(sh.head_dim), ctypes.c_double(scale), _p(k_asm), _p(v_bits), _p(q_arg),
       ctypes.c_int(n), _p(row_q), _p(row_h), _p(row_pos), _p(out), _p(lse))
    return out, lse


def request_rows(w, r: int):
    """All (query token, head) rows of request r as (row_q, row_h, row_pos)."""
    j0, j1 = int(w.recompute_off[r]), int(w.recompute_off[r + 1])
    H = w.shape.num_q_heads
    jj = np.repeat(np.arange(j0, j1, dtype=np.int32), H)
    hh = np.tile(np.arange(H, dtype=np.int32), j1 - j0)
    pp = np.repeat(w.recompute_pos[j0:j1].astype(np.int32), H)
    return jj, hh, pp


def full_layer(w, k_pool_bits, v_pool_bits, q_bits, k_new_bits, v_new_bits, inv_freq=None):
    """Whole hot path of one layer through the oracle: per request the assembled
    KV, and O [n_q, H_q, D] / LSE [n_q, H_q] for every recompute row."""
    sh = w.shape
    out = np.zeros((w.n_q, sh.num_q_heads, sh.head_dim), np.float64)
    lse = np.zeros((w.n_q, sh.num_q_heads), np.float64)
    asm = []
    for r in range(w.batch):
        a = assemble(w, r, k_pool_bits, v_pool_bits, k_new_bits, v_new_bits, inv_freq)
        asm.append(a)
        jj, hh, pp = request_rows(w, r)
        if len(jj):
            o, l = attention_rows(w, a.k, a.v_bits, q_bits, jj, hh, pp)
            out[jj, hh] = o
            lse[jj, hh] = l
    return asm, out, lse
