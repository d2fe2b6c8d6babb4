"""CPU-only checks of the library boundary: exported symbols, host placement vs the oracle,
and every validation error, none of which launches a kernel."""
import copy
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import tessera_oracle as orc
from paper_2609_32999_b200 import binding as tb
from paper_2609_32999_b200 import workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "tessera.h")).read()
    declared = re.findall(r"TESSERA_API\s+\w+\s+(tessera_\w+)\s*\(", hdr)
    assert len(declared) >= 11 and set(declared) == set(tb.EXPORTS)
    lib = ctypes.CDLL(tb.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


@pytest.mark.parametrize("make", [lambda: wl.config(1), lambda: wl.config(2), lambda: wl.adversarial(),
                                  lambda: wl.config(3), lambda: wl.config(5, requests_override=4)])
def test_host_placement_matches_oracle(make):
    w = make()
    plan = tb.Plan(w, host_only=True)
    page_off, pages, src_slot = plan.block_table()
    st, o_off, o_pages, o_src, _ = orc.placement(w)
    assert st == 0
    assert np.array_equal(page_off, o_off)
    assert np.array_equal(pages, o_pages)
    assert np.array_equal(src_slot, o_src)
    assert plan.info.total_tokens == w.total_tokens and plan.info.n_q == w.n_q
    assert plan.info.cached_tokens == w.cached_tokens and plan.info.qk_pairs == w.qk_pairs
    assert plan.info.gather_bytes == wl.gather_bytes(w) and plan.info.attn_flops == wl.attention_flops(w)
    plan.destroy()


def test_host_only_plan_refuses_device_calls():
    plan = tb.Plan(wl.config(1), host_only=True)
    with pytest.raises(tb.TesseraError) as e:
        plan.kv_compose(None, None, stream=0)
    assert e.value.status == tb.INVALID_ARG and "HOST_ONLY" in str(e.value)
    for call in (lambda: plan.kv_compose_from_fp8(None, None, 1.0, 1.0, None, None, stream=0),
                 lambda: plan.kv_retain_fp8(None, None, None, None, 1.0, 1.0, stream=0),
                 lambda: plan.kv_compose_from(None, None, None, None, stream=0),
                 lambda: plan.rope_shift(None, stream=0),
                 lambda: plan.rope_fresh(None, None, stream=0),
                 lambda: plan.extend_write(None, None, None, None, None, stream=0),
                 lambda: plan.kv_compose_k8(None, None, None, None, 1.0, stream=0),
                 lambda: plan.partial_prefill_attn_k8(None, 1.0, None, None, 1.0, None, None, None, stream=0),
                 lambda: plan.composed_prefill_host_tier(None, None, None, None, None, None, None, None, stream=0),
                 lambda: plan.composed_prefill_host(None, None, None, None, None, None, stream=0),
                 lambda: plan.partial_prefill_attn(None, None, None, None, None, None, None, stream=0)):
        with pytest.raises(tb.TesseraError) as e:
            call()
        assert e.value.status == tb.INVALID_ARG


def _base():
    shape = wl.ModelShape(4, 2, 64, 16, 1e4)
    return wl.build_workload("v", shape, [[4, wl.unit(40, "a", recompute=(0, 1)), wl.unit(20, "b"), 2],
                                          [wl.unit(20, "b", recompute=(0,)), 3]],
                             np.random.default_rng(0))


def _mut(**kw):
    w = copy.deepcopy(_base())
    for k, v in kw.items():
        setattr(w, k, np.asarray(v, dtype=np.int32) if not isinstance(v, (int, wl.ModelShape)) else v)
    return w


def test_validation_errors():
    w = _base()
    assert tb.plan_create_status(w) == tb.OK
    assert orc.placement(w)[0] == 0
    # recompute positions out of order
    rp = w.recompute_pos.copy(); rp[0], rp[1] = rp[1], rp[0]
    assert tb.plan_create_status(_mut(recompute_pos=rp)) == tb.UNSORTED_POSITIONS
    # a position nobody supplies: drop the first recompute row (position 0 of request 0)
    assert tb.plan_create_status(_mut(recompute_pos=w.recompute_pos[1:],
                                      recompute_off=w.recompute_off - np.array([0, 1, 1]))) == tb.UNCOVERED_POSITION
    # two units on one position
    tp = w.unit_target_pos.copy(); tp[1] -= 5
    assert tb.plan_create_status(_mut(unit_target_pos=tp)) == tb.UNIT_OVERLAP
    # unit leaves the request
    tp = w.unit_target_pos.copy(); tp[1] += 100
    assert tb.plan_create_status(_mut(unit_target_pos=tp)) == tb.UNIT_OVERLAP
    # page ids
    up = w.unit_pages.copy(); up[0] = w.num_pool_pages
    assert tb.plan_create_status(_mut(unit_pages=up)) == tb.PAGE_OUT_OF_RANGE
    fp = w.free_pages.copy(); fp[0] = w.unit_pages[0]
    assert tb.plan_create_status(_mut(free_pages=fp)) == tb.PAGE_OUT_OF_RANGE
    fp = w.free_pages.copy(); fp[1] = fp[0]
    assert tb.plan_create_status(_mut(free_pages=fp)) == tb.PAGE_OUT_OF_RANGE
    assert tb.plan_create_status(_mut(free_pages=w.free_pages[:2])) == tb.OUT_OF_PAGES
    # malformed descriptor
    assert tb.plan_create_status(_mut(unit_page_off=w.unit_page_off[::-1].copy())) == tb.INVALID_ARG
    st = w.unit_cached_stride.copy(); st[0] = 2
    assert tb.plan_create_status(_mut(unit_cached_stride=st)) == tb.INVALID_ARG
    # shapes
    for bad in (wl.ModelShape(4, 3, 64, 16, 1e4), wl.ModelShape(4, 2, 96, 16, 1e4), wl.ModelShape(4, 2, 64, 12, 1e4),
                wl.ModelShape(4, 2, 64, 16, 1e4, rope_pairing=2), wl.ModelShape(64, 2, 64, 16, 1e4)):
        assert tb.plan_create_status(_mut(shape=bad)) == tb.UNSUPPORTED_SHAPE
    assert "page" in tb.last_error() or "head" in tb.last_error() or "group" in tb.last_error()


def test_empty_batch_and_empty_request():
    shape = wl.ModelShape(4, 2, 64, 16, 1e4)
    w = wl.build_workload("empty", shape, [], np.random.default_rng(0))
    plan = tb.Plan(w, host_only=True)
    assert plan.info.total_tokens == 0 and plan.info.n_q == 0
    w = wl.build_workload("one-empty", shape, [[], [3]], np.random.default_rng(0))
    plan = tb.Plan(w, host_only=True)
    page_off, pages, src = plan.block_table()
    assert list(page_off) == [0, 0, 1] and list(src) == [-1, -1, -1]


def test_source_offset_and_target_stride_in_host_plan():
    """Units read from the middle of a page (retention) and written without rotation."""
    shape = wl.ModelShape(4, 2, 64, 16, 1e4)
    i32 = lambda x: np.asarray(x, np.int32)
    w = wl.Workload(name="retain", shape=shape, seq_len=i32([40]), unit_off=i32([0, 1]), unit_len=i32([40]),
                    unit_cached_pos=i32([21]), unit_cached_stride=i32([1]), unit_target_pos=i32([0]),
                    unit_page_off=i32([0, 3]), unit_pages=i32([7, 3, 9]), recompute_off=i32([0, 0]),
                    recompute_pos=i32([]), free_pages=i32([12, 11, 10]), num_pool_pages=16,
                    unit_src_offset=i32([5]), unit_target_stride=i32([0]))
    plan = tb.Plan(w, host_only=True)
    page_off, pages, src = plan.block_table()
    st, o_off, o_pages, o_src, _ = orc.placement(w)
    assert st == 0 and np.array_equal(src, o_src) and np.array_equal(pages, o_pages)
    want = [[7, 3, 9][(5 + i) // 16] * 16 + (5 + i) % 16 for i in range(40)]
    assert src.tolist() == want
    assert plan.info.n_rope_rows == 40                      # one shift per token: -(21 + i)
    # un-rotated form in the oracle: delta = -(cached_pos + i)
    t = wl.make_tensors(w)
    a = orc.assemble(w, 0, orc.bits(t.k_pool), orc.bits(t.v_pool), orc.bits(t.k_new), orc.bits(t.v_new))
    assert a.delta.tolist() == [-(21 + i) for i in range(40)]
    # wrong page count for the offset, bad offset, bad stride
    ok = copy.deepcopy(w); ok.unit_src_offset = i32([0])                    # 40 tokens from 0 also span 3 pages
    assert tb.plan_create_status(ok) == tb.OK
    bad = copy.deepcopy(w); bad.unit_src_offset = i32([12])                 # 12 + 40 = 52 tokens need 4 pages, 3 given
    assert tb.plan_create_status(bad) == tb.INVALID_ARG
    bad = copy.deepcopy(w); bad.unit_src_offset = i32([16])
    assert tb.plan_create_status(bad) == tb.INVALID_ARG
    bad = copy.deepcopy(w); bad.unit_target_stride = i32([2])
    assert tb.plan_create_status(bad) == tb.INVALID_ARG


def test_capture_descriptor_validation_and_row_count():
    """Units marked for capture by tessera_extend_write: page count, full recomputation, page clashes."""
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    i32 = lambda x: np.asarray(x, np.int32)
    w0 = wl.build_workload("cap", shape, [[wl.unit(100, "a", recompute=(0, 1)), wl.unit(70, "b", cached=False), 3]],
                           np.random.default_rng(1), spare_pages=8)
    used = -(-int(w0.seq_len[0]) // 64)
    spare = w0.free_pages[used:].tolist()

    def with_capture(off, pages, pool=0):
        w = copy.copy(w0)
        w.unit_retain_page_off, w.unit_retain_pages, w.retain_pool_pages = i32(off), i32(pages), pool
        return w

    ok = with_capture([0, 0, 2], spare[:2])
    plan = tb.Plan(ok, host_only=True)
    assert plan.info.retained_tokens == 70
    assert tb.plan_create_status(with_capture([0, 0, 2], [0, 1], pool=2)) == tb.OK                 # separate cache pool
    assert tb.plan_create_status(with_capture([0, 2, 2], spare[:2])) == tb.INVALID_ARG             # unit a is not fully recomputed
    assert tb.plan_create_status(with_capture([0, 0, 1], spare[:1])) == tb.INVALID_ARG             # 70 tokens need 2 pages
    assert tb.plan_create_status(with_capture([0, 0, 2], [int(w0.unit_pages[0]), spare[0]])) == tb.PAGE_OUT_OF_RANGE   # a source page
    assert tb.plan_create_status(with_capture([0, 0, 2], [int(w0.free_pages[0]), spare[0]])) == tb.PAGE_OUT_OF_RANGE   # a destination page
    assert tb.plan_create_status(with_capture([0, 0, 2], [spare[0], spare[0]])) == tb.PAGE_OUT_OF_RANGE                # listed twice
    assert tb.plan_create_status(with_capture([0, 0, 2], [0, 2], pool=2)) == tb.PAGE_OUT_OF_RANGE                      # outside the cache pool


def test_llama31_scaled_frequencies_match_the_library_rule():
    """The helper's table against the model library's own Llama-3 frequency initialisation."""
    import torch
    from transformers import LlamaConfig
    from transformers.modeling_rope_utils import ROPE_INIT_FUNCTIONS
    from paper_2609_32999_b200 import rope_scaling as rs
    scaling = {"rope_type": "llama3", "factor": 8.0, "low_freq_factor": 1.0, "high_freq_factor": 4.0,
               "original_max_position_embeddings": 8192, "rope_theta": 500000.0}
    try:
        cfg = LlamaConfig(hidden_size=4096, num_attention_heads=32, rope_theta=500000.0, max_position_embeddings=131072,
                          rope_scaling=dict(scaling))
    except TypeError:
        cfg = LlamaConfig(hidden_size=4096, num_attention_heads=32, max_position_embeddings=131072, rope_parameters=dict(scaling))
    want, _ = ROPE_INIT_FUNCTIONS["llama3"](cfg, "cpu")
    got = rs.llama31_inv_freq(128, 500000.0)
    assert np.allclose(got, want.double().numpy(), rtol=1e-6)
    plain = rs.default_inv_freq(128, 500000.0)
    assert np.array_equal(got[:20], plain[:20]) and np.allclose(got[-10:], plain[-10:] / 8.0)      # fast pairs kept, slow pairs 8x slower
    # and a plan takes the table
    w = wl.config(2)
    assert tb.Plan(w, host_only=True, inv_freq=got).info.n_rope_rows == 10
