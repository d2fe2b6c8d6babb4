"""Overlapped host tier: cached units in a pinned host pool, pulled over the link chunk by chunk by a
small reader launch while attention of the chunks already there runs.  The result must be the bits of
the unoverlapped path, and the oracle's within tolerance."""
import copy

import numpy as np
import pytest
import torch

from oracle import tessera_oracle as orc
from paper_2609_32999_b200 import binding as tb
from paper_2609_32999_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _host_tier_plan(w):
    w2 = copy.copy(w)
    w2.num_source_pages = w.num_pool_pages
    return tb.Plan(w2)


def _poisoned_like(t):
    pv = torch.tensor(gu.POISON, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    k, v = torch.empty_like(t.k_pool), torch.empty_like(t.v_pool)
    k[:] = pv
    v[:] = pv
    return k, v


def _same_bits(a, b):
    """torch.equal on the raw bits (the poison pattern is a NaN, which never compares equal as a number)."""
    return torch.equal(a.view(torch.int16), b.view(torch.int16))


@pytest.mark.parametrize("make,readers", [(lambda: wl.config(3, requests_override=6), 0),
                                          (lambda: wl.config(3, requests_override=6), 3),
                                          (lambda: wl.config(2), 0),                           # one request, split-KV attention
                                          (lambda: wl.adversarial(seed=9, shape=wl.ModelShape(32, 8, 128, 64, 500000.0)), 1),
                                          (lambda: wl.config(1), 0)])
def test_overlapped_host_tier_matches_plain_path_and_oracle(make, readers):
    w = make()
    t = wl.make_tensors(w, device=DEV, seed=12)
    host_k, host_v = t.k_pool.cpu().pin_memory(), t.v_pool.cpu().pin_memory()
    plan = _host_tier_plan(w)
    sh = w.shape
    # reference: the zero-copy gather + one attention call on separate, poisoned pools
    k_ref, v_ref = _poisoned_like(t)
    out_ref = torch.zeros(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=DEV)
    lse_ref = torch.zeros(w.n_q, sh.num_q_heads, dtype=torch.float32, device=DEV)
    plan.kv_compose_from(host_k, host_v, k_ref, v_ref)
    plan.partial_prefill_attn(k_ref, v_ref, t.q, t.k_new, t.v_new, out_ref, lse_ref)
    # overlapped path, twice in a row (the second call queues behind the first on both streams)
    k_st, v_st = _poisoned_like(t)
    out = torch.zeros_like(out_ref)
    lse = torch.zeros_like(lse_ref)
    for _ in range(2):
        plan.composed_prefill_host_tier(host_k, host_v, k_st, v_st, t.q, t.k_new, t.v_new, out, lse, reader_blocks=readers)
    torch.cuda.synchronize()
    assert plan.status() == 0
    assert _same_bits(k_st, k_ref) and _same_bits(v_st, v_ref)
    assert torch.equal(out, out_ref) and torch.equal(lse, lse_ref)
    # and against the oracle, like every other path
    g = gu.LayerRun()
    g.w, g.t, g.plan = w, t, plan
    g.page_off, g.pages, g.src_slot = plan.block_table()
    g.k_before, g.v_before = orc.bits(host_k), orc.bits(host_v)
    g.k_after, g.v_after = orc.bits(k_st), orc.bits(v_st)
    g.kn_bits, g.vn_bits, g.q_bits = orc.bits(t.k_new), orc.bits(t.v_new), orc.bits(t.q)
    g.out_f, g.lse_f = out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    gu.check_placement(g)
    asm, _, _ = gu.check_assembled(g)
    gu.check_attention(g, asm)
    mask = np.ones(w.num_pool_pages, bool)
    mask[g.pages] = False
    assert np.all(g.k_after[mask] == gu.POISON) and np.all(g.v_after[mask] == gu.POISON)


def test_overlapped_host_tier_with_8bit_units():
    """e4m3 units in the host pool: half the bytes over the link, expanded by the 8-bit gather kernel."""
    ks, vs = 1 / 64, 1 / 32
    w = wl.config(3, requests_override=5)
    t = wl.make_tensors(w, device=DEV, seed=21)
    k8 = orc.e4m3_encode((t.k_pool.float().cpu().numpy() / np.float32(ks)).astype(np.float32))
    v8 = orc.e4m3_encode((t.v_pool.float().cpu().numpy() / np.float32(vs)).astype(np.float32))
    host_k8, host_v8 = torch.from_numpy(k8).pin_memory(), torch.from_numpy(v8).pin_memory()
    plan = _host_tier_plan(w)
    sh = w.shape
    k_ref, v_ref = _poisoned_like(t)
    out_ref = torch.zeros(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=DEV)
    plan.kv_compose_from_fp8(host_k8, host_v8, ks, vs, k_ref, v_ref)
    plan.partial_prefill_attn(k_ref, v_ref, t.q, t.k_new, t.v_new, out_ref, None)
    k_st, v_st = _poisoned_like(t)
    out = torch.zeros_like(out_ref)
    plan.composed_prefill_host_tier(host_k8, host_v8, k_st, v_st, t.q, t.k_new, t.v_new, out, None,
                                    src_format=1, k_scale=ks, v_scale=vs)
    torch.cuda.synchronize()
    assert plan.status() == 0
    assert _same_bits(k_st, k_ref) and _same_bits(v_st, v_ref) and torch.equal(out, out_ref)
    g = gu.LayerRun()
    g.w, g.t, g.plan = w, t, plan
    g.page_off, g.pages, g.src_slot = plan.block_table()
    g.k_before, g.v_before, g.src_fmt, g.k_scale, g.v_scale = k8, v8, 1, ks, vs
    g.k_after, g.v_after = orc.bits(k_st), orc.bits(v_st)
    g.kn_bits, g.vn_bits, g.q_bits = orc.bits(t.k_new), orc.bits(t.v_new), orc.bits(t.q)
    g.out_f, g.lse_f = out.float().cpu().numpy().astype(np.float64), None
    asm, _, _ = gu.check_assembled(g)
    gu.check_attention(g, asm)


def test_overlapped_host_tier_rejects_bad_arguments():
    w = wl.config(1)
    t = wl.make_tensors(w, device=DEV, seed=2)
    hk, hv = t.k_pool.cpu().pin_memory(), t.v_pool.cpu().pin_memory()
    out = torch.zeros_like(t.q)
    with pytest.raises(tb.TesseraError):                      # plan without a separate source pool
        tb.Plan(w).composed_prefill_host_tier(hk, hv, t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out)
    plan = _host_tier_plan(w)
    with pytest.raises(tb.TesseraError):                      # more reader blocks than half the SMs
        plan.composed_prefill_host_tier(hk, hv, t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, reader_blocks=1000)
    with pytest.raises(tb.TesseraError):
        plan.composed_prefill_host_tier(hk, hv, t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, src_format=2)
    with pytest.raises(tb.TesseraError):
        plan.composed_prefill_host_tier(hk, hv, t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, src_format=1, k_scale=0.0)
