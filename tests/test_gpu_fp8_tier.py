"""GPU parity of the 8-bit (e4m3) storage tier: expanding an 8-bit source pool into a request's 16-bit
pages and retaining 16-bit pages as 8-bit units, against the oracle's codec and assembly."""
import copy
import dataclasses

import numpy as np
import pytest
import torch

from oracle import tessera_oracle as orc
from paper_2609_32999_b200 import binding as tb
from paper_2609_32999_b200 import workloads as wl
from tests import gpu_util as gu
from tests.test_gpu_parity import _retention_workloads

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
NAN8 = 0x7f                      # e4m3 NaN: the poison of 8-bit pools (no kernel produces it from finite data)


def _codes_of(pool_bf16, scale):
    """Host-side input generation: the e4m3 codes nearest to pool / scale."""
    x = pool_bf16.float().cpu().numpy() / np.float32(scale)
    return orc.e4m3_encode(x.astype(np.float32))


def _to_dev(codes):
    return torch.from_numpy(codes).to(DEV)


@pytest.mark.parametrize("fuse,pinned,scales", [(True, False, (1 / 64, 1 / 32)), (True, False, (0.013, 0.021)),
                                                (False, False, (1 / 64, 1 / 32)), (True, True, (0.013, 0.021))])
def test_expand_8bit_source_pool(fuse, pinned, scales):
    ks, vs = scales
    w = wl.config(3, requests_override=4)
    t = wl.make_tensors(w, device=DEV, seed=21)
    k8, v8 = _codes_of(t.k_pool, ks), _codes_of(t.v_pool, vs)
    assert not np.any((k8 & 0x7f) == NAN8)
    w2 = copy.copy(w)
    w2.num_source_pages = w.num_pool_pages
    plan = tb.Plan(w2)
    pv = torch.tensor(gu.POISON, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    t.k_pool[:] = pv
    t.v_pool[:] = pv
    k8_t, v8_t = torch.from_numpy(k8), torch.from_numpy(v8)
    k8_t, v8_t = (k8_t.pin_memory(), v8_t.pin_memory()) if pinned else (k8_t.to(DEV), v8_t.to(DEV))
    plan.kv_compose_from_fp8(k8_t, v8_t, ks, vs, t.k_pool, t.v_pool, fuse_rope=fuse)
    if not fuse:
        plan.rope_shift(t.k_pool)
    torch.cuda.synchronize()
    g = gu.LayerRun()
    g.w, g.t, g.plan = w, t, plan
    g.page_off, g.pages, g.src_slot = plan.block_table()
    if fuse:
        g.k_before, g.v_before, g.src_fmt, g.k_scale, g.v_scale = k8, v8, 1, ks, vs
    else:
        # without the fused rotation the call is "expand, then shift in place": the 16-bit value
        # c * scale exists in the page before it is rotated (exactly, the scales being powers of two
        # here), so the reference is the 16-bit path applied to a pool of exactly those values
        def as16(c8, sc):
            exact = orc.e4m3_decode(c8) * float(np.float32(sc))
            b16 = torch.from_numpy(exact).to(torch.bfloat16)
            assert np.array_equal(b16.double().numpy(), exact)
            return orc.bits(b16)
        g.k_before, g.v_before = as16(k8, ks), as16(v8, vs)
    g.k_after, g.v_after = orc.bits(t.k_pool), orc.bits(t.v_pool)
    g.kn_bits, g.vn_bits = orc.bits(t.k_new), orc.bits(t.v_new)
    gu.check_placement(g)
    asm, kmx, kmean = gu.check_assembled(g, scattered=False)
    assert kmx > 0                                              # rotated keys were compared
    if fuse:
        n_diff, n_all = g.double_rounding
        print("8-bit expansion, scales %r: %d of %d expanded elements differ from the single-rounding "
              "definition (one bf16 step each)" % (scales, n_diff, n_all))
        assert n_all > 0 and (n_diff == 0 or not gu._is_pow2(ks))
    mask = np.ones(w.num_pool_pages, bool)
    mask[g.pages] = False
    assert np.all(g.k_after[mask] == gu.POISON) and np.all(g.v_after[mask] == gu.POISON)
    # the attention path on top of the expanded pages
    out = torch.empty_like(t.q)
    lse = torch.zeros(w.n_q, w.shape.num_q_heads, dtype=torch.float32, device=DEV)
    plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, lse)
    torch.cuda.synchronize()
    assert plan.status() == 0
    g.k_after, g.v_after = orc.bits(t.k_pool), orc.bits(t.v_pool)
    g.q_bits, g.out_f, g.lse_f = orc.bits(t.q), out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    asm, _, _ = gu.check_assembled(g)
    gu.check_attention(g, asm)


def _half_spacing(y):
    """Half the distance between the two e4m3 values that bracket |y| (|y| < 448)."""
    table = orc.e4m3_decode(np.arange(0x7f, dtype=np.uint8))
    hi = np.searchsorted(table, np.abs(y), side="right")
    return (table[np.minimum(hi, 0x7e)] - table[hi - 1]) / 2


def test_retain_as_8bit_unit_then_reuse_it():
    """A freshly computed unit leaves a finished request's 16-bit pages as an 8-bit, position-free cache
    entry and is reused in another prompt.  Every stage starts from data the oracle (or the seeded
    generator) made on the host."""
    ks, vs = 1 / 32, 0.019
    A, R, B = _retention_workloads()
    tA = wl.make_tensors(A, device=DEV, seed=31)
    kA, vA, _ = gu.host_assembled_pools(A, tA)                 # the request's pages as the oracle leaves them
    R2, B2 = copy.copy(R), copy.copy(B)
    R2.num_source_pages = B2.num_source_pages = A.num_pool_pages
    planR = tb.Plan(R2)
    shape8 = tuple(tA.k_pool.shape)
    k8 = torch.full(shape8, NAN8, dtype=torch.uint8, device=DEV)
    v8 = torch.full(shape8, NAN8, dtype=torch.uint8, device=DEV)
    planR.kv_retain_fp8(kA, vA, k8, v8, ks, vs)
    torch.cuda.synchronize()
    page_off, pages, _ = planR.block_table()
    st, o_off, o_pages, _, _ = orc.placement(R)
    assert st == 0 and np.array_equal(pages, o_pages)
    k8_h, v8_h = k8.cpu().numpy(), v8.cpu().numpy()
    mask = np.ones(A.num_pool_pages, bool)
    mask[pages] = False
    assert np.all(k8_h[mask] == NAN8) and np.all(v8_h[mask] == NAN8)      # only destination pages were written
    a = orc.assemble(R, 0, orc.bits(kA), orc.bits(vA), orc.bits(tA.k_new), orc.bits(tA.v_new))
    T, Bp = int(R.seq_len[0]), R.shape.page_size
    row = R.shape.num_kv_heads * R.shape.head_dim
    p = np.arange(T)
    slots = pages[p // Bp].astype(np.int64) * Bp + p % Bp
    inv_k, inv_v = np.float32(1) / np.float32(ks), np.float32(1) / np.float32(vs)
    # V: the decision is taken on the fp32 product, on both sides -> identical codes
    v_want = orc.e4m3_encode(orc.bf16_bits_to_f64(a.v_bits).astype(np.float32).reshape(T, row) * inv_v)
    assert np.array_equal(v8_h.reshape(-1, row)[slots], v_want)
    # K: rotated in fp32 on the GPU, in fp64 by the oracle -> the stored value is the nearest code of the
    # oracle's value up to the fp32 rotation error (1e-5 relative)
    y = a.k.reshape(T, row) * float(inv_k)
    got = orc.e4m3_decode(k8_h.reshape(-1, row)[slots])
    assert np.isfinite(got).all() and np.abs(y).max() < 448
    slack = np.abs(got - y) - _half_spacing(y)
    assert slack.max() <= 1e-5 * np.abs(y).max() + 1e-7
    k_want = orc.e4m3_encode(y.astype(np.float32))
    assert np.mean(k8_h.reshape(-1, row)[slots] != k_want) < 2e-3       # differences only at near-ties
    # reuse: an 8-bit pool made on the host - every cached row quantised by the oracle's codec, the
    # retained unit as the oracle retains it - expanded into another prompt and attended over
    k8_img = _codes_of(tA.k_pool, ks).reshape(-1, row)
    v8_img = _codes_of(tA.v_pool, vs).reshape(-1, row)
    k8_img[slots], v8_img[slots] = k_want, v_want
    k8_img, v8_img = k8_img.reshape(shape8), v8_img.reshape(shape8)
    planB = tb.Plan(B2)
    pv = torch.tensor(gu.POISON, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    tB = dataclasses.replace(tA, k_pool=torch.full_like(tA.k_pool, 0), v_pool=torch.full_like(tA.v_pool, 0))
    tB.k_pool[:] = pv
    tB.v_pool[:] = pv
    planB.kv_compose_from_fp8(_to_dev(k8_img), _to_dev(v8_img), ks, vs, tB.k_pool, tB.v_pool)
    out = torch.zeros(B.n_q, B.shape.num_q_heads, B.shape.head_dim, dtype=torch.bfloat16, device=DEV)
    planB.partial_prefill_attn(tB.k_pool, tB.v_pool, tB.q, tB.k_new, tB.v_new, out, None)
    torch.cuda.synchronize()
    assert planB.status() == 0
    g = gu.LayerRun()
    g.w, g.t, g.plan = B, tB, planB
    g.page_off, g.pages, g.src_slot = planB.block_table()
    g.k_before, g.v_before, g.src_fmt, g.k_scale, g.v_scale = k8_img, v8_img, 1, ks, vs
    g.k_after, g.v_after = orc.bits(tB.k_pool), orc.bits(tB.v_pool)
    g.kn_bits, g.vn_bits, g.q_bits = orc.bits(tB.k_new), orc.bits(tB.v_new), orc.bits(tB.q)
    g.out_f, g.lse_f = out.float().cpu().numpy().astype(np.float64), None
    gu.check_placement(g)
    asm, _, _ = gu.check_assembled(g)
    gu.check_attention(g, asm)


def test_8bit_calls_reject_bad_arguments():
    w = wl.config(1)
    t = wl.make_tensors(w, device=DEV, seed=2)
    k8 = torch.zeros(tuple(t.k_pool.shape), dtype=torch.uint8, device=DEV)
    with pytest.raises(tb.TesseraError):                      # plan without a separate source pool
        tb.Plan(w).kv_compose_from_fp8(k8, k8, 1.0, 1.0, t.k_pool, t.v_pool)
    w2 = copy.copy(w)
    w2.num_source_pages = w.num_pool_pages
    plan = tb.Plan(w2)
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(tb.TesseraError):
            plan.kv_compose_from_fp8(k8, k8, bad, 1.0, t.k_pool, t.v_pool)
        with pytest.raises(tb.TesseraError):
            plan.kv_retain_fp8(t.k_pool, t.v_pool, k8, k8, 1.0, bad)


def test_saturation_and_special_values_when_retaining():
    """Values beyond +-448 * scale saturate, NaN becomes the NaN code, zeros keep their sign."""
    shape = wl.ModelShape(8, 2, 64, 16, 10000.0)
    rng = np.random.default_rng(4)
    w = wl.build_workload("sat", shape, [[wl.unit(40, "a")]], rng)
    t = wl.make_tensors(w, device=DEV, seed=9)
    special = torch.tensor([1e6, -1e6, 448.0, 449.0, 0.0, -0.0, float("nan"), float("inf"), -float("inf"), 2.0 ** -9, 2.0 ** -10, 3 * 2.0 ** -11],
                           dtype=torch.float32, device=DEV).to(torch.bfloat16)
    src_page = int(w.unit_pages[0])
    t.v_pool[src_page, 0, 0, :special.numel()] = special
    t.k_pool[src_page, 0, 0, :special.numel()] = special
    w2 = copy.copy(w)
    w2.num_source_pages = w.num_pool_pages
    # no rotation requested: K goes through the same scale-and-round as V
    plan = tb.Plan(w2)
    k8 = torch.full(tuple(t.k_pool.shape), NAN8, dtype=torch.uint8, device=DEV)
    v8 = torch.full(tuple(t.k_pool.shape), NAN8, dtype=torch.uint8, device=DEV)
    plan.kv_retain_fp8(t.k_pool, t.v_pool, k8, v8, 1.0, 1.0, fuse_rope=False)
    torch.cuda.synchronize()
    _, pages, _ = plan.block_table()
    got_v = v8[int(pages[0]), int(w.unit_target_pos[0]), 0, :special.numel()].cpu().numpy()
    got_k = k8[int(pages[0]), int(w.unit_target_pos[0]), 0, :special.numel()].cpu().numpy()
    want = orc.e4m3_encode(special.float().cpu().numpy())
    assert np.array_equal(got_v, want) and np.array_equal(got_k, want)
    assert want.tolist()[:9] == [0x7e, 0xfe, 0x7e, 0x7e, 0x00, 0x80, 0x7f, 0x7e, 0xfe]
