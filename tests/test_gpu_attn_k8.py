"""GPU parity of tessera_partial_prefill_attn_k8 (attention over 8-bit key pages).  The quantisation of
queries and keys is part of the method: the oracle attends, in fp64, over the DECODED operands (codes
times their scales), and the codes themselves are compared with the oracle's codec bit for bit."""
import copy
import dataclasses

import numpy as np
import pytest
import torch

from oracle import tessera_oracle as orc
from paper_2609_32999_b200 import binding as tb
from paper_2609_32999_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
NAN8 = 0x7f


def _host_made_pools(w, t, k_scale):
    """Pools as the oracle leaves them after gather + shift + scatter, with the assembled keys stored as
    e4m3 codes of (key / k_scale) by the oracle's codec.  Returns k_pool8 (device uint8), v_pool (device
    bf16) and {request: (decoded fp64 keys, v bits)}."""
    sh = w.shape
    row = sh.num_kv_heads * sh.head_dim
    kb, vb, knb, vnb = (orc.bits(x) for x in (t.k_pool, t.v_pool, t.k_new, t.v_new))
    st, page_off, pages, _, _ = orc.placement(w)
    assert st == 0
    k8 = np.full((w.num_pool_pages * sh.page_size, row), NAN8, np.uint8)
    v_img = vb.copy().reshape(-1, row)
    inv = np.float32(1) / np.float32(k_scale)
    stored = {}
    B = sh.page_size
    for r in range(w.batch):
        a = orc.assemble(w, r, kb, vb, knb, vnb)
        T = int(w.seq_len[r])
        if T == 0:
            continue
        p = np.arange(T)
        slots = pages[page_off[r] + p // B].astype(np.int64) * B + p % B
        codes = orc.e4m3_encode(a.k.reshape(T, row).astype(np.float32) * inv)
        k8[slots] = codes
        v_img[slots] = a.v_bits.reshape(T, row)
        stored[r] = ((orc.e4m3_decode(codes) * float(np.float32(k_scale))).reshape(a.k.shape), a.v_bits)
    k8_dev = torch.from_numpy(k8.reshape(w.num_pool_pages, sh.page_size, sh.num_kv_heads, sh.head_dim)).to(DEV)
    v_dev = torch.from_numpy(v_img.view(np.int16).reshape(vb.shape)).view(torch.bfloat16).to(DEV)
    return k8_dev, v_dev, stored


def _decoded_queries(t, q_scale):
    inv = np.float32(1) / np.float32(q_scale)
    codes = orc.e4m3_encode(t.q.float().cpu().numpy() * inv)
    return codes, orc.e4m3_decode(codes) * float(np.float32(q_scale))


def _check(w, out, lse, stored, q_dec, rows=None):
    out_f = out.float().cpu().numpy().astype(np.float64)
    lse_f = lse.cpu().numpy().astype(np.float64)
    errs, lerr = [], []
    for r, (k, v_bits) in stored.items():
        jj, hh, pp = orc.request_rows(w, r) if rows is None else rows[r]
        if len(jj) == 0:
            continue
        o, l = orc.attention_rows(w, k, v_bits, q_dec, jj, hh, pp)
        errs.append(np.abs(out_f[jj, hh] - o).ravel())
        lerr.append(np.abs(lse_f[jj, hh] - l))
    e = np.concatenate(errs)
    assert np.isfinite(e).all()
    assert e.max() <= gu.MAX_ABS and e.mean() <= gu.MEAN_ABS, "8-bit-key attention: max %.4g mean %.4g" % (e.max(), e.mean())
    assert np.concatenate(lerr).max() <= 5e-3
    return float(e.max()), float(e.mean())


@pytest.mark.parametrize("make,scales", [(lambda: wl.config(3, requests_override=3), (1 / 32, 1 / 32)),
                                         (lambda: wl.config(2), (0.03, 0.017)),                  # split along the keys, odd scales
                                         (lambda: wl.adversarial(seed=9, shape=wl.ModelShape(32, 8, 128, 64, 500000.0)), (1 / 16, 1 / 64)),
                                         (lambda: wl.adversarial(seed=44, shape=wl.ModelShape(40, 8, 128, 16, 500000.0)), (1 / 32, 1 / 32))])
def test_attention_over_8bit_keys_matches_fp64_attention_over_the_decoded_operands(make, scales):
    w = make()
    ks, qs = scales
    t = wl.make_tensors(w, device=DEV, seed=81)
    k8, v_pool, stored = _host_made_pools(w, t, ks)
    _, q_dec = _decoded_queries(t, qs)
    plan = tb.Plan(w)
    sh = w.shape
    out = torch.zeros(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(w.n_q, sh.num_q_heads, dtype=torch.float32, device=DEV)
    plan.partial_prefill_attn_k8(k8, ks, v_pool, t.q, qs, None, None, out, lse)
    torch.cuda.synchronize()
    assert plan.status() == 0
    mx, mean = _check(w, out, lse, stored, q_dec)
    # the quantisation is real: against the un-quantised operands the result is visibly different
    a = orc.assemble(w, 0, orc.bits(t.k_pool), orc.bits(t.v_pool), orc.bits(t.k_new), orc.bits(t.v_new))
    jj, hh, pp = orc.request_rows(w, 0)
    if len(jj):
        o_plain, _ = orc.attention_rows(w, a.k, a.v_bits, orc.bits(t.q), jj, hh, pp)
        assert np.abs(out.float().cpu().numpy()[jj, hh] - o_plain).mean() > 2 * mean


def test_fresh_rows_are_quantised_with_the_oracles_codec_and_queries_too():
    """k_new is written into the 8-bit pool as e4m3_rne(k_new * fp32(1 / k_scale)); V rows are bit copies;
    the attention result equals the one on pools that already held those codes."""
    w = wl.config(3, requests_override=2)
    ks, qs = 0.021, 1 / 32
    t = wl.make_tensors(w, device=DEV, seed=82)
    k8_full, v_full, stored = _host_made_pools(w, t, ks)
    plan = tb.Plan(w)
    sh = w.shape
    row = sh.num_kv_heads * sh.head_dim
    # start from the host-made pools with the fresh rows wiped, let the call scatter them
    st, page_off, pages, _, _ = orc.placement(w)
    B = sh.page_size
    slots = []
    for r in range(w.batch):
        pos = w.recompute_pos[w.recompute_off[r]:w.recompute_off[r + 1]].astype(np.int64)
        slots.append(pages[page_off[r] + pos // B].astype(np.int64) * B + pos % B)
    slots = torch.from_numpy(np.concatenate(slots)).to(DEV)
    k8 = k8_full.clone().view(-1, row)
    v = v_full.clone().view(-1, row)
    k8[slots] = NAN8
    v[slots] = torch.tensor(gu.POISON, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    k8, v = k8.view_as(k8_full), v.view_as(v_full)
    out = torch.zeros(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=DEV)
    ref = torch.zeros_like(out)
    lse = torch.zeros(w.n_q, sh.num_q_heads, dtype=torch.float32, device=DEV)
    plan.partial_prefill_attn_k8(k8, ks, v, t.q, qs, t.k_new, t.v_new, out, lse)
    plan.partial_prefill_attn_k8(k8_full, ks, v_full, t.q, qs, None, None, ref, None)
    torch.cuda.synchronize()
    assert plan.status() == 0
    want = orc.e4m3_encode(t.k_new.float().cpu().numpy().reshape(-1, row) * (np.float32(1) / np.float32(ks)))
    assert np.array_equal(k8.view(-1, row)[slots].cpu().numpy(), want)
    assert torch.equal(v.view(-1, row)[slots].view(torch.int16), t.v_new.reshape(-1, row).view(torch.int16))
    assert torch.equal(k8, k8_full) and torch.equal(v.view(torch.int16), v_full.view(torch.int16))
    assert torch.equal(out, ref)
    _check(w, out, lse, stored, _decoded_queries(t, qs)[1])


def test_8bit_key_pages_composed_on_the_gpu_then_attended():
    """The whole 8-bit-key path on the GPU: tessera_kv_compose_k8 rotates and quantises the cached keys into
    the request's 8-bit key pages and copies the values into the 16-bit pool; the attention call scatters
    the fresh rows and attends."""
    w = wl.config(3, requests_override=2)
    ks, qs = 0.027, 1 / 32
    t = wl.make_tensors(w, device=DEV, seed=83)
    w2 = copy.copy(w)
    w2.num_source_pages = w.num_pool_pages
    plan = tb.Plan(w2)
    sh = w.shape
    row = sh.num_kv_heads * sh.head_dim
    k8 = torch.full(tuple(t.k_pool.shape), NAN8, dtype=torch.uint8, device=DEV)
    src_k, src_v = t.k_pool.clone(), t.v_pool.clone()
    pv = torch.tensor(gu.POISON, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    t.v_pool[:] = pv
    plan.kv_compose_k8(src_k, src_v, k8, t.v_pool, ks)
    torch.cuda.synchronize()
    # cached rows: V bit copies; K the nearest code of the oracle's rotated key up to the fp32 rotation error
    kb, vb = orc.bits(src_k), orc.bits(src_v)
    zeros = np.zeros((max(w.n_q, 1), row), np.uint16)
    st, page_off, pages, _, _ = orc.placement(w)
    B = sh.page_size
    inv = float(np.float32(1) / np.float32(ks))
    table = orc.e4m3_decode(np.arange(0x7f, dtype=np.uint8))
    k8_h, v_h = k8.cpu().numpy().reshape(-1, row), orc.bits(t.v_pool).reshape(-1, row)
    n_diff = n_all = 0
    for r in range(w.batch):
        a = orc.assemble(w, r, kb, vb, zeros, zeros)
        T = int(w.seq_len[r])
        p = np.arange(T)
        slots = pages[page_off[r] + p // B].astype(np.int64) * B + p % B
        cached = np.ones(T, bool)
        cached[w.recompute_pos[w.recompute_off[r]:w.recompute_off[r + 1]]] = False
        # (recomputed positions inside cached units are copied too and overwritten later; they are not compared)
        assert np.array_equal(v_h[slots][cached], a.v_bits.reshape(T, row)[cached])
        y = a.k.reshape(T, row)[cached] * inv
        got = orc.e4m3_decode(k8_h[slots][cached])
        hi = np.searchsorted(table, np.abs(y), side="right")
        half = (table[np.minimum(hi, 0x7e)] - table[hi - 1]) / 2
        assert np.isfinite(got).all() and (np.abs(got - y) - half).max() <= 1e-5 * np.abs(y).max() + 1e-7
        want = orc.e4m3_encode(y.astype(np.float32))
        n_diff += int((k8_h[slots][cached] != want).sum())
        n_all += want.size
    assert n_diff < 2e-3 * n_all                                              # differences only at near-ties
    mask = np.ones(w.num_pool_pages, bool)
    mask[pages] = False
    assert np.all(k8.cpu().numpy()[mask] == NAN8) and np.all(orc.bits(t.v_pool)[mask] == gu.POISON)
    out = torch.zeros(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=DEV)
    lse = torch.zeros(w.n_q, sh.num_q_heads, dtype=torch.float32, device=DEV)
    plan.partial_prefill_attn_k8(k8, ks, t.v_pool, t.q, qs, t.k_new, t.v_new, out, lse)
    torch.cuda.synchronize()
    assert plan.status() == 0
    # The oracle attends over ITS OWN assembled keys quantised by its codec (no oracle input comes from a
    # kernel); the GPU's near-tie code differences counted above are absorbed by the tolerance.
    _, _, stored = _host_made_pools(w, dataclasses.replace(t, k_pool=src_k, v_pool=src_v), ks)
    e_max, e_mean = _check(w, out, lse, stored, _decoded_queries(t, qs)[1])
    assert e_max > 0


def test_8bit_key_attention_rejects_bad_arguments():
    w = wl.config(1)                                                            # head_dim 64
    t = wl.make_tensors(w, device=DEV, seed=2)
    k8 = torch.zeros(tuple(t.k_pool.shape), dtype=torch.uint8, device=DEV)
    out = torch.zeros_like(t.q)
    with pytest.raises(tb.TesseraError) as e:
        tb.Plan(w).partial_prefill_attn_k8(k8, 1.0, t.v_pool, t.q, 1.0, None, None, out)
    assert e.value.status == tb.UNSUPPORTED_SHAPE
    w = wl.config(2)
    t = wl.make_tensors(w, device=DEV, seed=2)
    k8 = torch.zeros(tuple(t.k_pool.shape), dtype=torch.uint8, device=DEV)
    out = torch.zeros_like(t.q)
    for bad in (0.0, -1.0, float("inf"), float("nan")):
        with pytest.raises(tb.TesseraError):
            tb.Plan(w).partial_prefill_attn_k8(k8, bad, t.v_pool, t.q, 1.0, None, None, out)
