"""GPU parity of tessera_extend_write: the write side of the extend pass in one kernel - fresh keys
rotated into the request's slots, values copied, queries rotated in place, and the un-rotated rows of
captured units written to cache pages - against the oracle, plus the capture -> reuse chain."""
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
i32 = lambda x: np.asarray(x, np.int32)


def _rotate_rows_host(bits, positions, shape):
    """fp64 rotation of every head vector of rows [n][H][D] (bf16 bits) for its position (the oracle's
    routine), returned unrounded."""
    x = orc.bf16_bits_to_f64(bits)
    out = np.empty_like(x)
    for j, p in enumerate(positions):
        for h in range(x.shape[1]):
            out[j, h] = orc.rope_rotate(x[j, h], float(p), shape.rope_theta, pairing=shape.rope_pairing)
    return out


def _run(w, seed, k_cache=None, v_cache=None, poison=True):
    """compose (fused) -> extend_write -> attention without its own scatter.  Returns a LayerRun whose
    kn_bits are the RAW fresh keys, so that check_assembled rotates them in the oracle."""
    t = wl.make_tensors(w, device=DEV, seed=seed)
    plan = tb.Plan(w)
    page_off, pages, src_slot = plan.block_table()
    if poison and len(pages):
        idx = torch.from_numpy(pages.astype(np.int64)).to(DEV)
        pv = torch.tensor(gu.POISON, dtype=torch.int16, device=DEV).view(torch.bfloat16)
        t.k_pool[idx] = pv
        t.v_pool[idx] = pv
    g = gu.LayerRun()
    g.w, g.t, g.plan = w, t, plan
    g.page_off, g.pages, g.src_slot = page_off, pages, src_slot
    g.k_before, g.v_before = orc.bits(t.k_pool).copy(), orc.bits(t.v_pool).copy()
    g.q_raw_bits, g.kn_bits, g.vn_bits = orc.bits(t.q).copy(), orc.bits(t.k_new).copy(), orc.bits(t.v_new).copy()
    g.fresh_k_raw = True
    plan.kv_compose(t.k_pool, t.v_pool, fuse_rope=True)
    kc = t.k_pool if k_cache is None else k_cache
    vc = t.v_pool if v_cache is None else v_cache
    plan.extend_write(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, kc, vc)
    sh = w.shape
    g.out = torch.zeros(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=DEV)
    g.lse = torch.zeros(w.n_q, sh.num_q_heads, dtype=torch.float32, device=DEV)
    plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, None, None, g.out, g.lse)
    torch.cuda.synchronize()
    g.status = plan.status()
    g.k_after, g.v_after = orc.bits(t.k_pool), orc.bits(t.v_pool)
    g.out_f = g.out.float().cpu().numpy().astype(np.float64)
    g.lse_f = g.lse.cpu().numpy().astype(np.float64)
    # inputs of the kernel that must not change
    assert np.array_equal(orc.bits(t.k_new), g.kn_bits) and np.array_equal(orc.bits(t.v_new), g.vn_bits)
    # rotated queries: within the rotated-key tolerance of the fp64 rotation of the raw queries
    q_want = _rotate_rows_host(g.q_raw_bits, w.recompute_pos, sh)
    q_got = orc.bf16_bits_to_f64(orc.bits(t.q))
    if w.n_q:
        d = np.abs(q_got - q_want)
        assert d.max() <= gu.MAX_ABS and d.mean() <= gu.MEAN_ABS
        zero = np.nonzero(w.recompute_pos == 0)[0]
        assert np.array_equal(orc.bits(t.q)[zero], g.q_raw_bits[zero])          # position 0: bit copy
    # the oracle attends with the queries rotated and rounded once on the host
    g.q_bits = orc.bits(torch.from_numpy(q_want).to(torch.bfloat16)) if w.n_q else g.q_raw_bits
    return g


@pytest.mark.parametrize("make", [lambda: wl.config(1), lambda: wl.config(3, requests_override=3),
                                  lambda: wl.adversarial(seed=9, shape=wl.ModelShape(32, 8, 128, 64, 500000.0)),
                                  lambda: wl.adversarial(seed=31, shape=wl.ModelShape(8, 2, 64, 16, 10000.0, rope_pairing=1)),
                                  lambda: wl.config(5, requests_override=2)])
def test_extend_write_then_attention_matches_oracle(make):
    w = make()
    g = _run(w, seed=71)
    assert g.status == 0
    gu.check_placement(g)
    asm, kmx, kmean = gu.check_assembled(g)          # fresh K rows: rotated raw keys (tolerance); V rows: bit copies
    assert kmx > 0
    gu.check_untouched(g)
    gu.check_attention(g, asm)


def test_fused_write_equals_rotate_then_scatter_bit_for_bit():
    """The same arithmetic as tessera_rope_fresh followed by the attention call's own scatter."""
    w = wl.config(3, requests_override=4)
    a = wl.make_tensors(w, device=DEV, seed=5)
    b = wl.make_tensors(w, device=DEV, seed=5)
    plan = tb.Plan(w)
    out_a, out_b = torch.zeros_like(a.q), torch.zeros_like(a.q)
    plan.kv_compose(a.k_pool, a.v_pool)
    plan.rope_fresh(a.q, a.k_new)
    plan.partial_prefill_attn(a.k_pool, a.v_pool, a.q, a.k_new, a.v_new, out_a, None)
    plan.kv_compose(b.k_pool, b.v_pool)
    plan.extend_write(b.k_pool, b.v_pool, b.q, b.k_new, b.v_new)
    plan.partial_prefill_attn(b.k_pool, b.v_pool, b.q, None, None, out_b, None)
    torch.cuda.synchronize()
    assert plan.status() == 0
    assert torch.equal(a.k_pool, b.k_pool) and torch.equal(a.v_pool, b.v_pool)
    assert torch.equal(a.q, b.q) and torch.equal(out_a, out_b)


def _with_capture(w, units, separate_pool):
    """Copy of workload `w` that captures the listed unit indices into spare pages (the tail of the
    free list, or pages 0.. of a separate cache pool)."""
    B = w.shape.page_size
    used = int(sum(-(-int(t) // B) for t in w.seq_len))
    spare = w.free_pages[used:].tolist()
    off, pages, nxt = [0], [], 0
    for u in range(len(w.unit_len)):
        if u in units:
            n = -(-int(w.unit_len[u]) // B)
            pages += list(range(nxt, nxt + n)) if separate_pool else spare[nxt:nxt + n]
            nxt += n
        off.append(len(pages))
    assert separate_pool or nxt <= len(spare)
    w2 = copy.copy(w)
    w2.unit_retain_page_off, w2.unit_retain_pages = i32(off), i32(pages)
    w2.retain_pool_pages = nxt + 2 if separate_pool else 0
    return w2


@pytest.mark.parametrize("separate_pool", [False, True])
def test_capture_writes_raw_rows_bit_for_bit(separate_pool):
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    rng = np.random.default_rng(23)
    segs = [[37, wl.unit(200, "x", recompute=(0, 1)), wl.unit(150, "U", cached=False), wl.unit(70, "y", cached_pos=3),
             wl.unit(64, "V", cached=False), 9],
            [wl.unit(129, "W", cached=False), 3]]
    w0 = wl.build_workload("capture", shape, segs, rng, spare_pages=12)
    w = _with_capture(w0, {1, 3, 4}, separate_pool)
    kc = vc = None
    if separate_pool:
        pv = torch.tensor(gu.POISON, dtype=torch.int16, device=DEV).view(torch.bfloat16)
        kc = torch.empty(w.retain_pool_pages, shape.page_size, 8, 128, dtype=torch.bfloat16, device=DEV)
        vc = torch.empty_like(kc)
        kc[:] = pv
        vc[:] = pv
    g = _run(w, seed=72, k_cache=kc, v_cache=vc, poison=False)
    assert g.status == 0 and g.plan.info.retained_tokens == 150 + 64 + 129
    gu.check_placement(g)
    asm, _, _ = gu.check_assembled(g)
    gu.check_attention(g, asm)
    row = 8 * 128
    B = shape.page_size
    kc_bits = (orc.bits(kc) if separate_pool else g.k_after).reshape(-1, row)
    vc_bits = (orc.bits(vc) if separate_pool else g.v_after).reshape(-1, row)
    written = np.zeros(kc_bits.shape[0], bool)
    for u in (1, 3, 4):
        r = int(np.searchsorted(w.unit_off, u, side="right") - 1)
        j0 = int(w.recompute_off[r])
        pos = w.recompute_pos[j0:int(w.recompute_off[r + 1])]
        for i in range(int(w.unit_len[u])):
            j = j0 + int(np.searchsorted(pos, w.unit_target_pos[u] + i))
            slot = int(w.unit_retain_pages[w.unit_retain_page_off[u] + i // B]) * B + i % B
            assert np.array_equal(kc_bits[slot], g.kn_bits[j].ravel()), (u, i)       # the raw key, untouched
            assert np.array_equal(vc_bits[slot], g.vn_bits[j].ravel()), (u, i)
            written[slot] = True
    # nothing else in the cache pool changed
    if separate_pool:
        assert np.all(kc_bits[~written] == gu.POISON) and np.all(vc_bits[~written] == gu.POISON)
    else:
        dest = np.zeros(kc_bits.shape[0], bool)
        for pg in g.pages:
            dest[int(pg) * B:(int(pg) + 1) * B] = True
        keep = ~written & ~dest
        assert np.array_equal(kc_bits[keep], g.k_before.reshape(-1, row)[keep])
        assert np.array_equal(vc_bits[keep], g.v_before.reshape(-1, row)[keep])


def test_capture_is_refused_for_units_that_are_not_fully_recomputed():
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    w0 = wl.build_workload("bad", shape, [[wl.unit(100, "a", recompute=(0, 1)), wl.unit(70, "b", cached=False), 3]],
                           np.random.default_rng(1), spare_pages=8)
    assert tb.plan_create_status(_with_capture(w0, {1}, False)) == tb.OK
    assert tb.plan_create_status(_with_capture(w0, {0}, False)) == tb.INVALID_ARG        # a cached unit with 2 fresh rows
    bad = _with_capture(w0, {1}, False)
    bad.unit_retain_pages = i32([int(w0.unit_pages[0])] * len(bad.unit_retain_pages))    # a source page of the batch
    assert tb.plan_create_status(bad) == tb.PAGE_OUT_OF_RANGE
    bad = _with_capture(w0, {1}, True)
    bad.retain_pool_pages = 1                                                            # 2 pages needed
    assert tb.plan_create_status(bad) == tb.PAGE_OUT_OF_RANGE


def test_capture_then_reuse_chain_against_the_raw_key():
    """Miss -> captured unit -> later hit, all on the GPU, compared with the oracle started from the
    ORIGINAL un-rotated key: (1) the direct capture of this file (raw bits kept, one rounding at reuse)
    and (2) the un-rotate path (fresh key rotated and rounded, read back from the request's pages,
    rotated back and rounded, rotated again at reuse and rounded).  Both must stay within the rotated-key
    tolerance; the errors of both are printed."""
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    rng = np.random.default_rng(17)
    B = shape.page_size
    pos_u, len_u, tgt = 37 + 200, 150, 1011
    A0 = wl.build_workload("A", shape, [[37, wl.unit(200, "x", recompute=(0, 1)), wl.unit(len_u, "U", cached=False), 9]],
                           rng, spare_pages=40)
    used = -(-int(A0.seq_len[0]) // B)
    spare = A0.free_pages[used:]
    n_cache = -(-len_u // B)
    A = _with_capture(A0, {1}, False)
    cache_pages = A.unit_retain_pages.tolist()
    T_b = tgt + len_u + 5
    reuse = lambda pages: wl.Workload(
        name="reuse", shape=shape, seq_len=i32([T_b]), unit_off=i32([0, 1]), unit_len=i32([len_u]),
        unit_cached_pos=i32([0]), unit_cached_stride=i32([0]), unit_target_pos=i32([tgt]),
        unit_page_off=i32([0, n_cache]), unit_pages=i32(pages), recompute_off=i32([0, tgt + 5]),
        recompute_pos=i32(list(range(tgt)) + list(range(tgt + len_u, T_b))),
        free_pages=i32(spare[2 * n_cache:2 * n_cache + -(-T_b // B)]), num_pool_pages=A.num_pool_pages)
    tA = wl.make_tensors(A, device=DEV, seed=31)
    j0 = int(np.searchsorted(A.recompute_pos, pos_u))
    k_raw = orc.bf16_bits_to_f64(orc.bits(tA.k_new)[j0:j0 + len_u])                      # the original key, [len][H][D]
    want = np.stack([[orc.rope_rotate(k_raw[i, h], tgt + i, shape.rope_theta) for h in range(8)] for i in range(len_u)])
    row = 8 * 128

    def reused_keys(t, pages):
        wB = reuse(pages)
        planB = tb.Plan(wB)
        planB.kv_compose(t.k_pool, t.v_pool)
        torch.cuda.synchronize()
        _, pg, _ = planB.block_table()
        p = tgt + np.arange(len_u)
        slots = pg[p // B].astype(np.int64) * B + p % B
        return orc.bf16_bits_to_f64(orc.bits(t.k_pool).reshape(-1, row)[slots]).reshape(len_u, 8, 128)

    # (1) direct capture
    t1 = wl.make_tensors(A, device=DEV, seed=31)
    planA = tb.Plan(A)
    planA.kv_compose(t1.k_pool, t1.v_pool)
    planA.extend_write(t1.k_pool, t1.v_pool, t1.q, t1.k_new, t1.v_new, t1.k_pool, t1.v_pool)
    e1 = np.abs(reused_keys(t1, cache_pages) - want)
    # (2) un-rotate path: rotate fresh rows, scatter through the attention call, retain from the request's pages
    t2 = wl.make_tensors(A, device=DEV, seed=31)
    planA0 = tb.Plan(A0)
    planA0.kv_compose(t2.k_pool, t2.v_pool)
    planA0.rope_fresh(t2.q, t2.k_new)
    planA0.partial_prefill_attn(t2.k_pool, t2.v_pool, t2.q, t2.k_new, t2.v_new, torch.zeros_like(t2.q), None)
    first, last = pos_u // B, (pos_u + len_u - 1) // B
    R = wl.Workload(name="retain", shape=shape, seq_len=i32([len_u]), unit_off=i32([0, 1]), unit_len=i32([len_u]),
                    unit_cached_pos=i32([pos_u]), unit_cached_stride=i32([1]), unit_target_pos=i32([0]),
                    unit_page_off=i32([0, last - first + 1]), unit_pages=i32(A0.free_pages[first:last + 1]),
                    recompute_off=i32([0, 0]), recompute_pos=i32([]), free_pages=i32(spare[n_cache:2 * n_cache]),
                    num_pool_pages=A.num_pool_pages, unit_src_offset=i32([pos_u % B]), unit_target_stride=i32([0]))
    tb.Plan(R).kv_compose(t2.k_pool, t2.v_pool)
    e2 = np.abs(reused_keys(t2, spare[n_cache:2 * n_cache].tolist()) - want)
    print("capture -> reuse, error against the rotated original key: direct capture max %.4g mean %.4g | "
          "un-rotate path (three roundings) max %.4g mean %.4g" % (e1.max(), e1.mean(), e2.max(), e2.mean()))
    assert e1.max() <= gu.MAX_ABS and e1.mean() <= gu.MEAN_ABS
    assert e2.max() <= 2 * gu.MAX_ABS and e2.mean() <= 2 * gu.MEAN_ABS
    assert e1.mean() < e2.mean()
