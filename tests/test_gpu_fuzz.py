"""Seeded random layouts through the whole path: head_dim, page size, group size (also ones that do not
divide the tile), pairing, fused / unfused shift, cached and uncached units at random cached positions and
strides, scattered recompute offsets - each compared with the oracle in full."""
import copy

import numpy as np
import pytest
import torch

from paper_2609_32999_b200 import binding as tb
from paper_2609_32999_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _random_workload(rng, tag):
    D = int(rng.choice([64, 128]))
    page = int(rng.choice([8, 16, 32, 64, 128]))
    hkv = int(rng.choice([1, 2, 4, 8]))
    g = int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8, 16]))
    shape = wl.ModelShape(hkv * g, hkv, D, page, float(rng.choice([1e4, 5e5])), rope_pairing=int(rng.integers(0, 2)))
    reqs = []
    for r in range(int(rng.integers(1, 7))):
        segs = []
        if rng.random() < 0.5:
            segs.append(int(rng.integers(1, 40)))
        for u in range(int(rng.integers(0, 5))):
            L = int(rng.integers(1, 700))
            cached = rng.random() < 0.8
            rec = tuple(sorted(set(int(x) for x in rng.integers(0, L, size=int(rng.integers(0, 6)))))) if cached else ()
            segs.append(wl.unit(L, (tag, r, u), cached=cached, cached_pos=int(rng.integers(0, 300)),
                                stride=int(rng.integers(0, 2)), recompute=rec))
        if rng.random() < 0.7 or not segs:
            segs.append(int(rng.integers(1, 90)))
        reqs.append(segs)
    return wl.build_workload("fuzz-%s" % tag, shape, reqs, rng)


@pytest.mark.parametrize("seed", [11, 12, 13, 14])
def test_random_layouts_full_parity(seed):
    rng = np.random.default_rng(seed)
    for it in range(6):
        w = _random_workload(rng, "%d-%d" % (seed, it))
        g = gu.run_layer(w, seed=seed * 100 + it, fuse=bool(rng.integers(0, 2)))
        assert g.status == 0
        gu.check_placement(g)
        asm, _, _ = gu.check_assembled(g)
        gu.check_untouched(g)
        if w.n_q:
            gu.check_attention(g, asm)


@pytest.mark.parametrize("seed", [21, 22])
def test_random_layouts_through_the_fused_write_side_with_capture(seed):
    """The same random layouts through tessera_extend_write (un-rotated fresh keys, every uncached unit
    captured into spare pages of the same pool) and attention without its own scatter."""
    from tests.test_gpu_extend_write import _run, _with_capture
    rng = np.random.default_rng(seed)
    for it in range(5):
        w0 = _random_workload(rng, "%d-%d" % (seed, it))
        uncached = {u for u in range(len(w0.unit_len)) if w0.unit_page_off[u + 1] == w0.unit_page_off[u] and w0.unit_len[u] > 0}
        B = w0.shape.page_size
        need = sum(-(-int(w0.unit_len[u]) // B) for u in uncached)
        # grow the pool by the pages the captured units need: they are appended to the free list, behind the
        # destination pages, which is where _with_capture takes the cache pages from
        w0 = copy.copy(w0)
        extra = np.arange(w0.num_pool_pages, w0.num_pool_pages + need, dtype=np.int32)
        w0.free_pages = np.concatenate([w0.free_pages, extra]).astype(np.int32)
        w0.num_pool_pages += need
        w = _with_capture(w0, uncached, False) if need else w0
        g = _run(w, seed=seed * 100 + it)
        assert g.status == 0
        gu.check_placement(g)
        asm, _, _ = gu.check_assembled(g)
        if w.n_q:
            gu.check_attention(g, asm)
        if need:
            row = w.shape.num_kv_heads * w.shape.head_dim
            kc, vc = g.k_after.reshape(-1, row), g.v_after.reshape(-1, row)
            for u in uncached:
                r = int(np.searchsorted(w.unit_off, u, side="right") - 1)
                j0 = int(w.recompute_off[r])
                pos = w.recompute_pos[j0:int(w.recompute_off[r + 1])]
                for i in range(int(w.unit_len[u])):
                    j = j0 + int(np.searchsorted(pos, w.unit_target_pos[u] + i))
                    slot = int(w.unit_retain_pages[w.unit_retain_page_off[u] + i // B]) * B + i % B
                    assert np.array_equal(kc[slot], g.kn_bits[j].ravel()) and np.array_equal(vc[slot], g.vn_bits[j].ravel())


@pytest.mark.parametrize("seed", [31])
def test_random_layouts_through_the_overlapped_host_tier(seed):
    """Random layouts with the units in a pinned host pool: the overlapped path must leave the bits of
    compose-from-host followed by one attention call."""
    rng = np.random.default_rng(seed)
    for it in range(5):
        w = _random_workload(rng, "%d-%d" % (seed, it))
        t = wl.make_tensors(w, device="cuda:0", seed=seed * 100 + it)
        hk, hv = t.k_pool.cpu().pin_memory(), t.v_pool.cpu().pin_memory()
        w2 = copy.copy(w)
        w2.num_source_pages = w.num_pool_pages
        plan = tb.Plan(w2)
        sh = w.shape
        ka, va, kb, vb = t.k_pool.clone(), t.v_pool.clone(), t.k_pool.clone(), t.v_pool.clone()
        oa = torch.zeros(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device="cuda:0")
        ob = torch.zeros_like(oa)
        plan.kv_compose_from(hk, hv, ka, va)
        plan.partial_prefill_attn(ka, va, t.q, t.k_new, t.v_new, oa, None)
        plan.composed_prefill_host_tier(hk, hv, kb, vb, t.q, t.k_new, t.v_new, ob, None, reader_blocks=int(rng.integers(0, 9)))
        torch.cuda.synchronize()
        assert plan.status() == 0
        assert torch.equal(ka.view(torch.int16), kb.view(torch.int16)) and torch.equal(va.view(torch.int16), vb.view(torch.int16))
        assert torch.equal(oa, ob)
