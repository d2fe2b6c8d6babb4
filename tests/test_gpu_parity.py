"""GPU parity: the CUDA library against the fp64 oracle on the same seeded bytes, through the C ABI."""
import math

import numpy as np
import pytest
import torch

from oracle import tessera_oracle as orc
from paper_2609_32999_b200 import binding as tb
from paper_2609_32999_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _full_check(w, fuse=True, seed=None):
    g = gu.run_layer(w, fuse=fuse, seed=seed)
    assert g.status == 0
    gu.check_placement(g)
    asm, kmx, kmean = gu.check_assembled(g)
    gu.check_untouched(g)
    amx, amean = gu.check_attention(g, asm)                       # whole path vs unrounded oracle keys
    gu.check_attention_alone(w, seed=seed)                         # attention kernel alone, on oracle-made pages
    return g, (kmx, kmean, amx, amean)


@pytest.mark.parametrize("idx", [1, 2, 3])
def test_config_full_parity(idx):
    _full_check(wl.config(idx))


def test_adversarial_shapes_and_shifts():
    """Negative shifts, non-zero cached positions, keys cached without rotation, a unit used twice,
    ragged pages, an uncached unit, an empty-ish request; small head_dim path and the Llama shape."""
    _full_check(wl.adversarial())
    _full_check(wl.adversarial(seed=9, shape=wl.ModelShape(32, 8, 128, 64, 500000.0)))
    _full_check(wl.adversarial(seed=10, shape=wl.ModelShape(16, 2, 128, 64, 500000.0)))
    _full_check(wl.adversarial(seed=11, shape=wl.ModelShape(8, 8, 128, 64, 10000.0)))


def test_unfused_compose_then_shift_equals_fused():
    w = wl.config(3, requests_override=4)
    a = gu.run_layer(w, fuse=True, seed=5, attention=False)
    b = gu.run_layer(w, fuse=False, seed=5, attention=False)
    assert np.array_equal(a.k_before, b.k_before)
    assert np.array_equal(a.k_after, b.k_after) and np.array_equal(a.v_after, b.v_after)
    gu.check_assembled(b, scattered=False)


def test_zero_shift_is_bit_copy():
    """A unit reused at the position it was cached at must come through bit for bit - including signed
    zeros whose pair partner is negative (a multiply-add by cos = 1, sin = 0 would turn -0.0 into +0.0)
    and infinities (0 x Inf would give NaN)."""
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    segs = [wl.unit(300, "a", cached_pos=0, recompute=(0,)), wl.unit(200, "b", cached_pos=300, recompute=(0,)), 5]
    w = wl.build_workload("zero", shape, [segs], np.random.default_rng(1))
    for fuse in (True, False):
        t = wl.make_tensors(w, device="cuda:0", seed=13)
        neg0 = torch.tensor(-0.0, dtype=torch.bfloat16, device="cuda:0")
        t.k_pool[:, :, :, 0:3] = neg0                                   # -0.0 in the first half ...
        t.k_pool[:, :, :, 64:67] = -t.k_pool[:, :, :, 64:67].abs() - 1  # ... with a negative partner
        t.k_pool[:, :, :, 70:72] = neg0                                 # -0.0 in the second half, positive partner
        t.k_pool[:, :, :, 6:8] = t.k_pool[:, :, :, 6:8].abs() + 1
        t.k_pool[:, :, :, 10] = float("inf")                            # an infinity next to an ordinary partner
        g = gu.run_layer(w, t=t, fuse=fuse, attention=False, poison=False)
        asm, mx, mean = gu.check_assembled(g, scattered=False)
        assert mx == 0.0 and np.all(asm[0].delta == 0)
        row = shape.num_kv_heads * shape.head_dim
        dst = g.k_after.reshape(-1, row)[gu.dest_slots(g, 0)][: 500]
        assert np.all(dst.reshape(500, 8, 128)[:, :, 0:3] == 0x8000) and np.all(dst.reshape(500, 8, 128)[:, :, 70:72] == 0x8000)
        assert np.all(dst.reshape(500, 8, 128)[:, :, 10] == 0x7f80)


def test_uniform_softmax_lse_and_mean():
    """K == 0: LSE = ln(p + 1) and O = mean of V[0..p] - shows the causal limit and page skipping
    exactly, which the absolute tolerance alone cannot at long context."""
    for w in (wl.config(1), wl.config(2), wl.adversarial(seed=9, shape=wl.ModelShape(32, 8, 128, 64, 500000.0))):
        t = wl.make_tensors(w, device="cuda:0")
        t.k_pool.zero_(); t.k_new.zero_()
        D = w.shape.head_dim
        sl = torch.arange(w.num_pool_pages * w.shape.page_size, device="cuda:0")
        v = torch.nn.functional.one_hot(sl % D, D).to(torch.bfloat16)          # V[slot] = e_(slot mod D)
        t.v_pool.copy_(v.view(w.num_pool_pages, w.shape.page_size, 1, D).expand_as(t.v_pool))
        t.v_new.zero_()
        g = gu.run_layer(w, t=t, poison=False)
        assert g.status == 0
        asm, _, _ = gu.check_assembled(g)
        for r, a in asm.items():
            jj, hh, pp = orc.request_rows(w, r)
            if len(jj) == 0:
                continue
            assert np.max(np.abs(g.lse_f[jj, hh] - np.log(pp + 1.0))) < 2e-4
            o, _ = orc.attention_rows(w, a.k, a.v_bits, g.q_bits, jj, hh, pp)
            # outputs are counts / (p + 1): exact up to the final bf16 rounding (relative 2^-8)
            assert np.all(np.abs(g.out_f[jj, hh] - o) <= np.abs(o) * 2.0 ** -8 + 1e-6)


def test_needle_on_each_side_of_causal_limit_and_page_boundary():
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    T = 64 * 5
    w = wl.build_workload("needle", shape, [[wl.unit(T, "a", cached=False)]], np.random.default_rng(3))
    dev = "cuda:0"
    for needle in (62, 63, 64, 65, 127, 128, 129, 255, 256, 257):
        t = wl.make_tensors(w, device=dev)
        t.q.zero_(); t.q[:, :, 0] = 8.0
        t.k_new.zero_(); t.k_new[needle, :, 0] = 64.0
        t.v_new.zero_(); t.v_new[needle, :, 1] = 1.0
        g = gu.run_layer(w, t=t, poison=True)
        col = g.out_f[:, :, 1]
        assert np.all(col[:needle] == 0.0), needle
        assert np.all(col[needle:] > 0.99), needle


def test_deterministic_and_null_lse():
    w = wl.config(3, requests_override=3)
    a = gu.run_layer(w, seed=1)
    b = gu.run_layer(w, seed=1, with_lse=False)
    assert torch.equal(a.out, b.out)
    assert np.array_equal(a.k_after, b.k_after)


def test_explicit_inv_freq_overrides_theta():
    w = wl.config(1)
    D = w.shape.head_dim
    inv = (w.shape.rope_theta ** (-2.0 * np.arange(D // 2) / D)) * 0.5       # scaled frequencies
    plan = tb.Plan(w, inv_freq=inv)
    g = gu.run_layer(w, plan=plan, attention=False)
    sh = w.shape
    row = sh.num_kv_heads * sh.head_dim
    a = orc.assemble(w, 0, g.k_before, g.v_before, g.kn_bits, g.vn_bits, inv_freq=inv)
    gk = orc.bf16_bits_to_f64(g.k_after.reshape(-1, row)[gu.dest_slots(g, 0)])
    rot = a.k_exact == 0
    rot[w.recompute_pos] = False
    d = np.abs(gk[rot] - a.k.reshape(-1, row)[rot])
    assert d.max() <= gu.MAX_ABS and d.mean() <= gu.MEAN_ABS
    wrong = orc.assemble(w, 0, g.k_before, g.v_before, g.kn_bits, g.vn_bits)
    assert np.abs(gk[rot] - wrong.k.reshape(-1, row)[rot]).max() > 0.5


def test_host_buffer_entry_point_matches_device_calls():
    w = wl.config(2)
    g = gu.run_layer(w, seed=2)
    t = wl.make_tensors(w, device="cuda:0", seed=2)
    plan = tb.Plan(w)
    qh, kh, vh = (x.cpu().pin_memory() for x in (t.q, t.k_new, t.v_new))
    oh = torch.empty_like(qh).pin_memory()
    lh = torch.empty(w.n_q, w.shape.num_q_heads, dtype=torch.float32).pin_memory()
    plan.composed_prefill_host(t.k_pool, t.v_pool, qh, kh, vh, oh, lh)
    assert torch.equal(oh, g.out.cpu())
    assert torch.equal(lh, g.lse.cpu())


@pytest.mark.parametrize("idx,layer,n_random", [(4, 0, 4096), (4, 15, 4096), (4, 31, 4096), (5, 5, 4096)])
def test_full_size_sampled(idx, layer, n_random):
    """Configurations too large for the oracle in full: gather compared in full (bit-exact V, block
    table, exact K rows, tolerance on rotated K), attention on the first and last q tile of every
    checked request plus n_random random (request, row, head) triples.  Config 4 is checked on its
    first, middle and last layer (each layer has its own K / V / Q draw)."""
    w = wl.config(idx)
    g = gu.run_layer(w, layer=layer)
    assert g.status == 0
    gu.check_placement(g)
    gu.check_untouched(g)
    rng = np.random.default_rng(100 * idx + layer)
    reqs = list(range(w.batch)) if idx == 4 else sorted(rng.choice(w.batch, size=8, replace=False).tolist())
    asm, kmx, kmean = gu.check_assembled(g, requests=reqs)
    tile_tokens = 128 // (w.shape.num_q_heads // w.shape.num_kv_heads)
    rows = {r: gu.sample_rows(w, r, rng, -(-n_random // len(reqs)), tile_tokens) for r in reqs}
    assert sum(len(v[0]) for v in rows.values()) >= n_random
    gu.check_attention(g, asm, rows_by_request=rows)


def _uniform_softmax_exact(w, seed):
    """K == 0 everywhere: every visible key gets the same weight, so LSE = ln(p + 1) and O = (sum of the
    visible V rows) / (p + 1) whatever the tiling - a dropped, doubled or wrongly masked key or page
    shows up directly.  V rows are one-hot (cached: by slot, fresh: by row index), so the sums are small
    integers.  The expected values are prefix sums over the oracle's assembled V; no oracle attention is
    needed, so this runs at any length."""
    dev = "cuda:0"
    t = wl.make_tensors(w, device=dev, seed=seed)
    D = w.shape.head_dim
    t.k_pool.zero_(); t.k_new.zero_()
    sl = torch.arange(w.num_pool_pages * w.shape.page_size, device=dev)
    v = torch.nn.functional.one_hot(sl % D, D).to(torch.bfloat16)               # V[slot] = e_(slot mod D)
    t.v_pool.copy_(v.view(w.num_pool_pages, w.shape.page_size, 1, D).expand_as(t.v_pool))
    jq = torch.arange(w.n_q, device=dev)
    vn = torch.nn.functional.one_hot((jq * 5 + 3) % D, D).to(torch.bfloat16)    # V_new[j] = e_((5j + 3) mod D)
    t.v_new.copy_(vn.view(w.n_q, 1, D).expand_as(t.v_new))
    g = gu.run_layer(w, t=t, poison=False)
    assert g.status == 0
    gu.check_placement(g)
    asm, _, _ = gu.check_assembled(g)
    gq = w.shape.num_q_heads // w.shape.num_kv_heads
    worst_lse = worst_o = 0.0
    for r, a in asm.items():
        j0, j1 = int(w.recompute_off[r]), int(w.recompute_off[r + 1])
        if j1 == j0:
            continue
        pos = w.recompute_pos[j0:j1].astype(np.int64)
        prefix = np.cumsum(orc.bf16_bits_to_f64(a.v_bits), axis=0)              # [T, H_kv, D]: sum of V[0..p]
        want = prefix[pos] / (pos + 1.0)[:, None, None]                         # [n, H_kv, D]
        want = np.repeat(want, gq, axis=1)                                      # query head h reads KV head h // g
        got = g.out_f[j0:j1]
        err = np.abs(got - want) - (np.abs(want) * 2.0 ** -8 + 1e-6)           # exact up to the final bf16 rounding
        worst_o = max(worst_o, float(err.max()))
        lse_err = np.abs(g.lse_f[j0:j1] - np.log(pos + 1.0)[:, None])
        worst_lse = max(worst_lse, float(lse_err.max()))
    assert worst_lse < 2e-4, "LSE differs from ln(p + 1) by %.3g" % worst_lse
    assert worst_o <= 0.0, "O differs from the mean of the visible V rows by %.3g beyond rounding" % worst_o
    return g


def test_uniform_softmax_exact_on_one_full_length_request():
    """One request of config 4 in full (33 024 tokens, all 2 304 query rows, 258 key steps per work item,
    two work items per thread block): the path the headline number takes, checked exactly."""
    w = wl.config(4, requests_override=1)
    assert int(w.seq_len[0]) == 33024 and w.n_q == 2304
    g = _uniform_softmax_exact(w, seed=41)
    assert g.plan.info.n_attn_items == 36 * 8                       # no split along the keys


def test_uniform_softmax_exact_on_scattered_rows_with_eight_heads_per_group():
    """Requests shaped like config 5: 8 query heads per KV head (16 tokens per tile), recompute rows
    scattered inside the cached units, uncached units recomputed in full."""
    w = wl.config(5, requests_override=3)
    uncached = [u for u in range(len(w.unit_len)) if w.unit_page_off[u + 1] == w.unit_page_off[u]]
    assert uncached and w.shape.num_q_heads // w.shape.num_kv_heads == 8
    _uniform_softmax_exact(w, seed=42)


@pytest.mark.parametrize("n_requests", [1, 3])
def test_needles_at_long_context_around_page_step_and_ring_boundaries(n_requests):
    """Keys with an overwhelming logit at positions just before / at / after a page boundary (multiples
    of 64), a 128-key step boundary and a wrap of the kernel's four-slot K/V ring (every 256 keys), more
    than 32 K tokens into the context.  A query row at position p must see exactly the needles at
    positions <= p: with k visible needles each gets weight 1/k in its own output column, an invisible
    one exactly 0.  One request is split along the keys (too few work items for the GPU), three are not."""
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    rng = np.random.default_rng(6)
    ctx = 32768 + 700
    lo, hi = 32768 - 200, 32768 + 200                                   # recomputed window inside the cached unit
    reqs = [[5, wl.unit(ctx, ("ctx", r), recompute=range(lo - 5, hi - 5)), 40] for r in range(n_requests)]
    w = wl.build_workload("needles", shape, reqs, rng)
    needles = [32703, 32704, 32705, 32767, 32768, 32769, 32831, 32832, 32895, 32896, 32897]
    dev = "cuda:0"
    t = wl.make_tensors(w, device=dev, seed=8)
    t.k_pool.zero_(); t.v_pool.zero_(); t.k_new.zero_(); t.v_new.zero_()
    t.q.zero_(); t.q[:, :, 0] = 8.0
    for r in range(n_requests):
        j0, j1 = int(w.recompute_off[r]), int(w.recompute_off[r + 1])
        pos = w.recompute_pos[j0:j1]
        for i, n in enumerate(needles):
            j = j0 + int(np.searchsorted(pos, n))
            assert pos[j - j0] == n
            t.k_new[j, :, 0] = 64.0
            t.v_new[j, :, 1 + i] = 1.0
    g = gu.run_layer(w, t=t, poison=True)
    assert g.status == 0
    items = g.plan.info.n_attn_items
    assert (items < 148) == (n_requests == 1)
    for r in range(n_requests):
        j0, j1 = int(w.recompute_off[r]), int(w.recompute_off[r + 1])
        pos = w.recompute_pos[j0:j1]
        seen = np.searchsorted(np.array(needles), pos, side="right")            # needles at positions <= p
        for i in range(len(needles)):
            col = g.out_f[j0:j1, :, 1 + i]
            vis = seen > i
            assert np.all(col[~vis] == 0.0), (r, needles[i])
            want = 1.0 / seen[vis]
            assert np.all(np.abs(col[vis] - want[:, None]) <= want[:, None] * 2.0 ** -7), (r, needles[i])
        assert np.all(g.out_f[j0:j1][seen == 0] == 0.0)


def _retention_workloads():
    """A: a request with an uncached unit U at an unaligned position.  R: the plan that retains U from
    A's pages into fresh cache pages in un-rotated form.  B: a later request that reuses the retained U
    (cached without rotation) at another position."""
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    rng = np.random.default_rng(17)
    pos_u, len_u = 37 + 200, 150
    A = wl.build_workload("A", shape, [[37, wl.unit(200, "x", recompute=(0, 1)), wl.unit(len_u, "U", cached=False), 9]],
                          rng, spare_pages=40)
    B_ = shape.page_size
    used = -(-int(A.seq_len[0]) // B_)
    spare = A.free_pages[used:]
    first, last = pos_u // B_, (pos_u + len_u - 1) // B_
    n_cache = -(-len_u // B_)
    i32 = lambda x: np.asarray(x, np.int32)
    R = wl.Workload(name="retain", shape=shape, seq_len=i32([len_u]), unit_off=i32([0, 1]), unit_len=i32([len_u]),
                    unit_cached_pos=i32([pos_u]), unit_cached_stride=i32([1]), unit_target_pos=i32([0]),
                    unit_page_off=i32([0, last - first + 1]), unit_pages=i32(A.free_pages[first:last + 1]),
                    recompute_off=i32([0, 0]), recompute_pos=i32([]), free_pages=i32(spare[:n_cache]),
                    num_pool_pages=A.num_pool_pages, unit_src_offset=i32([pos_u % B_]), unit_target_stride=i32([0]))
    tgt = 11
    T_b = tgt + len_u + 5
    B = wl.Workload(name="reuse", shape=shape, seq_len=i32([T_b]), unit_off=i32([0, 1]), unit_len=i32([len_u]),
                    unit_cached_pos=i32([0]), unit_cached_stride=i32([0]), unit_target_pos=i32([tgt]),
                    unit_page_off=i32([0, n_cache]), unit_pages=i32(spare[:n_cache]),
                    recompute_off=i32([0, tgt + 5 + 2]),
                    recompute_pos=i32(list(range(tgt)) + [tgt, tgt + 1] + list(range(tgt + len_u, T_b))),
                    free_pages=i32(spare[n_cache:n_cache + -(-T_b // B_)]), num_pool_pages=A.num_pool_pages)
    return A, R, B


def test_retain_fresh_unit_then_reuse_it():
    """Store side of the cache: a freshly computed unit is written back un-rotated from the request's
    pages (source offset inside a page, shift = -(position) per token), then reused elsewhere.  Every
    stage starts from pages the ORACLE assembled on the host, never from pages a kernel wrote."""
    import dataclasses
    A, R, B = _retention_workloads()
    a = gu.run_layer(A, seed=31)
    assert a.status == 0
    gu.check_attention(a, gu.check_assembled(a)[0])
    # retain: the request's pages as the oracle leaves them (rotated keys rounded once on the host)
    tA = wl.make_tensors(A, device="cuda:0", seed=31)
    kA, vA, _ = gu.host_assembled_pools(A, tA)
    tR = dataclasses.replace(tA, k_pool=kA, v_pool=vA)
    r = gu.run_layer(R, t=dataclasses.replace(tR, k_pool=kA.clone(), v_pool=vA.clone()), poison=False, attention=False)
    gu.check_placement(r)
    asm_r, kmx, kmean = gu.check_assembled(r)
    gu.check_untouched(r)
    assert set(asm_r[0].delta.tolist()) == set(range(-(237 + 149), -236))
    # the retained keys are the fresh keys un-rotated: compare with the oracle applied to k_new of A
    j0 = int(np.searchsorted(A.recompute_pos, 237))
    fresh = orc.bf16_bits_to_f64(orc.bits(tA.k_new)[j0:j0 + 150])
    for i in (0, 63, 149):
        want = np.stack([orc.rope_rotate(fresh[i, h], -(237 + i), 500000.0) for h in range(8)])
        assert np.max(np.abs(want - asm_r[0].k[i])) < 1e-9
    # reuse the retained unit (as the oracle retained it, rounded on the host) in another prompt
    kR, vR, _ = gu.host_assembled_pools(R, tR)
    b = gu.run_layer(B, t=dataclasses.replace(tR, k_pool=kR, v_pool=vR), poison=False)
    assert b.status == 0
    gu.check_placement(b)
    asm_b, _, _ = gu.check_assembled(b)
    gu.check_attention(b, asm_b)


def test_split_kv_single_request_with_wide_tiles():
    """A lone long request is split along the key axis into parts merged afterwards; tiles whose rows
    are far apart have rows that see no key at all in the later parts."""
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    rng = np.random.default_rng(5)
    segs = [7] + [wl.unit(700, ("u", i), recompute=(0, 1, 2, 350)) for i in range(6)] + [40]
    w = wl.build_workload("split", shape, [segs], rng)
    g = gu.run_layer(w, seed=77)
    assert g.status == 0
    asm, _, _ = gu.check_assembled(g)
    gu.check_attention(g, asm)
    gu.check_attention_alone(w, seed=77)
    assert tb.Plan(w, host_only=True).info.n_attn_items > 8 * 2      # the items really were split


def test_bounded_wait_gives_up_and_leaves_the_context_usable():
    """A wait on a barrier that nobody completes must run out, report its code and return: the same
    mechanism guards every mbarrier wait of the attention kernel."""
    st, code, cyc = tb.selftest_bounded_wait(3_000_000)            # about 1.5 ms of SM cycles
    assert st == tb.DEVICE_TIMEOUT and code == 42
    assert 3_000_000 <= cyc[0] < 30_000_000                          # gave up after the limit, not much later
    assert cyc[1] < 100_000 and cyc[2] == 0                          # later waits return at once, none "succeeded"
    g = gu.run_layer(wl.config(1))                                   # the context is still fine
    assert g.status == 0
    gu.check_attention(g, gu.check_assembled(g)[0])


def test_host_tier_compose_reads_a_pinned_host_pool():
    """Local-hit path: the cached units sit in pinned host memory (a separate source pool) and the
    gather kernel reads them over the interconnect; the device copies of the sources are wiped first."""
    import copy
    w = wl.config(3, requests_override=4)
    dev = "cuda:0"
    t = wl.make_tensors(w, device=dev, seed=12)
    host_k, host_v = t.k_pool.cpu().pin_memory(), t.v_pool.cpu().pin_memory()
    w2 = copy.copy(w)
    w2.num_source_pages = w.num_pool_pages
    plan = tb.Plan(w2)
    pv = torch.tensor(gu.POISON, dtype=torch.int16, device=dev).view(torch.bfloat16)
    t.k_pool[:] = pv
    t.v_pool[:] = pv
    with pytest.raises(tb.TesseraError):
        plan.kv_compose(t.k_pool, t.v_pool)                  # such a plan needs the _from entry point
    plan.kv_compose_from(host_k, host_v, t.k_pool, t.v_pool)
    torch.cuda.synchronize()
    g = gu.LayerRun()
    g.w, g.t, g.plan = w, t, plan
    g.page_off, g.pages, g.src_slot = plan.block_table()
    g.k_before, g.v_before = orc.bits(host_k), orc.bits(host_v)
    g.k_after, g.v_after = orc.bits(t.k_pool), orc.bits(t.v_pool)
    g.kn_bits, g.vn_bits = orc.bits(t.k_new), orc.bits(t.v_new)
    gu.check_placement(g)
    asm, kmx, kmean = gu.check_assembled(g, scattered=False)
    # nothing but destination pages was written
    mask = np.ones(w.num_pool_pages, bool)
    mask[g.pages] = False
    assert np.all(g.k_after[mask] == gu.POISON) and np.all(g.v_after[mask] == gu.POISON)
    # and the attention path works on top of it
    out = torch.empty_like(t.q)
    plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, out, None)
    torch.cuda.synchronize()
    g.k_after, g.v_after = orc.bits(t.k_pool), orc.bits(t.v_pool)
    g.q_bits, g.out_f, g.lse_f = orc.bits(t.q), out.float().cpu().numpy().astype(np.float64), None
    asm, _, _ = gu.check_assembled(g)
    gu.check_attention(g, asm)


@pytest.mark.parametrize("hq,hkv", [(16, 8), (16, 1), (2, 2)])
def test_other_group_sizes_on_the_tensor_core_path(hq, hkv):
    """g = 2, 16 and 1 query heads per KV head (tiles of 64, 8 and 128 tokens)."""
    w = wl.adversarial(seed=20 + hq, shape=wl.ModelShape(hq, hkv, 128, 64, 500000.0))
    g, _ = _full_check(w)
    assert g.plan.info.attn_kernel == 1


def test_batches_without_queries_or_without_requests():
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    dev = "cuda:0"
    # every position cached, nothing recomputed: attention is a no-op that still returns OK
    w = wl.build_workload("noq", shape, [[wl.unit(100, "a"), wl.unit(70, "b", cached_pos=5)]], np.random.default_rng(1))
    g = gu.run_layer(w)
    assert g.status == 0 and w.n_q == 0
    gu.check_assembled(g)
    gu.check_untouched(g)
    # empty batch
    w = wl.build_workload("empty", shape, [], np.random.default_rng(1))
    t = wl.make_tensors(w, device=dev)
    plan = tb.Plan(w)
    before = t.k_pool.clone()
    plan.kv_compose(t.k_pool, t.v_pool)
    plan.rope_shift(t.k_pool)
    plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, torch.empty_like(t.q), None)
    plan.composed_prefill_host(t.k_pool, t.v_pool, t.q.cpu(), t.k_new.cpu(), t.v_new.cpu(), t.q.cpu(), None)
    torch.cuda.synchronize()
    assert torch.equal(before, t.k_pool) and plan.status() == 0


@pytest.mark.parametrize("make", [lambda: wl.config(1), lambda: wl.config(3, requests_override=2),
                                  lambda: wl.adversarial(seed=9, shape=wl.ModelShape(32, 8, 128, 64, 500000.0))])
def test_rope_fresh_rotates_queries_and_keys_at_target_positions(make):
    w = make()
    dev = "cuda:0"
    t = wl.make_tensors(w, device=dev, seed=44)
    q0, k0 = orc.bf16_bits_to_f64(orc.bits(t.q)), orc.bf16_bits_to_f64(orc.bits(t.k_new))
    plan = tb.Plan(w)
    plan.rope_fresh(t.q, t.k_new)
    plan.rope_fresh(None, None)                                     # nothing to do is fine
    torch.cuda.synchronize()
    q1, k1 = orc.bf16_bits_to_f64(orc.bits(t.q)), orc.bf16_bits_to_f64(orc.bits(t.k_new))
    theta = w.shape.rope_theta
    rng = np.random.default_rng(0)
    errs = []
    for j in rng.choice(w.n_q, size=min(w.n_q, 40), replace=False):
        p = int(w.recompute_pos[j])
        for h in range(w.shape.num_q_heads):
            errs.append(np.abs(orc.rope_rotate(q0[j, h], p, theta) - q1[j, h]))
        for h in range(w.shape.num_kv_heads):
            errs.append(np.abs(orc.rope_rotate(k0[j, h], p, theta) - k1[j, h]))
    e = np.concatenate(errs)
    assert e.max() <= gu.MAX_ABS and e.mean() <= gu.MEAN_ABS
    # position 0 rows are bit copies
    zero = np.nonzero(w.recompute_pos == 0)[0]
    for j in zero:
        assert np.array_equal(q0[j], q1[j]) and np.array_equal(k0[j], k1[j])


@pytest.mark.parametrize("shape", [wl.ModelShape(8, 2, 64, 16, 10000.0, rope_pairing=1),
                                   wl.ModelShape(32, 8, 128, 64, 500000.0, rope_pairing=1)])
def test_interleaved_rope_pairing(shape):
    """Pairs (2m, 2m + 1) instead of (m, m + D/2): gather + shift, standalone shift and fresh rotation."""
    w = wl.adversarial(seed=31, shape=shape)
    _full_check(w)
    _full_check(w, fuse=False)
    dev = "cuda:0"
    t = wl.make_tensors(w, device=dev, seed=45)
    q0, k0 = orc.bf16_bits_to_f64(orc.bits(t.q)), orc.bf16_bits_to_f64(orc.bits(t.k_new))
    tb.Plan(w).rope_fresh(t.q, t.k_new)
    torch.cuda.synchronize()
    q1, k1 = orc.bf16_bits_to_f64(orc.bits(t.q)), orc.bf16_bits_to_f64(orc.bits(t.k_new))
    errs = []
    for j in range(0, w.n_q, 3):
        p = int(w.recompute_pos[j])
        errs.append(np.abs(orc.rope_rotate(q0[j, 0], p, shape.rope_theta, pairing=1) - q1[j, 0]))
        errs.append(np.abs(orc.rope_rotate(k0[j, 1], p, shape.rope_theta, pairing=1) - k1[j, 1]))
    e = np.concatenate(errs)
    assert e.max() <= gu.MAX_ABS and e.mean() <= gu.MEAN_ABS
    # and it really differs from the half-split result
    wrong = orc.rope_rotate(q0[5, 0], int(w.recompute_pos[5]), shape.rope_theta, pairing=0)
    assert np.abs(wrong - q1[5, 0]).max() > 0.1 or int(w.recompute_pos[5]) == 0


@pytest.mark.parametrize("shape", [wl.ModelShape(4, 4, 64, 8, 10000.0), wl.ModelShape(16, 1, 64, 128, 10000.0),
                                   wl.ModelShape(8, 4, 128, 32, 500000.0), wl.ModelShape(32, 8, 128, 64, 500000.0)])
def test_degenerate_layouts(shape):
    """One-token requests, one-token units, a unit that exactly fills a page, a request made of a single
    recomputed token, page sizes 8 / 32 / 64 / 128."""
    B = shape.page_size
    reqs = [[1],                                                        # a single fresh token
            [wl.unit(1, "one", cached_pos=3), 1],                       # one cached token + one fresh
            [wl.unit(B, "page", recompute=(0,)), wl.unit(B, "page2", cached_pos=7, recompute=(B - 1,)), 1],
            [2, wl.unit(2 * B + 1, "long", cached_pos=1, stride=0, recompute=(0, 2 * B)), 1]]
    w = wl.build_workload("degenerate", shape, reqs, np.random.default_rng(3))
    _full_check(w)


def test_sharp_softmax_with_frequent_reference_refresh():
    """Large logits (queries scaled by 6): the reference maximum is overtaken again and again, so the
    refresh path (true maximum, accumulator rescale in TMEM, probabilities redone) runs often."""
    w = wl.config(3, requests_override=3)
    t = wl.make_tensors(w, device="cuda:0", seed=61)
    t.q.mul_(6.0)
    g = gu.run_layer(w, t=t)
    assert g.status == 0
    gu.check_assembled(g)
    # with logits this large the single bf16 rounding of a rotated key moves a logit by up to
    # |q| * 2^-9 * sqrt(D), so the meaningful comparison is the kernel on keys stored exactly as the
    # oracle sees them (assembled and rounded on the host)
    assert np.isfinite(g.lse_f).all() and np.abs(g.out_f).max() < 8.0
    shape = w.shape
    t2 = wl.make_tensors(w, device="cuda:0", seed=61)
    t2.q.mul_(6.0)
    k_pool, v_pool, stored = gu.host_assembled_pools(w, t2)
    plan = tb.Plan(w)
    out = torch.zeros_like(t2.q)
    plan.partial_prefill_attn(k_pool, v_pool, t2.q, None, None, out, None)
    torch.cuda.synchronize()
    out_f = out.float().cpu().numpy().astype(np.float64)
    errs = []
    for r, (k, v_bits) in stored.items():
        jj, hh, pp = orc.request_rows(w, r)
        o, _ = orc.attention_rows(w, k, v_bits, orc.bits(t2.q), jj, hh, pp)
        errs.append(np.abs(out_f[jj, hh] - o).ravel())
    e = np.concatenate(errs)
    assert e.max() <= gu.MAX_ABS and e.mean() <= gu.MEAN_ABS


@pytest.mark.parametrize("page", [8, 16, 32, 128])
def test_tensor_core_path_with_other_page_sizes(page):
    """A 128-key step is 16, 8, 4 or 1 pages instead of 2."""
    shape = wl.ModelShape(32, 8, 128, page, 500000.0)
    g, _ = _full_check(wl.adversarial(seed=40 + page, shape=shape))
    assert g.plan.info.attn_kernel == 1
    w = wl.build_workload("long", shape, [[9, wl.unit(900, "a", recompute=(0, 1, 450)), wl.unit(333, "b", cached_pos=4), 17],
                                          [wl.unit(333, "b", cached_pos=4, recompute=(5,)), 3]], np.random.default_rng(page))
    _full_check(w)


def test_residency_decided_by_the_reuse_score_policy():
    """Config 3 with hits and misses chosen by the score-based admission rule: missed records are
    recomputed in full inside the same extend pass."""
    w = wl.config(3, requests_override=3, policy="reuse")
    _full_check(w)


@pytest.mark.parametrize("hq,hkv,D", [(40, 8, 128), (24, 8, 128), (28, 4, 128), (12, 2, 64)])
def test_group_sizes_that_do_not_divide_the_tile(hq, hkv, D):
    """g = 5, 3, 7, 6 query heads per KV head (Qwen-style head counts): a tile holds floor(128 / g)
    tokens and the remaining MMA rows are zero padding."""
    shape = wl.ModelShape(hq, hkv, D, 64 if D == 128 else 16, 500000.0)
    g, _ = _full_check(wl.adversarial(seed=50 + hq, shape=shape))
    assert g.plan.info.attn_kernel == 1
    w = wl.build_workload("mid", shape, [[3, wl.unit(700, "a", recompute=range(9)), wl.unit(300, "b", cached=False), 41]],
                          np.random.default_rng(hq))
    _full_check(w)


def test_output_buffer_aligned_to_16_bytes_only():
    """`out` need only be 16-byte aligned: the kernel's 32-byte stores fall back to 16-byte ones and
    the result is the same, bit for bit."""
    w = wl.config(2)
    t = wl.make_tensors(w, device="cuda:0", seed=3)
    plan = tb.Plan(w)
    plan.kv_compose(t.k_pool, t.v_pool)
    sh = w.shape
    n = w.n_q * sh.num_q_heads * sh.head_dim
    ref = torch.zeros(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device="cuda:0")
    raw = torch.zeros(n + 8, dtype=torch.bfloat16, device="cuda:0")
    off = raw[8:].view(w.n_q, sh.num_q_heads, sh.head_dim)
    assert ref.data_ptr() % 32 == 0 and off.data_ptr() % 32 == 16
    plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, ref, None)
    plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new, t.v_new, off, None)
    torch.cuda.synchronize()
    assert plan.status() == 0
    assert torch.equal(ref, off) and float(ref.float().abs().sum()) > 0
    # a non-split batch takes the direct epilogue (config 2 is split along the keys and merged afterwards)
    w3 = wl.config(3, requests_override=4)
    t3 = wl.make_tensors(w3, device="cuda:0", seed=4)
    p3 = tb.Plan(w3)
    p3.kv_compose(t3.k_pool, t3.v_pool)
    sh3 = w3.shape
    ref3 = torch.zeros(w3.n_q, sh3.num_q_heads, sh3.head_dim, dtype=torch.bfloat16, device="cuda:0")
    raw3 = torch.zeros(ref3.numel() + 8, dtype=torch.bfloat16, device="cuda:0")
    off3 = raw3[8:].view_as(ref3)
    p3.partial_prefill_attn(t3.k_pool, t3.v_pool, t3.q, t3.k_new, t3.v_new, ref3, None)
    p3.partial_prefill_attn(t3.k_pool, t3.v_pool, t3.q, t3.k_new, t3.v_new, off3, None)
    torch.cuda.synchronize()
    assert p3.status() == 0 and off3.data_ptr() % 32 == 16
    assert torch.equal(ref3, off3) and float(ref3.float().abs().sum()) > 0


def test_many_uneven_items_per_thread_block():
    """The persistent attention kernel walks many items per thread block: 240 short requests with one,
    two or three query tiles (so single-tile items are mixed in), tiles of different lengths and keys
    from 60 to 1 000 - every barrier phase carries over from item to item."""
    shape = wl.ModelShape(32, 8, 128, 64, 500000.0)
    rng = np.random.default_rng(123)
    reqs = []
    for r in range(240):
        ctx = int(rng.integers(50, 900))
        tail = int(rng.integers(1, 70))
        reqs.append([int(rng.integers(0, 4)), wl.unit(ctx, ("u", r), recompute=(0, 1, ctx // 2)), tail])
    w = wl.build_workload("many", shape, reqs, rng)
    plan = tb.Plan(w, host_only=True)
    assert plan.info.attn_kernel == 1 and plan.info.n_attn_items > 148 * 10
    g = gu.run_layer(w, seed=99)
    assert g.status == 0
    gu.check_placement(g)
    asm, _, _ = gu.check_assembled(g)
    gu.check_untouched(g)
    gu.check_attention(g, asm)
