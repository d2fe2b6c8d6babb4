"""Shared driver of the GPU parity tests: run the library on a workload, run the oracle on the
very same bytes, compare element by element."""
from __future__ import annotations

import numpy as np
import torch

from oracle import tessera_oracle as orc
from paper_2609_32999_b200 import binding as tb
from paper_2609_32999_b200 import workloads as wl

MAX_ABS, MEAN_ABS = 2e-2, 2e-3          # tolerance of bf16 attention outputs and re-rotated keys
POISON = 0x7FC1                         # a NaN pattern no kernel produces


class LayerRun:
    pass


def run_layer(w, t=None, fuse=True, layer=0, seed=None, poison=True, with_lse=True, plan=None,
              attention=True, scatter=True):
    """Runs compose (+ shift) (+ attention) through the C ABI on cuda:0.  Returns an object holding
    the pools before (host bits) and after (host bits), out, lse and the plan's tables."""
    dev = "cuda:0"
    if t is None:
        t = wl.make_tensors(w, layer=layer, device=dev, seed=seed)
    own_plan = plan is None
    plan = plan or tb.Plan(w)
    page_off, pages, src_slot = plan.block_table()
    if poison and len(pages):
        idx = torch.from_numpy(pages.astype(np.int64)).to(dev)
        pv = torch.tensor(POISON, dtype=torch.int16, device=dev).view(torch.bfloat16)
        t.k_pool[idx] = pv
        t.v_pool[idx] = pv
    g = LayerRun()
    g.w, g.t, g.plan = w, t, plan
    g.page_off, g.pages, g.src_slot = page_off, pages, src_slot
    g.k_before, g.v_before = orc.bits(t.k_pool).copy(), orc.bits(t.v_pool).copy()
    if fuse:
        plan.kv_compose(t.k_pool, t.v_pool, fuse_rope=True)
    else:
        plan.kv_compose(t.k_pool, t.v_pool, fuse_rope=False)
        plan.rope_shift(t.k_pool)
    sh = w.shape
    g.out = torch.zeros(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=dev)
    g.lse = torch.zeros(w.n_q, sh.num_q_heads, dtype=torch.float32, device=dev) if with_lse else None
    if attention:
        plan.partial_prefill_attn(t.k_pool, t.v_pool, t.q, t.k_new if scatter else None,
                                  t.v_new if scatter else None, g.out, g.lse)
    torch.cuda.synchronize()
    g.status = plan.status()
    g.k_after, g.v_after = orc.bits(t.k_pool), orc.bits(t.v_pool)
    g.q_bits, g.kn_bits, g.vn_bits = orc.bits(t.q), orc.bits(t.k_new), orc.bits(t.v_new)
    g.out_f = g.out.float().cpu().numpy().astype(np.float64)
    g.lse_f = g.lse.cpu().numpy().astype(np.float64) if with_lse else None
    g.own_plan = own_plan
    return g


def dest_slots(g, r):
    B = g.w.shape.page_size
    T = int(g.w.seq_len[r])
    p = np.arange(T)
    return g.pages[g.page_off[r] + p // B].astype(np.int64) * B + p % B


def check_placement(g):
    st, o_off, o_pages, o_src, _ = orc.placement(g.w)
    assert st == 0
    assert np.array_equal(g.page_off, o_off) and np.array_equal(g.pages, o_pages)
    assert np.array_equal(g.src_slot, o_src)


def check_assembled(g, requests=None, scattered=True):
    """Destination pages vs the oracle's assembled KV.  Returns (assembled list, max, mean) where
    max / mean are over all rotated key elements.  g.src_fmt = 1 (with g.k_scale / g.v_scale): the
    sources in g.k_before / g.v_before are e4m3 codes of an 8-bit pool."""
    w = g.w
    sh = w.shape
    row = sh.num_kv_heads * sh.head_dim
    ka = g.k_after.reshape(-1, row)
    va = g.v_after.reshape(-1, row)
    asm = {}
    errs = []
    for r in (range(w.batch) if requests is None else requests):
        a = orc.assemble(w, r, g.k_before, g.v_before, g.kn_bits, g.vn_bits, src_fmt=getattr(g, "src_fmt", 0),
                         k_scale=getattr(g, "k_scale", 1.0), v_scale=getattr(g, "v_scale", 1.0),
                         fresh_k_raw=getattr(g, "fresh_k_raw", False))
        asm[r] = a
        T = int(w.seq_len[r])
        if T == 0:
            continue
        slots = dest_slots(g, r)
        gv, gk = va[slots], ka[slots]
        if not scattered:      # only cached rows are comparable when the fresh rows were not written
            keep = np.ones(T, bool)
            keep[w.recompute_pos[w.recompute_off[r]:w.recompute_off[r + 1]]] = False
            tok0 = int(np.sum(w.seq_len[:r]))
            keep &= g.src_slot[tok0:tok0 + T] >= 0
        else:
            keep = np.ones(T, bool)
        ex = (a.k_exact != 0) & keep
        if getattr(g, "src_fmt", 0) == 1:
            # 8-bit sources: the oracle rounds the exact product code * scale once; the library rounds
            # the fp32 product.  The two agree bit for bit when the scale is a power of two (the product
            # is then exact in fp32); otherwise they may differ by one bf16 step at a double-rounding tie.
            cached_rows = keep & (g.src_slot[int(np.sum(w.seq_len[:r])):int(np.sum(w.seq_len[:r])) + T] >= 0)
            fresh_rows = keep & ~cached_rows
            assert np.array_equal(gv[fresh_rows], a.v_bits.reshape(T, row)[fresh_rows])
            _expanded_rows_equal(g, gv[cached_rows], a.v_bits.reshape(T, row)[cached_rows], g.v_scale, "V (request %d)" % r)
            _expanded_rows_equal(g, gk[ex & cached_rows], a.k_bits.reshape(T, row)[ex & cached_rows], g.k_scale, "K (request %d)" % r)
            assert np.array_equal(gk[ex & fresh_rows], a.k_bits.reshape(T, row)[ex & fresh_rows])
        else:
            assert np.array_equal(gv[keep], a.v_bits.reshape(T, row)[keep]), "V rows must be bit copies (request %d)" % r
            assert np.array_equal(gk[ex], a.k_bits.reshape(T, row)[ex]), "exact K rows differ (request %d)" % r
        rot = (a.k_exact == 0) & keep
        if rot.any():
            d = np.abs(orc.bf16_bits_to_f64(gk[rot]) - a.k.reshape(T, row)[rot])
            errs.append(d.ravel())
    if errs:
        e = np.concatenate(errs)
        mx, mean = float(e.max()), float(e.mean())
        assert mx <= MAX_ABS, "rotated keys: max-abs %.4g" % mx
        assert mean <= MEAN_ABS, "rotated keys: mean-abs %.4g" % mean
    else:
        mx = mean = 0.0
    return asm, mx, mean


def _is_pow2(x: float) -> bool:
    m, _ = np.frexp(np.float32(x))
    return float(m) == 0.5


def _expanded_rows_equal(g, got, want, scale, what):
    """Rows expanded from 8-bit codes: bit-exact for a power-of-two scale; otherwise any difference must
    be one bf16 step (the fp32 product landed on a tie the exact product is not on) and rare.  Counts
    are accumulated in g.double_rounding = [differing elements, compared elements]."""
    if not hasattr(g, "double_rounding"):
        g.double_rounding = [0, 0]
    g.double_rounding[1] += int(got.size)
    if _is_pow2(scale):
        assert np.array_equal(got, want), "expanded %s rows must be exact for a power-of-two scale" % what
        return
    diff = got != want
    n = int(diff.sum())
    g.double_rounding[0] += n
    if n:
        step = np.abs(got[diff].astype(np.int32) - want[diff].astype(np.int32))
        assert step.max() == 1, "expanded %s rows differ by more than one bf16 step" % what
        assert n <= 1e-3 * got.size + 2, "expanded %s rows: %d of %d elements differ" % (what, n, got.size)


def check_untouched(g):
    """Every page that is not a destination page keeps its bits (sources and canaries)."""
    w = g.w
    mask = np.ones(w.num_pool_pages, bool)
    mask[g.pages] = False
    assert np.array_equal(g.k_after[mask], g.k_before[mask]), "a non-destination K page changed"
    assert np.array_equal(g.v_after[mask], g.v_before[mask]), "a non-destination V page changed"


def check_attention(g, asm, rows_by_request=None):
    """Attention outputs of the whole path vs the oracle, which attends over its own unrounded fp64
    keys.  rows_by_request: {r: (row_q, row_h, row_pos)} or None for every row."""
    w = g.w
    sh = w.shape
    row = sh.num_kv_heads * sh.head_dim
    all_err, all_lse = [], []
    for r, a in asm.items():
        if rows_by_request is None:
            jj, hh, pp = orc.request_rows(w, r)
        else:
            jj, hh, pp = rows_by_request[r]
        if len(jj) == 0:
            continue
        k = a.k
        o, l = orc.attention_rows(w, k, a.v_bits, g.q_bits, jj, hh, pp)
        all_err.append(np.abs(g.out_f[jj, hh] - o).ravel())
        if g.lse_f is not None:
            all_lse.append(np.abs(g.lse_f[jj, hh] - l))
    e = np.concatenate(all_err)
    mx, mean = float(e.max()), float(e.mean())
    assert np.isfinite(e).all(), "non-finite attention output"
    assert mx <= MAX_ABS, "attention: max-abs %.4g" % mx
    assert mean <= MEAN_ABS, "attention: mean-abs %.4g" % mean
    if all_lse:
        le = float(np.concatenate(all_lse).max())
        assert le <= 2e-2, "LSE: max-abs %.4g" % le
    return mx, mean


def sample_rows(w, r, rng, n_random, tile_tokens):
    """First and last q tile of request r plus n_random random (row, head) pairs."""
    j0, j1 = int(w.recompute_off[r]), int(w.recompute_off[r + 1])
    H = w.shape.num_q_heads
    js = list(range(j0, min(j0 + tile_tokens, j1))) + list(range(max(j1 - tile_tokens, j0), j1))
    jj = np.repeat(np.array(js, np.int32), H)
    hh = np.tile(np.arange(H, dtype=np.int32), len(js))
    if n_random and j1 > j0:
        rj = rng.integers(j0, j1, size=n_random).astype(np.int32)
        rh = rng.integers(0, H, size=n_random).astype(np.int32)
        jj, hh = np.concatenate([jj, rj]), np.concatenate([hh, rh])
    return jj, hh, w.recompute_pos[jj].astype(np.int32)


def host_assembled_pools(w, t):
    """The state of the pools after gather + shift + scatter as the ORACLE computes it, with rotated keys
    rounded to bf16 on the host: destination pages filled from oracle.assemble, everything else left
    as generated.  Returns (k_pool, v_pool) device tensors and {request: fp64 K actually stored}."""
    sh = w.shape
    row = sh.num_kv_heads * sh.head_dim
    kb, vb, knb, vnb = (orc.bits(x) for x in (t.k_pool, t.v_pool, t.k_new, t.v_new))
    st, page_off, pages, _, _ = orc.placement(w)
    assert st == 0
    k_img, v_img = kb.copy().reshape(-1, row), vb.copy().reshape(-1, row)
    stored = {}
    B = sh.page_size
    for r in range(w.batch):
        a = orc.assemble(w, r, kb, vb, knb, vnb)
        T = int(w.seq_len[r])
        if T == 0:
            continue
        p = np.arange(T)
        slots = pages[page_off[r] + p // B].astype(np.int64) * B + p % B
        k_round = torch.from_numpy(a.k.reshape(T, row)).to(torch.bfloat16)          # one rounding, on the host
        k_bits = k_round.view(torch.int16).numpy().view(np.uint16).copy()
        ex = a.k_exact != 0
        k_bits[ex] = a.k_bits.reshape(T, row)[ex]                                    # bit copies stay bit copies
        k_img[slots] = k_bits
        v_img[slots] = a.v_bits.reshape(T, row)
        stored[r] = (orc.bf16_bits_to_f64(k_bits).reshape(a.k.shape), a.v_bits)
    dev = t.k_pool.device
    to_dev = lambda img: torch.from_numpy(img.view(np.int16).reshape(kb.shape)).view(torch.bfloat16).to(dev)
    return to_dev(k_img), to_dev(v_img), stored


def check_attention_alone(w, seed=None, layer=0):
    """The attention kernel by itself: pages assembled by the oracle on the host (rotated keys rounded
    once to bf16), attention on the GPU without any gather or scatter, compared with the oracle
    attending over exactly those stored keys."""
    dev = "cuda:0"
    t = wl.make_tensors(w, layer=layer, device=dev, seed=seed)
    k_pool, v_pool, stored = host_assembled_pools(w, t)
    plan = tb.Plan(w)
    sh = w.shape
    out = torch.zeros(w.n_q, sh.num_q_heads, sh.head_dim, dtype=torch.bfloat16, device=dev)
    lse = torch.zeros(w.n_q, sh.num_q_heads, dtype=torch.float32, device=dev)
    plan.partial_prefill_attn(k_pool, v_pool, t.q, None, None, out, lse)
    torch.cuda.synchronize()
    assert plan.status() == 0
    out_f = out.float().cpu().numpy().astype(np.float64)
    lse_f = lse.cpu().numpy().astype(np.float64)
    q_bits = orc.bits(t.q)
    errs, lerr = [], []
    for r, (k, v_bits) in stored.items():
        jj, hh, pp = orc.request_rows(w, r)
        if len(jj) == 0:
            continue
        o, l = orc.attention_rows(w, k, v_bits, q_bits, jj, hh, pp)
        errs.append(np.abs(out_f[jj, hh] - o).ravel())
        lerr.append(np.abs(lse_f[jj, hh] - l))
    if not errs:
        return 0.0, 0.0
    e = np.concatenate(errs)
    assert np.isfinite(e).all()
    assert e.max() <= MAX_ABS and e.mean() <= MEAN_ABS, "attention alone: max %.4g mean %.4g" % (e.max(), e.mean())
    assert np.concatenate(lerr).max() <= 5e-3, "attention alone: LSE max-abs %.4g" % np.concatenate(lerr).max()
    return float(e.max()), float(e.mean())
