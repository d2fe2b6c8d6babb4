"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each one is chosen so that a
plausible slip in the oracle (wrong sign, wrong pairing, wrong frequency, an
off-by-one in the causal limit, a transposed head mapping, a wrong slot) fails it.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import tessera_oracle as orc
from paper_2609_32999_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------- RoPE

@pytest.mark.parametrize("D,theta", [(64, 1e4), (128, 5e5), (8, 100.0)])
def test_rope_composition(D, theta):
    """R(d) R(p) k == R(p + d) k, including negative d and d == 0."""
    rng = np.random.default_rng(1)
    for p, d in [(0, 17), (100, -100), (150, -100), (31999, 1025), (12, 0), (7, -7), (5, -9)]:
        k = rng.standard_normal(D)
        a = orc.rope_rotate(orc.rope_rotate(k, p, theta), d, theta)
        b = orc.rope_rotate(k, p + d, theta)
        assert np.max(np.abs(a - b)) < 1e-10
    k = rng.standard_normal(D)
    assert np.array_equal(orc.rope_rotate(k, 0, theta), k)


def test_rope_relative_position_invariance():
    """<R(m) q, R(n) k> == <q, R(n - m) k>."""
    rng = np.random.default_rng(2)
    D, theta = 128, 5e5
    for m, n in [(3, 10), (1000, 4), (0, 0), (511, 33023)]:
        q, k = rng.standard_normal(D), rng.standard_normal(D)
        lhs = orc.rope_rotate(q, m, theta) @ orc.rope_rotate(k, n, theta)
        rhs = q @ orc.rope_rotate(k, n - m, theta)
        assert abs(lhs - rhs) < 1e-9


def test_rope_one_hot_closed_form():
    """k = e_m (first half) -> cos(p w_m) at m, +sin(p w_m) at m + D/2, zero elsewhere;
    k = e_{m + D/2} -> -sin at m, cos at m + D/2.  Fixes direction, pairing, frequency."""
    D, theta, p = 16, 10000.0, 5
    for m in range(D // 2):
        w = 1.0 / (theta ** (2.0 * m / D))
        e = np.zeros(D); e[m] = 1.0
        r = orc.rope_rotate(e, p, theta)
        exp = np.zeros(D); exp[m] = math.cos(p * w); exp[m + D // 2] = math.sin(p * w)
        assert np.allclose(r, exp, atol=1e-14)
        e = np.zeros(D); e[m + D // 2] = 1.0
        r = orc.rope_rotate(e, p, theta)
        exp = np.zeros(D); exp[m] = -math.sin(p * w); exp[m + D // 2] = math.cos(p * w)
        assert np.allclose(r, exp, atol=1e-14)
    # the first pair turns by exactly p radians (w_0 = 1), the last by p * theta^-(D-2)/D
    e = np.zeros(D); e[0] = 1.0
    assert abs(orc.rope_rotate(e, 1, theta)[D // 2] - math.sin(1.0)) < 1e-15


def test_rope_2d_is_rotation_matrix():
    """D = 2: a single pair with w = 1 -> the 2-D counter-clockwise rotation matrix."""
    for ang in [0.3, -1.2, 2.0]:
        R = np.array([[math.cos(ang), -math.sin(ang)], [math.sin(ang), math.cos(ang)]])
        v = np.array([0.7, -1.9])
        assert np.allclose(orc.rope_rotate(v, ang, 12345.0), R @ v, atol=1e-15)


def test_rope_preserves_pair_norms():
    rng = np.random.default_rng(3)
    D = 64
    k = rng.standard_normal(D)
    r = orc.rope_rotate(k, 977, 1e4)
    assert np.allclose(k[:32] ** 2 + k[32:] ** 2, r[:32] ** 2 + r[32:] ** 2, atol=1e-12)


def test_rope_matches_library_rotary():
    """Same numbers as the rotary routine of the model family the paper serves
    (half-split pairing, rotate_half convention), evaluated in fp64."""
    from transformers.models.llama.modeling_llama import apply_rotary_pos_emb
    D, theta = 128, 5e5
    rng = np.random.default_rng(4)
    x = rng.standard_normal((1, 1, 6, D))                       # [batch, heads, seq, D]
    pos = np.array([0, 1, 17, 511, 4096, 33023], dtype=np.float64)
    inv = 1.0 / (theta ** (np.arange(0, D, 2, dtype=np.float64) / D))
    fr = np.outer(pos, inv)
    emb = np.concatenate([fr, fr], axis=-1)
    cos, sin = torch.from_numpy(np.cos(emb))[None], torch.from_numpy(np.sin(emb))[None]
    xt = torch.from_numpy(x)
    q_emb, _ = apply_rotary_pos_emb(xt, xt, cos, sin)
    for i, p in enumerate(pos):
        ours = orc.rope_rotate(x[0, 0, i], p, theta)
        assert np.max(np.abs(ours - q_emb[0, 0, i].numpy())) < 1e-10   # angle ulp at 3e4 rad


def test_rope_explicit_inv_freq_and_interleaved():
    D, theta = 32, 1e4
    rng = np.random.default_rng(5)
    k = rng.standard_normal(D)
    inv = theta ** (-2.0 * np.arange(D // 2) / D)
    assert np.allclose(orc.rope_rotate(k, 9, theta), orc.rope_rotate(k, 9, 1.0, inv_freq=inv), atol=1e-14)
    # interleaved pairing is the half-split rotation on a permuted vector
    perm = np.concatenate([np.arange(0, D, 2), np.arange(1, D, 2)])
    a = orc.rope_rotate(k, 9, theta, pairing=1)
    b = orc.rope_rotate(k[perm], 9, theta, pairing=0)
    assert np.allclose(a[perm], b, atol=1e-14)


def test_paper_position_example_negative_shift():
    """Sec. 2.2's example: a document cached at 150-249 reused at 50-149 needs a
    shift of -100 on every key; shifting equals rotating the raw key at the target."""
    row = [l for l in open(os.path.join(GOLDEN, "fig1_doc_b_positions.txt")) if not l.startswith("#")][0]
    c0, c1, t0, t1 = map(int, row.split())
    assert c1 - c0 == t1 - t0 == 99 and t0 - c0 == -100
    shape = wl.ModelShape(2, 1, 16, 16, 10000.0)
    rng = np.random.default_rng(6)
    w = wl.build_workload("docB", shape,
                          [[t0, wl.unit(c1 - c0 + 1, "B", cached_pos=c0), 3]], rng)
    t = wl.make_tensors(w)
    kp = orc.bits(t.k_pool).copy()
    a0 = orc.assemble(w, 0, kp, orc.bits(t.v_pool), orc.bits(t.k_new), orc.bits(t.v_new))
    assert set(a0.delta[t0:t1 + 1]) == {-100}
    # independent check of the values: unrotate pool content by its cached position, rotate at target
    st, page_off, pages, src_slot, fresh = orc.placement(w)
    assert st == 0
    pool = orc.bf16_bits_to_f64(kp).reshape(-1, 1, 16)
    for p in (t0, t0 + 37, t1):
        i = p - t0
        cached = pool[src_slot[p], 0]
        raw_key = orc.rope_rotate(cached, -(c0 + i), 10000.0)
        direct = orc.rope_rotate(raw_key, p, 10000.0)
        assert np.max(np.abs(direct - a0.k[p, 0])) < 1e-10


def test_fresh_keys_handed_over_unrotated_are_rotated_for_their_positions():
    """Sec. 6.1: the forward path captures pre-RoPE keys; Sec. 5.3: the request itself sees them rotated
    for their positions.  With fresh_k_raw the oracle's assembled key at a recomputed position p must be
    the library rotary routine applied to the raw key at position p (every head), a bit copy at p = 0,
    and cached rows must not change."""
    from transformers.models.llama.modeling_llama import apply_rotary_pos_emb
    shape = wl.ModelShape(4, 2, 32, 8, 10000.0)
    w = wl.build_workload("raw", shape, [[3, wl.unit(20, "a", cached_pos=4, recompute=(0, 7)), wl.unit(9, "b", cached=False), 2]],
                          np.random.default_rng(4))
    t = wl.make_tensors(w, seed=6)
    kb, vb, knb, vnb = (orc.bits(x) for x in (t.k_pool, t.v_pool, t.k_new, t.v_new))
    plain = orc.assemble(w, 0, kb, vb, knb, vnb)
    raw = orc.assemble(w, 0, kb, vb, knb, vnb, fresh_k_raw=True)
    D, theta = 32, 10000.0
    inv = 1.0 / (theta ** (np.arange(0, D, 2, dtype=np.float64) / D))
    k_new = orc.bf16_bits_to_f64(knb)                                        # [n_q, H_kv, D]
    fresh = np.zeros(int(w.seq_len[0]), bool)
    for j, p in enumerate(w.recompute_pos.tolist()):
        fresh[p] = True
        emb = np.concatenate([p * inv, p * inv])[None, None, None]
        cos, sin = torch.from_numpy(np.cos(emb)), torch.from_numpy(np.sin(emb))
        x = torch.from_numpy(k_new[j][None, :, None, :])                      # [1, heads, 1, D]
        want, _ = apply_rotary_pos_emb(x, x, cos[0], sin[0])
        assert np.max(np.abs(want[0, :, 0].numpy() - raw.k[p])) < 1e-12, p
        assert raw.delta[p] == p and raw.k_exact[p] == (1 if p == 0 else 0)
        assert np.array_equal(raw.v_bits[p], vnb[j])
    assert fresh[0] and np.array_equal(raw.k[0], k_new[0])                    # position 0: untouched
    assert np.array_equal(raw.k[~fresh], plain.k[~fresh]) and np.array_equal(raw.v_bits, plain.v_bits)
    assert np.abs(raw.k[fresh][1:] - plain.k[fresh][1:]).max() > 0.1          # and it really differs from the rotated-input reading


# ---------------------------------------------------------------------- placement

def _placement_by_hand(w):
    """Per-token restatement used only here: walk every unit token by token."""
    B = w.shape.page_size
    src = []
    for r in range(w.batch):
        s = [-1] * int(w.seq_len[r])
        for u in range(w.unit_off[r], w.unit_off[r + 1]):
            pg = w.unit_pages[w.unit_page_off[u]:w.unit_page_off[u + 1]]
            if len(pg) == 0:
                continue
            for i in range(w.unit_len[u]):
                page, off = divmod(i, B)
                s[w.unit_target_pos[u] + i] = int(pg[page]) * B + off
        src.extend(s)
    return np.array(src, np.int32)


@pytest.mark.parametrize("make", [lambda: wl.config(1), lambda: wl.config(2), lambda: wl.adversarial(),
                                  lambda: wl.config(3, requests_override=3)])
def test_placement(make):
    w = make()
    st, page_off, pages, src_slot, fresh = orc.placement(w)
    assert st == 0
    B = w.shape.page_size
    need = [-(-int(t) // B) for t in w.seq_len]
    assert list(np.diff(page_off)) == need
    assert np.array_equal(pages, w.free_pages[: sum(need)])          # consumed in order
    assert np.array_equal(src_slot, _placement_by_hand(w))
    # every position has exactly one supplier class and recompute indices are a bijection
    assert np.all((src_slot >= 0) | (fresh >= 0))
    assert sorted(fresh[fresh >= 0]) == list(range(w.n_q))
    # destination pages never alias source pages
    assert not (set(pages.tolist()) & set(w.unit_pages.tolist()))


def _read_placement_golden():
    """Parses tests/golden/placement_slots.txt into a list of (name, Workload, expected dict)."""
    cases, cur = [], None
    for line in open(os.path.join(GOLDEN, "placement_slots.txt")):
        line = line.split("#")[0].strip()
        if not line:
            continue
        key, *rest = line.split()
        if key == "case":
            cur = {"name": rest[0], "units": []}
            cases.append(cur)
        elif key == "unit":
            k = rest.index("pages")
            cur["units"].append(([int(x) for x in rest[:k]], [int(x) for x in rest[k + 1:]]))
        else:
            cur[key] = [int(x) for x in rest]
    out = []
    i32 = lambda x: np.asarray(x, np.int32)
    for c in cases:
        B = c["B"][0]
        shape = wl.ModelShape(4, 2, 64, B, 1e4)
        ulen = [u[0][0] for u in c["units"]]
        pages = [p for u in c["units"] for p in u[1]]
        poff = np.cumsum([0] + [len(u[1]) for u in c["units"]])
        w = wl.Workload(name=c["name"], shape=shape, seq_len=i32(c["seq_len"]), unit_off=i32([0, len(ulen)]),
                        unit_len=i32(ulen), unit_cached_pos=i32([0] * len(ulen)), unit_cached_stride=i32([1] * len(ulen)),
                        unit_target_pos=i32([u[0][1] for u in c["units"]]), unit_page_off=i32(poff), unit_pages=i32(pages),
                        recompute_off=i32([0, len(c["recompute"])]), recompute_pos=i32(c["recompute"]),
                        free_pages=i32(c["free"]), num_pool_pages=max(pages + c["free"]) + 1,
                        unit_src_offset=i32([u[0][2] for u in c["units"]]))
        out.append((c["name"], w, c))
    return out


def test_placement_against_hand_written_golden():
    """Literal slot numbers worked out by hand (tests/golden/placement_slots.txt), with and without a
    source offset: the oracle's slot arithmetic against something that is not its own formula."""
    cases = _read_placement_golden()
    assert len(cases) >= 4
    for name, w, c in cases:
        st, page_off, pages, src, fresh = orc.placement(w)
        assert st == 0, name
        assert pages.tolist() == c["block_table"], name
        assert src.tolist() == c["src_slot"], name
        B = w.shape.page_size
        dst = [int(pages[p // B]) * B + p % B for p in range(int(w.seq_len[0]))]
        assert dst == c["dst_slot"], name
        assert [p for p in range(len(fresh)) if fresh[p] >= 0] == c["recompute"], name


def test_retained_form_is_the_unrotated_key():
    """Store side (Sec. 5.3: the miss prefill keeps an unrotated copy for the cache; Sec. 6.1: pre-RoPE
    keys are captured).  A unit whose keys sit in a request's pages rotated at positions p0 + i, retained
    with target stride 0 at target position 0, must come out as R(-(p0 + i)) applied to each stored key,
    i.e. as the key before any rotation: assembling it and rotating back by +(p0 + i) returns the stored
    key, and the per-token shifts are exactly -(p0 + i)."""
    shape = wl.ModelShape(4, 2, 16, 4, 100.0)
    i32 = lambda x: np.asarray(x, np.int32)
    p0, n = 6, 7                                                     # unit at positions 6..12 of the request
    w = wl.Workload(name="retain", shape=shape, seq_len=i32([n]), unit_off=i32([0, 1]), unit_len=i32([n]),
                    unit_cached_pos=i32([p0]), unit_cached_stride=i32([1]), unit_target_pos=i32([0]),
                    unit_page_off=i32([0, 3]), unit_pages=i32([5, 1, 3]), recompute_off=i32([0, 0]),
                    recompute_pos=i32([]), free_pages=i32([0, 2]), num_pool_pages=6,
                    unit_src_offset=i32([p0 % 4]), unit_target_stride=i32([0]))
    # pool rows are arbitrary bf16 numbers x_i (what the request's pages hold at positions p0 + i);
    # the retained row must be R(-(p0 + i)) x_i
    t = wl.make_tensors(w, seed=3)
    kb, vb = orc.bits(t.k_pool), orc.bits(t.v_pool)
    none = np.zeros((1, 2 * 16), np.uint16)
    a = orc.assemble(w, 0, kb, vb, none, none)
    assert a.delta.tolist() == [-(p0 + i) for i in range(n)]
    pool = orc.bf16_bits_to_f64(kb).reshape(-1, 2, 16)
    for i in range(n):
        si = p0 % 4 + i
        slot = [5, 1, 3][si // 4] * 4 + si % 4
        for h in range(2):
            want = orc.rope_rotate(pool[slot, h], -(p0 + i), 100.0)
            assert np.max(np.abs(want - a.k[i, h])) < 1e-12
            back = orc.rope_rotate(a.k[i, h], p0 + i, 100.0)           # rotating forward again returns the stored key
            assert np.max(np.abs(back - pool[slot, h])) < 1e-12
        assert np.array_equal(a.v_bits[i], vb.reshape(-1, 2, 16)[slot])
    # with target stride 1 (the default) the same descriptor shifts every token by the same -p0
    w1 = wl.Workload(**{**w.__dict__, "unit_target_stride": None})
    a1 = orc.assemble(w1, 0, kb, vb, none, none)
    assert a1.delta.tolist() == [-p0] * n
    # one worked number: pair 0 turns by exactly (shift) radians whatever theta is (w_0 = 1), so for
    # token 2 (shift -8) element 0 of head 0 is x cos 8 + y sin 8 with (x, y) = (elements 0 and 8)
    si = p0 % 4 + 2
    slot = [5, 1, 3][si // 4] * 4 + si % 4
    x, y = pool[slot, 0, 0], pool[slot, 0, 8]
    assert abs(a.k[2, 0, 0] - (x * math.cos(8.0) + y * math.sin(8.0))) < 1e-12
    assert abs(a.k[2, 0, 8] - (y * math.cos(8.0) - x * math.sin(8.0))) < 1e-12


def test_placement_rejects_bad_batches():
    shape = wl.ModelShape(2, 1, 16, 16, 1e4)
    rng = np.random.default_rng(0)
    w = wl.build_workload("gap", shape, [[4, wl.unit(20, "a"), 2]], rng)
    w.recompute_pos = w.recompute_pos[1:].copy()                      # position 0 now uncovered
    w.recompute_off = np.array([0, len(w.recompute_pos)], np.int32)
    assert orc.placement(w)[0] < 0
    w = wl.build_workload("few", shape, [[4, wl.unit(20, "a"), 2]], rng)
    w.free_pages = w.free_pages[:1].copy()
    assert orc.placement(w)[0] < 0
    w = wl.build_workload("overlap", shape, [[wl.unit(20, "a"), wl.unit(20, "b")]], rng)
    w.unit_target_pos = np.array([0, 10], np.int32)
    assert orc.placement(w)[0] < 0


# ---------------------------------------------------------------------- attention

def _tiny(seed=11, D=8):
    shape = wl.ModelShape(4, 2, D, 4, 100.0)
    rng = np.random.default_rng(seed)
    segs = [3, wl.unit(9, "a", cached_pos=2, recompute=(0, 4)), wl.unit(6, "b", cached=False),
            wl.unit(7, "c", cached_pos=0, stride=0, recompute=(6,)), 4]
    return wl.build_workload("tiny", shape, [segs], rng)


def test_attention_brute_force_tiny():
    """Triple loop written here from the definition, on T = 29, D = 8."""
    w = _tiny()
    t = wl.make_tensors(w, seed=99)
    kb, vb, qb, knb, vnb = (orc.bits(x) for x in (t.k_pool, t.v_pool, t.q, t.k_new, t.v_new))
    asm, out, lse = orc.full_layer(w, kb, vb, qb, knb, vnb)
    a = asm[0]
    V = orc.bf16_bits_to_f64(a.v_bits)
    Q = orc.bf16_bits_to_f64(qb)
    D, g = 8, 2
    for j, p in enumerate(w.recompute_pos):
        for h in range(4):
            s = [sum(Q[j, h, d] * a.k[t_, h // g, d] for d in range(D)) / math.sqrt(D) for t_ in range(p + 1)]
            z = sum(math.exp(x) for x in s)
            for d in range(D):
                o = sum(math.exp(s[t_]) / z * V[t_, h // g, d] for t_ in range(p + 1))
                assert abs(o - out[j, h, d]) < 1e-12
            assert abs(math.log(z) - lse[j, h]) < 1e-12


def test_attention_with_float64_queries_against_numpy_softmax():
    """The fp64-query form of the oracle's attention (used for 8-bit-key attention, whose decoded queries
    need not be bf16 numbers): brute force with numpy on a tiny case, and equal to the bf16-query form
    when the queries are bf16 numbers."""
    shape = wl.ModelShape(4, 2, 8, 4, 1e4)
    rng = np.random.default_rng(12)
    T = 19
    w = wl.build_workload("q64", shape, [[wl.unit(T, "a", cached=False)]], rng)
    k = rng.standard_normal((T, 2, 8))
    v = torch.from_numpy(rng.standard_normal((T, 2, 8))).to(torch.bfloat16)
    q = rng.standard_normal((T, 4, 8)) * 0.37                                  # not bf16 numbers
    jj, hh, pp = orc.request_rows(w, 0)
    o, l = orc.attention_rows(w, k, orc.bits(v), q, jj, hh, pp)
    vd = v.double().numpy()
    for i in range(len(jj)):
        p, h = int(pp[i]), int(hh[i])
        sc = (k[: p + 1, h // 2] @ q[jj[i], h]) / math.sqrt(8)
        wgt = np.exp(sc - sc.max()); wgt /= wgt.sum()
        assert np.max(np.abs(o[i] - wgt @ vd[: p + 1, h // 2])) < 1e-12
        assert abs(l[i] - (sc.max() + math.log(np.exp(sc - sc.max()).sum()))) < 1e-12
    qb = torch.from_numpy(q).to(torch.bfloat16)
    o1, l1 = orc.attention_rows(w, k, orc.bits(v), orc.bits(qb), jj, hh, pp)
    o2, l2 = orc.attention_rows(w, k, orc.bits(v), qb.double().numpy(), jj, hh, pp)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)


def test_partial_equals_rows_of_library_causal_attention():
    """Recompute set = all tokens reproduces ordinary causal prefill (library SDPA,
    fp64, KV heads repeated g times); any subset equals the matching rows."""
    shape = wl.ModelShape(4, 2, 16, 8, 1e4)
    rng = np.random.default_rng(21)
    T = 45
    w_full = wl.build_workload("full", shape, [[wl.unit(T, "a", cached=False)]], rng)
    t = wl.make_tensors(w_full, seed=5)
    bits5 = [orc.bits(x) for x in (t.k_pool, t.v_pool, t.q, t.k_new, t.v_new)]
    _, out, lse = orc.full_layer(w_full, *bits5)
    Q = torch.from_numpy(orc.bf16_bits_to_f64(bits5[2])).permute(1, 0, 2)[None]         # [1,H,T,D]
    K = torch.from_numpy(orc.bf16_bits_to_f64(bits5[3])).permute(1, 0, 2).repeat_interleave(2, 0)[None]
    V = torch.from_numpy(orc.bf16_bits_to_f64(bits5[4])).permute(1, 0, 2).repeat_interleave(2, 0)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(Q, K, V, is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.max(np.abs(ref - out)) < 1e-12
    # a partial mask over the same assembled KV: cached rows hold exactly k_new/v_new content
    sel = [0, 3, 4, 17, 44]
    a_k = orc.bf16_bits_to_f64(bits5[3])
    o2, l2 = orc.attention_rows(w_full, a_k, bits5[4], bits5[2],
                                np.repeat(sel, 4), np.tile(np.arange(4), len(sel)), np.repeat(sel, 4))
    assert np.max(np.abs(o2.reshape(len(sel), 4, 16) - ref[sel])) < 1e-12
    assert np.max(np.abs(l2.reshape(len(sel), 4) - lse[sel])) < 1e-12


def test_uniform_softmax_closed_form_and_causal_limit():
    """K == 0 -> LSE = ln(p + 1) exactly and O = mean of V[0..p]; with V[t, :, 0] = t this
    is p / 2: any off-by-one in the causal limit or a wrong kv head shows."""
    w = wl.config(1)
    sh = w.shape
    T = int(w.seq_len[0])
    k = np.zeros((T, sh.num_kv_heads, sh.head_dim))
    vt = torch.zeros(T, sh.num_kv_heads, sh.head_dim)
    vt[:, 0, 0] = torch.arange(T, dtype=torch.float32)
    vt[:, 1, 0] = -2 * torch.arange(T, dtype=torch.float32)
    vb = orc.bits(vt.to(torch.bfloat16))                 # integers below 512 are exact in bf16? no: use check
    V = orc.bf16_bits_to_f64(vb)
    t = wl.make_tensors(w)
    jj, hh, pp = orc.request_rows(w, 0)
    o, l = orc.attention_rows(w, k, vb, orc.bits(t.q), jj, hh, pp)
    g = sh.num_q_heads // sh.num_kv_heads
    for i in range(len(jj)):
        p = pp[i]
        assert abs(l[i] - math.log(p + 1)) < 1e-12
        assert abs(o[i, 0] - V[: p + 1, hh[i] // g, 0].mean()) < 1e-9


def test_needle_inside_and_outside_causal_limit():
    """One key with an overwhelming logit: it must dominate when at position <= p and be
    invisible at position p + 1."""
    shape = wl.ModelShape(1, 1, 8, 4, 1e4)
    rng = np.random.default_rng(8)
    T = 23
    w = wl.build_workload("needle", shape, [[wl.unit(T, "a", cached=False)]], rng)
    qf = torch.zeros(T, 1, 8); qf[:, 0, 0] = 8.0
    for needle in (9, 10, 11, 12):
        kf = torch.zeros(T, 1, 8); kf[needle, 0, 0] = 64.0
        vf = torch.zeros(T, 1, 8); vf[needle, 0, 1] = 1.0
        o, _ = orc.attention_rows(w, kf.double().numpy(), orc.bits(vf.to(torch.bfloat16)),
                                  orc.bits(qf.to(torch.bfloat16)), [10], [0], [10])
        if needle <= 10:
            assert o[0, 1] > 0.999999
        else:
            assert o[0, 1] == 0.0


def test_assemble_precedence_and_exact_rows():
    """Recomputed rows override cached rows; delta == 0 rows and V rows are bit copies."""
    w = wl.adversarial()
    t = wl.make_tensors(w, seed=3)
    kb, vb, qb, knb, vnb = (orc.bits(x) for x in (t.k_pool, t.v_pool, t.q, t.k_new, t.v_new))
    st, page_off, pages, src_slot, fresh = orc.placement(w)
    assert st == 0
    base = 0
    row = w.shape.num_kv_heads * w.shape.head_dim
    kflat, vflat = kb.reshape(-1, row), vb.reshape(-1, row)
    saw_zero_delta = saw_negative = False
    for r in range(w.batch):
        a = orc.assemble(w, r, kb, vb, knb, vnb)
        T = int(w.seq_len[r])
        for p in range(T):
            j, s = fresh[base + p], src_slot[base + p]
            if j >= 0:
                assert a.k_exact[p]
                assert np.array_equal(a.k_bits[p].ravel(), knb[j].ravel())
                assert np.array_equal(a.v_bits[p].ravel(), vnb[j].ravel())
            else:
                assert np.array_equal(a.v_bits[p].ravel(), vflat[s])
                if a.delta[p] == 0:
                    saw_zero_delta = True
                    assert a.k_exact[p] and np.array_equal(a.k_bits[p].ravel(), kflat[s])
                    assert np.array_equal(a.k[p].ravel(), orc.bf16_bits_to_f64(kflat[s]))
                saw_negative |= a.delta[p] < 0
        base += T
    assert saw_zero_delta and saw_negative


def test_kv_byte_model_closed_form():
    """Sec. 2.4: 2 L (H_kv/TP) d_h w; the paper's example (64 layers, 8 KV heads, d_h 128,
    16-bit) is 64 KiB per token per rank at TP = 4 ... and 256 KiB summed over 4 ranks."""
    assert wl.kv_bytes_per_token(64, 8, 128, 2, tp=4) * 4 == 256 * 1024
    assert wl.kv_bytes_per_token(1, 8, 128, 2) == 4096
    w = wl.config(2)
    assert w.total_tokens == 5312 and w.n_q == 352 and w.cached_tokens == 5120
    assert wl.gather_bytes(w) == 5120 * 8192


# ---------------------------------------------------------------- 8-bit (e4m3) storage form
def test_e4m3_decode_all_codes_against_library_and_closed_forms():
    codes = np.arange(256, dtype=np.uint8)
    v = orc.e4m3_decode(codes)
    lib = torch.arange(256, dtype=torch.uint8).view(torch.float8_e4m3fn).double().numpy()
    assert np.array_equal(np.isnan(v), np.isnan(lib)) and np.isnan(v).sum() == 2
    assert np.array_equal(v[~np.isnan(v)], lib[~np.isnan(lib)])
    assert v[0x38] == 1.0 and v[0x7e] == 448.0 and v[0x01] == 2.0 ** -9 and v[0x08] == 2.0 ** -6
    assert v[0xb8] == -1.0 and v[0x80] == 0.0 and np.signbit(v[0x80])
    assert np.all(np.diff(v[:0x7f]) > 0)                      # codes 0x00..0x7e ascend


def test_e4m3_encode_nearest_even_saturating():
    table = orc.e4m3_decode(np.arange(0x7f, dtype=np.uint8))
    # round trip of every finite code, both signs
    assert np.array_equal(orc.e4m3_encode(table.astype(np.float32)), np.arange(0x7f, dtype=np.uint8))
    assert np.array_equal(orc.e4m3_encode((-table).astype(np.float32)), np.arange(0x7f, dtype=np.uint8) | 0x80)
    # exact midpoints go to the even code; a hair to either side goes to the nearer one
    mid = ((table[:-1] + table[1:]) / 2).astype(np.float32)
    assert np.array_equal(mid.astype(np.float64), (table[:-1] + table[1:]) / 2)     # midpoints are floats
    lo = np.arange(0x7e, dtype=np.uint8)
    assert np.array_equal(orc.e4m3_encode(mid), np.where(lo % 2 == 0, lo, lo + 1))
    assert np.array_equal(orc.e4m3_encode(np.nextafter(mid, np.float32(0))), lo)
    assert np.array_equal(orc.e4m3_encode(np.nextafter(mid, np.float32(1e9))), lo + 1)
    # saturation and NaN
    big = np.array([448.0, 449.0, 464.0, 1e9, np.inf, -1e9, -np.inf, np.nan], np.float32)
    assert orc.e4m3_encode(big).tolist() == [0x7e, 0x7e, 0x7e, 0x7e, 0x7e, 0xfe, 0xfe, 0x7f]
    # library conversion (which does not saturate) on values inside the range
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(100000) * np.exp(rng.uniform(-12, 5, 100000))).astype(np.float32)
    x = x[np.abs(x) < 448]
    want = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(orc.e4m3_encode(x), want)


def test_assemble_from_8bit_pool_reduces_to_the_16bit_path():
    """Every e4m3 value (and its product with a power of two) is a bf16 value, so an 8-bit source pool
    with a power-of-two scale must assemble exactly like the 16-bit pool holding the same numbers."""
    w = wl.adversarial()
    t = wl.make_tensors(w, seed=5)
    rng = np.random.default_rng(2)
    knb, vnb = orc.bits(t.k_new), orc.bits(t.v_new)
    shape = tuple(t.k_pool.shape)
    k8 = rng.integers(0, 256, size=shape, dtype=np.uint8)
    v8 = rng.integers(0, 256, size=shape, dtype=np.uint8)
    k8[(k8 & 0x7f) == 0x7f] = 0x38                            # no NaN codes
    v8[(v8 & 0x7f) == 0x7f] = 0x38
    for scale in (1.0, 0.25):
        kb = orc.bits(torch.from_numpy(orc.e4m3_decode(k8) * scale).to(torch.bfloat16))
        vb = orc.bits(torch.from_numpy(orc.e4m3_decode(v8) * scale).to(torch.bfloat16))
        assert np.array_equal(orc.bf16_bits_to_f64(kb), orc.e4m3_decode(k8) * scale)     # exact in bf16
        for r in range(w.batch):
            a16 = orc.assemble(w, r, kb, vb, knb, vnb)
            a8 = orc.assemble(w, r, k8, v8, knb, vnb, src_fmt=1, k_scale=scale, v_scale=scale)
            assert np.array_equal(a16.v_bits, a8.v_bits) and np.array_equal(a16.k, a8.k)
            assert np.array_equal(a16.k_exact, a8.k_exact) and np.array_equal(a16.k_bits, a8.k_bits)
    # a scale that is not a power of two: the 16-bit row is the EXACT product code * float(scale) rounded
    # once to bf16.  Checked against exact rational arithmetic: the result must be the bf16 neighbour
    # nearest to the exact product, the even one on a tie.
    from fractions import Fraction
    a8 = orc.assemble(w, 0, k8, v8, knb, vnb, src_fmt=1, k_scale=0.3, v_scale=0.7)
    st, _, _, src_slot, fresh = orc.placement(w)
    row = w.shape.num_kv_heads * w.shape.head_dim
    p = next(p for p in range(int(w.seq_len[0])) if fresh[p] < 0)
    codes = v8.reshape(-1, row)[src_slot[p]]
    sc = Fraction(float(np.float32(0.7)))
    got = orc.bf16_bits_to_f64(a8.v_bits[p].ravel())
    for c, gv, gb in zip(codes.tolist(), got.tolist(), a8.v_bits[p].ravel().tolist()):
        exact = Fraction(float(orc.e4m3_decode(np.array([c], np.uint8))[0])) * sc
        if exact == 0:
            assert gv == 0.0
            continue
        up = orc.bf16_bits_to_f64(np.array([gb + 1], np.uint16))[0]      # next bf16 away from zero
        dn = orc.bf16_bits_to_f64(np.array([gb - 1], np.uint16))[0]      # next bf16 towards zero
        err = abs(Fraction(gv) - exact)
        for nb in (up, dn):
            e2 = abs(Fraction(float(nb)) - exact)
            assert err < e2 or (err == e2 and gb % 2 == 0), (c, gv, nb)


def test_f64_to_bf16_single_rounding():
    """The oracle's double -> bf16 rounding against the library's float -> bfloat16 conversion on values
    that are floats already (one rounding either way), plus the cases where rounding a double through
    float first would go wrong (a double just above / below a bf16 midpoint)."""
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(20000) * np.exp(rng.uniform(-30, 30, 20000))).astype(np.float32)
    want = orc.bits(torch.from_numpy(x).to(torch.bfloat16))
    assert np.array_equal(orc.f64_to_bf16_bits(x.astype(np.float64)), want)
    # 1 + 2^-8 is the midpoint between bf16 1.0 (0x3f80, even) and 1 + 2^-7 (0x3f81)
    mid = 1.0 + 2.0 ** -8
    assert orc.f64_to_bf16_bits(np.array([mid, mid + 2.0 ** -40, mid - 2.0 ** -40])).tolist() == [0x3f80, 0x3f81, 0x3f80]
    # 1 + 3 * 2^-8 is the midpoint between 0x3f81 (odd) and 0x3f82 (even): the tie goes up to the even one
    assert orc.f64_to_bf16_bits(np.array([1.0 + 3 * 2.0 ** -8])).tolist() == [0x3f82]
    # rounding through float first would turn mid + 2^-40 into the exact midpoint and lose the tie
    assert np.float32(mid + 2.0 ** -40) == np.float32(mid)
    assert orc.f64_to_bf16_bits(np.array([0.0, -0.0, np.inf, -np.inf, 2.0 ** -140, -1.5])).tolist() == \
        [0x0000, 0x8000, 0x7f80, 0xff80, 0x0000, 0xbfc0]
