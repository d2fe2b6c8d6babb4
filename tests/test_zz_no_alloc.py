"""The no-allocation RoPE shift against the plan-based one.

Some users of this library run where device allocation is not allowed (an engine that owns the
device through its own pool, a no-allocation phase).  They call tessera_rope_shift_static, whose
only scratch is a fixed array inside the library.  This file is collected last on purpose, so a run
that stops at the first failure has already exercised every other test."""
import numpy as np
import pytest
import torch

from oracle import tessera_oracle as orc
from paper_2609_32999_b200 import binding as tb
from paper_2609_32999_b200 import workloads as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _slots_and_shifts(w, page_off, pages):
    """Destination slot and shift amount of every cached-unit token (plain index arithmetic)."""
    B = w.shape.page_size
    slots, deltas = [], []
    for r in range(w.batch):
        for u in range(w.unit_off[r], w.unit_off[r + 1]):
            if w.unit_page_off[u + 1] == w.unit_page_off[u]:
                continue
            i = np.arange(w.unit_len[u])
            p = w.unit_target_pos[u] + i
            slots.append(pages[page_off[r] + p // B].astype(np.int64) * B + p % B)
            deltas.append(p - (w.unit_cached_pos[u] + w.unit_cached_stride[u] * i))
    slots, deltas = np.concatenate(slots), np.concatenate(deltas)
    shifts, idx = np.unique(deltas, return_inverse=True)
    return slots.astype(np.int32), idx.astype(np.int32), shifts.astype(np.int32)


def _oracle_rotated_k(w, plan, t0_bits, after_bits):
    """Every destination row of the rotated pool against the oracle's assembled keys (fp64)."""
    page_off, pages, _ = plan.block_table()
    sh = w.shape
    row = sh.num_kv_heads * sh.head_dim
    B = sh.page_size
    ka = after_bits.reshape(-1, row)
    zeros = np.zeros((max(w.n_q, 1), row), np.uint16)
    errs = []
    for r in range(w.batch):
        T = int(w.seq_len[r])
        if T == 0:
            continue
        a = orc.assemble(w, r, t0_bits[0], t0_bits[1], zeros, zeros)
        p = np.arange(T)
        slots = pages[page_off[r] + p // B].astype(np.int64) * B + p % B
        cached = np.ones(T, bool)
        cached[w.recompute_pos[w.recompute_off[r]:w.recompute_off[r + 1]]] = False     # fresh rows are not shifted
        ex = cached & (a.delta == 0)
        assert np.array_equal(ka[slots][ex], t0_bits[0].reshape(-1, row)[_src_slots(w, r)][ex])
        rot = cached & (a.delta != 0)
        if rot.any():
            errs.append(np.abs(orc.bf16_bits_to_f64(ka[slots][rot]) - a.k.reshape(T, row)[rot]).ravel())
    e = np.concatenate(errs)
    assert e.max() <= gu.MAX_ABS and e.mean() <= gu.MEAN_ABS
    return e.max(), e.mean()


def _src_slots(w, r):
    """Source slot of every position of request r (0 where no cached unit covers it)."""
    st, _, _, src, _ = orc.placement(w)
    assert st == 0
    t0 = int(np.sum(w.seq_len[:r]))
    return np.maximum(src[t0:t0 + int(w.seq_len[r])], 0)


def _prime(shape):
    """The library's first call on a device looks up the scratch array's address, and the CUDA runtime
    loads a kernel's code on its first launch; both happen once per process.  The no-allocation
    property is checked on calls after that."""
    dev = "cuda:0"
    pool = torch.zeros(2, shape.page_size, shape.num_kv_heads, shape.head_dim, dtype=torch.bfloat16, device=dev)
    one = torch.zeros(1, dtype=torch.int32, device=dev)
    tb.rope_shift_static(shape, pool, one, one, np.array([1], np.int32))
    torch.cuda.synchronize()


def _compare(w, seed):
    dev = "cuda:0"
    _prime(w.shape)
    plan = tb.Plan(w)
    page_off, pages, _ = plan.block_table()
    # existing entry points: unfused compose, then the plan-based shift
    ref = wl.make_tensors(w, device=dev, seed=seed)
    before = (orc.bits(ref.k_pool).copy(), orc.bits(ref.v_pool).copy())
    plan.kv_compose(ref.k_pool, ref.v_pool, fuse_rope=False)
    plan.rope_shift(ref.k_pool)
    # new entry point on identically composed pools
    new = wl.make_tensors(w, device=dev, seed=seed)
    plan.kv_compose(new.k_pool, new.v_pool, fuse_rope=False)
    slots, idx, shifts = _slots_and_shifts(w, page_off, pages)
    assert len(shifts) <= tb.STATIC_MAX_SHIFTS
    d_slots, d_idx = torch.from_numpy(slots).to(dev), torch.from_numpy(idx).to(dev)
    torch.cuda.synchronize()
    free0, alloc0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
    tb.rope_shift_static(w.shape, new.k_pool, d_slots, d_idx, shifts)
    torch.cuda.synchronize()
    # nothing was allocated on the device, by the driver or by torch's caching allocator
    assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
    # same table values, same fp32 arithmetic: identical bits to the plan-based shift
    assert torch.equal(ref.k_pool, new.k_pool)
    assert torch.equal(ref.v_pool, new.v_pool)
    # and within the rotated-key tolerance of the fp64 oracle
    _oracle_rotated_k(w, plan, before, orc.bits(new.k_pool))
    # the shift really happened: rotated rows differ from the merely copied ones
    plain = wl.make_tensors(w, device=dev, seed=seed)
    plan.kv_compose(plain.k_pool, plain.v_pool, fuse_rope=False)
    assert not torch.equal(plain.k_pool, new.k_pool)
    plan.destroy()


def test_static_shift_matches_plan_shift_twice_in_a_row():
    _compare(wl.adversarial(seed=9, shape=wl.ModelShape(32, 8, 128, 64, 500000.0)), seed=21)
    _compare(wl.config(1), seed=22)          # second call: other head_dim, other shifts, same scratch
    _compare(wl.config(2), seed=23)


def test_static_shift_skips_slots_outside_the_stated_pool():
    """Slot ids that are negative or at / beyond num_pool_slots are skipped on the device.  The bound
    passed is smaller than the real pool, so the 'outside' ids still point into allocated memory and a
    missing check would show up as changed rows rather than as a fault."""
    w = wl.config(1)
    dev = "cuda:0"
    t = wl.make_tensors(w, device=dev, seed=5)
    before = t.k_pool.clone()
    B = w.shape.page_size
    n_slots_real = w.num_pool_pages * B
    bound = n_slots_real // 2
    inside = torch.arange(3, bound, 7, dtype=torch.int32)
    outside = torch.cat([torch.arange(bound, n_slots_real, 5, dtype=torch.int32), torch.tensor([-1, -7], dtype=torch.int32)])
    slots = torch.cat([inside, outside]).to(dev)
    idx = torch.zeros_like(slots)
    tb.rope_shift_static(w.shape, t.k_pool, slots, idx, np.array([37], np.int32), num_pool_slots=bound)
    torch.cuda.synchronize()
    rows_before = before.view(n_slots_real, -1)
    rows_after = t.k_pool.view(n_slots_real, -1)
    touched = torch.zeros(n_slots_real, dtype=torch.bool)
    touched[inside.long()] = True
    touched = touched.to(dev)
    assert torch.equal(rows_after[~touched], rows_before[~touched])          # skipped and unlisted rows: bit-identical
    assert not torch.equal(rows_after[touched], rows_before[touched])        # listed rows inside the bound were rotated
    # a slot_shift entry outside the table is skipped as well
    t2 = before.clone()
    tb.rope_shift_static(w.shape, t2, inside.to(dev), torch.full_like(inside, 3).to(dev), np.array([37], np.int32))
    torch.cuda.synchronize()
    assert torch.equal(t2, before)


def test_static_shift_refuses_interleaved_pairing():
    w = wl.config(1)
    dev = "cuda:0"
    t = wl.make_tensors(w, device=dev)
    import dataclasses
    shape = dataclasses.replace(w.shape, rope_pairing=1)
    slots = torch.zeros(1, dtype=torch.int32, device=dev)
    with pytest.raises(tb.TesseraError) as e:
        tb.rope_shift_static(shape, t.k_pool, slots, slots, np.array([1], np.int32))
    assert e.value.status == tb.UNSUPPORTED_SHAPE


def test_static_shift_rejects_oversized_table():
    w = wl.config(1)
    dev = "cuda:0"
    t = wl.make_tensors(w, device=dev)
    before = t.k_pool.clone()
    n = tb.STATIC_MAX_SHIFTS + 1
    slots = torch.zeros(4, dtype=torch.int32, device=dev)
    with pytest.raises(tb.TesseraError) as e:
        tb.rope_shift_static(w.shape, t.k_pool, slots, slots, np.arange(n, dtype=np.int32))
    assert e.value.status == tb.UNSUPPORTED_SHAPE and str(tb.STATIC_MAX_SHIFTS) in str(e.value)
    torch.cuda.synchronize()
    assert torch.equal(before, t.k_pool)
