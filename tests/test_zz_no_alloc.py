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


def _compare(w, seed):
    dev = "cuda:0"
    plan = tb.Plan(w)
    page_off, pages, _ = plan.block_table()
    # existing entry points: unfused compose, then the plan-based shift
    ref = wl.make_tensors(w, device=dev, seed=seed)
    plan.kv_compose(ref.k_pool, ref.v_pool, fuse_rope=False)
    plan.rope_shift(ref.k_pool)
    # new entry point on identically composed pools
    new = wl.make_tensors(w, device=dev, seed=seed)
    plan.kv_compose(new.k_pool, new.v_pool, fuse_rope=False)
    slots, idx, shifts = _slots_and_shifts(w, page_off, pages)
    assert len(shifts) <= tb.STATIC_MAX_SHIFTS
    tb.rope_shift_static(w.shape, new.k_pool, torch.from_numpy(slots).to(dev), torch.from_numpy(idx).to(dev), shifts)
    torch.cuda.synchronize()
    a = orc.bf16_bits_to_f64(orc.bits(ref.k_pool))
    b = orc.bf16_bits_to_f64(orc.bits(new.k_pool))
    diff = np.abs(a - b)
    assert np.isfinite(b).all()
    assert diff.max() <= gu.MAX_ABS and diff.mean() <= gu.MEAN_ABS
    assert torch.equal(ref.v_pool, new.v_pool)
    # the shift really happened: rotated rows differ from the merely copied ones
    plain = wl.make_tensors(w, device=dev, seed=seed)
    plan.kv_compose(plain.k_pool, plain.v_pool, fuse_rope=False)
    assert not torch.equal(plain.k_pool, new.k_pool)
    plan.destroy()


def test_static_shift_matches_plan_shift_twice_in_a_row():
    _compare(wl.adversarial(seed=9, shape=wl.ModelShape(32, 8, 128, 64, 500000.0)), seed=21)
    _compare(wl.config(1), seed=22)          # second call: other head_dim, other shifts, same scratch
    _compare(wl.config(2), seed=23)


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
