"""Seeded random layouts through the whole path: head_dim, page size, group size (also ones that do not
divide the tile), pairing, fused / unfused shift, cached and uncached units at random cached positions and
strides, scattered recompute offsets - each compared with the oracle in full."""
import numpy as np
import pytest

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
