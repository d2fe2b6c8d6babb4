"""Seeded synthetic workloads for the composed-prefill hot path.

This module only *describes* batches (who is cached where, who lands where,
which positions are recomputed) and draws random bf16 tensors.  It contains
none of the method's arithmetic (no RoPE, no softmax, no slot computation), so
that both the CPU oracle and the CUDA library can be fed from it without
sharing any code of the method itself.

The five named workloads stand in for the paper's RAG datasets and agent-memory
traces (Sec. 6.1): the same shapes, popularity skew and length mix, but seeded
synthetic content.  Rotating i.i.d. N(0,1) pairs leaves them i.i.d. N(0,1), so
"keys cached rotated at positions 0..len-1" and "fresh keys already rotated at
their target positions" are both plain N(0,1) draws.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence

import numpy as np
import torch

BASE_SEED = 20260932


@dataclasses.dataclass
class ModelShape:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    rope_theta: float
    rope_pairing: int = 0          # 0 = half-split (i, i + D/2)
    sm_scale: float = 0.0          # 0 -> 1/sqrt(D)


@dataclasses.dataclass
class Workload:
    """One batch in the layout the C ABI takes (CSR over requests and units)."""
    name: str
    shape: ModelShape
    seq_len: np.ndarray             # [batch]
    unit_off: np.ndarray            # [batch+1]
    unit_len: np.ndarray            # [n_units]
    unit_cached_pos: np.ndarray     # [n_units]
    unit_cached_stride: np.ndarray  # [n_units] 1 = rotated at cached_pos+i, 0 = not rotated
    unit_target_pos: np.ndarray     # [n_units]
    unit_page_off: np.ndarray       # [n_units+1]
    unit_pages: np.ndarray          # source page ids
    recompute_off: np.ndarray       # [batch+1]
    recompute_pos: np.ndarray       # ascending per request
    free_pages: np.ndarray          # destination page ids, consumed in order
    num_pool_pages: int
    n_layers: int = 1
    unit_src_offset: Optional[np.ndarray] = None     # [n_units] token 0's offset inside its first source page
    unit_target_stride: Optional[np.ndarray] = None  # [n_units] 0 = every token rotated for target_pos
    num_source_pages: int = 0                        # > 0: unit_pages index a separate source pool (host tier)
    unit_retain_page_off: Optional[np.ndarray] = None  # [n_units+1] CSR: cache pages of units captured by extend_write
    unit_retain_pages: Optional[np.ndarray] = None
    retain_pool_pages: int = 0                       # > 0: the cache pages index a separate cache pool

    @property
    def batch(self) -> int:
        return int(self.seq_len.shape[0])

    @property
    def total_tokens(self) -> int:
        return int(self.seq_len.sum())

    @property
    def n_q(self) -> int:
        return int(self.recompute_pos.shape[0])

    @property
    def cached_tokens(self) -> int:
        n = 0
        for u in range(len(self.unit_len)):
            if self.unit_page_off[u + 1] > self.unit_page_off[u]:
                n += int(self.unit_len[u])
        return n

    @property
    def qk_pairs(self) -> int:
        """Unmasked (query token, key) pairs: sum over queries of position+1."""
        return int(self.recompute_pos.astype(np.int64).sum() + self.n_q)


def _i32(x) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(x, dtype=np.int32))


class _UnitSpec:
    __slots__ = ("uid", "length", "cached", "cached_pos", "stride", "recompute")

    def __init__(self, uid, length, cached=True, cached_pos=0, stride=1, recompute=()):
        self.uid = uid                # pool identity; equal uids share source pages
        self.length = int(length)
        self.cached = bool(cached)
        self.cached_pos = int(cached_pos)
        self.stride = int(stride)
        self.recompute = recompute    # offsets inside the unit that are recomputed


def build_workload(name: str, shape: ModelShape, requests: Sequence[Sequence[object]],
                   rng: np.random.Generator, n_layers: int = 1,
                   shuffle_pages: bool = True, spare_pages: int = 3) -> Workload:
    """Assemble a Workload from per-request segment lists.

    Each request is a list of segments in prompt order; a segment is either an
    int n (n request-specific tokens: instruction, separator, query; always
    recomputed) or a _UnitSpec.  Source pages are given to distinct cached unit
    ids in first-use order, destination pages come after them, and (optionally)
    all page ids are passed through one seeded permutation so that neither
    sources nor destinations are adjacent in the pool.
    """
    B = shape.page_size
    seq_len, unit_off = [], [0]
    u_len, u_cpos, u_stride, u_tpos, u_uid, u_cached = [], [], [], [], [], []
    rec_off, rec_pos = [0], []
    for segs in requests:
        pos = 0
        for s in segs:
            if isinstance(s, _UnitSpec):
                u_len.append(s.length); u_cpos.append(s.cached_pos); u_stride.append(s.stride)
                u_tpos.append(pos); u_uid.append(s.uid); u_cached.append(s.cached)
                offs = range(s.length) if not s.cached else sorted(set(int(o) for o in s.recompute))
                rec_pos.extend(pos + o for o in offs)
                pos += s.length
            else:
                n = int(s)
                rec_pos.extend(range(pos, pos + n))
                pos += n
        seq_len.append(pos)
        unit_off.append(len(u_len))
        rec_off.append(len(rec_pos))
    # source pages per distinct cached uid
    first_page = {}
    n_src = 0
    for uid, ln, c in zip(u_uid, u_len, u_cached):
        if c and uid not in first_page:
            first_page[uid] = n_src
            n_src += -(-ln // B)
    n_dst = sum(-(-t // B) for t in seq_len)
    total = n_src + n_dst + spare_pages
    perm = rng.permutation(total) if shuffle_pages else np.arange(total)
    u_page_off, u_pages = [0], []
    for uid, ln, c in zip(u_uid, u_len, u_cached):
        if c:
            f = first_page[uid]
            u_pages.extend(int(perm[f + k]) for k in range(-(-ln // B)))
        u_page_off.append(len(u_pages))
    free = [int(perm[n_src + k]) for k in range(n_dst + spare_pages)]
    return Workload(
        name=name, shape=shape, seq_len=_i32(seq_len), unit_off=_i32(unit_off),
        unit_len=_i32(u_len), unit_cached_pos=_i32(u_cpos), unit_cached_stride=_i32(u_stride),
        unit_target_pos=_i32(u_tpos), unit_page_off=_i32(u_page_off), unit_pages=_i32(u_pages),
        recompute_off=_i32(rec_off), recompute_pos=_i32(rec_pos), free_pages=_i32(free),
        num_pool_pages=total, n_layers=n_layers)


def zipf_ranks(rng: np.random.Generator, n: int, pool: int, s: float, distinct: bool) -> List[int]:
    """n draws of a rank in 1..pool with P(k) proportional to k^-s (inverse CDF on
    seeded uniforms); `distinct` redraws repeats inside one request."""
    w = np.arange(1, pool + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(w / w.sum())
    out: List[int] = []
    seen = set()
    while len(out) < n:
        k = int(np.searchsorted(cdf, rng.random(), side="left")) + 1
        k = min(k, pool)
        if distinct and k in seen:
            continue
        seen.add(k)
        out.append(k)
    return out


LLAMA8B = dict(num_q_heads=32, num_kv_heads=8, head_dim=128, page_size=64, rope_theta=500000.0)


def _policy_cache(policy: Optional[str], capacity_blocks: int, avg_blocks_per_request: float):
    """Residency model for configs 2-4: None = every unit is a hit (the configurations as stated);
    "reuse" = the paper's score-based admission / eviction (Sec. 5.2), "lru", "lfu" = baselines."""
    if policy is None:
        return None
    from . import residency as rs
    if policy == "reuse":
        return rs.ReuseScoreCache(capacity_blocks, rs.ReuseScoreCache.window_for(capacity_blocks, avg_blocks_per_request))
    if policy == "lru":
        return rs.LRUCache(capacity_blocks)
    if policy == "lfu":
        return rs.LFUCache(capacity_blocks)
    raise ValueError("policy must be None, 'reuse', 'lru' or 'lfu'")


def config(index: int, seed: Optional[int] = None, requests_override: Optional[int] = None,
           policy: Optional[str] = None, warm_requests: int = 400, capacity_fraction: float = 0.1) -> Workload:
    """The five benchmark configurations, index 1..5.

    With `policy` (configs 2-4) residency is no longer "everything cached": a cache holding
    `capacity_fraction` of the unit pool is warmed with `warm_requests` requests of the same
    popularity law, and the batch's units are hits only if resident; the others are uncached and
    fully recomputed (Sec. 5.3 "Preparation failures": computed from text).

    `requests_override` shrinks (or grows) the number of requests of the batched
    configurations (3, 4, 5) while keeping every per-request rule; it is how the
    multi-GPU bench gives each rank its own batch and how tests take a slice.
    """
    seed = BASE_SEED + index if seed is None else seed
    rng = np.random.default_rng(seed)
    if index == 1:
        shape = ModelShape(4, 2, 64, 16, 10000.0)
        segs = [16] + [_UnitSpec(("u", i), 64, recompute=range(4)) for i in range(4)] + [32]
        return build_workload("c1-tiny", shape, [segs], rng)
    if index == 2:
        shape = ModelShape(**LLAMA8B)
        cache = _policy_cache(policy, int(capacity_fraction * 1000 * 8), 10 * 8)
        for _ in range(warm_requests if cache else 0):
            cache.request([(k, 8) for k in zipf_ranks(rng, 10, 1000, 1.0, distinct=True)])
        ranks = zipf_ranks(rng, 10, 1000, 1.0, distinct=True)
        hits = cache.request([(k, 8) for k in ranks]) if cache else [True] * 10
        segs = [64] + [_UnitSpec(("c", k), 512, cached=h, recompute=range(16)) for k, h in zip(ranks, hits)] + [128]
        return build_workload("c2-rag-single", shape, [segs], rng)
    if index == 3:
        shape = ModelShape(**LLAMA8B)
        nreq = requests_override or 16
        rec_len = rng.integers(128, 385, size=5000)      # length fixed per pool id
        id_perm = rng.permutation(5000)
        blocks_of = lambda i: -(-int(rec_len[i]) // 64)
        cache = _policy_cache(policy, int(capacity_fraction * sum(blocks_of(i) for i in range(5000))), 20 * 4.5)
        for _ in range(warm_requests if cache else 0):
            cache.request([(int(id_perm[k - 1]), blocks_of(int(id_perm[k - 1]))) for k in zipf_ranks(rng, 20, 5000, 1.1, distinct=True)])
        reqs = []
        for _ in range(nreq):
            ranks = zipf_ranks(rng, 20, 5000, 1.1, distinct=True)
            ids = [int(id_perm[k - 1]) for k in ranks]
            hits = cache.request([(i, blocks_of(i)) for i in ids]) if cache else [True] * 20
            order = rng.permutation(20)
            segs = [256] + [_UnitSpec(("m", ids[o]), int(rec_len[ids[o]]), cached=hits[o], recompute=range(8))
                            for o in order] + [96]
            reqs.append(segs)
        return build_workload("c3-agent-memory", shape, reqs, rng)
    if index == 4:
        shape = ModelShape(**LLAMA8B)
        nreq = requests_override or 4
        id_perm = rng.permutation(4000)
        cache = _policy_cache(policy, int(capacity_fraction * 4000 * 8), 64 * 8)
        for _ in range(warm_requests if cache else 0):
            cache.request([(int(id_perm[k - 1]), 8) for k in zipf_ranks(rng, 64, 4000, 0.9, distinct=True)])
        reqs = []
        for _ in range(nreq):
            ranks = zipf_ranks(rng, 64, 4000, 0.9, distinct=True)
            hits = cache.request([(int(id_perm[k - 1]), 8) for k in ranks]) if cache else [True] * 64
            segs = [_UnitSpec(("c", int(id_perm[k - 1])), 512, cached=h, recompute=range(32)) for k, h in zip(ranks, hits)] + [256]
            reqs.append(segs)
        return build_workload("c4-long-rag", shape, reqs, rng, n_layers=32)
    if index == 5:
        shape = ModelShape(64, 8, 128, 64, 500000.0)
        nreq = requests_override or 32
        reqs = []
        uid = 0
        for _ in range(nreq):
            target = int(rng.integers(2048, 16385))
            lens = []
            left = target
            while left > 0:
                ln = int(rng.integers(256, 1025))
                ln = min(ln, left)
                if ln < 256 and lens:
                    lens[-1] += ln          # short tail merges into the previous unit
                else:
                    lens.append(ln)
                left -= ln
            segs = []
            for ln in lens:
                cached = rng.random() >= 0.2
                k = int(round(0.15 * ln))
                rec = np.sort(rng.choice(ln, size=k, replace=False)) if cached else ()
                segs.append(_UnitSpec(("x", uid), ln, cached=cached, recompute=rec))
                uid += 1
            segs.append(128)
            reqs.append(segs)
        return build_workload("c5-mixed-70b", shape, reqs, rng)
    raise ValueError("config index must be 1..5")


def adversarial(seed: int = 7, shape: Optional[ModelShape] = None) -> Workload:
    """Small batch exercising what the five configurations never do: units cached
    at non-zero positions, negative shifts, keys cached without rotation
    (stride 0), a unit used twice, unaligned targets, ragged last pages, an
    uncached unit and scattered recompute offsets."""
    rng = np.random.default_rng(seed)
    shape = shape or ModelShape(8, 2, 64, 16, 10000.0)
    r0 = [5,
          _UnitSpec("a", 37, cached_pos=150, recompute=(0, 1)),          # moves backwards: delta < 0
          3,
          _UnitSpec("b", 64, cached_pos=0, stride=0, recompute=(0,)),    # cached without rotation
          _UnitSpec("c", 21, cached_pos=9, recompute=(0, 5, 20)),
          _UnitSpec("d", 30, cached=False),
          11]
    r1 = [_UnitSpec("c", 21, cached_pos=9, recompute=()),                # target 0, delta = -9
          _UnitSpec("a", 37, cached_pos=150, recompute=(3, 36)),
          _UnitSpec("e", 16, cached_pos=37 + 21, recompute=(0,)),        # delta == 0: exact copy
          1]
    r2 = [2]                                                             # no unit at all
    return build_workload("adversarial", shape, [r0, r1, r2], rng)


def unit(length, uid=None, cached=True, cached_pos=0, stride=1, recompute=()):
    """Public constructor of a context-unit segment for build_workload()."""
    return _UnitSpec(uid if uid is not None else object(), length, cached, cached_pos, stride, recompute)


@dataclasses.dataclass
class LayerTensors:
    k_pool: torch.Tensor   # [num_pages, page, H_kv, D] bf16
    v_pool: torch.Tensor
    q: torch.Tensor        # [n_q, H_q, D]
    k_new: torch.Tensor    # [n_q, H_kv, D]
    v_new: torch.Tensor


def make_tensors(w: Workload, layer: int = 0, device: str = "cpu", seed: Optional[int] = None) -> LayerTensors:
    """N(0,1) bf16 tensors for one layer, drawn on `device` from a per-layer seed.
    CPU and CUDA generators give different streams; parity always reads back the
    very bytes the GPU consumed."""
    s = (BASE_SEED if seed is None else seed) * 1000003 + layer
    g = torch.Generator(device=device)
    g.manual_seed(s)
    sh = w.shape

    def draw(*dims):
        return torch.randn(*dims, generator=g, device=device, dtype=torch.float32).to(torch.bfloat16)

    pool_dims = (w.num_pool_pages, sh.page_size, sh.num_kv_heads, sh.head_dim)
    return LayerTensors(
        k_pool=draw(*pool_dims), v_pool=draw(*pool_dims),
        q=draw(max(w.n_q, 1), sh.num_q_heads, sh.head_dim)[: w.n_q],
        k_new=draw(max(w.n_q, 1), sh.num_kv_heads, sh.head_dim)[: w.n_q],
        v_new=draw(max(w.n_q, 1), sh.num_kv_heads, sh.head_dim)[: w.n_q])


# ---- byte / flop model used by the bench (Sec. 2.4's per-token KV size) --------

def kv_bytes_per_token(n_layers: int, num_kv_heads: int, head_dim: int, width_bytes: int, tp: int = 1) -> int:
    """KV state per token per rank: 2 * L * (H_kv / TP) * d_h * w  (Sec. 2.4)."""
    return 2 * n_layers * (num_kv_heads // tp) * head_dim * width_bytes


def gather_bytes(w: Workload) -> int:
    """Algorithmic bytes of gather + RoPE shift for one layer: every cached token's
    K and V row is read once and written once."""
    return 2 * w.cached_tokens * kv_bytes_per_token(1, w.shape.num_kv_heads, w.shape.head_dim, 2)


def attention_flops(w: Workload) -> int:
    """Algorithmic flops of the partial prefill for one layer: 4*D per unmasked
    (query, key) pair and query head (QK^T and PV, multiply-add = 2)."""
    return 4 * w.shape.head_dim * w.shape.num_q_heads * w.qk_pairs
