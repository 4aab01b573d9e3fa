"""Seeded synthetic inputs for the multi-tenant LoRA layer.

This module only *draws numbers*: it contains no part of the layer's arithmetic
(no products, no gradients), so that the CPU oracle and the CUDA path can both be fed
from it without sharing any of the method's code.  Everything is a pure function of
(seed, tensor id, element index): a 64-bit counter hash gives two uniforms per element,
Box-Muller turns them into a normal deviate, and the value is rounded to bf16
(round-to-nearest-even) because the layer's inputs are bf16 tensors.

The five workloads mirror the shapes of the paper's multi-task RLVR runs (Experimental
Setup: up to 32 concurrent tasks, 10 replicas, generation lengths up to 4096, decode
batches of one token per sequence); the paper's datasets themselves are not used.

Arrays are numpy: bf16 tensors are returned as ``uint16`` bit patterns (``*_bits``) and
the same values widened exactly to ``float32``.
"""
from __future__ import annotations

import concurrent.futures
import dataclasses
import math
import os
from typing import Dict, List, Optional

import numpy as np

BASE_SEED = 0x4D41524C  # "MARL"

# tensor ids of the counter hash
TID_W, TID_X, TID_DY, TID_A, TID_B, TID_TABLE, TID_RANKS, TID_PERTURB = 1, 2, 3, 4, 5, 6, 7, 8

_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_GOLD = np.uint64(0x9E3779B97F4A7C15)


def _mix64(z: np.ndarray) -> np.ndarray:
    """SplitMix64 finaliser, vectorised over a uint64 array (wraps modulo 2**64)."""
    z = (z ^ (z >> np.uint64(30))) * _M1
    z = (z ^ (z >> np.uint64(27))) * _M2
    return z ^ (z >> np.uint64(31))


def _stream_key(seed: int, tensor_id: int, sub: int = 0) -> np.uint64:
    k = (seed * 0x9E3779B97F4A7C15 + tensor_id * 0xD1B54A32D192ED03 + sub * 0x8CB92BA72F3D8DD7) & (2**64 - 1)
    with np.errstate(over="ignore"):
        return _mix64(np.array([k], dtype=np.uint64))[0]


def hash_u64(seed: int, tensor_id: int, index: np.ndarray, sub: int = 0) -> np.ndarray:
    """64 hashed bits per counter value ``index`` (any integer array)."""
    key = _stream_key(seed, tensor_id, sub)
    with np.errstate(over="ignore"):
        return _mix64(index.astype(np.uint64) * _GOLD + key)


def uniform01(seed: int, tensor_id: int, index: np.ndarray, sub: int = 0) -> np.ndarray:
    """Uniform doubles in (0, 1): top 53 bits of the hash, offset by half an ulp."""
    h = hash_u64(seed, tensor_id, index, sub)
    return ((h >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def f32_to_bf16_bits(v: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (1-8-7), round-to-nearest-even; returns uint16 bit patterns."""
    b = np.ascontiguousarray(v, dtype=np.float32).view(np.uint32)
    bias = np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))
    return ((b + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(seed: int, tensor_id: int, shape, sigma: float, sub: int = 0, chunk: int = 1 << 21):
    """bf16-rounded N(0, sigma^2) tensor -> (bits uint16, values float32), element i of the
    flattened tensor uses counters 2i and 2i+1.  Chunks are drawn on a thread pool (the result does
    not depend on the chunking: every element is a pure function of its index)."""
    n = int(np.prod(shape))
    bits = np.empty(n, dtype=np.uint16)

    def fill(lo):
        hi = min(n, lo + chunk)
        idx = np.arange(lo, hi, dtype=np.uint64)
        u1 = uniform01(seed, tensor_id, idx * np.uint64(2), sub)
        u2 = uniform01(seed, tensor_id, idx * np.uint64(2) + np.uint64(1), sub)
        z = np.sqrt(-2.0 * np.log(u1)) * np.cos((2.0 * math.pi) * u2)
        bits[lo:hi] = f32_to_bf16_bits((z * sigma).astype(np.float32))

    starts = list(range(0, n, chunk))
    if len(starts) <= 1:
        for lo in starts:
            fill(lo)
    else:
        with concurrent.futures.ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
            list(ex.map(fill, starts))
    bits = bits.reshape(shape)
    return bits, bf16_bits_to_f32(bits)


@dataclasses.dataclass
class Adapter:
    """One tenant's LoRA parameters: A is d_in x rank, B is rank x d_out, scale = alpha / rank."""
    tenant_id: int
    rank: int
    alpha: float
    A_bits: np.ndarray
    B_bits: np.ndarray

    @property
    def scale(self) -> float:
        return self.alpha / self.rank if self.rank > 0 else 0.0

    @property
    def A(self) -> np.ndarray:
        return bf16_bits_to_f32(self.A_bits)

    @property
    def B(self) -> np.ndarray:
        return bf16_bits_to_f32(self.B_bits)


@dataclasses.dataclass
class Projection:
    """One adapted projection: a frozen base weight shared by all tenants plus one adapter per tenant."""
    name: str
    d_in: int
    d_out: int
    W_bits: np.ndarray
    adapters: List[Adapter]
    x_bits: np.ndarray                  # [T][d_in]
    dy_bits: Optional[np.ndarray]       # [T_bwd][d_out] or None (forward-only workload)
    # Several projections over one input served as one layer (a pool over several projections): their widths.  W and
    # dy hold them side by side; an adapter of rank r then has A_bits [d_in][P r] (the A's side by side) and B_bits
    # [r][d_out] (the B's side by side), and output range p pairs columns p r .. (p+1) r of A with its columns of B.
    parts: Optional[List[int]] = None

    @property
    def W(self) -> np.ndarray:
        return bf16_bits_to_f32(self.W_bits)

    @property
    def x(self) -> np.ndarray:
        return bf16_bits_to_f32(self.x_bits)

    @property
    def dy(self) -> Optional[np.ndarray]:
        return None if self.dy_bits is None else bf16_bits_to_f32(self.dy_bits)


@dataclasses.dataclass
class Workload:
    """A mixed batch: the token-to-adapter segment table plus the projections it is run through.

    seg_offsets[S+1] / seg_slot[S] describe contiguous token ranges; slot j means the j-th
    adapter of every projection (slot -1 = base weight only).  ``T_bwd`` rows (a prefix of
    the batch) take part in the backward pass; 0 means forward only.
    """
    name: str
    T: int
    T_bwd: int
    seg_offsets: np.ndarray
    seg_slot: np.ndarray
    projections: List[Projection]
    n_tenants: int
    max_rank: int

    def tok_slot(self) -> np.ndarray:
        """Per-token slot by plain expansion of the table (input bookkeeping, not the method's index build)."""
        out = np.empty(self.T, dtype=np.int32)
        for s in range(len(self.seg_slot)):
            out[self.seg_offsets[s]:self.seg_offsets[s + 1]] = self.seg_slot[s]
        return out


def _make_adapters(seed, n, ranks, alphas, d_in, d_out, proj_index) -> List[Adapter]:
    out = []
    for t in range(n):
        r = int(ranks[t])
        a_bits, _ = normal_bf16(seed, TID_A, (d_in, r), 0.02, sub=proj_index * 4096 + t)
        b_bits, _ = normal_bf16(seed, TID_B, (r, d_out), 0.02, sub=proj_index * 4096 + t)
        out.append(Adapter(tenant_id=1000 + t, rank=r, alpha=float(alphas[t]), A_bits=a_bits, B_bits=b_bits))
    return out


def _make_projection(seed, name, d_in, d_out, n, ranks, alphas, T, T_bwd, proj_index, x_group) -> Projection:
    w_bits, _ = normal_bf16(seed, TID_W, (d_in, d_out), 0.02, sub=proj_index)
    x_bits, _ = normal_bf16(seed, TID_X, (T, d_in), 1.0, sub=x_group)
    dy_bits = None
    if T_bwd > 0:
        dy_bits, _ = normal_bf16(seed, TID_DY, (T_bwd, d_out), 1.0, sub=proj_index)
    return Projection(name, d_in, d_out, w_bits, _make_adapters(seed, n, ranks, alphas, d_in, d_out, proj_index),
                      x_bits, dy_bits)


def lognormal_segments(seed: int, T: int, n_tenants: int, sub: int = 0, shrink: int = 1):
    """Per-tenant training segments: lengths clip(round(exp(N(ln 1024, 0.6^2))), 128, 4096) drawn until
    they cover T tokens; the last one is shortened to fit and, if that leaves fewer than 128 tokens,
    merged into its predecessor.  Segment j (after a seeded shuffle of the order) belongs to tenant
    j mod n_tenants.  ``shrink`` divides median and clip bounds (scaled-down test cases)."""
    med, lo_len, hi_len = 1024.0 / shrink, max(1, 128 // shrink), max(1, 4096 // shrink)
    lens = []
    total, c = 0, 0
    while total < T:
        idx = np.array([2 * c, 2 * c + 1], dtype=np.uint64)
        u = uniform01(seed, TID_TABLE, idx, sub)
        z = math.sqrt(-2.0 * math.log(u[0])) * math.cos(2.0 * math.pi * u[1])
        L = int(min(hi_len, max(lo_len, round(math.exp(math.log(med) + 0.6 * z)))))
        lens.append(L)
        total += L
        c += 1
    lens[-1] -= total - T
    if lens[-1] < lo_len and len(lens) > 1:
        lens[-2] += lens[-1]
        lens.pop()
    S = len(lens)
    slots = np.arange(S, dtype=np.int64) % n_tenants
    # seeded Fisher-Yates shuffle of the (length, tenant) pairs
    order = np.arange(S)
    for i in range(S - 1, 0, -1):
        h = int(hash_u64(seed, TID_TABLE, np.array([1_000_000 + i], dtype=np.uint64), sub)[0])
        j = h % (i + 1)
        order[i], order[j] = order[j], order[i]
    lens = np.asarray(lens, dtype=np.int64)[order]
    slots = slots[order]
    offsets = np.zeros(S + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(lens)
    return offsets, slots.astype(np.int32)


def uniform_token_slots(seed: int, T: int, n_tenants: int, sub: int = 0) -> np.ndarray:
    """Decode batch: one tenant id per token, uniform over the tenants, unsorted."""
    h = hash_u64(seed, TID_TABLE, np.arange(T, dtype=np.uint64), sub + 77)
    return (h % np.uint64(n_tenants)).astype(np.int32)


def zipf_segments(seed: int, T: int, n_tenants: int, s: float = 1.1, max_len: int = 2048, sub: int = 0):
    # scaled-down callers pass a smaller max_len
    """Skewed mixed batch: each segment's tenant ~ Zipf(s) over the tenants (P(t) ~ (t+1)^-s) and its
    length is a log-uniform integer in [1, max_len]; the last segment is truncated to fit T."""
    p = np.arange(1, n_tenants + 1, dtype=np.float64) ** (-s)
    cdf = np.cumsum(p / p.sum())
    lens, slots = [], []
    total, c = 0, 0
    while total < T:
        u = uniform01(seed, TID_TABLE, np.array([2 * c, 2 * c + 1], dtype=np.uint64), sub + 31)
        t = int(min(n_tenants - 1, np.searchsorted(cdf, u[0], side="right")))
        L = int(min(max_len, max(1, math.floor(math.exp(u[1] * math.log(max_len + 1.0))))))
        L = min(L, T - total)
        lens.append(L)
        slots.append(t)
        total += L
        c += 1
    offsets = np.zeros(len(lens) + 1, dtype=np.int32)
    offsets[1:] = np.cumsum(lens)
    return offsets, np.asarray(slots, dtype=np.int32)


def per_token_table(tok_slot: np.ndarray):
    T = len(tok_slot)
    return np.arange(T + 1, dtype=np.int32), np.asarray(tok_slot, dtype=np.int32)


def make_workload(cfg: int, scale_down: int = 1, seed: Optional[int] = None) -> Workload:
    """Build workload ``cfg`` in 1..5.  ``scale_down`` > 1 divides the token count and the weight
    dimensions by that factor (kept multiples of 64) to get a same-structure case the oracle can
    finish quickly; 1 gives the full-size configuration."""
    seed = BASE_SEED + cfg if seed is None else seed
    sd = scale_down

    def dim(v):
        return max(64, (v // sd) // 64 * 64)

    if cfg == 1:
        K = N = dim(512)
        n, T = 4, max(8, 256 // sd)
        q = T // 4
        offsets = np.array([0, q, 2 * q, 3 * q, T], dtype=np.int32)
        slots = np.arange(4, dtype=np.int32)
        ranks, alphas = [8] * n, [16.0] * n
        projs = [_make_projection(seed, "proj", K, N, n, ranks, alphas, T, T, 0, 0)]
        return Workload("cfg1-tiny", T, T, offsets, slots, projs, n, 8)
    if cfg == 2:
        K = N = dim(4096)
        n, T = 32, max(8, 256 // sd)
        offsets, slots = per_token_table(uniform_token_slots(seed, T, n))
        ranks, alphas = [16] * n, [32.0] * n
        projs = [_make_projection(seed, "proj", K, N, n, ranks, alphas, T, 0, 0, 0)]
        return Workload("cfg2-decode", T, 0, offsets, slots, projs, n, 16)
    if cfg == 3:
        K, N = dim(4096), dim(11008)
        n, T = 10, 16384 // sd
        offsets, slots = lognormal_segments(seed, T, n, shrink=sd)
        ranks, alphas = [32] * n, [64.0] * n
        projs = [_make_projection(seed, "up", K, N, n, ranks, alphas, T, T, 0, 0)]
        return Workload("cfg3-train", T, T, offsets, slots, projs, n, 32)
    if cfg == 4:
        K = N = dim(5120)
        n, T = 32, 8192 // sd
        offsets, slots = zipf_segments(seed, T, n, max_len=max(1, 2048 // sd))
        rk = hash_u64(seed, TID_RANKS, np.arange(n, dtype=np.uint64)) % np.uint64(4)
        ranks = [int((8, 16, 32, 64)[int(v)]) for v in rk]
        alphas = [16.0] * n
        projs = [_make_projection(seed, "proj", K, N, n, ranks, alphas, T, T, 0, 0)]
        return Workload("cfg4-hetero", T, T, offsets, slots, projs, n, 64)
    if cfg == 5:
        H, F = dim(4096), dim(11008)
        n = 32
        Tt, Td = 4096 // sd, max(8, 256 // sd)
        o1, s1 = lognormal_segments(seed, Tt, n, shrink=sd)
        o2, s2 = per_token_table(uniform_token_slots(seed, Td, n))
        offsets = np.concatenate([o1, (o2[1:] + Tt).astype(np.int32)]).astype(np.int32)
        slots = np.concatenate([s1, s2]).astype(np.int32)
        T = Tt + Td
        ranks, alphas = [16] * n, [32.0] * n
        shapes = [("q", H, H, 0), ("k", H, H, 0), ("v", H, H, 0), ("o", H, H, 1),
                  ("gate", H, F, 2), ("up", H, F, 2), ("down", F, H, 3)]
        projs = [_make_projection(seed, nm, di, do, n, ranks, alphas, T, Tt, pi, xg)
                 for pi, (nm, di, do, xg) in enumerate(shapes)]
        return Workload("cfg5-layer", T, Tt, offsets, slots, projs, n, 16)
    raise ValueError(f"unknown config {cfg}")


def fuse_projections(w: Workload, names: Optional[List[str]] = None, segmented: bool = False) -> Workload:
    """Several projections that read the same x (q, k, v; gate, up) as ONE adapted projection, so that one layer call
    serves them all: the base weights side by side ([d_in][sum d_out]), A_t side by side ([d_in][P r]), B_t block
    diagonal ([P r][sum d_out], block p = B_t of projection p over that projection's output columns, zeros elsewhere).
    Then y = x W + s (x A) B of the fused projection is the concatenation of the P separate layer outputs; the same
    holds for dx (their sum), dA (side by side) and the diagonal blocks of dB.  Needs the same rank and alpha on
    every projection of a tenant (so that one scale s = alpha / r serves all: the fused adapter gets alpha P).
    segmented = True keeps the tenants' B matrices side by side instead ([r][sum d_out], rank r, alpha unchanged) and
    records the projections' widths in Projection.parts: the layout of a pool over several projections, which stores
    and streams none of the block-diagonal form's zeros."""
    projs = [p for p in w.projections if names is None or p.name in names]
    assert projs and all(p.d_in == projs[0].d_in and (p.x_bits is projs[0].x_bits or np.array_equal(p.x_bits, projs[0].x_bits))
                         for p in projs), "projections must share x"
    P = len(projs)
    offs = np.concatenate([[0], np.cumsum([p.d_out for p in projs])]).astype(np.int64)
    adapters = []
    for t, a0 in enumerate(projs[0].adapters):
        parts = [p.adapters[t] for p in projs]
        assert all(a.rank == a0.rank and a.alpha == a0.alpha and a.tenant_id == a0.tenant_id for a in parts)
        r = a0.rank
        A_bits = np.concatenate([a.A_bits for a in parts], axis=1)
        if segmented:
            adapters.append(Adapter(a0.tenant_id, r, a0.alpha, np.ascontiguousarray(A_bits),
                                    np.ascontiguousarray(np.concatenate([a.B_bits for a in parts], axis=1))))
            continue
        B_bits = np.zeros((P * r, int(offs[-1])), dtype=np.uint16)
        for i, a in enumerate(parts):
            B_bits[i * r:(i + 1) * r, offs[i]:offs[i + 1]] = a.B_bits
        adapters.append(Adapter(a0.tenant_id, P * r, a0.alpha * P, np.ascontiguousarray(A_bits), B_bits))
    dy_bits = None if projs[0].dy_bits is None else np.ascontiguousarray(np.concatenate([p.dy_bits for p in projs], axis=1))
    fused = Projection("+".join(p.name for p in projs), projs[0].d_in, int(offs[-1]),
                       np.ascontiguousarray(np.concatenate([p.W_bits for p in projs], axis=1)), adapters, projs[0].x_bits, dy_bits)
    if segmented:
        fused.parts = [p.d_out for p in projs]
        return Workload(w.name + "-fused", w.T, w.T_bwd, w.seg_offsets, w.seg_slot, [fused], w.n_tenants, w.max_rank)
    return Workload(w.name + "-fused", w.T, w.T_bwd, w.seg_offsets, w.seg_slot, [fused], w.n_tenants, P * w.max_rank)


SWEEP_NAME = r"^(decode|prefill|qkv|qkvsep|qkvseg|gateup|gateupsep|gateupseg|decode\d+x\d+)-(\d+)-(\d+)$"

# Variants of the configured workloads (same tensors, another pass or another table):
VARIANTS = {
    "cfg3-fwd": "cfg3, forward only",
    "cfg3-alltenants": "cfg3 with a table of the same recipe in which all 10 tenants appear (13 to 16 segments)",
    "cfg5-decode": "the decode part of cfg5 alone: its 256 decode tokens through the 7 projections, forward only",
    "cfg5-alltenants": "cfg5 whose 4096 training rows hold all 32 tenants (same recipe, lengths divided by 8)",
    "cfg5-fused": "cfg5 with q, k, v and gate, up each served by one pool over the projections (4 calls per pass instead of 7)",
    "cfg5-decode-fused": "cfg5-decode with q, k, v and gate, up each served by one pool over the projections",
}


def _fuse_layer(w: Workload, name: str) -> Workload:
    """q, k, v and gate, up of a decoder-layer workload as one projection each (a pool over the projections)."""
    by = {p.name: p for p in w.projections}
    projs = [fuse_projections(w, ["q", "k", "v"], segmented=True).projections[0], by["o"],
             fuse_projections(w, ["gate", "up"], segmented=True).projections[0], by["down"]]
    return Workload(name, w.T, w.T_bwd, w.seg_offsets, w.seg_slot, projs, w.n_tenants, w.max_rank)


def _table_with_all_tenants(seed: int, T: int, n: int, shrink: int, lo: int, hi: int):
    """First table of the lognormal recipe (sub-stream 1, 2, ...) with lo..hi segments in which every tenant appears."""
    for sub in range(1, 200):
        off, sl = lognormal_segments(seed, T, n, sub=sub, shrink=shrink)
        if lo <= len(sl) <= hi and len(set(sl.tolist())) == n:
            return off, sl
    raise RuntimeError("no table with every tenant present in the first 200 sub-streams")


def make_variant(name: str, base: Optional[Workload] = None) -> Workload:
    """See VARIANTS.  ``base`` may pass the already generated cfg3 / cfg5 workload (generation is the slow part); its
    tensors are shared, not copied."""
    if name not in VARIANTS:
        raise ValueError(f"unknown variant {name!r}")
    cfg = int(name[3])
    w = base if base is not None else make_workload(cfg)
    if name == "cfg5-fused":
        return _fuse_layer(w, name)
    if name == "cfg5-decode-fused":
        return _fuse_layer(make_variant("cfg5-decode", w), name)
    if name == "cfg3-fwd":
        projs = [dataclasses.replace(p, dy_bits=None) for p in w.projections]
        return Workload(name, w.T, 0, w.seg_offsets, w.seg_slot, projs, w.n_tenants, w.max_rank)
    if name == "cfg3-alltenants":
        off, sl = _table_with_all_tenants(BASE_SEED + 3, w.T, w.n_tenants, 1, 13, 16)
        return Workload(name, w.T, w.T_bwd, off, sl, w.projections, w.n_tenants, w.max_rank)
    if name == "cfg5-decode":
        Tt = w.T_bwd
        keep = [s for s in range(len(w.seg_slot)) if w.seg_offsets[s] >= Tt]
        off = np.array([int(w.seg_offsets[s]) - Tt for s in keep] + [w.T - Tt], dtype=np.int32)
        projs = [dataclasses.replace(p, x_bits=np.ascontiguousarray(p.x_bits[Tt:]), dy_bits=None) for p in w.projections]
        # projections that shared their input keep sharing it
        first = {}
        for p, p0 in zip(projs, w.projections):
            key = id(p0.x_bits)
            if key in first:
                p.x_bits = first[key]
            else:
                first[key] = p.x_bits
        return Workload(name, w.T - Tt, 0, off, w.seg_slot[keep].astype(np.int32), projs, w.n_tenants, w.max_rank)
    if name == "cfg5-alltenants":
        Tt = w.T_bwd
        o1, s1 = _table_with_all_tenants(BASE_SEED + 5, Tt, w.n_tenants, 8, 32, 64)
        keep = [s for s in range(len(w.seg_slot)) if w.seg_offsets[s] >= Tt]
        o2 = np.array([int(w.seg_offsets[s]) for s in keep] + [w.T], dtype=np.int32)
        off = np.concatenate([o1[:-1], o2]).astype(np.int32)
        sl = np.concatenate([s1, w.seg_slot[keep]]).astype(np.int32)
        return Workload(name, w.T, w.T_bwd, off, sl, w.projections, w.n_tenants, w.max_rank)
    raise ValueError(name)


def make_named_workload(name: str) -> Workload:
    """``cfgN`` gives make_workload(N).  Two forward-only families for sweeps over the rollout phases, both on a
    4096 x 4096 base weight with rank-16 adapters of scale 2:

    ``decode-T-n``   T decode tokens (one per sequence), tenant of each token uniform over n tenants, unsorted;
    ``decodeKxN-T-n``  the same over a K x N base weight (the projections of decoder layers of other sizes);
    ``prefill-T-n``  T prompt tokens in whole-prompt segments (lognormal lengths, median 1024, clipped to
                     [128, 4096]) dealt to n tenants in shuffled order;
    ``qkv-T-n`` / ``gateup-T-n``  a decode batch through the fused q+k+v (4096 x 12288) or gate+up (4096 x 22016)
                     projection (adapters fused block-diagonally), ``qkvsep`` / ``gateupsep`` through the same
                     projections one call each, ``qkvseg`` / ``gateupseg`` through one pool over the projections."""
    import re
    if name.startswith("cfg") and name[3:].isdigit():
        return make_workload(int(name[3:]))
    if name in VARIANTS:
        return make_variant(name)
    m = re.match(SWEEP_NAME, name)
    if not m:
        raise ValueError(f"unknown workload {name!r}")
    kind, T, n = m.group(1), int(m.group(2)), int(m.group(3))
    if T < 1 or n < 1 or n > 4096:
        raise ValueError(f"workload {name!r}: need T >= 1 and 1 <= tenants <= 4096")
    if kind in ("qkv", "qkvsep", "qkvseg", "gateup", "gateupsep", "gateupseg"):
        # projections of a 7B-shaped decoder layer that share their input, on a decode batch: q, k, v 4096 x 4096 or
        # gate, up 4096 x 11008, rank 16 each; "...sep" runs them as separate projections (one call each), without
        # the suffix they are fused into one (fuse_projections)
        seed = BASE_SEED + 102
        names, N = (("q", "k", "v"), 4096) if kind.startswith("qkv") else (("gate", "up"), 11008)
        offsets, slots = per_token_table(uniform_token_slots(seed, T, n))
        ranks, alphas = [16] * n, [32.0] * n
        projs = [_make_projection(seed, nm, 4096, N, n, ranks, alphas, T, 0, pi, 0) for pi, nm in enumerate(names)]
        for p in projs[1:]:
            p.x_bits = projs[0].x_bits
        w = Workload(name, T, 0, offsets, slots, projs, n, 16)
        if kind.endswith("sep"):
            return w
        f = fuse_projections(w, segmented=kind.endswith("seg"))
        f.name = name
        return f
    seed = BASE_SEED + 100 + (0 if kind.startswith("decode") else 1)
    K = N = 4096
    if kind.startswith("decode") and kind != "decode":
        K, N = (int(v) for v in kind[6:].split("x"))
        if K % 8 or N % 8 or K < 8 or N < 8:
            raise ValueError(f"workload {name!r}: K and N must be multiples of 8")
    if kind.startswith("decode"):
        offsets, slots = per_token_table(uniform_token_slots(seed, T, n))
    else:
        offsets, slots = lognormal_segments(seed, T, n)
    ranks, alphas = [16] * n, [32.0] * n
    projs = [_make_projection(seed, "proj", K, N, n, ranks, alphas, T, 0, 0, 0)]
    return Workload(name, T, 0, offsets, slots, projs, n, 16)


def small_random_case(seed: int, T: int, K: int, N: int, ranks, alphas=None, n_segments: int = 6,
                      with_base_only: bool = True, sigma_w: float = 0.02) -> Workload:
    """Small ragged case for tests: random segment boundaries (zero-length segments allowed), tenants may
    recur in non-adjacent segments, one tenant may get no tokens, optional slot -1 segment."""
    n = len(ranks)
    alphas = [16.0] * n if alphas is None else alphas
    cuts = np.sort(hash_u64(seed, TID_TABLE, np.arange(n_segments - 1, dtype=np.uint64), 5) % np.uint64(T + 1))
    offsets = np.concatenate([[0], cuts.astype(np.int64), [T]]).astype(np.int32)
    pick = hash_u64(seed, TID_TABLE, np.arange(n_segments, dtype=np.uint64), 6)
    lo = -1 if with_base_only else 0
    span = max(1, n - 1) - lo            # the last tenant never appears: exercises "registered but absent"
    slots = (pick % np.uint64(span)).astype(np.int64) + lo
    w_bits, _ = normal_bf16(seed, TID_W, (K, N), sigma_w)
    x_bits, _ = normal_bf16(seed, TID_X, (T, K), 1.0)
    dy_bits, _ = normal_bf16(seed, TID_DY, (T, N), 1.0)
    proj = Projection("proj", K, N, w_bits, _make_adapters(seed, n, ranks, alphas, K, N, 0), x_bits, dy_bits)
    return Workload(f"small-{seed}", T, T, offsets, slots.astype(np.int32), [proj], n, max(ranks) if ranks else 0)
