"""Seeded synthetic inputs for the KV-reuse hot path.

This module only *draws inputs*: token streams with shared prefixes, residency plans for the
index, pod loads, block-id lists and KV pool contents.  It holds none of the method's
arithmetic (no hashing of tokens, no index, no matching, no scoring, no copying) and is the
one module that both the GPU tests/benchmark and the CPU oracle's tests are allowed to share.

The traffic imitates the structure of the workloads the paper evaluates on (Section 3.2.5 and
Table 1: text-to-SQL style requests, i.e. long shared schema/system prompts followed by short
unique questions) and Llama-class KV shapes; no item of any public dataset is reproduced.

All randomness comes from one counter-based 64-bit generator (the published splitmix64
finaliser over ``seed`` and a counter), so any slice of any stream can be regenerated
independently - that is what lets a 100 GiB pool be checked without holding it on the host.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass, field
from typing import Optional

import numpy as np

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_SEEDMUL = np.uint64(0xD1B54A32D192ED03)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)

NO_BLOCK = 0xFFFFFFFF


def mix64(seed: int, counter) -> np.ndarray:
    """Counter-based generator: splitmix64's output function of (counter+1)*GOLD + seed*SEEDMUL."""
    c = np.asarray(counter, dtype=np.uint64)
    with np.errstate(over="ignore"):
        z = (c + np.uint64(1)) * _GOLD + np.uint64(seed & 0xFFFFFFFFFFFFFFFF) * _SEEDMUL
        z = (z ^ (z >> np.uint64(30))) * _C1
        z = (z ^ (z >> np.uint64(27))) * _C2
        z = z ^ (z >> np.uint64(31))
    return z


def pool_words(seed: int, first_word: int, n_words: int) -> np.ndarray:
    """Logical KV content: 64-bit word w of the block-major byte stream is mix64(seed, w)."""
    return mix64(seed, np.arange(first_word, first_word + n_words, dtype=np.uint64))


def pool_bytes(seed: int, first_byte: int, n_bytes: int) -> np.ndarray:
    """Bytes [first_byte, first_byte+n_bytes) of the little-endian logical stream (8-aligned)."""
    assert first_byte % 8 == 0 and n_bytes % 8 == 0
    return pool_words(seed, first_byte // 8, n_bytes // 8).astype("<u8").view(np.uint8)


class Stream:
    """Sequential reader over mix64(seed, 0), mix64(seed, 1), ..."""

    def __init__(self, seed: int, tag: int = 0):
        self.seed = seed * 1000003 + tag      # independent sub-stream per (seed, tag)
        self.pos = 0

    def u64(self, n: int) -> np.ndarray:
        out = mix64(self.seed, np.arange(self.pos, self.pos + n, dtype=np.uint64))
        self.pos += n
        return out

    def unit(self, n: int) -> np.ndarray:
        """Uniform doubles in [0, 1)."""
        return (self.u64(n) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)

    def randint(self, lo: int, hi: int, n: int) -> np.ndarray:
        """Uniform int64 in [lo, hi)."""
        return (lo + np.floor(self.unit(n) * (hi - lo))).astype(np.int64)

    def normal(self, n: int) -> np.ndarray:
        u1 = 1.0 - self.unit(n)
        u2 = self.unit(n)
        return np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)

    def permutation(self, n: int) -> np.ndarray:
        return np.argsort(self.u64(n), kind="stable").astype(np.int64)

    def zipf(self, k: int, s: float, n: int) -> np.ndarray:
        """Ranks 0..k-1 with probability proportional to 1/(rank+1)^s (s = 0: uniform)."""
        w = 1.0 / np.power(np.arange(1, k + 1, dtype=np.float64), s)
        cdf = np.cumsum(w) / np.sum(w)
        return np.minimum(np.searchsorted(cdf, self.unit(n), side="right"), k - 1).astype(np.int64)

    def keys(self, n: int) -> np.ndarray:
        """Random 64-bit keys avoiding the two reserved values 0 and ~0."""
        k = self.u64(n)
        bad = (k == np.uint64(0)) | (k == _M64)
        k[bad] = np.uint64(0x1234567)
        return k


# ------------------------------------------------------------------------------------------
# specifications


@dataclass
class RoutingSpec:
    """Requests + index content for hash -> match -> score."""

    name: str
    seed: int
    R: int
    block_tokens: int
    vocab: int
    len_dist: str                 # "uniform" | "loguniform" | "normal" | "fixed"
    len_lo: int
    len_hi: int
    len_mean: float = 0.0
    len_sd: float = 0.0
    n_prompts: int = 0            # shared prefixes
    prompt_lo: int = 0
    prompt_hi: int = 0            # inclusive
    share_prob: float = 0.0       # probability that a request starts with a shared prompt
    zipf_s: float = 0.0
    num_pods: int = 4
    capacity: int = 2048
    n_entries: int = 1024
    residency: str = "prefix_closed"   # | "random_nonzero"
    resident_q: float = 0.5
    id_space: int = 256           # block ids are drawn below this
    cached_frac: float = 0.0      # > 0: each request's own first blocks are cached (no prompts)
    load_hi: int = 256


@dataclass
class KVSpec:
    """Paged pool shape and the gather/scatter batches."""

    name: str
    seed: int
    layout: int                   # 0 block-major, 1 layer-major, 2 layer-major with split K and V
    num_layers: int
    num_kv_heads: int
    block_tokens: int
    head_dim: int
    elem_bytes: int
    num_blocks: int
    content: str = "mix64"        # | "normal_bf16"

    @property
    def tile_bytes(self) -> int:
        return 2 * self.num_kv_heads * self.block_tokens * self.head_dim * self.elem_bytes

    @property
    def block_bytes(self) -> int:
        return self.num_layers * self.tile_bytes

    @property
    def pool_bytes(self) -> int:
        return self.num_blocks * self.block_bytes


@dataclass
class RoutingWorkload:
    spec: RoutingSpec
    tokens: np.ndarray            # int32, all requests concatenated
    tok_off: np.ndarray           # int64 [R+1]
    src_tokens: np.ndarray        # int32: sequences whose full-block chains are cached
    src_tok_off: np.ndarray       # int64 [S+1]
    src_masks: np.ndarray         # uint64 per full block of the sources, source by source
    src_ids: np.ndarray           # uint32, same indexing
    filler_keys: np.ndarray       # uint64 random keys that match nothing
    filler_masks: np.ndarray
    filler_ids: np.ndarray
    pod_load: np.ndarray          # int32 [P]
    ready_mask: int
    block_table: Optional[np.ndarray] = None   # [R, blocks per request] (long-context case)
    prompt_of_request: Optional[np.ndarray] = None


def _lengths(spec: RoutingSpec, st: Stream) -> np.ndarray:
    if spec.len_dist == "uniform":
        return st.randint(spec.len_lo, spec.len_hi + 1, spec.R)
    if spec.len_dist == "loguniform":
        u = st.unit(spec.R)
        v = np.floor(np.exp(np.log(spec.len_lo) + u * (np.log(spec.len_hi) - np.log(spec.len_lo))))
        return np.clip(v, spec.len_lo, spec.len_hi).astype(np.int64)
    if spec.len_dist == "normal":
        v = np.rint(spec.len_mean + spec.len_sd * st.normal(spec.R))
        return np.clip(v, spec.len_lo, spec.len_hi).astype(np.int64)
    if spec.len_dist == "fixed":
        return np.full(spec.R, spec.len_lo, dtype=np.int64)
    raise ValueError(spec.len_dist)


def _offsets(lens: np.ndarray) -> np.ndarray:
    off = np.zeros(len(lens) + 1, dtype=np.int64)
    np.cumsum(lens, out=off[1:])
    return off


def _prefix_closed_masks(nblk: np.ndarray, P: int, q: float, st: Stream) -> np.ndarray:
    """Per source: pod p holds blocks [0, L_p); L_p = 0 w.p. 1-q, else uniform in [1, n]; one
    random pod holds the whole source.  Returns one mask per block, source by source."""
    S = len(nblk)
    resident = st.unit(S * P).reshape(S, P) < q
    upto = np.floor(st.unit(S * P).reshape(S, P) * nblk[:, None]).astype(np.int64) + 1
    upto = np.where(resident, upto, 0)
    full = st.randint(0, P, S)
    upto[np.arange(S), full] = nblk
    masks = []
    for s in range(S):
        i = np.arange(nblk[s], dtype=np.int64)[:, None]          # [n, 1]
        bits = (i < upto[s][None, :]).astype(np.uint64)          # [n, P]
        weights = np.left_shift(np.uint64(1), np.arange(P, dtype=np.uint64))
        masks.append((bits * weights[None, :]).sum(axis=1, dtype=np.uint64))
    return np.concatenate(masks) if masks else np.zeros(0, dtype=np.uint64)


def _random_nonzero_masks(n: int, P: int, st: Stream) -> np.ndarray:
    allm = (1 << P) - 1 if P < 64 else 0xFFFFFFFFFFFFFFFF
    m = st.u64(n) & np.uint64(allm)
    m[m == 0] = np.uint64(1)
    return m


def build_routing(spec: RoutingSpec) -> RoutingWorkload:
    B, P = spec.block_tokens, spec.num_pods
    st = Stream(spec.seed, 1)
    lens = _lengths(spec, st)
    tok_off = _offsets(lens)
    tokens = st.randint(0, spec.vocab, int(tok_off[-1])).astype(np.int32)
    block_table = None
    prompt_of_request = None

    if spec.cached_frac > 0.0:
        # every request is its own source: its first cached_frac of blocks are in the cache
        nblk_req = lens // B
        n_cached = np.floor(nblk_req * spec.cached_frac).astype(np.int64)
        src_lens = n_cached * B
        src_tok_off = _offsets(src_lens)
        src_tokens = np.concatenate(
            [tokens[tok_off[r]: tok_off[r] + src_lens[r]] for r in range(spec.R)]
        ).astype(np.int32)
        per = int(nblk_req.max())
        assert int(nblk_req.min()) == per, "long-context case uses equal-length requests"
        assert per * spec.R <= spec.id_space
        block_table = np.stack(
            [r * per + st.permutation(per) for r in range(spec.R)]
        ).astype(np.uint32)
        src_ids = np.concatenate(
            [block_table[r, : n_cached[r]] for r in range(spec.R)]
        ).astype(np.uint32)
        src_nblk = n_cached
    else:
        st = Stream(spec.seed, 7)             # prompts and who shares them
        plen = st.randint(spec.prompt_lo, spec.prompt_hi + 1, spec.n_prompts)
        src_tok_off = _offsets(plen)
        src_tokens = st.randint(0, spec.vocab, int(src_tok_off[-1])).astype(np.int32)
        shares = st.unit(spec.R) < spec.share_prob
        which = st.zipf(max(spec.n_prompts, 1), spec.zipf_s, spec.R)
        prompt_of_request = np.where(shares, which, -1)
        for r in range(spec.R):
            if shares[r] and spec.n_prompts > 0:
                j = int(which[r])
                k = int(min(plen[j], lens[r]))
                tokens[tok_off[r]: tok_off[r] + k] = src_tokens[src_tok_off[j]: src_tok_off[j] + k]
        src_nblk = plen // B
        total_src = int(src_nblk.sum())
        assert total_src <= spec.id_space, "prefix blocks need distinct pool ids"
        src_ids = st.permutation(spec.id_space)[:total_src].astype(np.uint32)

    total_src = int(src_nblk.sum())
    st = Stream(spec.seed, 5)                 # residency, filler entries, pod load
    if spec.residency == "prefix_closed":
        src_masks = _prefix_closed_masks(src_nblk, P, spec.resident_q, st)
    else:
        src_masks = _random_nonzero_masks(total_src, P, st)

    n_fill = max(spec.n_entries - total_src, 0)
    filler_keys = st.keys(n_fill)
    filler_masks = _random_nonzero_masks(n_fill, P, st)
    filler_ids = st.randint(0, spec.id_space, n_fill).astype(np.uint32)
    pod_load = st.randint(0, spec.load_hi, P).astype(np.int32)
    ready = (1 << P) - 1 if P < 64 else 0xFFFFFFFFFFFFFFFF
    return RoutingWorkload(spec, tokens, tok_off, src_tokens, src_tok_off, src_masks, src_ids,
                           filler_keys, filler_masks, filler_ids, pod_load, ready, block_table,
                           prompt_of_request)


# ------------------------------------------------------------------------------------------
# KV pool content and id lists


def bf16_normal_bits(seed: int, n: int) -> np.ndarray:
    """n bf16 bit patterns of N(0,1) draws (round-to-nearest-even from float32), as uint16."""
    x = Stream(seed, 2).normal(n).astype(np.float32).view(np.uint32)
    rounded = x + np.uint32(0x7FFF) + ((x >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def host_pool(kv: KVSpec) -> np.ndarray:
    """Whole pool as host bytes in its PHYSICAL layout (small pools only)."""
    assert kv.pool_bytes <= (2 << 30), "host_pool is for small pools"
    if kv.content == "normal_bf16":
        assert kv.elem_bytes == 2
        logical = bf16_normal_bits(kv.seed, kv.pool_bytes // 2).astype("<u2").view(np.uint8)
    else:
        logical = pool_bytes(kv.seed, 0, kv.pool_bytes)
    return to_physical(kv, np.ascontiguousarray(logical), kv.num_blocks)


def to_physical(kv: KVSpec, logical: np.ndarray, n: int) -> np.ndarray:
    """Block-major bytes of n blocks ([block][layer][K half][V half]) placed as a pool of n blocks
    in kv's physical layout.  Placement of generated content only."""
    if kv.layout == 0:
        return logical
    if kv.layout == 1:
        t = logical.reshape(n, kv.num_layers, kv.tile_bytes)
        return np.ascontiguousarray(t.transpose(1, 0, 2)).reshape(-1)
    t = logical.reshape(n, kv.num_layers, 2, kv.tile_bytes // 2)
    return np.ascontiguousarray(t.transpose(1, 2, 0, 3)).reshape(-1)       # [layer][K/V][block]


def logical_blocks(kv: KVSpec, ids) -> np.ndarray:
    """Content of the given blocks as a block-major mini-pool [len(ids) * block_bytes]."""
    assert kv.content == "mix64"
    from . import synth

    out = np.empty((len(ids), kv.block_bytes), dtype=np.uint8)
    for j, b in enumerate(ids):
        synth.fill_host(out[j], kv.seed, int(b) * kv.block_bytes)   # == pool_bytes(...), natively
    return out.reshape(-1)


def physical_blocks(kv: KVSpec, b0: int, b1: int) -> np.ndarray:
    """Generated content of blocks [b0, b1) laid out as a pool of b1 - b0 blocks in kv's
    PHYSICAL layout (what a slice of the real pool holds before anything is scattered)."""
    assert kv.content == "mix64"
    from . import synth

    n = b1 - b0
    logical = np.empty(n * kv.block_bytes, dtype=np.uint8)
    synth.fill_host(logical, kv.seed, b0 * kv.block_bytes)
    return to_physical(kv, logical, n)


def distinct_ids(seed: int, num_blocks: int, n: int) -> np.ndarray:
    """n block ids drawn uniformly without replacement."""
    assert n <= num_blocks
    return Stream(seed, 3).permutation(num_blocks)[:n].astype(np.uint32)


# ------------------------------------------------------------------------------------------
# the five configurations (seed = configuration number - 1)


def cfg1_routing() -> RoutingSpec:
    return RoutingSpec(name="cfg1-tiny", seed=0, R=8, block_tokens=16, vocab=32000,
                       len_dist="uniform", len_lo=64, len_hi=512, n_prompts=2, prompt_lo=128,
                       prompt_hi=128, share_prob=0.5, zipf_s=0.0, num_pods=4, capacity=2048,
                       n_entries=1024, residency="random_nonzero", id_space=256)


def cfg1_kv() -> KVSpec:
    return KVSpec(name="cfg1-tiny", seed=0, layout=0, num_layers=2, num_kv_heads=4,
                  block_tokens=16, head_dim=64, elem_bytes=2, num_blocks=256,
                  content="normal_bf16")


def cfg2_routing() -> RoutingSpec:
    return RoutingSpec(name="cfg2-llama3-8b", seed=1, R=64, block_tokens=16, vocab=128256,
                       len_dist="loguniform", len_lo=1024, len_hi=8192, n_prompts=32,
                       prompt_lo=512, prompt_hi=2048, share_prob=1.0, zipf_s=1.1, num_pods=16,
                       capacity=1 << 19, n_entries=200000, residency="prefix_closed",
                       resident_q=0.5, id_space=4096)


def cfg2_kv() -> KVSpec:
    return KVSpec(name="cfg2-llama3-8b", seed=1, layout=0, num_layers=32, num_kv_heads=8,
                  block_tokens=16, head_dim=128, elem_bytes=2, num_blocks=4096)


def cfg3_routing() -> RoutingSpec:
    return RoutingSpec(name="cfg3-routing-heavy", seed=2, R=4096, block_tokens=16, vocab=128256,
                       len_dist="normal", len_lo=256, len_hi=8192, len_mean=2048.0, len_sd=512.0,
                       n_prompts=256, prompt_lo=128, prompt_hi=1024, share_prob=0.6, zipf_s=1.0,
                       num_pods=64, capacity=1 << 21, n_entries=1 << 20,
                       residency="prefix_closed", resident_q=0.125, id_space=1 << 20)


def cfg4_kv() -> KVSpec:
    return KVSpec(name="cfg4-llama3-70b", seed=3, layout=1, num_layers=80, num_kv_heads=8,
                  block_tokens=16, head_dim=128, elem_bytes=2, num_blocks=20000)


def cfg5_routing() -> RoutingSpec:
    return RoutingSpec(name="cfg5-long-context-fp8", seed=4, R=32, block_tokens=32, vocab=128256,
                       len_dist="fixed", len_lo=128000, len_hi=128000, num_pods=32,
                       capacity=1 << 23, n_entries=1 << 22, residency="prefix_closed",
                       resident_q=0.5, id_space=128000, cached_frac=0.75)


def cfg5_kv() -> KVSpec:
    return KVSpec(name="cfg5-long-context-fp8", seed=4, layout=0, num_layers=28, num_kv_heads=4,
                  block_tokens=32, head_dim=128, elem_bytes=1, num_blocks=128000)


def scaled(spec, **changes):
    """A copy of a specification with some fields replaced (reduced sizes for CPU tests)."""
    return dataclasses.replace(spec, **changes)
