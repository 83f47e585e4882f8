"""Seeded synthetic inputs for the chunk-attention path.

This module only *draws inputs*: request shapes (prefix length, chunk length),
block tables, and 16-bit Q/K/V bit patterns.  It contains none of the method's
arithmetic (no attention, no cache indexing) so that the CPU oracle and the
CUDA library can both be fed from it without sharing any code of their own.

Workload shapes follow the paper's traffic: 32 heads x 128 (7B-class) or
40 heads x 128 (13B-class) decoder layers (Sec. 4.1, model settings), 30 end
devices per batch (Sec. 4.1, testbed), prompt chunks of 64..512 tokens
(Sec. 2.3 chunk-size study; Sec. 4.1 baselines use 128/256), prompts up to a
few thousand tokens (Table 3), and short linear draft sequences for
verification (Sec. 3.4).  The benchmark prompts themselves are not used; these
are stand-ins with the same shape statistics.

Every KV pool is filled with N(0,1) values in *all* slots, including slots
beyond a request's prefix and pages no request owns: stale data that the path
must mask out (attention) or overwrite (append).
"""
from __future__ import annotations

import concurrent.futures as _cf
import dataclasses
from typing import List, Sequence

import numpy as np

PAGE_SIZE = 16
SEED_BASE = 18989 * 10  # shapes: SEED_BASE + config#, values: + 100

_FILL_CHUNK = 1 << 24  # elements per independently seeded fill chunk


# --------------------------------------------------------------------------
# 16-bit encodings (data preparation only)
# --------------------------------------------------------------------------
def f32_to_bits(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round float32 values to fp16 / bf16 (nearest even) and return uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "fp16":
        return x.astype(np.float16).view(np.uint16)
    if dtype == "bf16":
        u = x.view(np.uint32)
        r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
        return r.astype(np.uint16)
    raise ValueError(f"dtype {dtype!r}")


def bits_to_f64(bits: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of fp16 / bf16 bit patterns to float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    if dtype == "fp16":
        return bits.view(np.float16).astype(np.float64)
    if dtype == "bf16":
        return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)
    raise ValueError(f"dtype {dtype!r}")


def normal_bits(n: int, dtype: str, seed: int, threads: int = 8) -> np.ndarray:
    """n values ~ N(0,1) rounded to `dtype`, as uint16 bits.

    The stream is defined per fixed-size chunk (chunk i uses the i-th child of
    SeedSequence(seed)), so the result does not depend on the thread count.
    """
    out = np.empty(n, dtype=np.uint16)
    nchunks = (n + _FILL_CHUNK - 1) // _FILL_CHUNK
    if nchunks == 0:
        return out
    children = np.random.SeedSequence(seed).spawn(nchunks)

    def fill(i: int) -> None:
        lo = i * _FILL_CHUNK
        hi = min(n, lo + _FILL_CHUNK)
        g = np.random.Generator(np.random.PCG64(children[i]))
        out[lo:hi] = f32_to_bits(g.standard_normal(hi - lo, dtype=np.float32), dtype)

    if nchunks == 1 or threads <= 1:
        for i in range(nchunks):
            fill(i)
    else:
        with _cf.ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(nchunks)))
    return out


def projection_inputs(seed: int, dtype: str, rows: int, hidden: int, features: int):
    """Layer input x [rows, hidden] ~ N(0,1) and projection weights w [features, hidden] ~ N(0, 1/hidden) (so that
    the projected values are ~ N(0,1) like the q/k/v of the other workloads), both as uint16 bits."""
    x = normal_bits(rows * hidden, dtype, seed + 21).reshape(rows, hidden)
    g = np.random.Generator(np.random.PCG64(seed + 22))
    w = np.empty((features, hidden), dtype=np.uint16)
    inv = np.float32(1.0 / np.sqrt(hidden))
    step = max(1, (1 << 24) // hidden)
    for lo in range(0, features, step):
        hi = min(features, lo + step)
        w[lo:hi] = f32_to_bits(g.standard_normal((hi - lo, hidden), dtype=np.float32) * inv, dtype)
    return x, w


# --------------------------------------------------------------------------
# Descriptors
# --------------------------------------------------------------------------
@dataclasses.dataclass
class CacheSpec:
    """Geometry of a K (or V) pool; strides are in elements, head_dim contiguous."""
    dtype: str
    num_heads: int
    head_dim: int
    num_pages: int
    layout: str            # "paged": [page][head][slot][d];  "contiguous": [token][head][d]
    page_size: int = PAGE_SIZE

    @property
    def stride_token(self) -> int:
        return self.head_dim if self.layout == "paged" else self.num_heads * self.head_dim

    @property
    def stride_head(self) -> int:
        return self.page_size * self.head_dim if self.layout == "paged" else self.head_dim

    @property
    def stride_page(self) -> int:
        return self.page_size * self.num_heads * self.head_dim

    @property
    def pool_elems(self) -> int:
        return self.num_pages * self.stride_page


@dataclasses.dataclass
class Step:
    """One call of the path: a ragged batch of chunks (Sec. 2.1, batched inference)."""
    prefix_len: np.ndarray   # int32 [R]  tokens already cached per request
    chunk_len: np.ndarray    # int32 [R]  rows sent up this step per request
    cu_chunk: np.ndarray     # int32 [R+1] exclusive prefix sum of chunk_len
    block_table: np.ndarray  # int32 [R, max_pages] physical page ids, -1 where unused
    q: np.ndarray            # uint16 [T, Hq, d]   Hq = G * H query heads (G = 1 in the paper's models)
    k_new: np.ndarray        # uint16 [T, H, d]
    v_new: np.ndarray        # uint16 [T, H, d]
    tree_mask: "np.ndarray | None" = None   # uint32 [T]: bit c = row sees chunk position c (chunks of <= 16 rows)

    @property
    def num_requests(self) -> int:
        return int(self.prefix_len.shape[0])

    @property
    def total_rows(self) -> int:
        return int(self.cu_chunk[-1])

    @property
    def max_pages(self) -> int:
        return int(self.block_table.shape[1])


@dataclasses.dataclass
class Scenario:
    name: str
    cache: CacheSpec
    k_pool: np.ndarray       # uint16 [pool_elems]
    v_pool: np.ndarray       # uint16 [pool_elems]
    steps: List[Step]
    note: str = ""


def _pages_for(tokens: int) -> int:
    return (int(tokens) + PAGE_SIZE - 1) // PAGE_SIZE


def _make_step(rng_vals_seed: int, dtype: str, H: int, d: int,
               prefix_len: Sequence[int], chunk_len: Sequence[int],
               block_table: np.ndarray, q_heads: int | None = None) -> Step:
    prefix_len = np.asarray(prefix_len, dtype=np.int32)
    chunk_len = np.asarray(chunk_len, dtype=np.int32)
    cu = np.zeros(len(chunk_len) + 1, dtype=np.int32)
    np.cumsum(chunk_len, out=cu[1:])
    T = int(cu[-1])
    n = T * H * d
    Hq = H if q_heads is None else int(q_heads)
    q = normal_bits(T * Hq * d, dtype, rng_vals_seed + 1).reshape(T, Hq, d)
    k = normal_bits(n, dtype, rng_vals_seed + 2).reshape(T, H, d)
    v = normal_bits(n, dtype, rng_vals_seed + 3).reshape(T, H, d)
    return Step(prefix_len, chunk_len, cu, np.ascontiguousarray(block_table, dtype=np.int32), q, k, v)


def _place_pages(shape_rng: np.random.Generator, tokens_per_request: Sequence[int],
                 slack_pages: int, shuffled: bool = True):
    """Give every request distinct physical pages drawn from one shared pool."""
    need = [_pages_for(t) for t in tokens_per_request]
    total = int(sum(need))
    num_pages = total + int(slack_pages)
    order = shape_rng.permutation(num_pages) if shuffled else np.arange(num_pages)
    max_pages = max(need + [1])
    table = np.full((len(need), max_pages), -1, dtype=np.int32)
    at = 0
    for r, n in enumerate(need):
        table[r, :n] = order[at:at + n]
        at += n
    return table, num_pages


def _scenario(name, dtype, H, d, layout, num_pages, steps, value_seed, note=""):
    cache = CacheSpec(dtype, H, d, num_pages, layout)
    k_pool = normal_bits(cache.pool_elems, dtype, value_seed + 11)
    v_pool = normal_bits(cache.pool_elems, dtype, value_seed + 12)
    return Scenario(name, cache, k_pool, v_pool, steps, note)


# --------------------------------------------------------------------------
# The five workloads
# --------------------------------------------------------------------------
def tiny(prompt: int = 256, chunk: int = 64, draft: int = 4, H: int = 8, d: int = 64,
         dtype: str = "fp16", seed: int = SEED_BASE + 1) -> Scenario:
    """One request; prompt processed as prompt/chunk chunks (prefix 0, chunk, 2*chunk, ...)
    over a contiguous [token][head][d] cache, then one `draft`-token verify chunk."""
    total = prompt + draft
    num_pages = _pages_for(total)
    table = np.arange(num_pages, dtype=np.int32)[None, :]
    steps = []
    for s, p in enumerate(range(0, prompt, chunk)):
        steps.append(_make_step(seed + 100 + 10 * s, dtype, H, d, [p], [min(chunk, prompt - p)], table))
    steps.append(_make_step(seed + 100 + 10 * len(steps), dtype, H, d, [prompt], [draft], table))
    return _scenario("tiny", dtype, H, d, "contiguous", num_pages, steps, seed + 100,
                     "1 request, chunked prompt then a draft-verify chunk, identity block table")


def llama7b_chunked(prompt: int = 2048, chunk: int = 256, H: int = 32, d: int = 128,
                    dtype: str = "fp16", seed: int = SEED_BASE + 2) -> Scenario:
    """One request, prompt chunked at `chunk`, paged cache with pages in shuffled physical order."""
    rng = np.random.Generator(np.random.PCG64(seed))
    table, num_pages = _place_pages(rng, [prompt], slack_pages=0)
    steps = []
    for s, p in enumerate(range(0, prompt, chunk)):
        steps.append(_make_step(seed + 100 + 10 * s, dtype, H, d, [p], [min(chunk, prompt - p)], table))
    return _scenario("llama7b_chunked", dtype, H, d, "paged", num_pages, steps, seed + 100,
                     "1 request, 7B-shaped layer, shuffled pages")


def ragged_prefill(num_requests: int = 30, max_prefix: int = 4096,
                   chunk_choices: Sequence[int] = (64, 128, 256, 512),
                   H: int = 32, d: int = 128, dtype: str = "fp16",
                   seed: int = SEED_BASE + 3) -> Scenario:
    """Prompt chunks from `num_requests` devices: prefix uniform over multiples of 16 in
    [0, max_prefix], chunk length drawn from `chunk_choices`, pages placed at random in one pool."""
    rng = np.random.Generator(np.random.PCG64(seed))
    prefix = PAGE_SIZE * rng.integers(0, max_prefix // PAGE_SIZE + 1, size=num_requests)
    chunk = rng.choice(np.asarray(chunk_choices), size=num_requests)
    table, num_pages = _place_pages(rng, prefix + chunk, slack_pages=max(8, num_requests))
    step = _make_step(seed + 100, dtype, H, d, prefix, chunk, table)
    return _scenario("ragged_prefill", dtype, H, d, "paged", num_pages, [step], seed + 100,
                     "ragged prefill batch, append in the same call")


TREE_MAX_ROWS = 16


def random_tree_masks(seed: int, chunk_len: Sequence[int]) -> np.ndarray:
    """One uint32 word per packed row.  For a chunk of at most TREE_MAX_ROWS rows the rows form a random token
    tree in topological order: node c hangs under a node drawn uniformly from {root, 0..c-1} and its word has
    bit c and its parent's bits set (a row sees its ancestors and itself; the root is the cached prefix, which is
    always visible).  Rows of longer chunks get the causal word (it is not consulted for them)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    words = []
    for C in np.asarray(chunk_len, dtype=np.int64):
        C = int(C)
        if C > TREE_MAX_ROWS:
            words.extend([0xFFFFFFFF] * C)
            continue
        mask = []
        for c in range(C):
            parent = int(rng.integers(-1, c))          # -1: hangs directly under the prefix
            mask.append((mask[parent] if parent >= 0 else 0) | (1 << c))
        words.extend(mask)
    return np.asarray(words, dtype=np.uint32)


def spec_verify(num_requests: int = 30, min_prefix: int = 512, max_prefix: int = 4096,
                max_draft: int = 8, H: int = 32, d: int = 128, dtype: str = "fp16",
                seed: int = SEED_BASE + 4, q_group: int = 1, tree: bool = False) -> Scenario:
    """Draft-verification batch: prefix uniform in [min_prefix, max_prefix] (any value, so
    appends start mid-page), draft length uniform in [1, max_draft].  q_group > 1 gives q_group query
    heads per K/V head; tree=True replaces the linear drafts by random token trees."""
    rng = np.random.Generator(np.random.PCG64(seed))
    prefix = rng.integers(min_prefix, max_prefix + 1, size=num_requests)
    chunk = rng.integers(1, max_draft + 1, size=num_requests)
    table, num_pages = _place_pages(rng, prefix + chunk, slack_pages=max(8, num_requests))
    step = _make_step(seed + 100, dtype, H, d, prefix, chunk, table, q_heads=H * q_group)
    if tree:
        step.tree_mask = random_tree_masks(seed + 200, chunk)
    return _scenario("spec_verify", dtype, H, d, "paged", num_pages, [step], seed + 100,
                     "speculative verification batch")


def mixed_13b(num_prefill: int = 8, prefill_chunk: int = 512, max_prefill_prefix: int = 8192,
              num_verify: int = 32, draft: int = 4, min_verify_prefix: int = 1024,
              max_verify_prefix: int = 8192, H: int = 40, d: int = 128, dtype: str = "bf16",
              seed: int = SEED_BASE + 5, q_group: int = 1, tree: bool = False) -> Scenario:
    """13B-shaped mixed batch: prefill chunks and verify chunks interleaved in one call
    over one paged pool.  q_group and tree as in spec_verify."""
    rng = np.random.Generator(np.random.PCG64(seed))
    p_pre = rng.integers(0, max_prefill_prefix + 1, size=num_prefill)
    p_ver = rng.integers(min_verify_prefix, max_verify_prefix + 1, size=num_verify)
    prefix = np.concatenate([p_pre, p_ver])
    chunk = np.concatenate([np.full(num_prefill, prefill_chunk), np.full(num_verify, draft)])
    order = rng.permutation(len(prefix))          # devices arrive in no particular order
    prefix, chunk = prefix[order], chunk[order]
    table, num_pages = _place_pages(rng, prefix + chunk, slack_pages=max(8, len(prefix)))
    step = _make_step(seed + 100, dtype, H, d, prefix, chunk, table, q_heads=H * q_group)
    if tree:
        step.tree_mask = random_tree_masks(seed + 200, chunk)
    return _scenario("mixed_13b", dtype, H, d, "paged", num_pages, [step], seed + 100,
                     "13B-shaped mixed prefill + verify batch")


WORKLOADS = {
    "tiny": tiny,
    "llama7b_chunked": llama7b_chunked,
    "ragged_prefill": ragged_prefill,
    "spec_verify": spec_verify,
    "mixed_13b": mixed_13b,
}
