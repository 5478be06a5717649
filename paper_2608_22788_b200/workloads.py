"""Seeded synthetic inputs for the decode-step hot path.

This module only *draws* inputs (sequence lengths, bf16 tensors, block tables,
logits, draft tokens).  It contains none of the method's arithmetic: no
attention, no softmax, no argmax.  Both the CPU oracle's tests and the CUDA
path's tests/bench build their inputs here so that both sides see the same
bits.

The paper measures rollouts on DeepScaleR / KodCode prompts with Qwen models
(Evaluation section, Appendix "experimental setup"); neither prompts, traces nor
weights are available, so these draws stand in for them.  Shapes follow the
rollout-step setting: per-sequence KV lengths, a paged cache addressed through a
block table, one draft length gamma per call (Section 3.4).

Conventions
-----------
* bf16 tensors are carried as ``numpy.uint16`` bit patterns.
* ``kv_lens[s]`` counts every key of sequence ``s`` *including* the ``q_len``
  tokens being scored in this step (their K/V are already in the cache).
* KV pool layouts: ``"HND"`` = ``[page, kv_head, token, dim]`` and ``"NHD"`` =
  ``[page, token, kv_head, dim]``; strides are reported in elements.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np

BF16_NAN_BITS = np.uint16(0x7FFF)  # a quiet NaN; used to poison bytes nobody may read


# --------------------------------------------------------------------------- #
# bf16 <-> float32 bit helpers (storage format only)
# --------------------------------------------------------------------------- #
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (round-to-nearest-even); returns uint16 bits."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    nan = np.isnan(x)
    rounded = ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)
    if nan.any():
        rounded = np.where(nan, BF16_NAN_BITS, rounded)
    return rounded


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Decode uint16 bfloat16 bit patterns to float32 (exact)."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def normal_bf16(shape: Sequence[int], seed: int, std: float = 1.0, threads: int = 8,
                chunk: int = 1 << 22) -> np.ndarray:
    """N(0, std^2) samples rounded to bf16, as uint16 bits.

    The flat array is cut into fixed-size chunks, each drawn from its own child
    of ``SeedSequence(seed)``; the result therefore does not depend on the
    number of worker threads.
    """
    n = int(np.prod(shape, dtype=np.int64))
    out = np.empty(n, dtype=np.uint16)
    nchunks = max(1, (n + chunk - 1) // chunk)
    children = np.random.SeedSequence(seed).spawn(nchunks)

    def work(i: int) -> None:
        lo = i * chunk
        hi = min(n, lo + chunk)
        rng = np.random.default_rng(children[i])
        x = rng.standard_normal(hi - lo, dtype=np.float32)
        if std != 1.0:
            x *= np.float32(std)
        # same rounding as f32_to_bf16_bits, in place (the draws are finite, so no NaN branch)
        u = x.view(np.uint32)
        lsb = (u >> np.uint32(16)) & np.uint32(1)
        u += lsb
        u += np.uint32(0x7FFF)
        u >>= np.uint32(16)
        out[lo:hi] = u

    if nchunks == 1 or threads <= 1:
        for i in range(nchunks):
            work(i)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(work, range(nchunks)))
    return out.reshape(tuple(shape))


# --------------------------------------------------------------------------- #
# sequence-length laws of the five workload configurations
# --------------------------------------------------------------------------- #
def lens_tiny() -> np.ndarray:
    return np.array([17, 64, 200, 513], dtype=np.int32)


def lens_bulk(seed: int = 0, n: int = 256) -> np.ndarray:
    """Bulk pool: lognormal, median 2048, sigma 0.8, clipped to [64, 16384]."""
    rng = np.random.default_rng([seed, 2])
    z = rng.standard_normal(n)
    L = np.rint(np.exp(math.log(2048.0) + 0.8 * z))
    return np.clip(L, 64, 16384).astype(np.int32)


def lens_tail(seed: int = 0, n: int = 8) -> np.ndarray:
    """Tail pool: uniform integers in [32768, 131072]."""
    rng = np.random.default_rng([seed, 3])
    return rng.integers(32768, 131072, size=n, endpoint=True).astype(np.int32)


def lens_verify(seed: int = 0, n: int = 16) -> np.ndarray:
    """Tail-pool speculative verify: 49152 +- 4096, uniform integers."""
    rng = np.random.default_rng([seed, 4])
    return rng.integers(49152 - 4096, 49152 + 4096, size=n, endpoint=True).astype(np.int32)


def lens_mixed(seed: int = 0, n: int = 1024, lo: int = 256, hi: int = 131072, alpha: float = 1.5,
               max_kv_bytes: float = 40e9, bytes_per_token: int = 4096) -> np.ndarray:
    """Uniform-routing mixed batch: Pareto(alpha) truncated to [lo, hi] by inverse CDF.

    If a draw's total KV exceeds ``max_kv_bytes`` the draw is repeated with the
    next seed.
    """
    s = seed
    while True:
        rng = np.random.default_rng([s, 5])
        u = rng.random(n)
        L = np.floor(lo * (1.0 - u * (1.0 - (lo / hi) ** alpha)) ** (-1.0 / alpha))
        L = np.clip(L, lo, hi).astype(np.int32)
        if float(L.sum()) * bytes_per_token <= max_kv_bytes:
            return L
        s += 1


def sweep_subset(pool_lens: np.ndarray, concurrency: int, draw: int, seed: int = 0) -> np.ndarray:
    """``concurrency`` lengths drawn without replacement from the fixed mixed pool."""
    rng = np.random.default_rng([seed, 6, concurrency, draw])
    idx = rng.choice(len(pool_lens), size=concurrency, replace=False)
    return np.asarray(pool_lens)[idx].astype(np.int32)


# --------------------------------------------------------------------------- #
# paged attention batch
# --------------------------------------------------------------------------- #
@dataclass
class AttnBatch:
    name: str
    num_seqs: int
    q_len: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    num_pages: int
    max_pages_per_seq: int
    layout: str
    scale: float
    kv_lens: np.ndarray          # int32 [B]
    block_table: np.ndarray      # int32 [B, max_pages_per_seq]
    q: Optional[np.ndarray]      # uint16 [B, q_len, Hq, D]
    k_pool: Optional[np.ndarray]  # uint16 [num_pages, ...] per layout
    v_pool: Optional[np.ndarray]
    seed: int = 0
    meta: dict = field(default_factory=dict)

    @property
    def kv_page_stride(self) -> int:
        return self.page_size * self.num_kv_heads * self.head_dim

    @property
    def kv_token_stride(self) -> int:
        return self.head_dim if self.layout == "HND" else self.num_kv_heads * self.head_dim

    @property
    def kv_head_stride(self) -> int:
        return self.page_size * self.head_dim if self.layout == "HND" else self.head_dim

    @property
    def pool_shape(self) -> tuple:
        if self.layout == "HND":
            return (self.num_pages, self.num_kv_heads, self.page_size, self.head_dim)
        return (self.num_pages, self.page_size, self.num_kv_heads, self.head_dim)

    @property
    def total_tokens(self) -> int:
        return int(self.kv_lens.astype(np.int64).sum())

    def algorithmic_bytes(self) -> int:
        """Bytes the step must move: every K and V element once, Q in, O out (bf16)."""
        kv = self.total_tokens * self.num_kv_heads * self.head_dim * 2 * 2
        qo = self.num_seqs * self.q_len * self.num_q_heads * self.head_dim * 2 * 2
        return kv + qo


def make_batch(name: str, kv_lens: Sequence[int], *, q_len: int = 1, num_q_heads: int = 32,
               num_kv_heads: int = 8, head_dim: int = 128, page_size: int = 64, seed: int = 0,
               layout: str = "HND", spare_frac: float = 0.05, poison: bool = False,
               fill: bool = True, scale: Optional[float] = None, threads: int = 8,
               extra_table_cols: int = 0) -> AttnBatch:
    """Build one paged-KV attention batch.

    Physical pages: a pool of ``sum(ceil(n_s / P))`` pages plus ``spare_frac``
    spare ones; one global random permutation assigns them to the sequences'
    logical pages, so that consecutive logical pages are not adjacent in memory.

    ``poison=True`` overwrites everything the computation must not depend on
    with NaN (spare pages, the unused tail of each last page) and sets unused
    block-table slots to -1.  With ``fill=False`` no tensor data is drawn (only
    lengths and the block table), for callers that fill the pools elsewhere.
    """
    assert layout in ("HND", "NHD")
    kv_lens = np.asarray(kv_lens, dtype=np.int32)
    B = int(kv_lens.shape[0])
    P = int(page_size)
    pages_per_seq = (kv_lens.astype(np.int64) + P - 1) // P
    used = int(pages_per_seq.sum())
    num_pages = used + max(1, int(math.ceil(used * spare_frac)))
    max_pages = int(pages_per_seq.max()) + int(extra_table_cols) if B > 0 else 1
    max_pages = max(max_pages, 1)

    rng = np.random.default_rng([seed, 11])
    perm = rng.permutation(num_pages).astype(np.int32)
    block_table = np.full((B, max_pages), -1 if poison else 0, dtype=np.int32)
    cursor = 0
    for s in range(B):
        c = int(pages_per_seq[s])
        block_table[s, :c] = perm[cursor:cursor + c]
        cursor += c
    spare_pages = perm[cursor:]

    b = AttnBatch(name=name, num_seqs=B, q_len=int(q_len), num_q_heads=int(num_q_heads),
                  num_kv_heads=int(num_kv_heads), head_dim=int(head_dim), page_size=P,
                  num_pages=num_pages, max_pages_per_seq=max_pages, layout=layout,
                  scale=float(scale if scale is not None else 1.0 / math.sqrt(head_dim)),
                  kv_lens=kv_lens, block_table=block_table, q=None, k_pool=None, v_pool=None,
                  seed=seed)
    b.meta["spare_pages"] = spare_pages
    if not fill:
        return b

    b.q = normal_bf16((B, q_len, num_q_heads, head_dim), seed=seed * 1000 + 1, threads=threads)
    b.k_pool = normal_bf16(b.pool_shape, seed=seed * 1000 + 2, threads=threads)
    b.v_pool = normal_bf16(b.pool_shape, seed=seed * 1000 + 3, threads=threads)
    if poison:
        poison_unused(b)
    return b


def poison_unused(b: AttnBatch) -> None:
    """NaN-fill spare pages and the token slots past each sequence's end."""
    P = b.page_size
    for pool in (b.k_pool, b.v_pool):
        pool[b.meta["spare_pages"]] = BF16_NAN_BITS
        for s in range(b.num_seqs):
            n = int(b.kv_lens[s])
            r = n % P
            if n > 0 and r != 0:
                last = int(b.block_table[s, (n - 1) // P])
                if b.layout == "HND":
                    pool[last, :, r:, :] = BF16_NAN_BITS
                else:
                    pool[last, r:, :, :] = BF16_NAN_BITS


def contiguous_kv(b: AttnBatch, s: int) -> tuple:
    """Gather sequence ``s`` out of the pages into dense ``[n, Hkv, D]`` uint16 arrays."""
    n = int(b.kv_lens[s])
    P = b.page_size
    npg = (n + P - 1) // P
    pages = b.block_table[s, :npg]
    outs = []
    for pool in (b.k_pool, b.v_pool):
        x = pool[pages]
        if b.layout == "HND":
            x = np.transpose(x, (0, 2, 1, 3))
        x = x.reshape(npg * P, b.num_kv_heads, b.head_dim)[:n]
        outs.append(np.ascontiguousarray(x))
    return outs[0], outs[1]


# named configurations ------------------------------------------------------ #
def config_tiny(seed: int = 0, layout: str = "HND", poison: bool = False, q_len: int = 1) -> AttnBatch:
    return make_batch("tiny", lens_tiny(), q_len=q_len, num_q_heads=8, num_kv_heads=2, head_dim=64,
                      page_size=16, seed=seed, layout=layout, poison=poison, spare_frac=0.25)


def config_bulk(seed: int = 0, fill: bool = True, **kw) -> AttnBatch:
    return make_batch("bulk", lens_bulk(seed), seed=seed, fill=fill, **kw)


def config_tail(seed: int = 0, fill: bool = True, **kw) -> AttnBatch:
    return make_batch("tail", lens_tail(seed), seed=seed, fill=fill, **kw)


def config_verify(gamma: int, seed: int = 0, fill: bool = True, **kw) -> AttnBatch:
    return make_batch(f"verify_g{gamma}", lens_verify(seed), q_len=1 + gamma, seed=seed, fill=fill, **kw)


def config_mixed(seed: int = 0, fill: bool = True, **kw) -> AttnBatch:
    return make_batch("mixed", lens_mixed(seed), seed=seed, fill=fill, **kw)


# --------------------------------------------------------------------------- #
# speculative-verify logits and drafts
# --------------------------------------------------------------------------- #
VOCAB = 151936


def make_logits(num_seqs: int, gamma: int, vocab: int = VOCAB, seed: int = 0, std: float = 2.0,
                threads: int = 8) -> np.ndarray:
    """bf16 logits ``[B, gamma+1, V]`` drawn N(0, std^2) (std = 2), as uint16 bits."""
    return normal_bf16((num_seqs, gamma + 1, vocab), seed=seed * 1000 + 7, std=std, threads=threads)


def make_draft(row_best: np.ndarray, vocab: int, seed: int = 0):
    """Draft tokens that follow ``row_best`` up to a seeded cut point.

    ``row_best`` is an int array ``[B, gamma+1]`` supplied by the caller (the
    per-row best token; this module does not compute it).  For each sequence a
    cut ``c`` is drawn uniformly from ``{0..gamma}``: ``draft[:c]`` equals
    ``row_best[:c]``; ``draft[c]`` (when ``c < gamma``) is shifted so that it
    surely differs; later positions are a mix of random tokens and tokens that
    *do* equal ``row_best`` -- so counting matches and taking the longest
    matching prefix give different answers.  Returns ``(draft, cut)``.
    """
    row_best = np.asarray(row_best)
    B, g1 = row_best.shape
    gamma = g1 - 1
    rng = np.random.default_rng([seed, 13])
    cut = rng.integers(0, gamma, size=B, endpoint=True).astype(np.int32)
    draft = np.empty((B, gamma), dtype=np.int32)
    for b in range(B):
        for i in range(gamma):
            if i < cut[b]:
                draft[b, i] = row_best[b, i]
            elif i == cut[b]:
                draft[b, i] = (int(row_best[b, i]) + 1 + int(rng.integers(0, max(1, vocab - 1)))) % vocab
                if draft[b, i] == row_best[b, i]:
                    draft[b, i] = (int(row_best[b, i]) + 1) % vocab
            elif rng.random() < 0.5:
                draft[b, i] = row_best[b, i]
            else:
                draft[b, i] = int(rng.integers(0, vocab))
    return draft, cut
