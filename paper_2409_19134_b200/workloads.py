"""Seeded synthetic inputs for partitioned decode attention.

This module only *generates inputs*: ragged per-user lengths, paged KV pools
with shuffled page tables, and queries.  It holds none of the method's
arithmetic (no scores, no softmax, no merge) so that both the CUDA path and
the CPU oracle can be fed the very same bytes without sharing any code of
the computation itself.

Layout produced (the layout the C-ABI consumes):
  k_pool, v_pool : [num_pages, num_kv_heads, page_size, head_dim]
  page_indptr    : int32 [batch+1]   prefix sums of pages owned by each user
  page_indices   : int32 [page_indptr[-1]]  physical page of each logical page
  seq_lens       : int32 [batch]     tokens actually cached (0 = empty)
Token t of user u lives at pool[page_indices[page_indptr[u] + t // P], kvh, t % P, :].

Every slot that no token occupies (unreferenced pages, the tail of a user's
last page, slack pages) is filled with NaN, so that a reader that touches
them poisons its result.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, Optional, Tuple

import numpy as np
import torch

PAGE_SIZE = 16


@dataclass
class PagedKV:
    """One KV partition (the private prompt cache or the public generated-token cache)."""
    k_pool: torch.Tensor
    v_pool: torch.Tensor
    page_indptr: torch.Tensor   # int32 [B+1]
    page_indices: torch.Tensor  # int32 [total pages]
    seq_lens: torch.Tensor      # int32 [B]

    @property
    def num_pages(self) -> int:
        return int(self.k_pool.shape[0])

    def to(self, device) -> "PagedKV":
        return PagedKV(*(t.to(device) for t in
                         (self.k_pool, self.v_pool, self.page_indptr, self.page_indices, self.seq_lens)))


@dataclass
class Workload:
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_size: int
    dtype: torch.dtype
    sm_scale: float
    q: torch.Tensor            # [B, Hq, D]
    priv: PagedKV              # private ("input") partition: prompt KV
    pub: PagedKV               # public ("output") partition: generated-token KV
    seed: int = 0

    def to(self, device) -> "Workload":
        return Workload(self.name, self.batch, self.num_q_heads, self.num_kv_heads, self.head_dim,
                        self.page_size, self.dtype, self.sm_scale, self.q.to(device),
                        self.priv.to(device), self.pub.to(device), self.seed)

    @property
    def elem_size(self) -> int:
        return 4 if self.dtype == torch.float32 else 2

    def kv_bytes(self) -> int:
        """Bytes of K and V rows that hold cached tokens, both partitions."""
        toks = int(self.priv.seq_lens.sum().item()) + int(self.pub.seq_lens.sum().item())
        return toks * 2 * self.num_kv_heads * self.head_dim * self.elem_size


# Length recipes: ("const", v) | ("uniform", lo, hi) inclusive | ("lognormal", median, sigma, lo, hi)
CONFIGS: Dict[str, dict] = {
    # tiny MHA partitioned decode, fp32
    "c1_tiny_mha": dict(batch=4, hq=8, hkv=8, d=64, dtype="f32", lin=("const", 256), lout=("const", 32), seed=0),
    # Llama-2-7B-shaped layer decode step (MHA)
    "c2_llama2_7b": dict(batch=32, hq=32, hkv=32, d=128, dtype="bf16",
                         lin=("uniform", 512, 4096), lout=("uniform", 1, 512), seed=1),
    # Llama-3-8B-shaped GQA decode step
    "c3_llama3_8b_gqa": dict(batch=128, hq=32, hkv=8, d=128, dtype="bf16",
                             lin=("uniform", 2048, 8192), lout=("uniform", 1, 1024), seed=2),
    # long-prompt split-K stress
    "c4_long_prompt": dict(batch=8, hq=32, hkv=8, d=128, dtype="bf16",
                           lin=("uniform", 32768, 131072), lout=("uniform", 1, 256), seed=3),
    # many-user service batch (public partitions may be empty)
    "c5_many_user": dict(batch=512, hq=64, hkv=8, d=128, dtype="bf16",
                         lin=("lognormal", 1024, 0.8, 16, 16384), lout=("uniform", 0, 2048), seed=4),
}


def _draw_lengths(rng: np.random.Generator, spec: Tuple, n: int) -> np.ndarray:
    kind = spec[0]
    if kind == "const":
        return np.full(n, int(spec[1]), dtype=np.int64)
    if kind == "uniform":
        return rng.integers(int(spec[1]), int(spec[2]) + 1, size=n, dtype=np.int64)
    if kind == "lognormal":
        _, median, sigma, lo, hi = spec
        x = rng.lognormal(mean=math.log(median), sigma=sigma, size=n)
        return np.clip(np.rint(x), lo, hi).astype(np.int64)
    raise ValueError(f"unknown length recipe {spec!r}")


def make_lengths(cfg: dict, seed: Optional[int] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Private and public token counts per user; one NumPy generator, private drawn first."""
    rng = np.random.default_rng(cfg["seed"] if seed is None else seed)
    lin = _draw_lengths(rng, cfg["lin"], cfg["batch"])
    lout = _draw_lengths(rng, cfg["lout"], cfg["batch"])
    return lin, lout


def _torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


_FILL_CHUNK_PAGES = 2048  # fixed, so that the bytes do not depend on how much memory is free


def _randn_into(dst: torch.Tensor, gen: torch.Generator) -> None:
    """Fill dst (any float dtype) with N(0,1) drawn in fp32 and rounded to dst's dtype."""
    flat = dst.view(dst.shape[0], -1)
    for s in range(0, flat.shape[0], _FILL_CHUNK_PAGES):
        e = min(s + _FILL_CHUNK_PAGES, flat.shape[0])
        flat[s:e] = torch.randn((e - s, flat.shape[1]), generator=gen, device=dst.device,
                                dtype=torch.float32).to(dst.dtype)


def make_paged_kv(seq_lens: np.ndarray, num_kv_heads: int, head_dim: int, dtype: torch.dtype,
                  rng: np.random.Generator, gen: torch.Generator, device,
                  page_size: int = PAGE_SIZE, over_alloc: float = 0.10,
                  slack_pages: Optional[np.ndarray] = None, poison: bool = True) -> PagedKV:
    """Build one partition: a global pool whose pages are handed out in a seeded random order.

    slack_pages[u] extra pages are listed in user u's table beyond what seq_lens[u] needs
    (allocated but unused capacity); they stay NaN.
    """
    B = len(seq_lens)
    need = (seq_lens + page_size - 1) // page_size
    cap = need + (slack_pages if slack_pages is not None else 0)
    indptr = np.zeros(B + 1, dtype=np.int64)
    np.cumsum(cap, out=indptr[1:])
    total = int(indptr[-1])
    num_pages = max(1, int(math.ceil(total * (1.0 + over_alloc))) + 1)
    perm = rng.permutation(num_pages)
    indices = perm[:total].astype(np.int32)

    shape = (num_pages, num_kv_heads, page_size, head_dim)
    k_pool = torch.empty(shape, dtype=dtype, device=device)
    v_pool = torch.empty(shape, dtype=dtype, device=device)
    _randn_into(k_pool, gen)
    _randn_into(v_pool, gen)

    if poison:
        nan = float("nan")
        dead = [perm[total:]]
        slot = np.arange(page_size)
        tail_pages, tail_valid = [], []
        for u in range(B):
            pages_u = indices[indptr[u]:indptr[u + 1]]
            if cap[u] > need[u]:
                dead.append(pages_u[need[u]:])
            r = int(seq_lens[u] % page_size)
            if need[u] > 0 and r != 0:
                tail_pages.append(int(pages_u[need[u] - 1]))
                tail_valid.append(r)
        dead_idx = torch.from_numpy(np.concatenate(dead).astype(np.int64)).to(device)
        if dead_idx.numel():
            k_pool[dead_idx] = nan
            v_pool[dead_idx] = nan
        if tail_pages:
            tp = torch.tensor(tail_pages, dtype=torch.int64, device=device)
            mask = torch.from_numpy(slot[None, :] >= np.asarray(tail_valid)[:, None]).to(device)
            mask = mask[:, None, :, None]
            for pool in (k_pool, v_pool):
                blk = pool[tp]
                blk = torch.where(mask, torch.full_like(blk, nan), blk)
                pool[tp] = blk

    return PagedKV(k_pool, v_pool,
                   torch.from_numpy(indptr.astype(np.int32)).to(device),
                   torch.from_numpy(indices).to(device),
                   torch.from_numpy(seq_lens.astype(np.int32)).to(device))


def make_workload(cfg, seed: Optional[int] = None, device="cpu", over_alloc: float = 0.10,
                  slack: bool = False, poison: bool = True, sm_scale: Optional[float] = None,
                  lengths: Optional[Tuple[np.ndarray, np.ndarray]] = None) -> Workload:
    """Build a full workload from a named config (or a dict with the same keys).

    Lengths come from NumPy's default_rng(seed); values from a torch.Generator on `device`
    seeded with the same number.  `lengths` overrides the drawn lengths (edge-case tests).
    """
    name = cfg if isinstance(cfg, str) else cfg.get("name", "custom")
    cfg = CONFIGS[cfg] if isinstance(cfg, str) else cfg
    seed = cfg.get("seed", 0) if seed is None else seed
    dtype = _torch_dtype(cfg["dtype"])
    B, hq, hkv, d = cfg["batch"], cfg["hq"], cfg["hkv"], cfg["d"]
    lin, lout = lengths if lengths is not None else make_lengths(cfg, seed)
    lin = np.asarray(lin, dtype=np.int64)
    lout = np.asarray(lout, dtype=np.int64)
    assert len(lin) == B and len(lout) == B

    rng = np.random.default_rng([seed, 0x5bd])  # page shuffles: a stream of their own
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    q = torch.randn((B, hq, d), generator=gen, device=device, dtype=torch.float32).to(dtype)
    slack_in = rng.integers(0, 3, size=B) if slack else None
    slack_out = rng.integers(0, 3, size=B) if slack else None
    priv = make_paged_kv(lin, hkv, d, dtype, rng, gen, device, over_alloc=over_alloc,
                         slack_pages=slack_in, poison=poison)
    pub = make_paged_kv(lout, hkv, d, dtype, rng, gen, device, over_alloc=over_alloc,
                        slack_pages=slack_out, poison=poison)
    scale = (1.0 / math.sqrt(d)) if sm_scale is None else float(sm_scale)
    return Workload(name, B, hq, hkv, d, PAGE_SIZE, dtype, scale, q, priv, pub, seed)


def gather_dense(part: PagedKV, user: int, kv_head: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """Pure indexing helper: the [len, D] K and V rows of one user and KV head, in token order."""
    P = part.k_pool.shape[2]
    n = int(part.seq_lens[user])
    lo = int(part.page_indptr[user])
    npg = (n + P - 1) // P
    pages = part.page_indices[lo:lo + npg].long()
    k = part.k_pool[pages, kv_head].reshape(npg * P, -1)[:n]
    v = part.v_pool[pages, kv_head].reshape(npg * P, -1)[:n]
    return k, v
