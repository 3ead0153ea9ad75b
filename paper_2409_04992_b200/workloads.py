"""Seeded synthetic inputs for decode attention over a KV cache.

This module only draws random tensors, lengths and block tables and lays them out in
memory.  It holds none of the attention arithmetic, which is why both the CUDA tests and
the independent CPU checker may take their inputs from it.

The shapes are those of a 13B-class decoder as the paper evaluates it (Sec. IV-C, IV-D,
V-A): 40 heads of dimension 128, fp16 everywhere, so one (token, head) is 256 B of K and
256 B of V.  The five standard workloads stand in for the paper's OPT-13B runs on dataset
samples, whose values do not change what the path costs.

Conventions
-----------
* ``seq_lens[b]`` counts the new token: the caches arrive holding ``seq_lens[b]-1`` tokens,
  the append fills position ``seq_lens[b]-1``, attention covers ``[0, seq_lens[b])``.
* contiguous caches are ``[B, H, s_max, D]``; paged pools are ``[P, H, T, D]`` for K and for
  V with one ``block_table [B, M]`` (logical block -> physical block) shared by both.
* The block table is one random permutation over all blocks of the pool, so sequences
  interleave physically; unused table entries are -1; a few spare blocks belong to nobody.
* With ``poison=True`` every cache slot that attention must not read (padding, the tail of
  each sequence's last block, spare blocks) and the slot the append must fill hold the fp16
  NaN pattern 0x7E00, so a stray read or a missing append contaminates the output.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import torch

HEADS_13B = 40
HEAD_DIM_13B = 128
BASE_SEED = 240904992
NAN_BITS = 0x7E00


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and distribution of one decode step's inputs."""

    name: str
    index: int                      # position in the standard list; enters the seed
    batch: int
    len_lo: int                     # seq_lens ~ uniform{len_lo..len_hi}, new token counted
    len_hi: int
    layout: str                     # "contiguous" | "paged"
    s_max: int = 0                  # contiguous: padded capacity per sequence
    block_tokens: int = 0           # paged: tokens per block (T)
    heads: int = HEADS_13B
    head_dim: int = HEAD_DIM_13B
    layers: int = 1
    peaked_fraction: float = 0.0    # share of key rows multiplied by peaked_gain
    peaked_gain: float = 4.0
    spare_blocks: int = 3

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.head_dim)

    @property
    def paged(self) -> bool:
        return self.layout == "paged"

    @property
    def max_blocks_per_seq(self) -> int:
        return -(-self.len_hi // self.block_tokens) if self.paged else 0

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


#: The five standard workloads (13B-class shapes).
STANDARD: List[Workload] = [
    Workload("ctx1k_b1_contiguous", 0, batch=1, len_lo=1024, len_hi=1024,
             layout="contiguous", s_max=1024),
    Workload("ctx2k-4k_b16_contiguous", 1, batch=16, len_lo=2048, len_hi=4096,
             layout="contiguous", s_max=4096),
    Workload("ctx16k_b64_paged16", 2, batch=64, len_lo=16384, len_hi=16384,
             layout="paged", block_tokens=16),
    Workload("ctx128k_b8_paged64_peaked", 3, batch=8, len_lo=131072, len_hi=131072,
             layout="paged", block_tokens=64, peaked_fraction=0.01),
    Workload("decode13b_40layers_b16_ctx4k-8k_paged32", 4, batch=16, len_lo=4096, len_hi=8192,
             layout="paged", block_tokens=32, layers=40),
]


def by_name(name: str) -> Workload:
    for w in STANDARD:
        if w.name == name or str(w.index) == name:
            return w
    raise KeyError(f"unknown workload {name!r}; have {[w.name for w in STANDARD]}")


@dataclasses.dataclass
class Case:
    """One layer's tensors for one decode step (all on one device)."""

    workload: Workload
    layer: int
    q: torch.Tensor                 # fp16 [B,H,D]
    k_new: torch.Tensor             # fp16 [B,H,D]
    v_new: torch.Tensor             # fp16 [B,H,D]
    k_cache: torch.Tensor           # fp16 [B,H,s_max,D] or [P,H,T,D]
    v_cache: torch.Tensor
    seq_lens: torch.Tensor          # int32 [B]
    block_table: Optional[torch.Tensor]   # int32 [B,M] or None
    seq_lens_host: List[int]
    scale: float

    @property
    def max_seq_len(self) -> int:
        return max(self.seq_lens_host) if self.seq_lens_host else 0

    @property
    def kv_tokens(self) -> int:
        """Cached positions attended this step, summed over sequences (one layer)."""
        return int(sum(self.seq_lens_host))

    @property
    def kv_bytes_read(self) -> int:
        """fp16 K and V bytes the step must read: 2 * D * 2 B per (token, head)."""
        return kv_bytes_per_token(self.workload.heads, self.workload.head_dim) * self.kv_tokens


def kv_bytes_per_token(heads: int = HEADS_13B, head_dim: int = HEAD_DIM_13B) -> int:
    """Bytes of K plus V one cached position holds across all heads of one layer (fp16)."""
    return heads * head_dim * 2 * 2


def kv_cache_bytes(batch: int, tokens: int, layers: int, heads: int = HEADS_13B,
                   head_dim: int = HEAD_DIM_13B) -> int:
    """Whole-model fp16 KV footprint: batch * tokens * layers positions."""
    return batch * tokens * layers * kv_bytes_per_token(heads, head_dim)


def draw_seq_lens(w: Workload) -> List[int]:
    """Lengths depend on the workload only (every layer sees the same sequences)."""
    g = torch.Generator(device="cpu")
    g.manual_seed(BASE_SEED + w.index)
    return torch.randint(w.len_lo, w.len_hi + 1, (w.batch,), generator=g).tolist()


def _fill_normal(t: torch.Tensor, gen: torch.Generator, row_gain_fraction: float = 0.0,
                 row_gain: float = 1.0, chunk_rows: int = 1 << 20) -> None:
    """t[...] = fp16(N(0,1)) drawn in fp32, chunked; optionally a share of rows times a gain."""
    dim = t.shape[-1]
    flat = t.view(-1, dim)
    for start in range(0, flat.shape[0], chunk_rows):
        rows = min(chunk_rows, flat.shape[0] - start)
        x = torch.randn((rows, dim), dtype=torch.float32, device=t.device, generator=gen)
        if row_gain_fraction > 0.0:
            pick = torch.rand((rows, 1), dtype=torch.float32, device=t.device,
                              generator=gen) < row_gain_fraction
            x = torch.where(pick, x * row_gain, x)
        flat[start:start + rows] = x.to(torch.float16)


def _poison(t: torch.Tensor) -> None:
    t.view(torch.int16).fill_(NAN_BITS)


def generate(w: Workload, layer: int = 0, device: str = "cpu", poison: bool = True,
             seq_lens: Optional[List[int]] = None) -> Case:
    """Draw one layer's inputs.  Same (workload, layer, device type) => same bits."""
    dev = torch.device(device)
    lens = list(seq_lens) if seq_lens is not None else draw_seq_lens(w)
    if len(lens) != w.batch:
        raise ValueError("seq_lens must have one entry per sequence")
    seed = BASE_SEED + w.index + 1000 * layer
    cpu_gen = torch.Generator(device="cpu")
    cpu_gen.manual_seed(seed + 7)
    gen = torch.Generator(device=dev)
    gen.manual_seed(seed)
    B, H, D = w.batch, w.heads, w.head_dim

    small = [torch.empty((B, H, D), dtype=torch.float16, device=dev) for _ in range(3)]
    for t in small:
        if t.numel():
            _fill_normal(t, gen)
    q, k_new, v_new = small

    table = None
    if not w.paged:
        if any(n > w.s_max for n in lens):
            raise ValueError("a sequence is longer than s_max")
        shape = (B, H, w.s_max, D)
    else:
        T = w.block_tokens
        need = [-(-n // T) for n in lens]
        P = sum(need) + w.spare_blocks
        M = max(w.max_blocks_per_seq, max(need, default=0), 1)
        perm = torch.randperm(P, generator=cpu_gen).to(torch.int32)
        table = torch.full((B, M), -1, dtype=torch.int32)
        at = 0
        for b, n in enumerate(need):
            table[b, :n] = perm[at:at + n]
            at += n
        spare = perm[at:]
        shape = (P, H, T, D)
    k_cache = torch.empty(shape, dtype=torch.float16, device=dev)
    v_cache = torch.empty(shape, dtype=torch.float16, device=dev)
    if k_cache.numel():
        _fill_normal(k_cache, gen, w.peaked_fraction, w.peaked_gain)
        _fill_normal(v_cache, gen)

    if poison:
        for cache in (k_cache, v_cache):
            if not w.paged:
                for b, n in enumerate(lens):
                    _poison(cache[b, :, max(n - 1, 0):, :])
            else:
                T = w.block_tokens
                for b, n in enumerate(lens):
                    if n > 0:
                        _poison(cache[int(table[b, (n - 1) // T]), :, (n - 1) % T:, :])
                for p in spare.tolist():
                    _poison(cache[p])

    return Case(workload=w, layer=layer, q=q, k_new=k_new, v_new=v_new,
                k_cache=k_cache, v_cache=v_cache,
                seq_lens=torch.tensor(lens, dtype=torch.int32, device=dev),
                block_table=None if table is None else table.to(dev),
                seq_lens_host=lens, scale=w.scale)


@dataclasses.dataclass
class GroupedCase:
    """Inputs of the grouped-head / multi-token variant: `base` holds caches, lengths and the
    block table for `base.workload.heads` KV heads (its own q, k_new, v_new are not used)."""

    base: Case
    q: torch.Tensor                 # fp16 [B,Tq,Hq,D]
    k_new: torch.Tensor             # fp16 [B,Tq,Hkv,D], token-major as the bulk append takes it
    v_new: torch.Tensor
    new_lens: torch.Tensor          # int32 [B]: min(Tq, seq_len), the tokens this step appends

    @property
    def q_tokens(self) -> int:
        return self.q.shape[1]


def generate_grouped(w: Workload, q_tokens: int, q_heads: int, layer: int = 0, device: str = "cpu",
                     seq_lens: Optional[List[int]] = None) -> GroupedCase:
    """`w.heads` is the number of KV heads; q_heads must be a multiple of it.  Same arguments,
    same bits."""
    if q_heads % w.heads != 0:
        raise ValueError("q_heads must be a multiple of the workload's (KV) heads")
    base = generate(w, layer, device, seq_lens=seq_lens)
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(BASE_SEED + w.index + 1000 * layer + 500)
    q = torch.empty((w.batch, q_tokens, q_heads, w.head_dim), dtype=torch.float16, device=dev)
    k_new = torch.empty((w.batch, q_tokens, w.heads, w.head_dim), dtype=torch.float16, device=dev)
    v_new = torch.empty_like(k_new)
    for t in (q, k_new, v_new):
        if t.numel():
            _fill_normal(t, gen)
    new_lens = torch.tensor([min(q_tokens, n) for n in base.seq_lens_host], dtype=torch.int32, device=dev)
    return GroupedCase(base=base, q=q, k_new=k_new, v_new=v_new, new_lens=new_lens)


def gather_rows(case: Case, b: int, h: int):
    """The K and V rows of one (sequence, head) as contiguous [L,D] tensors (memory movement
    only: contiguous slice, or a walk of the block table)."""
    n = case.seq_lens_host[b]
    if case.block_table is None:
        return case.k_cache[b, h, :n].contiguous(), case.v_cache[b, h, :n].contiguous()
    T = case.workload.block_tokens
    blocks = case.block_table[b, : -(-n // T)].long()
    k = case.k_cache[blocks, h].reshape(-1, case.workload.head_dim)[:n].contiguous()
    v = case.v_cache[blocks, h].reshape(-1, case.workload.head_dim)[:n].contiguous()
    return k, v


@dataclasses.dataclass
class SparfState:
    """Extra per-layer state of the sparse (SparF) path for a paged case."""

    kt_pool: torch.Tensor           # fp16 [Pk,H,D,Tk]: the embedding-major copy of K
    kt_block_table: torch.Tensor    # int32 [B,Mk]: logical Tk-token group -> block of kt_pool
    v_sum: torch.Tensor             # fp32 [B,H,D]: running sum of each sequence's V rows
    k_tokens: torch.Tensor          # int32 [B]: tokens to keep per sequence
    k_tokens_host: List[int]

    @property
    def kt_block_tokens(self) -> int:
        return self.kt_pool.shape[3]


def _relayout_kt(case: Case, kt_tokens: int, cpu_gen: torch.Generator):
    """The K pool re-laid embedding-major in groups of kt_tokens tokens under a table of its
    own (memory movement only; slots past a sequence's end carry the NaN poison)."""
    w = case.workload
    T, H, D = w.block_tokens, w.heads, w.head_dim
    dev = case.k_cache.device
    need = [-(-n // kt_tokens) for n in case.seq_lens_host]
    Pk = sum(need) + w.spare_blocks
    Mk = max(-(-w.len_hi // kt_tokens), max(need, default=0), 1)
    perm = torch.randperm(Pk, generator=cpu_gen).to(torch.int32)
    kt_table = torch.full((w.batch, Mk), -1, dtype=torch.int32)
    kt_pool = torch.empty((Pk, H, D, kt_tokens), dtype=torch.float16, device=dev)
    _poison(kt_pool)
    at = 0
    for b, n in enumerate(need):
        kt_table[b, :n] = perm[at:at + n]
        at += n
        if n == 0:
            continue
        blocks = case.block_table[b, : -(-case.seq_lens_host[b] // T)].long()
        rows = case.k_cache[blocks].permute(1, 3, 0, 2).reshape(H, D, -1)          # [H, D, tokens]
        padded = torch.empty((H, D, n * kt_tokens), dtype=torch.float16, device=dev)
        _poison(padded)
        padded[:, :, : rows.shape[2]] = rows
        kt_pool[kt_table[b, :n].long().to(dev)] = padded.view(H, D, n, kt_tokens).permute(2, 0, 1, 3)
    return kt_pool, kt_table.to(dev)


def make_sparf_state(case: Case, keep_fraction: float = 0.125,
                     kt_block_tokens: Optional[int] = None) -> SparfState:
    """The embedding-major K copy is a pure re-layout of the K pool (poison included), in
    groups of kt_block_tokens tokens (default: the K/V block size, sharing the K/V table).
    v_sum is an input of the algorithm (it enters as the mean value vector): it is drawn as
    N(0, L) per element, the distribution of a sum of L unit normals, not computed from V."""
    if case.block_table is None:
        raise ValueError("the sparse path is defined on the paged layout")
    w = case.workload
    dev = case.q.device
    gen = torch.Generator(device=dev)
    gen.manual_seed(BASE_SEED + 5000 + w.index + 1000 * case.layer)
    if kt_block_tokens is None or kt_block_tokens == w.block_tokens:
        kt_pool, kt_table = case.k_cache.transpose(2, 3).contiguous(), case.block_table
    else:
        if kt_block_tokens % w.block_tokens:
            raise ValueError("kt_block_tokens must be a multiple of the K/V block size")
        cpu_gen = torch.Generator(device="cpu")
        cpu_gen.manual_seed(BASE_SEED + 6000 + w.index + 1000 * case.layer)
        kt_pool, kt_table = _relayout_kt(case, kt_block_tokens, cpu_gen)
    lens = torch.tensor(case.seq_lens_host, dtype=torch.float32, device=dev)
    v_sum = torch.randn((w.batch, w.heads, w.head_dim), dtype=torch.float32, device=dev,
                        generator=gen) * lens.clamp(min=1).sqrt()[:, None, None]
    keep = [0 if n == 0 else max(1, -(-n * int(round(keep_fraction * 1024)) // 1024))
            for n in case.seq_lens_host]
    return SparfState(kt_pool=kt_pool, kt_block_table=kt_table, v_sum=v_sum.contiguous(),
                      k_tokens=torch.tensor(keep, dtype=torch.int32, device=dev),
                      k_tokens_host=keep)
