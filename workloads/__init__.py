"""Seeded synthetic inputs for paged GQA decode attention.

This module only *makes inputs* (lengths, block tables, random bf16 pools, NaN
poison in the places that must never be read) and copies parts of them between
devices.  It holds none of the attention arithmetic and is the one module that
both the CUDA tests/benchmark and the CPU oracle's callers may import.

The shapes stand in for long agent trajectories served by an LLM inference
service (the paper, Sec. 3.2 and Sec. 4: hundreds of concurrent sessions that
share one long initial prompt, contexts that grow by multi-thousand-token
feedback prompts up to 131,072 tokens).  No dataset or benchmark item is
involved: every value is drawn from a seeded generator.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np
import torch

HQ, HKV, D = 48, 8, 128


@dataclass
class Case:
    """One decode-attention problem.  Tensors live on ``device``."""
    name: str
    q: torch.Tensor            # bf16 [B, Hq, D]
    k_pages: torch.Tensor      # bf16 [num_pages, Hkv, P, D] (logical shape; strides may differ)
    v_pages: torch.Tensor      # bf16, same shape/strides as k_pages
    block_table: torch.Tensor  # int32 [B, max_pages], unused entries = -1
    seq_lens: torch.Tensor     # int32 [B]
    window: int
    scale: float
    lens: np.ndarray = field(repr=False, default=None)  # host copy of seq_lens (int64)
    # 8-bit cache only: the pools then hold E4M3 codes (torch.uint8) and these are the fp32 [Hkv]
    # dequantisation factors (K = k_scale[g] * e4m3(code)); None for a bf16 cache
    k_scale: Optional[torch.Tensor] = None
    v_scale: Optional[torch.Tensor] = None

    @property
    def B(self) -> int:
        return self.q.shape[0]

    @property
    def P(self) -> int:
        return self.k_pages.shape[2]

    def attended_tokens(self) -> np.ndarray:
        """Tokens each sequence attends (exact count, not rounded to pages)."""
        L = self.lens.astype(np.int64)
        w = self.window
        n = np.where((w > 0) & (w < L), w, L)
        return np.maximum(n, 0)

    def algorithmic_bytes(self, out_itemsize: int = 4) -> int:
        """Bytes the operation must move: attended K+V rows, block-table entries
        touched, seq_len, q, out and lse.  Split-K partials are overhead and are
        not counted."""
        Hq, Dh = self.q.shape[1], self.q.shape[2]
        Hkv = self.k_pages.shape[1]
        n = self.attended_tokens()
        L = np.maximum(self.lens.astype(np.int64), 0)
        lo = L - n
        P = self.P
        pages_touched = np.where(n > 0, (L - 1) // P - lo // P + 1, 0)
        per_seq = (n * (2 * Hkv * Dh * self.k_pages.element_size()) + pages_touched * 4 + 4
                   + Hq * Dh * 2 + Hq * Dh * out_itemsize + Hq * 4)
        scales = 2 * Hkv * 4 if self.k_scale is not None else 0
        return int(per_seq.sum()) + scales


    def unique_kv_bytes(self) -> int:
        """Bytes of the K+V rows attended by at least one sequence, each physical row counted once
        (sequences that share pages -- a common prefix -- read the same rows): what has to come from
        HBM at least once per call, where ``algorithmic_bytes`` counts every sequence's reads."""
        Hkv, Dh = self.k_pages.shape[1], self.k_pages.shape[3]
        P = self.P
        n = self.attended_tokens()
        L = np.maximum(self.lens.astype(np.int64), 0)
        bt = self.block_table.cpu().numpy().astype(np.int64)
        rows_in_page = np.zeros(int(self.k_pages.shape[0]), dtype=np.int64)   # most rows any sequence attends
        for b in range(len(L)):
            if n[b] <= 0:
                continue
            lo = int(L[b] - n[b])
            first, last = lo // P, (int(L[b]) - 1) // P
            pages = bt[b, first:last + 1]
            cnt = np.full(len(pages), P, dtype=np.int64)
            cnt[0] -= lo - first * P
            cnt[-1] -= (last + 1) * P - int(L[b])
            np.maximum.at(rows_in_page, pages, cnt)
        return int(rows_in_page.sum()) * 2 * Hkv * Dh * self.k_pages.element_size()


def _randn_bf16(shape, gen: torch.Generator, device) -> torch.Tensor:
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32).to(torch.bfloat16)


E4M3_NAN = 0x7F


def _randn_e4m3(shape, gen: torch.Generator, device, inv_scale: torch.Tensor) -> torch.Tensor:
    """Random E4M3 codes (uint8): N(0,1) draws times ``inv_scale`` (broadcast), cast by torch.  This
    only makes inputs: both the CUDA path and the oracle take the codes as given."""
    x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32) * inv_scale
    return x.clamp_(-448.0, 448.0).to(torch.float8_e4m3fn).view(torch.uint8)


def default_kv_scales(Hkv: int):
    """The fixed, deliberately not power-of-two factors the 8-bit workloads use: with them the
    dequantised cache is again ~N(0,1) and the stored magnitudes stay below 448."""
    g = np.arange(Hkv, dtype=np.float32)
    return (np.float32(0.02) + np.float32(0.003) * g).astype(np.float32), \
           (np.float32(0.025) - np.float32(0.001) * g).astype(np.float32)


def build_case(name: str, lens: Sequence[int], P: int, seed: int, device="cpu", *,
               Hq: int = HQ, Hkv: int = HKV, Dh: int = D, window: int = 0,
               scale: Optional[float] = None, shuffle: bool = True,
               pool_pages: Optional[int] = None, shared_prefix_tokens: int = 0,
               layout: str = "head_major", poison: bool = True,
               pad_table_to: Optional[int] = None, fill_chunk_pages: int = 16384,
               kv_dtype: str = "bf16") -> Case:
    """Build one problem.

    lens                  context length of each sequence (current token included)
    shuffle               physical page ids are a random permutation of the pool
                          (False: sequence pages laid out contiguously in order)
    pool_pages            size of the physical pool (default: exactly the pages
                          referenced); extra pages are NaN-filled
    shared_prefix_tokens  the first this-many tokens of every sequence use the
                          SAME physical pages (must be a multiple of P)
    layout                "head_major": memory order [page, kv_head, token, d];
                          "token_major": memory order [page, token, kv_head, d]
                          (same logical shape, different strides)
    poison                NaN in page tails past each sequence's end, in unused
                          pool pages; block-table padding is -1 either way
    kv_dtype              "bf16", or "fp8": pools of E4M3 codes (uint8) with the per-KV-head
                          factors of default_kv_scales(); NaN is then the code 0x7F
    """
    rng = np.random.default_rng(seed)
    gen = torch.Generator(device=device)
    gen.manual_seed(seed)
    lens = np.asarray(lens, dtype=np.int64)
    B = len(lens)
    if shared_prefix_tokens % P:
        raise ValueError("shared prefix must be whole pages")
    pre_pages = shared_prefix_tokens // P
    npg = np.maximum((lens + P - 1) // P, 0)
    if pre_pages and (lens < shared_prefix_tokens).any():
        raise ValueError("every sequence must contain the shared prefix")
    own = npg - pre_pages if pre_pages else npg
    referenced = int(own.sum()) + pre_pages
    pool = referenced if pool_pages is None else int(pool_pages)
    if pool < referenced:
        raise ValueError("pool smaller than the pages referenced")
    pool = max(pool, 1)
    ids = rng.permutation(pool)[:referenced] if shuffle else np.arange(referenced)
    max_pages = int(max(int(npg.max()) if B else 1, 1))
    if pad_table_to is not None:
        max_pages = max(max_pages, int(pad_table_to))
    bt = np.full((B, max_pages), -1, dtype=np.int32)
    cursor = pre_pages
    for b in range(B):
        if pre_pages:
            bt[b, :pre_pages] = ids[:pre_pages]
        k = int(own[b])
        bt[b, pre_pages:pre_pages + k] = ids[cursor:cursor + k]
        cursor += k

    if layout == "head_major":
        phys = (pool, Hkv, P, Dh)
        to_logical = lambda t: t
    elif layout == "token_major":
        phys = (pool, P, Hkv, Dh)
        to_logical = lambda t: t.permute(0, 2, 1, 3)
    else:
        raise ValueError(layout)

    if kv_dtype not in ("bf16", "fp8"):
        raise ValueError(kv_dtype)
    fp8 = kv_dtype == "fp8"
    nan = E4M3_NAN if fp8 else float("nan")
    pool_dtype = torch.uint8 if fp8 else torch.bfloat16
    k_scale = v_scale = None
    if fp8:
        k_scale, v_scale = (torch.from_numpy(a).to(device) for a in default_kv_scales(Hkv))
    head_shape = (1, Hkv, 1, 1) if layout == "head_major" else (1, 1, Hkv, 1)
    pools = []
    for which in range(2):
        if poison and pool > referenced:
            t = torch.full(phys, nan, dtype=pool_dtype, device=device)
        else:
            t = torch.empty(phys, dtype=pool_dtype, device=device)
        ids_t = torch.from_numpy(np.ascontiguousarray(ids)).to(device)
        for s in range(0, referenced, fill_chunk_pages):
            sel = ids_t[s:s + fill_chunk_pages]
            if fp8:
                inv = (1.0 / (k_scale if which == 0 else v_scale)).reshape(head_shape)
                t[sel] = _randn_e4m3((len(sel),) + phys[1:], gen, device, inv)
            else:
                t[sel] = _randn_bf16((len(sel),) + phys[1:], gen, device)
        pools.append(t)
    k_pages, v_pages = (to_logical(t) for t in pools)

    if poison:
        # rows past a sequence's end inside its last page must never be read
        for b in range(B):
            L = int(lens[b])
            if L > 0 and L % P and not (pre_pages and L <= shared_prefix_tokens):
                page = int(bt[b, (L - 1) // P])
                k_pages[page, :, L % P:, :] = nan
                v_pages[page, :, L % P:, :] = nan

    q = _randn_bf16((B, Hq, Dh), gen, device)
    return Case(
        name=name, q=q, k_pages=k_pages, v_pages=v_pages,
        block_table=torch.from_numpy(bt).to(device),
        seq_lens=torch.from_numpy(lens.astype(np.int32)).to(device),
        window=int(window), scale=float(scale if scale is not None else 1.0 / math.sqrt(Dh)),
        lens=lens.copy(), k_scale=k_scale, v_scale=v_scale)


# ----------------------------------------------------------------------------
# The five workload recipes.
# ----------------------------------------------------------------------------

def lengths_c2(seed: int = 1, B: int = 64) -> np.ndarray:
    return np.random.default_rng(seed).integers(1024, 16385, size=B)


def lengths_c3(seed: int = 2, B: int = 256) -> np.ndarray:
    u = np.random.default_rng(seed).uniform(math.log(512.0), math.log(32768.0), size=B)
    return np.clip(np.floor(np.exp(u)).astype(np.int64), 512, 32768)


def lengths_c5(seed: int = 4, B: int = 128, prefix: int = 16384, max_suffix: int = 8192) -> np.ndarray:
    return prefix + np.random.default_rng(seed).integers(0, max_suffix + 1, size=B)


def c1(device="cpu") -> Case:
    """1 sequence x 512 tokens, page 16, contiguous block table, seed 0, and three
    key rows multiplied by 20 (all KV heads) to stress softmax stability."""
    case = build_case("c1", [512], 16, 0, device, shuffle=False)
    hot = np.random.default_rng(0).choice(512, size=3, replace=False)
    for t in hot:
        page = int(case.block_table[0, t // 16])
        row = case.k_pages[page, :, t % 16, :].float() * 20.0
        case.k_pages[page, :, t % 16, :] = row.to(torch.bfloat16)
    return case


def c2(device="cpu", B: int = 64, kv_dtype: str = "bf16") -> Case:
    """64 sequences, lengths uniform in [1024, 16384], page 16, block tables dealt
    from one random permutation of an exact-size pool, seed 1."""
    return build_case("c2", lengths_c2(1, B), 16, 1, device, kv_dtype=kv_dtype)


def c3(device="cpu", B: int = 256, pool_bytes: float = 20e9, kv_dtype: str = "bf16") -> Case:
    """256 sequences, lengths log-uniform in [512, 32768], page 16, referenced pages
    scattered through a ~20 GB pool (K + V) whose other pages are NaN, seed 2."""
    lens = lengths_c3(2, B)
    page_bytes = 2 * HKV * 16 * D * 2   # the pool keeps its page count when the cache is 8-bit
    referenced = int(((lens + 15) // 16).sum())
    pool = max(int(pool_bytes // page_bytes), referenced)
    return build_case("c3", lens, 16, 2, device, pool_pages=pool, kv_dtype=kv_dtype)


def c4(device="cpu", B: int = 8, L: int = 131072, kv_dtype: str = "bf16") -> Case:
    """8 sequences x 131,072 tokens, page 64, shuffled pool, seed 3."""
    return build_case("c4", [L] * B, 64, 3, device, kv_dtype=kv_dtype)


def c5(device="cpu", window: int = 0, B: int = 128, kv_dtype: str = "bf16") -> Case:
    """128 sequences sharing a 16,384-token prefix (same physical pages in every
    block table) plus unique suffixes uniform in [0, 8192], page 16, seed 4;
    window = 0 (full) or 8192."""
    return build_case("c5b" if window else "c5a", lengths_c5(4, B), 16, 4, device,
                      shared_prefix_tokens=16384, window=window, kv_dtype=kv_dtype)


RECIPES = {"c1": c1, "c2": c2, "c3": c3, "c4": c4,
           "c5a": lambda device="cpu", **kw: c5(device, 0, **kw),
           "c5b": lambda device="cpu", **kw: c5(device, 8192, **kw)}


# ----------------------------------------------------------------------------
# Moving parts of a case to the host (for the CPU oracle's callers).
# ----------------------------------------------------------------------------

def host_subcase(case: Case, seq_ids: Sequence[int]) -> Case:
    """A CPU copy of the chosen sequences only: their pages are gathered into a
    compact head-major pool and the block table is renumbered to match.  Pure
    copying; values are untouched."""
    seq_ids = list(seq_ids)
    P = case.P
    lens = case.lens[seq_ids]
    npg = np.maximum((lens + P - 1) // P, 0)
    bt_host = case.block_table[seq_ids].cpu().numpy()
    used = np.unique(np.concatenate([bt_host[i, :npg[i]] for i in range(len(seq_ids))]
                                    + [np.zeros(0, np.int32)]))
    remap = {int(p): i for i, p in enumerate(used)}
    new_bt = np.full_like(bt_host, -1)
    for i in range(len(seq_ids)):
        new_bt[i, :npg[i]] = [remap[int(p)] for p in bt_host[i, :npg[i]]]
    sel = torch.from_numpy(used.astype(np.int64)).to(case.k_pages.device)
    if len(used) == 0:
        sel = torch.zeros(1, dtype=torch.int64, device=case.k_pages.device)
    k = case.k_pages.index_select(0, sel).contiguous().cpu()
    v = case.v_pages.index_select(0, sel).contiguous().cpu()
    return Case(name=case.name + "/sub", q=case.q[seq_ids].cpu(), k_pages=k, v_pages=v,
                block_table=torch.from_numpy(new_bt), seq_lens=torch.from_numpy(lens.astype(np.int32)),
                window=case.window, scale=case.scale, lens=lens.copy(),
                k_scale=None if case.k_scale is None else case.k_scale.cpu(),
                v_scale=None if case.v_scale is None else case.v_scale.cpu())


def to_device(case: Case, device) -> Case:
    """Copy a case to another device, keeping the pools' strides."""
    def mv(t):
        if t.is_contiguous():
            return t.to(device)
        # keep memory order: move the underlying dense buffer, then re-view
        order = sorted(range(t.dim()), key=lambda i: -t.stride(i))
        dense = t.permute(order).contiguous().to(device)
        inv = [order.index(i) for i in range(t.dim())]
        return dense.permute(inv)
    return Case(name=case.name, q=case.q.to(device), k_pages=mv(case.k_pages), v_pages=mv(case.v_pages),
                block_table=case.block_table.to(device), seq_lens=case.seq_lens.to(device),
                window=case.window, scale=case.scale, lens=case.lens.copy(),
                k_scale=None if case.k_scale is None else case.k_scale.to(device),
                v_scale=None if case.v_scale is None else case.v_scale.to(device))
