"""Seeded synthetic inputs shaped like the paper's decode / prefill workloads.

This module only makes data: random tensors, sequence lengths, page tables and
storage-dtype rounding.  It contains none of the attention arithmetic and it
imports neither the CUDA binding nor the CPU oracle, so both sides can be fed the
very same host buffers.

Tensors are numpy arrays in their storage dtype: ``float32``, or ``uint16`` holding
bf16 bit patterns (numpy has no bf16).  ``to_torch`` reinterprets them for the GPU.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace
from typing import Dict, Optional, Tuple

import numpy as np

_CHUNK = 1 << 24  # elements drawn per independent Philox stream


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even), returned as uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (r >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def as_f64(a: np.ndarray) -> np.ndarray:
    """Exact widening of a storage array (float32 or bf16 bits) to float64."""
    if a.dtype == np.uint16:
        return bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


def normal(seed: int, shape, std: float = 1.0, dtype: str = "bf16") -> np.ndarray:
    """i.i.d. N(0, std^2) values, deterministic in (seed, shape), in the storage dtype.

    The stream is cut into fixed chunks, chunk c drawn from Philox(key=seed, counter
    block c), so the result does not depend on the number of worker threads.
    """
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16 if dtype == "bf16" else np.float32)

    def fill(c: int):
        lo, hi = c * _CHUNK, min(n, (c + 1) * _CHUNK)
        g = np.random.Generator(np.random.Philox(key=seed, counter=[0, 0, c, 0]))
        x = g.standard_normal(hi - lo, dtype=np.float32)
        if std != 1.0:
            x *= np.float32(std)
        out[lo:hi] = f32_to_bf16_bits(x) if dtype == "bf16" else x

    chunks = range((n + _CHUNK - 1) // _CHUNK)
    if len(chunks) <= 1:
        for c in chunks:
            fill(c)
    else:
        with ThreadPoolExecutor(max_workers=16) as ex:
            list(ex.map(fill, chunks))
    return out.reshape(shape)


def to_torch(a: np.ndarray, device=None):
    """numpy storage array -> torch tensor (uint16 bit patterns become bfloat16)."""
    import torch
    t = torch.from_numpy(a)
    if a.dtype == np.uint16:
        t = t.view(torch.bfloat16)
    return t.to(device) if device is not None else t


@dataclass(frozen=True)
class DecodeConfig:
    """One decode workload. ``lengths`` None means every sequence has ``kv_len`` tokens."""
    name: str
    batch: int
    n_q: int
    n_k: int
    n_v: int
    d_qk: int
    d_v: int
    kv_len: int
    dtype: str = "bf16"            # storage dtype of q and the cache
    seed: int = 0
    page_size: int = 0             # 0 = contiguous [batch, head, seq, dim]
    len_range: Optional[Tuple[int, int]] = None  # uniform integer lengths in [lo, hi]

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(self.d_qk))

    def gqa_twin(self) -> "DecodeConfig":
        """The comparison shape: same Q and V heads, K given as many heads as V (n_k = n_v)."""
        return replace(self, name=self.name + "_gqa", n_k=self.n_v)


# The five configurations the benchmark definition lists (decode ones here, prefill below).
CFG1 = DecodeConfig("cfg1_small_f32", batch=1, n_q=16, n_k=2, n_v=4, d_qk=64, d_v=64, kv_len=512,
                    dtype="f32", seed=0)
CFG2 = DecodeConfig("cfg2_b16_4k", batch=16, n_q=16, n_k=2, n_v=4, d_qk=128, d_v=128, kv_len=4096,
                    seed=2000)
CFG3 = DecodeConfig("cfg3_b4_32k", batch=4, n_q=32, n_k=4, n_v=8, d_qk=128, d_v=128, kv_len=32768,
                    seed=3000)
CFG5 = DecodeConfig("cfg5_paged_varlen", batch=64, n_q=32, n_k=4, n_v=8, d_qk=128, d_v=128,
                    kv_len=65536, seed=5000, page_size=16, len_range=(1024, 65536))
# The paper's own efficiency experiment: SIGMA-1.5B heads against the 16/16 GQA standard model.
SIGMA15B = DecodeConfig("sigma1p5b", batch=1, n_q=32, n_k=4, n_v=16, d_qk=64, d_v=64, kv_len=32768,
                        seed=6000)
DECODE_CONFIGS: Dict[str, DecodeConfig] = {c.name: c for c in (CFG1, CFG2, CFG3, CFG5, SIGMA15B)}


@dataclass(frozen=True)
class PrefillConfig:
    name: str
    batch: int
    seq: int
    n_q: int
    n_k: int
    n_v: int
    d_qk: int
    d_v: int
    d_model: int
    d_aug: int
    seed: int = 4000
    h_std: float = 0.02

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(self.d_qk))


CFG4 = PrefillConfig("cfg4_prefill_8k", batch=2, seq=8192, n_q=32, n_k=4, n_v=8, d_qk=128, d_v=128,
                     d_model=2048, d_aug=3072)


@dataclass
class DecodeInputs:
    cfg: DecodeConfig
    q: np.ndarray                 # [batch, n_q, d_qk]
    k: np.ndarray                 # contiguous [batch, n_k, S, d_qk] or paged [pages, n_k, page, d_qk]
    v: np.ndarray
    seqlens: np.ndarray           # int32 [batch]
    k_strides: Tuple[int, int, int]  # elements: (blk, head, tok)
    v_strides: Tuple[int, int, int]
    page_table: Optional[np.ndarray] = None  # int32 [batch, max_pages_per_seq]
    num_pages: int = 0
    max_seqlen: int = 0
    extra: dict = field(default_factory=dict)


def draw_lengths(cfg: DecodeConfig) -> np.ndarray:
    if cfg.len_range is None:
        return np.full(cfg.batch, cfg.kv_len, dtype=np.int32)
    g = np.random.Generator(np.random.Philox(key=cfg.seed + 7))
    lo, hi = cfg.len_range
    return g.integers(lo, hi + 1, size=cfg.batch).astype(np.int32)


def shuffled_page_table(seqlens: np.ndarray, page_size: int, seed: int, spare_pages: int = 0,
                        unused: int = 0):
    """Every sequence gets ceil(len / page_size) distinct physical pages drawn from one
    seeded permutation of the pool; table entries past a sequence's last page hold ``unused``."""
    pages_per = (seqlens.astype(np.int64) + page_size - 1) // page_size
    num_pages = int(pages_per.sum()) + spare_pages
    g = np.random.Generator(np.random.Philox(key=seed + 11))
    perm = g.permutation(num_pages).astype(np.int32)
    table = np.full((len(seqlens), int(pages_per.max()) if len(seqlens) else 0), unused, dtype=np.int32)
    at = 0
    for b, n in enumerate(pages_per):
        table[b, :n] = perm[at:at + n]
        at += int(n)
    return table, num_pages


def make_decode_inputs(cfg: DecodeConfig, seqlens: Optional[np.ndarray] = None) -> DecodeInputs:
    """q, K, V i.i.d. N(0,1) in the config's storage dtype; tensor t uses seed cfg.seed + t."""
    if seqlens is None:
        seqlens = draw_lengths(cfg)
    seqlens = np.ascontiguousarray(seqlens, dtype=np.int32)
    q = normal(cfg.seed + 0, (cfg.batch, cfg.n_q, cfg.d_qk), dtype=cfg.dtype)
    if cfg.page_size == 0:
        S = cfg.kv_len
        k = normal(cfg.seed + 1, (cfg.batch, cfg.n_k, S, cfg.d_qk), dtype=cfg.dtype)
        v = normal(cfg.seed + 2, (cfg.batch, cfg.n_v, S, cfg.d_v), dtype=cfg.dtype)
        return DecodeInputs(cfg, q, k, v, seqlens,
                            (cfg.n_k * S * cfg.d_qk, S * cfg.d_qk, cfg.d_qk),
                            (cfg.n_v * S * cfg.d_v, S * cfg.d_v, cfg.d_v), max_seqlen=S)
    ps = cfg.page_size
    table, num_pages = shuffled_page_table(seqlens, ps, cfg.seed)
    k = normal(cfg.seed + 1, (num_pages, cfg.n_k, ps, cfg.d_qk), dtype=cfg.dtype)
    v = normal(cfg.seed + 2, (num_pages, cfg.n_v, ps, cfg.d_v), dtype=cfg.dtype)
    return DecodeInputs(cfg, q, k, v, seqlens,
                        (cfg.n_k * ps * cfg.d_qk, ps * cfg.d_qk, cfg.d_qk),
                        (cfg.n_v * ps * cfg.d_v, ps * cfg.d_v, cfg.d_v),
                        page_table=table, num_pages=num_pages, max_seqlen=int(table.shape[1]) * ps)


def paginate(inp: DecodeInputs, page_size: int, seed: int, identity: bool = False) -> DecodeInputs:
    """Re-lay a contiguous cache into pages (pure byte movement): same tokens, new addresses."""
    cfg = inp.cfg
    assert inp.page_table is None
    S = inp.k.shape[2]
    pages_per_seq = (S + page_size - 1) // page_size
    lens_full = np.full(cfg.batch, pages_per_seq * page_size, dtype=np.int32)
    if identity:
        table = np.arange(cfg.batch * pages_per_seq, dtype=np.int32).reshape(cfg.batch, pages_per_seq)
        num_pages = cfg.batch * pages_per_seq
    else:
        table, num_pages = shuffled_page_table(lens_full, page_size, seed, spare_pages=3)
    k = np.zeros((num_pages, cfg.n_k, page_size, cfg.d_qk), dtype=inp.k.dtype)
    v = np.zeros((num_pages, cfg.n_v, page_size, cfg.d_v), dtype=inp.v.dtype)
    for b in range(cfg.batch):
        for p in range(pages_per_seq):
            lo, hi = p * page_size, min(S, (p + 1) * page_size)
            k[table[b, p], :, : hi - lo] = inp.k[b, :, lo:hi]
            v[table[b, p], :, : hi - lo] = inp.v[b, :, lo:hi]
    return DecodeInputs(replace(cfg, page_size=page_size), inp.q, k, v, inp.seqlens,
                        (cfg.n_k * page_size * cfg.d_qk, page_size * cfg.d_qk, cfg.d_qk),
                        (cfg.n_v * page_size * cfg.d_v, page_size * cfg.d_v, cfg.d_v),
                        page_table=table, num_pages=num_pages, max_seqlen=pages_per_seq * page_size)


@dataclass
class PrefillInputs:
    cfg: PrefillConfig
    h: np.ndarray        # [batch*seq, d_model]
    W_Q: np.ndarray      # [n_q*d_qk, d_model]   (nn.Linear layout: [out, in])
    W_gate: np.ndarray   # [d_aug, n_q*d_qk]
    W_up: np.ndarray     # [d_aug, n_q*d_qk]
    W_down: np.ndarray   # [n_q*d_qk, d_aug]
    k_new: np.ndarray    # [batch, seq, n_k, d_qk]
    v_new: np.ndarray    # [batch, seq, n_v, d_v]
    q_direct: np.ndarray  # [batch, seq, n_q, d_qk] N(0,1) queries for a peaked softmax


def make_prefill_inputs(cfg: PrefillConfig) -> PrefillInputs:
    """Hidden states N(0, h_std^2); weights N(0, 1/fan_in); K, V and the direct q N(0,1); all bf16."""
    T = cfg.batch * cfg.seq
    d_q0 = cfg.n_q * cfg.d_qk
    s = cfg.seed
    return PrefillInputs(
        cfg,
        h=normal(s + 0, (T, cfg.d_model), std=cfg.h_std),
        W_Q=normal(s + 1, (d_q0, cfg.d_model), std=cfg.d_model ** -0.5),
        W_gate=normal(s + 2, (cfg.d_aug, d_q0), std=d_q0 ** -0.5),
        W_up=normal(s + 3, (cfg.d_aug, d_q0), std=d_q0 ** -0.5),
        W_down=normal(s + 4, (d_q0, cfg.d_aug), std=cfg.d_aug ** -0.5),
        k_new=normal(s + 5, (cfg.batch, cfg.seq, cfg.n_k, cfg.d_qk)),
        v_new=normal(s + 6, (cfg.batch, cfg.seq, cfg.n_v, cfg.d_v)),
        q_direct=normal(s + 7, (cfg.batch, cfg.seq, cfg.n_q, cfg.d_qk)),
    )
