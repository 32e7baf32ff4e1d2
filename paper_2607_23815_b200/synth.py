"""Seeded synthetic inputs for the paged-KV attention path.

This module only draws numbers and lays out batches (lengths, page placement,
block tables).  It contains none of the attention / append arithmetic, so both
the CPU oracle's tests and the CUDA path's tests may take their inputs from it.

Values are produced by a counter-based generator keyed on *logical*
coordinates (tensor tag, sequence uid, token position, head, dim).  Re-drawing
the K/V of a sequence prefix (after an eviction, or for a from-scratch prefill
of prefix+suffix) therefore reproduces the same numbers, which is what the
"reuse == recompute" checks rely on (paper Section 2.1, prefix caching: the KV
entries of an identical prompt prefix are identical).

The workload shapes follow the paper's evaluation (Section 7.2, Table 2: tuple
contexts of a few hundred to a few thousand tokens, short operator
instructions, answers of at most 8 tokens for predicates) with i.i.d. N(0,1)
bf16 values standing in for real activations.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import numpy as np
import torch

# tensor tags
TAG_Q, TAG_K, TAG_V, TAG_LEN_A, TAG_LEN_B, TAG_PERM, TAG_MISC = 1, 2, 3, 4, 5, 6, 7

_MASK64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Python int -> two's complement signed 64-bit value."""
    x &= _MASK64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_M1 = _s64(0xBF58476D1CE4E5B9)
_M2 = _s64(0x94D049BB133111EB)
_C_UID = _s64(0xD6E8FEB86659FD93)
_C_POS = _s64(0xA0761D6478BD642F)
_C_ELT = _s64(0xE7037ED1A0B428DB)


def _lsr(z: torch.Tensor, k: int) -> torch.Tensor:
    return (z >> k) & ((1 << (64 - k)) - 1)


def _mix64(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 output function on int64 tensors (wrap-around arithmetic)."""
    z = z + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _M1
    z = (z ^ _lsr(z, 27)) * _M2
    return z ^ _lsr(z, 31)


def _mix64_int(z: int) -> int:
    z = (z + 0x9E3779B97F4A7C15) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


def hash_u64(seed: int, tag: int, index: int) -> int:
    """Scalar hash used for lengths and other per-item draws."""
    return _mix64_int(_mix64_int((seed << 8) ^ tag) ^ ((index * 0xD6E8FEB86659FD93) & _MASK64))


def uniform_int(seed: int, tag: int, index: int, lo: int, hi: int) -> int:
    """Inclusive discrete uniform in [lo, hi] (modulo bias < 2^-40, ignored)."""
    return lo + hash_u64(seed, tag, index) % (hi - lo + 1)


def normal_bf16(seed: int, tag: int, uid: int, pos0: int, n_tokens: int, n_heads: int,
                head_dim: int, device="cpu") -> torch.Tensor:
    """N(0,1) values rounded to bf16, shape [n_tokens][n_heads][head_dim].

    Element (t, h, d) depends only on (seed, tag, uid, pos0 + t, h, d).
    """
    if n_tokens == 0:
        return torch.empty((0, n_heads, head_dim), dtype=torch.bfloat16, device=device)
    base = _s64(_mix64_int(_mix64_int((seed << 8) ^ tag) ^ ((uid * 0xD6E8FEB86659FD93) & _MASK64)))
    pos = torch.arange(pos0, pos0 + n_tokens, dtype=torch.int64, device=device)
    row = _mix64(pos * _C_POS + base)                                   # [T]
    elt = torch.arange(n_heads * head_dim, dtype=torch.int64, device=device) * _C_ELT
    bits = _mix64(row[:, None] ^ elt[None, :])                          # [T][H*D]
    u1 = (_lsr(bits, 40).to(torch.float32) + 1.0) * (1.0 / 16777216.0)  # (0, 1]
    u2 = ((bits >> 8) & 0xFFFFFF).to(torch.float32) * (1.0 / 16777216.0)
    z = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
    return z.to(torch.bfloat16).reshape(n_tokens, n_heads, head_dim)


def page_permutation(seed: int, num_pages: int) -> np.ndarray:
    """Seeded permutation of the pool's page ids (argsort of hashed keys)."""
    idx = torch.arange(num_pages, dtype=torch.int64)
    base = _s64(_mix64_int((seed << 8) ^ TAG_PERM))
    keys = _mix64(idx * _C_UID + base)
    return torch.argsort(keys, stable=True).numpy().astype(np.int32)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor -> numpy uint16 bit patterns (exact, on the host)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def bits_to_bf16(bits: np.ndarray, device="cpu") -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).to(device)


# --------------------------------------------------------------------------- #
# workload shapes
# --------------------------------------------------------------------------- #
@dataclasses.dataclass(frozen=True)
class Geometry:
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    page_size: int = 16

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def scale(self) -> float:
        return float(np.float32(1.0 / math.sqrt(self.head_dim)))

    @property
    def kv_bytes_per_token(self) -> int:
        """Per-layer K+V bytes of one token in bf16."""
        return 2 * self.n_kv_heads * self.head_dim * 2


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    geom: Geometry
    num_pages: int
    n_extend: int = 0
    prefix_range: tuple = (0, 0)
    extend_range: tuple = (0, 0)
    n_decode: int = 0
    ctx_range: tuple = (0, 0)
    seed: int = 260723815


_LLAMA8B = Geometry(32, 8, 128)
_LLAMA70B = Geometry(64, 8, 128)

WORKLOADS = {
    # tiny correctness case: reuse must equal a from-scratch prefill
    "tiny": Workload("tiny", Geometry(4, 2, 64), 256, n_extend=8, prefix_range=(32, 128),
                     extend_range=(16, 48), seed=260723815 + 0),
    # downstream operator's suffix over an upstream tuple's pages
    "extend_8b": Workload("extend_8b", _LLAMA8B, 32768, n_extend=64, prefix_range=(512, 2048),
                          extend_range=(64, 256), seed=260723815 + 1),
    # short semantic-operator answers decoded over the same pages
    "decode_8b": Workload("decode_8b", _LLAMA8B, 65536, n_decode=256, ctx_range=(1024, 4096),
                          seed=260723815 + 2),
    # sem_map feeding sem_filter: one mixed step
    "pipeline_step": Workload("pipeline_step", _LLAMA8B, 65536, n_extend=48, prefix_range=(256, 3072),
                              extend_range=(32, 192), n_decode=192, ctx_range=(512, 4088),
                              seed=260723815 + 3),
    # long-document reuse
    "long_doc_70b": Workload("long_doc_70b", _LLAMA70B, 40960, n_extend=32, prefix_range=(8192, 16384),
                             extend_range=(128, 512), seed=260723815 + 4),
}


def scaled(w: Workload, **kw) -> Workload:
    return dataclasses.replace(w, **kw)


@dataclasses.dataclass
class Sequence:
    uid: int
    prefix_len: int          # tokens already in the pool before this step (P, or C-1 ... see kind)
    new_len: int             # tokens appended this step (E for extend, 1 for decode)
    pages: List[int]         # physical page ids, logical block order

    @property
    def total_len(self) -> int:
        return self.prefix_len + self.new_len


def draw_lengths(w: Workload):
    """Per-sequence (prefix, extend) pairs and decode context lengths."""
    ext = [(uniform_int(w.seed, TAG_LEN_A, i, *w.prefix_range),
            uniform_int(w.seed, TAG_LEN_B, i, *w.extend_range)) for i in range(w.n_extend)]
    dec = [uniform_int(w.seed, TAG_LEN_A, 1_000_000 + i, *w.ctx_range) for i in range(w.n_decode)]
    return ext, dec


def pages_needed(length: int, page_size: int) -> int:
    return (length + page_size - 1) // page_size


def block_table(rows: List[List[int]], max_pages: Optional[int] = None) -> np.ndarray:
    """Pad page-id lists to a rectangular int32 table with -1."""
    width = max([len(r) for r in rows] + [1]) if max_pages is None else max_pages
    bt = np.full((len(rows), width), -1, dtype=np.int32)
    for i, r in enumerate(rows):
        bt[i, :len(r)] = r
    return bt
