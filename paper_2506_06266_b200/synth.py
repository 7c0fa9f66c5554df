"""Seeded synthetic inputs for Cartridge decode attention.

This module only draws random numbers and shapes.  It holds none of the attention arithmetic and
imports neither the CUDA binding nor the CPU oracle, so both sides can be fed from it.

The recipes stand in for the paper's throughput protocol (App. A.3: a batch of randomly initialised
Cartridges of a given size pre-loaded on the GPU, tokens appended to the KV cache while decoding)
at Llama-3B / Llama-8B attention shapes; no dataset or trained weight is involved.

Values: float32 N(0,1) rounded to nearest-even bf16.  Integers (suffix lengths, which Cartridges a
request composes) come from ``numpy.random.default_rng``.  Every draw has its own sub-seed derived
from the workload seed so that a tensor can be regenerated alone.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional, Tuple

import numpy as np
import torch

# sub-stream offsets added to a workload's seed
SUB_CARTRIDGE = 0      # + cartridge index * 2 (K), +1 (V) inside a 1e6-wide block
SUB_SUFFIX = 10
SUB_Q = 20
SUB_LENGTHS = 30
SUB_APPEND = 40
SUB_OUTLIER = 50


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def normal_bf16(shape, seed: int, device="cpu") -> torch.Tensor:
    """N(0,1) drawn in float32 and rounded to bf16 (round to nearest even)."""
    dev = torch.device(device)
    x = torch.randn(tuple(shape), generator=_gen(seed, dev), device=dev, dtype=torch.float32)
    return x.to(torch.bfloat16)


def normal_bf16_chunked(shape, seed: int, device, chunk_elems: int = 1 << 28) -> torch.Tensor:
    """Like normal_bf16 but fills a large tensor piecewise along dim 0 so that the float32
    temporary stays small; piece i uses seed + 7919 * i."""
    out = torch.empty(tuple(shape), device=device, dtype=torch.bfloat16)
    rows = shape[0]
    per_row = int(np.prod(shape[1:])) if len(shape) > 1 else 1
    step = max(1, chunk_elems // max(per_row, 1))
    for i, r0 in enumerate(range(0, rows, step)):
        r1 = min(rows, r0 + step)
        out[r0:r1] = normal_bf16((r1 - r0,) + tuple(shape[1:]), seed + 7919 * i, device)
    return out


def bits(t: torch.Tensor) -> np.ndarray:
    """The bf16 bit patterns of a tensor as a uint16 numpy array (copied to the host)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def outlier_channels(n_layers: int, n_kv_heads: int, head_dim: int, seed: int, prob: float
                     ) -> np.ndarray:
    """Boolean [L][Hkv][D]: which key channels are outliers.  A channel is a (layer, KV head, dim)
    triple, fixed across tokens and requests, as a property of a model would be."""
    rng = np.random.default_rng(seed + SUB_OUTLIER)
    return rng.random((n_layers, n_kv_heads, head_dim)) < prob


def scale_key_channels(k: torch.Tensor, mask_lhd: np.ndarray, factor: float) -> torch.Tensor:
    """Multiply the masked channels of k ([L][Hkv][n][D]) by ``factor`` (a power of two keeps
    bf16 values exact)."""
    m = torch.from_numpy(mask_lhd).to(k.device)
    mult = torch.where(m, torch.tensor(float(factor)), torch.tensor(1.0)).to(torch.bfloat16)
    return k * mult[:, :, None, :].to(k.device)


@dataclass(frozen=True)
class Workload:
    """One synthetic serving scenario.

    cartridges: 'private' -- every request has its own Cartridge of p tokens;
                'shared'  -- all requests attend to one Cartridge stored once;
                'pool'    -- ``pool`` Cartridges; each request composes ``compose`` distinct
                             members, order kept;
                'none'    -- suffix only.
    Suffix lengths are uniform integers in [suffix_lo, suffix_hi] (both inclusive).
    """
    name: str
    seed: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    batch: int
    p: int
    suffix_lo: int
    suffix_hi: int
    cartridges: str = "private"
    pool: int = 0
    compose: int = 1
    outlier_prob: float = 0.0
    outlier_factor: float = 8.0
    decode_steps: int = 1
    head_dim: int = 128

    @property
    def scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))

    @property
    def n_cartridges(self) -> int:
        return {"private": self.batch, "shared": 1, "pool": self.pool, "none": 0}[self.cartridges]

    def suffix_lengths(self) -> np.ndarray:
        rng = np.random.default_rng(self.seed + SUB_LENGTHS)
        return rng.integers(self.suffix_lo, self.suffix_hi + 1, size=self.batch).astype(np.int64)

    def request_parts(self) -> List[List[int]]:
        """For each request, the ordered Cartridge indices it attends to."""
        if self.cartridges == "private":
            return [[b] for b in range(self.batch)]
        if self.cartridges == "shared":
            return [[0] for _ in range(self.batch)]
        if self.cartridges == "none":
            return [[] for _ in range(self.batch)]
        rng = np.random.default_rng(self.seed + SUB_LENGTHS + 1)
        return [list(map(int, rng.choice(self.pool, self.compose, replace=False)))
                for _ in range(self.batch)]

    def kv_tokens(self) -> np.ndarray:
        """KV tokens each request attends to (Cartridge tokens + suffix) before any decode append."""
        parts = self.request_parts()
        return np.asarray([len(pp) * self.p for pp in parts], dtype=np.int64) + self.suffix_lengths()

    def kv_bytes_per_token_layer(self) -> int:
        return 2 * self.n_kv_heads * self.head_dim * 2

    # ---- tensors -------------------------------------------------------------------------
    def cartridge_kv(self, index: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
        """(K, V) bf16 [L][Hkv][p][D] of Cartridge ``index``."""
        shape = (self.n_layers, self.n_kv_heads, self.p, self.head_dim)
        base = self.seed * 1_000_003 + SUB_CARTRIDGE + 2 * index
        k = normal_bf16_chunked(shape, base, device)
        v = normal_bf16_chunked(shape, base + 1, device)
        if self.outlier_prob > 0:
            k = scale_key_channels(k, self.outlier_mask(), self.outlier_factor)
        return k, v

    def suffix_kv(self, request: int, length: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
        """(K, V) bf16 [L][T][Hkv][D]: the suffix tokens of a request, token-major per layer."""
        shape = (self.n_layers, length, self.n_kv_heads, self.head_dim)
        base = self.seed * 1_000_003 + 500_000 + SUB_SUFFIX + 2 * request
        k = normal_bf16(shape, base, device)
        v = normal_bf16(shape, base + 1, device)
        if self.outlier_prob > 0:
            m = torch.from_numpy(self.outlier_mask()).to(k.device)
            mult = torch.where(m, torch.tensor(float(self.outlier_factor)), torch.tensor(1.0))
            k = k * mult.to(torch.bfloat16).to(k.device)[:, None, :, :]
        return k, v

    def queries(self, step: int, device="cpu") -> torch.Tensor:
        """bf16 [L][B][Hq][D]: the query of every request at every layer for decode step ``step``."""
        shape = (self.n_layers, self.batch, self.n_q_heads, self.head_dim)
        return normal_bf16(shape, self.seed * 1_000_003 + 700_000 + SUB_Q + step, device)

    def appended_kv(self, step: int, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
        """(K, V) bf16 [L][B][Hkv][D]: the token each request appends at decode step ``step``."""
        shape = (self.n_layers, self.batch, self.n_kv_heads, self.head_dim)
        base = self.seed * 1_000_003 + 800_000 + SUB_APPEND + 2 * step
        k = normal_bf16(shape, base, device)
        v = normal_bf16(shape, base + 1, device)
        if self.outlier_prob > 0:
            m = torch.from_numpy(self.outlier_mask()).to(k.device)
            mult = torch.where(m, torch.tensor(float(self.outlier_factor)), torch.tensor(1.0))
            k = k * mult.to(torch.bfloat16).to(k.device)[:, None, :, :]
        return k, v

    def outlier_mask(self) -> np.ndarray:
        return outlier_channels(self.n_layers, self.n_kv_heads, self.head_dim, self.seed,
                                self.outlier_prob)


# The five workloads the benchmark contract names (seeds 1001..1005).
def config1() -> Workload:
    return Workload("c1_single_layer_b4", 1001, 1, 24, 8, 4, 512, 64, 64)


def config2() -> Workload:
    return Workload("c2_llama3b_b64_p2048", 1002, 28, 24, 8, 64, 2048, 1, 512,
                    outlier_prob=0.001)


def config3() -> Workload:
    return Workload("c3_llama8b_b128_shared_p4096", 1003, 32, 32, 8, 128, 4096, 1, 1024,
                    cartridges="shared", decode_steps=64)


def config4() -> Workload:
    return Workload("c4_llama8b_b96_compose2of16_p2048", 1004, 32, 32, 8, 96, 2048, 1, 512,
                    cartridges="pool", pool=16, compose=2)


def config5_full() -> Workload:
    return Workload("c5_full_context_b8_n100k", 1005, 32, 32, 8, 8, 100_000, 256, 256)


def config5_cartridge() -> Workload:
    return Workload("c5_cartridge_b256_p2048", 1005, 32, 32, 8, 256, 2048, 256, 256)


def shrink(w: Workload, **kw) -> Workload:
    """A smaller workload of the same structure (for tests the oracle finishes in seconds)."""
    return replace(w, **kw)
