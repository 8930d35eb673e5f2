"""Seeded synthetic workloads for the EchoKV decode path.

This module only *draws inputs*: shapes, seeds, value distributions and page
orders.  It holds none of the method's arithmetic (no reconstruction, no
softmax) and is the one module that both the CPU oracle's tests and the CUDA
library's tests use, so that both sides see bit-identical stored values.

Recipe (stands in for the paper's LongBench / RULER-driven serving workloads,
whose items are not reproduced here; shapes follow the paper's backbones,
Appendix "Compression-Ratio Configurations": GQA 8 KV heads x 128, and the
Llama-2-7B MHA shape):
  anchor-layer K, V      ~ N(0, 1)
  compressed-layer K, V  = rho * anchor + sqrt(1 - rho^2) * N(0, 1)  (fp32, then
                           one rounding to the storage dtype), so that the layers
                           are similar the way the paper's inter-layer
                           similarity premise assumes
  queries                ~ N(0, 1)
  predictors Wk, Wv      Xavier-uniform U(-a, a), a = sqrt(6 / (D_in + D_drop)),
                           independent per layer and per K / V
  pages                  identity order or a seeded random permutation
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    dtype: str            # "bf16" | "fp32": storage type of cache, weights, q
    batch: int
    context: int          # L: tokens in the cache at the decode step (newest included)
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_retained_heads: int  # r; m = r * head_dim
    rho: float             # correlation of a compressed layer to its anchor
    n_layers: int = 2
    group_size: int = 2    # S
    page_tokens: int = 16
    random_pages: bool = False
    seed: int = 1000
    n_retained_dims: int = 0   # if non-zero: m itself, in flat dims (need not end on a head boundary)
    save_k: bool = False       # compressed layers keep their keys whole; only the values are evicted and predicted

    @property
    def D(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def m(self) -> int:
        return self.n_retained_dims if self.n_retained_dims else self.n_retained_heads * self.head_dim

    @property
    def mk(self) -> int:
        """K dims a compressed layer stores."""
        return self.D if (self.save_k and self.m < self.D) else self.m

    @property
    def d_in(self) -> int:
        return self.D + self.m

    @property
    def d_drop(self) -> int:
        return self.D - self.m

    @property
    def pages_per_seq(self) -> int:
        return (self.context + self.page_tokens - 1) // self.page_tokens

    def is_anchor(self, layer: int) -> bool:
        return layer % self.group_size == 0

    def anchor_of(self, layer: int) -> int:
        return layer - layer % self.group_size

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five benchmark configurations, in order.
C0 = Workload("c0_tiny_fp32", "fp32", 1, 512, 8, 8, 64, 4, 0.8, seed=1000)
C1 = Workload("c1_llama2_7b_layer", "bf16", 8, 8192, 32, 32, 128, 16, 0.8, seed=1001)
C2 = Workload("c2_llama3_8b_gqa_layer", "bf16", 16, 32768, 32, 8, 128, 2, 0.7, seed=1002)
C3 = Workload("c3_llama2_7b_32layers", "bf16", 4, 16384, 32, 32, 128, 16, 0.8,
              n_layers=32, group_size=4, random_pages=True, seed=1003)


def c4_point(ratio_pct: int, context: int, batch: int) -> Workload:
    """One point of the Llama-3-8B-shaped sweep: ratio_pct of the layer's KV
    heads are discarded (25 / 50 / 75)."""
    r = {25: 6, 50: 4, 75: 2}[ratio_pct]
    return Workload("c4_r%d_L%d_B%d" % (ratio_pct, context, batch), "bf16", batch, context,
                    32, 8, 128, r, 0.7, seed=1004)


CONFIGS = {"c0": C0, "c1": C1, "c2": C2, "c3": C3}


def torch_dtype(w: Workload) -> torch.dtype:
    return torch.bfloat16 if w.dtype == "bf16" else torch.float32


def _gen(seed: int, *stream: int, device="cpu") -> torch.Generator:
    """Independent sub-stream per (seed, tensor id, layer, ...).  A CUDA generator draws a
    different (equally deterministic) sequence than the CPU one: workloads too large to draw on
    the host are drawn on the device and read back where the oracle needs them."""
    s = seed
    for v in stream:
        s = (s * 1000003 + 7919 * (v + 1)) % (2 ** 62)
    g = torch.Generator(device=device)
    g.manual_seed(s)
    return g


T_ANCHOR_K, T_ANCHOR_V, T_NOISE_K, T_NOISE_V, T_WK, T_WV, T_Q, T_PAGES = range(8)


def normal(shape, seed: int, *stream: int, device="cpu") -> torch.Tensor:
    return torch.randn(shape, generator=_gen(seed, *stream, device=device), dtype=torch.float32, device=device)


def xavier_uniform(d_out: int, d_in: int, seed: int, *stream: int, device="cpu") -> torch.Tensor:
    a = math.sqrt(6.0 / (d_in + d_out))
    u = torch.rand((d_out, d_in), generator=_gen(seed, *stream, device=device), dtype=torch.float32, device=device)
    return (u * 2.0 - 1.0) * a


def anchor_cache(w: Workload, layer: int, kind: str, batch_index: int | None = None, device="cpu") -> torch.Tensor:
    """fp32 pre-rounding N(0,1) cache of anchor layer `layer`: [B, L, D]
    (or [L, D] for one sequence).  kind is "k" or "v"."""
    tid = T_ANCHOR_K if kind == "k" else T_ANCHOR_V
    if batch_index is None:
        return torch.stack([anchor_cache(w, layer, kind, b, device) for b in range(w.batch)])
    return normal((w.context, w.D), w.seed, tid, layer, batch_index, device=device)


def layer_cache(w: Workload, layer: int, kind: str, batch_index: int, width: int | None = None,
                anchor_f32: torch.Tensor | None = None, device="cpu") -> torch.Tensor:
    """Stored-precision cache of `layer` for one sequence: [L, width].

    An anchor layer is N(0,1); a compressed layer is rho * anchor + sqrt(1 -
    rho^2) * N(0,1), mixed in fp32 on the flattened feature axis.  `width`
    limits the result to the first `width` flat dims (a compressed layer only
    stores m of them).
    """
    width = w.D if width is None else width
    a_layer = w.anchor_of(layer)
    if anchor_f32 is None:
        anchor_f32 = anchor_cache(w, a_layer, kind, batch_index, device)
    if layer == a_layer:
        x = anchor_f32[:, :width]
    else:
        tid = T_NOISE_K if kind == "k" else T_NOISE_V
        noise = normal((w.context, w.D), w.seed, tid, layer, batch_index, device=device)[:, :width]
        x = w.rho * anchor_f32[:, :width] + math.sqrt(1.0 - w.rho * w.rho) * noise
    return x.to(torch_dtype(w)).contiguous()


def predictor_weights(w: Workload, layer: int, kind: str, device="cpu") -> torch.Tensor:
    """Stored-precision predictor of a compressed layer: [D_drop, D_in],
    columns = the D anchor dims then the m local dims."""
    tid = T_WK if kind == "k" else T_WV
    return xavier_uniform(w.d_drop, w.d_in, w.seed, tid, layer, device=device).to(torch_dtype(w)).contiguous()


def queries(w: Workload, layer: int, device="cpu") -> torch.Tensor:
    """Stored-precision decode queries: [B, H_q, d]."""
    return normal((w.batch, w.n_q_heads, w.head_dim), w.seed, T_Q, layer, device=device).to(torch_dtype(w)).contiguous()


def block_table(w: Workload, n_pages_total: int | None = None) -> torch.Tensor:
    """int32 [B, pages_per_seq]: page ids of each sequence, identity order or a
    seeded random permutation of all pages of the pool."""
    n = w.batch * w.pages_per_seq
    n_pages_total = n if n_pages_total is None else n_pages_total
    if n_pages_total < n:
        raise ValueError("pool too small")
    if w.random_pages:
        perm = torch.randperm(n_pages_total, generator=_gen(w.seed, T_PAGES))[:n]
    else:
        perm = torch.arange(n)
    return perm.to(torch.int32).reshape(w.batch, w.pages_per_seq).contiguous()


def to_numpy_stored(x: torch.Tensor) -> np.ndarray:
    """Stored tensor -> numpy without changing a bit: bf16 becomes its uint16
    bit pattern, fp32 stays float32."""
    x = x.cpu()
    if x.dtype == torch.bfloat16:
        return x.contiguous().view(torch.int16).numpy().view(np.uint16)
    return x.contiguous().numpy()


def paged_pool(w: Workload, seqs: list[torch.Tensor], table: torch.Tensor, n_pages_total: int,
               width: int) -> torch.Tensor:
    """Lay per-sequence caches [L, width] out as a page pool
    [n_pages_total, page_tokens, width] following `table` (host tensor).
    Slots that hold no token are zero."""
    P = w.page_tokens
    pool = torch.zeros((n_pages_total, P, width), dtype=seqs[0].dtype)
    for b, x in enumerate(seqs):
        L = x.shape[0]
        n_full = L // P
        ids = table[b, :n_full].long()
        if n_full:
            pool[ids] = x[:n_full * P].reshape(n_full, P, width)
        if L % P:
            pool[int(table[b, n_full]), :L % P] = x[n_full * P:]
    return pool
