"""Seeded synthetic inputs for the loop-r prefill step.

This module only makes inputs.  It holds none of the method's arithmetic (no token scoring,
no column selection, no quantizer, no attention): the test oracle and the CUDA library both
consume what it produces and neither depends on the other.

The inputs stand in for the paper's workloads (pretrained looped Transformers of width 2048
with 16 heads of 128, 4 loops, Section 5.1 and Appendix E), which are not available here.
They reproduce the structure the paper reports in Section 3: hidden-state change that
concentrates on a shrinking, nested set of token rows (Section 3.1), attention mass that
concentrates on a few persistent key columns (Section 3.2), and cross-loop K/V residuals that
are small next to the full states (Section 3.3).

Recipe (one layer):
  G^(1) ~ N(0, 1)                                             [L, d]
  G^(r) = G^(r-1) + Delta^(r);  rows of the nested changed set C_r get N(0, delta_hi),
          the rest N(0, delta_lo)   (second argument = standard deviation)
  W_q, W_k, W_v ~ N(0, w_std)                                  [d, d]
  Q^(r), K^(r), V^(r) = G^(r) W   (optionally after RMS normalisation of the rows)
  "heavy" key positions: a fixed random subset of heavy_frac*L positions whose key rows are
          multiplied by heavy_scale in every loop and every head
  storage rounding: bf16 configurations round G, Q, K, V to bf16 (round to nearest even);
          arrays are returned as float32 holding exactly representable values.
Random numbers come from numpy's counter-based Philox generator keyed by
(seed, layer, stream id), so the values do not depend on the machine.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Optional

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    L: int
    n_heads: int
    head_dim: int
    n_loops: int
    dtype: str                      # "f32" | "bf16": storage type of hidden states, Q, K, V
    changed_fracs: tuple            # fraction of rows changed entering loop r, r = 2..R
    delta_hi: float
    delta_lo: float
    w_std: float
    heavy_frac: float
    heavy_scale: float
    token_frac: float               # token budget as a fraction of L (same for every sparse loop)
    col_budget: int
    q_block: int
    bits: int
    group: int
    n_layers: int = 1
    rmsnorm: bool = False
    eps: float = 1e-6

    @property
    def d(self) -> int:
        return self.n_heads * self.head_dim

    @property
    def k_tokens(self) -> int:
        return int(np.floor(self.token_frac * self.L + 0.5))

    @property
    def sm_scale(self) -> float:
        return 1.0 / float(np.sqrt(self.head_dim))

    def n_changed(self, r: int) -> int:
        return int(np.floor(self.changed_fracs[r - 2] * self.L + 0.5))


def config1() -> Workload:
    """Tiny single-layer check (fp32, L=512, 4 heads of 64, R=2)."""
    return Workload("c1_tiny", L=512, n_heads=4, head_dim=64, n_loops=2, dtype="f32",
                    changed_fracs=(0.25,), delta_hi=0.5, delta_lo=1e-3, w_std=256 ** -0.5,
                    heavy_frac=0.0, heavy_scale=1.0, token_frac=0.25, col_budget=64, q_block=64,
                    bits=4, group=64)


def config2(L: int = 8192, n_heads: int = 16) -> Workload:
    """One layer of the 2.6B-shaped block (bf16, 16 heads of 128, R=4)."""
    return Workload("c2_layer", L=L, n_heads=n_heads, head_dim=128, n_loops=4, dtype="bf16",
                    changed_fracs=(0.30, 0.15, 0.08), delta_hi=0.3, delta_lo=1e-3,
                    w_std=(n_heads * 128) ** -0.5, heavy_frac=0.02, heavy_scale=8.0,
                    token_frac=0.15, col_budget=512, q_block=1024, bits=4, group=128)


def config3(L: int = 32768, n_layers: int = 48) -> Workload:
    """48-layer stack of the same block, L=32768, token budget 10%, column budget 1024."""
    return Workload("c3_stack", L=L, n_heads=16, head_dim=128, n_loops=4, dtype="bf16",
                    changed_fracs=(0.30, 0.15, 0.08), delta_hi=0.3, delta_lo=1e-3, w_std=0.02,
                    heavy_frac=0.02, heavy_scale=8.0, token_frac=0.10, col_budget=1024,
                    q_block=1024, bits=4, group=128, n_layers=n_layers, rmsnorm=True)


def config5(L: int = 131072, n_layers: int = 48) -> Workload:
    """Long-context memory configuration (prefill part)."""
    return replace(config3(L, n_layers), name="c5_long", col_budget=2048)


def sweep_point(n_loops: int, token_frac: float, col_budget: int, bits: int, L: int = 8192) -> Workload:
    """One point of the sparsity/depth sweep: changed fraction 0.40 * 0.5^(r-2)."""
    fr = tuple(0.40 * 0.5 ** (r - 2) for r in range(2, n_loops + 1))
    return replace(config2(L), name=f"c4_R{n_loops}_t{token_frac}_c{col_budget}_b{bits}", n_loops=n_loops,
                   changed_fracs=fr, token_frac=token_frac, col_budget=col_budget, bits=bits)


# ----------------------------------------------------------------------------------------------
def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounded = ((u + 0x7FFF + ((u >> 16) & 1)) >> 16) << 16
    return rounded.astype(np.uint32).view(np.float32).reshape(x.shape)


def _rng(seed: int, layer: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 20) ^ (layer << 8) ^ stream, 0x5EED]))


@dataclass
class LayerInputs:
    workload: Workload
    G: List[np.ndarray]             # R arrays [L, d]
    Q: List[np.ndarray]             # R arrays [L, H, dh]
    K: List[np.ndarray]
    V: List[np.ndarray]
    changed_rows: List[np.ndarray]  # planted changed-row sets for loops 2..R (nested, ascending)
    heavy_cols: np.ndarray


def make_layer_inputs(w: Workload, seed: int = 0, layer: int = 0) -> LayerInputs:
    """Host (numpy) generator: all loops of one layer."""
    L, d, H, dh = w.L, w.d, w.n_heads, w.head_dim
    store = (lambda a: a.astype(np.float32)) if w.dtype == "f32" else round_to_bf16

    g = _rng(seed, layer, 1).standard_normal((L, d), dtype=np.float32)
    Wq = (_rng(seed, layer, 2).standard_normal((d, d), dtype=np.float32) * np.float32(w.w_std))
    Wk = (_rng(seed, layer, 3).standard_normal((d, d), dtype=np.float32) * np.float32(w.w_std))
    Wv = (_rng(seed, layer, 4).standard_normal((d, d), dtype=np.float32) * np.float32(w.w_std))

    # nested changed-row sets: one random permutation, prefixes of decreasing length
    perm = _rng(seed, 0, 5).permutation(L)
    changed = [np.sort(perm[: w.n_changed(r)]) for r in range(2, w.n_loops + 1)]
    n_heavy = int(np.floor(w.heavy_frac * L + 0.5))
    heavy = np.sort(_rng(seed, 0, 6).permutation(L)[:n_heavy])

    G, Q, K, V = [], [], [], []
    for r in range(1, w.n_loops + 1):
        if r > 1:
            rr = _rng(seed, layer, 16 + r)
            delta = rr.standard_normal((L, d), dtype=np.float32) * np.float32(w.delta_lo)
            rows = changed[r - 2]
            delta[rows] = rr.standard_normal((len(rows), d), dtype=np.float32) * np.float32(w.delta_hi)
            g = g + delta
        g = store(g)
        x = g
        if w.rmsnorm:
            x = g / np.sqrt(np.mean(g.astype(np.float64) ** 2, axis=1, keepdims=True) + 1e-6).astype(np.float32)
        q = store(x @ Wq).reshape(L, H, dh)
        k = (x @ Wk).reshape(L, H, dh)
        if n_heavy:
            k[heavy] *= np.float32(w.heavy_scale)
        k = store(k)
        v = store(x @ Wv).reshape(L, H, dh)
        G.append(g); Q.append(q); K.append(k); V.append(v)
    return LayerInputs(w, G, Q, K, V, changed, heavy)


# ----------------------------------------------------------------------------------------------
# Device-side generator for the stack configurations (too large for host numpy in reasonable time).
# Same recipe as make_layer_inputs, drawn with torch's seeded CUDA generator.
# ----------------------------------------------------------------------------------------------
class DeviceStack:
    """Synthetic 48-layer stack inputs on the GPU.

    stack_hidden()        -> [G^(1) .. G^(R)], each [L, d] in storage type: the stack-level hidden state
                             that token selection scores (one selection per loop, shared by all layers).
    layer(l)              -> LayerGen with .qkv1() (all rows, loop 1), .hidden(r) ([L, d]) and
                             .rows(r, active_idx) (Q, K, V of the active rows of loop r).
    Each layer's input replaces the recurrence by the same lazy-update generator
    (Y^(r) = Y^(r-1) + Delta^(r) on the shared nested changed-row sets); Q/K/V are projections of the
    RMS-normalised rows with per-layer weights N(0, w_std).
    """

    def __init__(self, w: Workload, seed: int = 0, device="cuda:0"):
        import torch
        self.w, self.seed, self.device, self.torch = w, seed, device, torch
        self.dt = torch.float32 if w.dtype == "f32" else torch.bfloat16
        perm = _rng(seed, 0, 5).permutation(w.L)
        self.changed = [torch.from_numpy(np.sort(perm[: w.n_changed(r)])).to(device)
                        for r in range(2, w.n_loops + 1)]
        n_heavy = int(np.floor(w.heavy_frac * w.L + 0.5))
        self.heavy = torch.from_numpy(np.sort(_rng(seed, 0, 6).permutation(w.L)[:n_heavy])).to(device)

    def _gen(self, layer: int, stream: int):
        g = self.torch.Generator(device=self.device)
        g.manual_seed((self.seed << 20) ^ (layer << 8) ^ stream)
        return g

    def _delta(self, layer: int, r: int):
        torch, w = self.torch, self.w
        g = self._gen(layer, 16 + r)
        delta = torch.randn(w.L, w.d, generator=g, device=self.device) * w.delta_lo
        rows = self.changed[r - 2]
        delta[rows] = torch.randn(len(rows), w.d, generator=g, device=self.device) * w.delta_hi
        return delta

    def _chain(self, layer: int):
        """Yields the storage-rounded hidden state of loops 1..R as float32 tensors."""
        torch, w = self.torch, self.w
        y = torch.randn(w.L, w.d, generator=self._gen(layer, 1), device=self.device).to(self.dt).float()
        yield y
        for r in range(2, w.n_loops + 1):
            y = (y + self._delta(layer, r)).to(self.dt).float()
            yield y

    def stack_hidden(self):
        return [y.to(self.dt) for y in self._chain(10_000)]

    def layer(self, layer: int):
        return LayerGen(self, layer)


class LayerGen:
    def __init__(self, stack: DeviceStack, layer: int):
        torch, w = stack.torch, stack.w
        self.s, self.layer_id = stack, layer
        mk = lambda sid: (torch.randn(w.d, w.d, generator=stack._gen(layer, sid), device=stack.device)
                          * w.w_std).to(stack.dt)
        self.Wq, self.Wk, self.Wv = mk(2), mk(3), mk(4)
        self._hidden = list(stack._chain(layer))            # R float32 tensors [L, d]

    def hidden(self, r: int):
        return self._hidden[r - 1].to(self.s.dt)

    def _project(self, x, pos):
        torch, w, s = self.s.torch, self.s.w, self.s
        if w.rmsnorm:
            x = x * torch.rsqrt(x.pow(2).mean(dim=1, keepdim=True) + 1e-6)
        x = x.to(s.dt)
        q = (x @ self.Wq).view(-1, w.n_heads, w.head_dim)
        k = (x @ self.Wk).float()
        if len(s.heavy):
            is_heavy = torch.isin(pos, s.heavy)
            k = torch.where(is_heavy[:, None], k * w.heavy_scale, k)
        k = k.to(s.dt).view(-1, w.n_heads, w.head_dim)
        v = (x @ self.Wv).view(-1, w.n_heads, w.head_dim)
        return q.contiguous(), k.contiguous(), v.contiguous()

    def qkv1(self):
        torch, w = self.s.torch, self.s.w
        return self._project(self._hidden[0], torch.arange(w.L, device=self.s.device))

    def rows(self, r: int, active_idx):
        pos = active_idx.long()
        return self._project(self._hidden[r - 1][pos], pos)

    def release(self):
        self._hidden = None
