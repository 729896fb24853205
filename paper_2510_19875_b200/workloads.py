"""Seeded synthetic Q/K/V with the shapes and structure of long-context attention layers.

Input synthesis only: nothing of the mask-estimation or attention arithmetic lives here, so the
CPU oracle and the CUDA library can both be fed the same bytes from this module.

Every tensor is drawn as float32 standard normal from ``numpy`` PCG64 streams keyed by
``(seed, tensor, batch, head)``, the structure below is added in float32, and bf16 workloads are
rounded once (nearest-even) at the end. Layout ``[batch, heads, T, d]``, contiguous.

Structure (all optional, combined per workload):
  sink    per kv head a unit vector u; ``K[g, 0] = 4 sqrt(d) u`` and ``Q[h, t] += 2 u`` for every t.
  local   per kv head and 256-token window w a vector s ~ N(0, I); ``Q[h, t] += s[w(t)]``,
          ``K[g, j] += 0.5 s[w(j)]``.
  anchors per kv head 64 distinct positions in [1, T); per q head each token is chosen with
          probability 0.1 and, if an anchor lies before it, is rotated to cosine 0.8 with one such
          anchor's key (norm kept).
  needle  per kv head one key block in [1, N_k / 2) whose keys all point along a unit vector n
          (norms kept); the last 128 queries of the group's heads are rotated to cosine 0.9 with n.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field, replace

import numpy as np

_Q, _K, _V, _AUX = 0, 1, 2, 3


@dataclass(frozen=True)
class WorkloadSpec:
    name: str
    seed: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    T: int
    d: int
    block: int
    k_top: int
    dtype: str  # "f32" | "bf16"
    sink: bool = False
    local: bool = False
    anchors: bool = False
    needle: bool = False

    def scaled(self, **kw) -> "WorkloadSpec":
        """Same recipe at other sizes (used for test-sized and sweep variants)."""
        return replace(self, **kw)

    @property
    def n_blocks(self) -> int:
        return -(-self.T // self.block)

    @property
    def n_rows(self) -> int:
        return self.batch * self.n_q_heads * self.n_blocks


# The five workload shapes; "sweep" is instantiated per T with ``scaled(T=...)``.
SPECS = {
    "single_head_fp32": WorkloadSpec("single_head_fp32", 0, 1, 1, 1, 2048, 64, 32, 8, "f32"),
    "gqa_layer_16k": WorkloadSpec("gqa_layer_16k", 1, 1, 32, 8, 16384, 128, 64, 16, "bf16", sink=True, local=True),
    "cot_layer_128k": WorkloadSpec("cot_layer_128k", 2, 1, 32, 8, 131072, 128, 64, 32, "bf16", sink=True, anchors=True),
    "needle_stack_32k": WorkloadSpec("needle_stack_32k", 100, 28, 28, 4, 32768, 128, 64, 16, "bf16", needle=True),
    "sweep": WorkloadSpec("sweep", 3, 1, 32, 8, 4096, 128, 64, 32, "bf16", sink=True),
}
SWEEP_T = (4096, 16384, 65536, 262144, 1048576)


@dataclass
class Workload:
    spec: WorkloadSpec
    q: np.ndarray  # float32, or uint16 holding bf16 bits
    k: np.ndarray
    v: np.ndarray
    notes: dict = field(default_factory=dict)  # planted positions, for reports

    def torch_tensors(self, device="cpu", pin=False):
        """(q, k, v) as torch tensors of the workload's dtype sharing these bytes (CPU) or copied."""
        import torch

        out = []
        for a in (self.q, self.k, self.v):
            t = torch.from_numpy(a.view(np.int16) if a.dtype == np.uint16 else a)
            if a.dtype == np.uint16:
                t = t.view(torch.bfloat16)
            if pin:
                t = t.pin_memory()
            out.append(t.to(device) if str(device) != "cpu" else t)
        return tuple(out)


def _rng(seed: int, *key: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, *key])))


def _unit(x: np.ndarray) -> np.ndarray:
    return x / np.linalg.norm(x, axis=-1, keepdims=True)


def _rotate_towards(x: np.ndarray, target_unit: np.ndarray, cos: float) -> np.ndarray:
    """Rows of x turned to the given cosine with target_unit, keeping their norms."""
    norm = np.linalg.norm(x, axis=-1, keepdims=True)
    perp = x - (x * target_unit).sum(-1, keepdims=True) * target_unit
    perp = _unit(perp)
    return (norm * (cos * target_unit + np.sqrt(1.0 - cos * cos) * perp)).astype(np.float32)


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 (round to nearest even), returned as uint16 bit patterns."""
    import torch

    return torch.from_numpy(np.ascontiguousarray(x)).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def generate(spec: WorkloadSpec, with_v: bool = True) -> Workload:
    B, H, G, T, d = spec.batch, spec.n_q_heads, spec.n_kv_heads, spec.T, spec.d
    hpg = H // G
    out_dt = np.float32 if spec.dtype == "f32" else np.uint16
    q = np.empty((B, H, T, d), out_dt)
    k = np.empty((B, G, T, d), out_dt)
    v = np.empty((B, G, T, d) if with_v else (0,), out_dt)
    cast = (lambda a: a) if spec.dtype == "f32" else to_bf16_bits
    notes: dict = {}
    n_blocks = spec.n_blocks
    def fill_group(b: int, g: int) -> None:
        seed = spec.seed + b  # stacks: one independent seed per layer
        aux = _rng(seed, _AUX, 0, g)
        kg = _rng(seed, _K, 0, g).standard_normal((T, d), dtype=np.float32)
        sink_u = _unit(aux.standard_normal(d).astype(np.float32)) if spec.sink else None
        win = None
        if spec.local:
            n_win = -(-T // 256)
            win = aux.standard_normal((n_win, d)).astype(np.float32)
            kg += 0.5 * win[np.arange(T) // 256]
        if spec.sink:
            kg[0] = 4.0 * np.sqrt(np.float32(d)) * sink_u
        anchor_pos = None
        if spec.anchors:
            n_anchor = min(64, T - 1)
            anchor_pos = np.sort(aux.choice(np.arange(1, T), size=n_anchor, replace=False))
            notes[("anchors", b, g)] = anchor_pos
        needle_dir = None
        if spec.needle:
            blk = int(aux.integers(1, max(2, n_blocks // 2)))
            needle_dir = _unit(aux.standard_normal(d).astype(np.float32))
            lo, hi = blk * spec.block, min(T, (blk + 1) * spec.block)
            kg[lo:hi] = np.linalg.norm(kg[lo:hi], axis=-1, keepdims=True) * needle_dir
            notes[("needle_block", b, g)] = blk
        k[b, g] = cast(kg)
        if with_v:
            v[b, g] = cast(_rng(seed, _V, 0, g).standard_normal((T, d), dtype=np.float32))
        for h in range(g * hpg, (g + 1) * hpg):
            qh = _rng(seed, _Q, 0, h).standard_normal((T, d), dtype=np.float32)
            if spec.local:
                qh += win[np.arange(T) // 256]
            if spec.sink:
                qh += 2.0 * sink_u
            if spec.anchors:
                hr = _rng(seed, _AUX, 1, h)
                chosen = np.nonzero(hr.random(T) < 0.1)[0]
                before = np.searchsorted(anchor_pos, chosen, side="left")  # anchors strictly before t
                chosen, before = chosen[before > 0], before[before > 0]
                pick = np.minimum((hr.random(chosen.shape[0]) * before).astype(np.int64), before - 1)
                target = _unit(kg[anchor_pos[pick]])
                qh[chosen] = _rotate_towards(qh[chosen], target, 0.8)
            if spec.needle:
                lo = max(0, T - 128)
                qh[lo:] = _rotate_towards(qh[lo:], needle_dir, 0.9)
            q[b, h] = cast(qh)

    # kv groups are independent streams: fill them on a few threads (numpy releases the GIL)
    groups = [(b, g) for b in range(B) for g in range(G)]
    n_workers = max(1, min(len(groups), os.cpu_count() or 1, 16))
    if n_workers == 1:
        for bg in groups:
            fill_group(*bg)
    else:
        with ThreadPoolExecutor(n_workers) as pool:
            list(pool.map(lambda bg: fill_group(*bg), groups))
    return Workload(spec, q, k, v, notes)
