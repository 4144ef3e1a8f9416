"""Seeded Gaussian-mixture key/value/query streams shaped like long-decoding KV caches.

A *unit* is one (sequence, layer, KV head): the granularity at which the paper
partitions a cache into clusters (Section 4.1, Eq. 1-3).  Units are independent, so
every unit owns one ``torch.Generator`` seeded from (config id, unit index); any
subset of units reproduces the same numbers as the full batch.

Recipe (per unit):
  * ``n_mix`` component means ~ N(0, 1) per dimension; keys = mean[c] + sigma_k * N(0, 1)
    with c uniform; in the bf16 configs ``n_outlier`` fixed channels of every key are
    multiplied by ``outlier_scale``; values ~ N(0, 1).
  * decode step t (1-based): the means have moved -- "line": by ``drift_step * t`` along
    one fixed unit direction; "walk": every mean has taken t random-direction steps of
    length ``drift_step`` and ``new_count`` fresh N(0, 1) means join every ``new_every``
    steps.  The step's key is drawn from the moved mixture, its value ~ N(0, 1), and each
    of the G query heads is a uniformly chosen current mean + sigma_q * N(0, 1) (no
    outlier scaling).
  * keys and values are rounded to the storage dtype here, queries to bf16-representable
    fp32 in the bf16 configs, so both consumers see identical numbers.

Nothing in this file computes a distance, a centroid, a score or a softmax.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterable, List, Sequence, Tuple

import torch

_DECODE_BLOCK = 256  # the stream is always generated in blocks of this many steps


@dataclass(frozen=True)
class WorkloadConfig:
    cfg_id: int
    name: str
    B: int
    L: int
    Hq: int
    Hkv: int
    d: int
    kv_dtype: str          # "f32" | "bf16" | "fp8" (bf16 rows handed over, stored as e4m3 bytes with a scale per row)
    n_prefill: int
    steps: int
    M0: int                # clusters per unit at build time
    T: int                 # k-means (Lloyd) iterations
    budget: int            # token budget per decode step
    n_mix: int
    init_mode: str         # "kmeanspp" | "random"
    max_clusters: int
    sigma_k: float = 0.5
    sigma_q: float = 0.3
    n_outlier: int = 0
    outlier_scale: float = 8.0
    drift: str = "line"    # "line" | "walk"
    drift_step: float = 0.01
    new_every: int = 0
    new_count: int = 0
    split_size_factor: float = 2.0   # gamma
    split_var_factor: float = 2.0    # alpha
    split_min_size: int = 8
    split_iters: int = 8
    update_mode: str = "adaptive"    # "adaptive" | "static" | "local" | "delayed" (how the partition follows the decode stream)
    local_max: int = 64              # "local": size above which a cluster born during decoding splits
    buf_max: int = 64                # "delayed": buffered entries per unit that force a split

    @property
    def U(self) -> int:
        return self.B * self.L * self.Hkv

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def max_tokens(self) -> int:
        return self.n_prefill + self.steps

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.kv_dtype == "f32" else torch.bfloat16

    def scaled(self, **kw) -> "WorkloadConfig":
        """A copy with some fields replaced (smaller test-size variants of a config)."""
        from dataclasses import replace
        return replace(self, **kw)


CONFIGS = {
    1: WorkloadConfig(1, "tiny-fp32", B=1, L=1, Hq=4, Hkv=1, d=64, kv_dtype="f32",
                      n_prefill=2048, steps=512, M0=64, T=10, budget=256, n_mix=16,
                      init_mode="kmeanspp", max_clusters=256),
    2: WorkloadConfig(2, "llama3-8b-8k", B=1, L=32, Hq=32, Hkv=8, d=128, kv_dtype="bf16",
                      n_prefill=8192, steps=4096, M0=256, T=10, budget=1024, n_mix=64,
                      init_mode="random", max_clusters=1024, n_outlier=4),
    3: WorkloadConfig(3, "low-prefill-shift", B=1, L=32, Hq=32, Hkv=8, d=128, kv_dtype="bf16",
                      n_prefill=1024, steps=32768, M0=64, T=10, budget=2048, n_mix=64,
                      init_mode="random", max_clusters=4096, n_outlier=4,
                      drift="walk", drift_step=0.02, new_every=4096, new_count=8),
    4: WorkloadConfig(4, "long-prefill-32k", B=1, L=32, Hq=32, Hkv=8, d=128, kv_dtype="bf16",
                      n_prefill=32768, steps=2048, M0=1024, T=20, budget=2048, n_mix=64,
                      init_mode="random", max_clusters=2048, n_outlier=4),
    5: WorkloadConfig(5, "batched-serving", B=16, L=28, Hq=28, Hkv=4, d=128, kv_dtype="bf16",
                      n_prefill=16384, steps=4096, M0=512, T=10, budget=1024, n_mix=64,
                      init_mode="random", max_clusters=1024, n_outlier=4),
}


def unit_seed(cfg_id: int, unit: int) -> int:
    """Seed of one unit's generator: distinct per (config, unit), stable across subsets."""
    return 1000003 * cfg_id + 7919 * unit + 17


def _round_storage(x: torch.Tensor, cfg: WorkloadConfig) -> torch.Tensor:
    return x.to(cfg.torch_dtype)


def _round_query(x: torch.Tensor, cfg: WorkloadConfig) -> torch.Tensor:
    if cfg.kv_dtype != "f32":
        return x.to(torch.bfloat16).to(torch.float32)
    return x


class UnitStream:
    """Prefill block and decode stream of one unit.  Calls must be made in order:
    ``prefill()`` once, then ``decode(n)`` repeatedly; the decode stream is produced in
    fixed blocks of 256 steps internally so the numbers do not depend on how the caller
    slices it."""

    def __init__(self, cfg: WorkloadConfig, unit: int, device: str = "cpu"):
        self.cfg = cfg
        self.unit = unit
        self.device = torch.device(device)
        self.g = torch.Generator(device=self.device)
        self.g.manual_seed(unit_seed(cfg.cfg_id, unit))
        d = cfg.d
        n_new_total = cfg.new_count * (cfg.steps // cfg.new_every) if cfg.new_every else 0
        self.means = torch.zeros(cfg.n_mix + n_new_total, d, device=self.device)
        self.means[: cfg.n_mix] = self._randn(cfg.n_mix, d)
        self.n_active = cfg.n_mix
        direction = self._randn(d)
        self.direction = direction / direction.norm()
        self.scale = torch.ones(d, device=self.device)
        if cfg.n_outlier:
            perm = torch.randperm(d, generator=self.g, device=self.device)
            self.scale[perm[: cfg.n_outlier]] = cfg.outlier_scale
        self.t = 0                      # decode steps produced so far
        self._buf: List[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]] = []
        self._buf_pos = 0
        self._prefilled = False

    def _randn(self, *shape) -> torch.Tensor:
        return torch.randn(*shape, generator=self.g, device=self.device)

    def _randint(self, high: int, shape) -> torch.Tensor:
        return torch.randint(high, shape, generator=self.g, device=self.device)

    def prefill(self) -> Tuple[torch.Tensor, torch.Tensor]:
        assert not self._prefilled
        self._prefilled = True
        cfg = self.cfg
        comp = self._randint(cfg.n_mix, (cfg.n_prefill,))
        K = self.means[comp] + cfg.sigma_k * self._randn(cfg.n_prefill, cfg.d)
        K = K * self.scale
        V = self._randn(cfg.n_prefill, cfg.d)
        return _round_storage(K, cfg), _round_storage(V, cfg)

    def _block(self) -> None:
        """Produce the next block of decode steps into the buffer."""
        cfg = self.cfg
        nb = _DECODE_BLOCK
        if cfg.new_every:
            nb = min(nb, cfg.new_every - (self.t % cfg.new_every))
        na = self.n_active
        steps = torch.arange(self.t + 1, self.t + nb + 1, device=self.device, dtype=torch.float32)
        if cfg.drift == "line":
            # means_t = means_0 + drift_step * t * direction
            shift = (cfg.drift_step * steps)[:, None] * self.direction[None, :]      # [nb, d]
            kc = self._randint(na, (nb,))
            k_mean = self.means[kc] + shift
            qc = self._randint(na, (nb, cfg.G))
            q_mean = self.means[qc] + shift[:, None, :]
        else:
            inc = self._randn(nb, na, cfg.d)
            inc = inc / inc.norm(dim=-1, keepdim=True)
            path = self.means[:na][None] + cfg.drift_step * torch.cumsum(inc, dim=0)  # [nb, na, d]
            kc = self._randint(na, (nb,))
            ar = torch.arange(nb, device=self.device)
            k_mean = path[ar, kc]
            qc = self._randint(na, (nb, cfg.G))
            q_mean = path[ar[:, None], qc]
            self.means[:na] = path[-1]
        k = (k_mean + cfg.sigma_k * self._randn(nb, cfg.d)) * self.scale
        v = self._randn(nb, cfg.d)
        q = q_mean + cfg.sigma_q * self._randn(nb, cfg.G, cfg.d)
        self.t += nb
        if cfg.new_every and self.t % cfg.new_every == 0 and self.n_active + cfg.new_count <= self.means.shape[0]:
            self.means[self.n_active: self.n_active + cfg.new_count] = self._randn(cfg.new_count, cfg.d)
            self.n_active += cfg.new_count
        self._buf.append((_round_query(q, cfg), _round_storage(k, cfg), _round_storage(v, cfg)))

    def decode(self, n: int) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
        """Next ``n`` decode steps: q [n, G, d] fp32, k [n, d], v [n, d] (storage dtype)."""
        qs, ks, vs = [], [], []
        need = n
        while need > 0:
            if not self._buf:
                self._block()
                self._buf_pos = 0
            q, k, v = self._buf[0]
            avail = q.shape[0] - self._buf_pos
            take = min(avail, need)
            sl = slice(self._buf_pos, self._buf_pos + take)
            qs.append(q[sl]); ks.append(k[sl]); vs.append(v[sl])
            self._buf_pos += take
            need -= take
            if self._buf_pos == q.shape[0]:
                self._buf.pop(0)
                self._buf_pos = 0
        return torch.cat(qs), torch.cat(ks), torch.cat(vs)


def make_prefill(streams: Sequence[UnitStream]) -> Tuple[torch.Tensor, torch.Tensor]:
    """Stack the prefill blocks of several units: K, V of shape [U, n_prefill, d]."""
    ks, vs = zip(*(s.prefill() for s in streams))
    return torch.stack(ks).contiguous(), torch.stack(vs).contiguous()


def make_decode_chunk(streams: Sequence[UnitStream], n: int) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """Next ``n`` steps of several units, step-major: q [n, U, G, d], k [n, U, d], v [n, U, d]."""
    qs, ks, vs = zip(*(s.decode(n) for s in streams))
    return (torch.stack(qs, dim=1).contiguous(), torch.stack(ks, dim=1).contiguous(),
            torch.stack(vs, dim=1).contiguous())
