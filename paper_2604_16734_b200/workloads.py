"""Seeded synthetic workloads shaped like the paper's image, tiled-image and video inputs.

This module only *generates inputs* (post-projection q/k/v tensors) and chunk
schedules.  It contains none of the method's arithmetic (no attention, no
scoring, no selection) and is the one module shared by the CUDA path and the
CPU oracle: both sides read the arrays produced here.

The paper evaluates on public image/video suites with trained models
(Sec. 4.1); neither is available offline, so these generators reproduce only the
*shape* of those inputs: vision tokens first (a patch grid per image tile or
video frame, Eq. 3), text tokens last, and block boundaries aligned to
tiles / frames (Sec. 3.1).  Values are smooth spatial fields (Gaussian-blurred
white noise) so that neighbouring patches are redundant, with temporal AR(1)
correlation across video frames.

Everything is drawn from ``torch.Generator`` objects seeded from
``BASE_SEED + 1000 * config_index + layer`` (per-layer draws) and
``BASE_SEED + 1000 * config_index + 999`` (draws shared by all layers), on
whichever device is asked for.  CPU and CUDA generators give different
streams; parity tests always hand the *same* generated arrays to both sides.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Tuple

import torch

BASE_SEED = 260416734


@dataclasses.dataclass(frozen=True)
class WorkloadConfig:
    """One synthetic workload: model attention shape, prefix structure, chunking and budget."""

    name: str
    index: int                  # position in the benchmark's config list (seeds depend on it)
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str                  # "fp32" | "bf16"
    grid: Tuple[int, int]       # patch grid (h, w) of one tile / frame (Eq. 3)
    n_units: int                # tiles or frames
    n_text: int
    chunk: int                  # block size b (Alg. 1)
    budget: int                 # memory budget M = B entries per (layer, kv-head) (Alg. 1)
    kind: str                   # "image" | "tiles" | "video"
    rho: float = 0.0            # AR(1) coefficient across frames (video)
    scene_cut: int = 0          # fresh field every scene_cut frames (0 = never)
    shared_rank: int = 0        # rank of the component shared by all tiles ("tiles")
    noise_std: float = 0.3
    blur_sigma: float = 2.0
    mix_layers: bool = True     # per-layer random orthogonal mixing of the channels
    obs_window: int = 32

    @property
    def n_vision(self) -> int:
        return self.grid[0] * self.grid[1] * self.n_units

    @property
    def n_tokens(self) -> int:
        return self.n_vision + self.n_text

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def torch_dtype(self) -> torch.dtype:
        return torch.float32 if self.dtype == "fp32" else torch.bfloat16

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "fp32" else 2

    def chunks(self) -> List[Tuple[int, int]]:
        """(pos0, n) for every block: vision tokens in blocks of ``chunk`` (short last
        block if it does not divide), then the text prompt as block(s) of its own."""
        out = []
        p = 0
        for total in (self.n_vision, self.n_text):
            r = total
            while r > 0:
                n = min(self.chunk, r)
                out.append((p, n))
                p += n
                r -= n
        return out

    def chunks_hybrid(self) -> List[Tuple[int, int]]:
        """Hybrid schedule (the paper's default, Sec. 5 "Budgeting"): the first min(B, n_vision) tokens in one pass,
        the rest of the vision tokens in blocks of ``chunk``, then the text prompt."""
        first = min(self.budget, self.n_vision)
        out = [(0, first)]
        p = first
        for end in (self.n_vision, self.n_tokens):
            while p < end:
                n = min(self.chunk, end - p)
                out.append((p, n))
                p += n
        return out

    def scaled(self, **kw) -> "WorkloadConfig":
        return dataclasses.replace(self, **kw)


CONFIGS = {
    "C1": WorkloadConfig("C1", 0, 1, 4, 1, 64, "fp32", (24, 24), 1, 32, 64, 128, "image",
                         mix_layers=False),
    "C2": WorkloadConfig("C2", 1, 32, 32, 32, 128, "bf16", (24, 24), 1, 64, 128, 192, "image"),
    "C3": WorkloadConfig("C3", 2, 28, 28, 4, 128, "bf16", (24, 24), 5, 128, 576, 1024, "tiles",
                         shared_rank=8),
    "C4": WorkloadConfig("C4", 3, 32, 32, 8, 128, "bf16", (14, 14), 64, 128, 196, 2048, "video",
                         rho=0.9),
    "C5": WorkloadConfig("C5", 4, 32, 32, 8, 128, "bf16", (12, 12), 256, 256, 1024, 4096, "video",
                         rho=0.95, scene_cut=32),
    # The axis of the paper's block-size study (Sec. 5 "Block size and structural alignment", Table 4: blocks of 256 / 512 / 784 / 1024 at a budget of
    # 2048 on roughly 8k vision tokens in 28x28 tiles), with the attention shape of a 7B model with grouped heads:
    # 28 layers, 28 query / 4 kv heads, d = 128; 10 tiles of 784 tokens + 128 text tokens.  The block size and the
    # budget are meant to be overridden (``scaled(chunk=..., budget=...)``, ``bench.py --block / --budget``).
    "T4": WorkloadConfig("T4", 5, 28, 28, 4, 128, "bf16", (28, 28), 10, 128, 784, 2048, "tiles",
                         shared_rank=8),
}


def _blur_matrix(n: int, sigma: float, device, dtype=torch.float64) -> torch.Tensor:
    """n x n matrix applying a 1-D Gaussian blur with reflect ('dcba|abcd|dcba') padding."""
    radius = int(math.ceil(4.0 * sigma))
    offs = torch.arange(-radius, radius + 1, dtype=dtype)
    wts = torch.exp(-0.5 * (offs / sigma) ** 2)
    wts = wts / wts.sum()
    m = torch.zeros(n, n, dtype=dtype)
    period = 2 * n
    for i in range(n):
        for o, wt in zip(range(-radius, radius + 1), wts.tolist()):
            j = (i + o) % period
            if j >= n:
                j = period - 1 - j
            m[i, j] += wt
    return m.to(device)


class Workload:
    """Generator of per-layer (q, k, v) for one config.

    ``layer(l)`` returns q ``[N][Hq][d]``, k ``[N][Hkv][d]``, v ``[N][Hkv][d]`` in the
    config's dtype (values already rounded to it, so both consumers see identical inputs).
    """

    def __init__(self, cfg: WorkloadConfig, device="cpu", seed: Optional[int] = None):
        self.cfg = cfg
        self.device = torch.device(device)
        self.seed = BASE_SEED if seed is None else seed
        self._base = None

    # -- random helpers -------------------------------------------------------------
    def _gen(self, stream: int) -> torch.Generator:
        g = torch.Generator(device=self.device)
        g.manual_seed(self.seed + 1000 * self.cfg.index + stream)
        return g

    def _randn(self, gen, *shape) -> torch.Tensor:
        return torch.randn(*shape, generator=gen, device=self.device, dtype=torch.float32)

    def _blur_field(self, gen, units: int, channels: int) -> torch.Tensor:
        """[units][h*w][channels]: white noise blurred on the patch grid, unit std per channel."""
        h, w = self.cfg.grid
        x = self._randn(gen, units, h, w, channels)
        bh = _blur_matrix(h, self.cfg.blur_sigma, self.device).float()
        bw = _blur_matrix(w, self.cfg.blur_sigma, self.device).float()
        x = torch.einsum("ij,ujkc->uikc", bh, x)
        x = torch.einsum("kl,uilc->uikc", bw, x)
        x = x.reshape(units, h * w, channels)
        x = x / x.std(dim=1, keepdim=True).clamp_min(1e-6)
        return x

    # -- structure shared by all layers ----------------------------------------------
    def _base_fields(self):
        """Noise-free vision fields for Q, K, V ([N_vis][D] each), shared by all layers."""
        if self._base is not None:
            return self._base
        cfg = self.cfg
        gen = self._gen(999)
        out = []
        for width in (cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim,
                      cfg.n_kv_heads * cfg.head_dim):
            if cfg.kind == "image":
                f = self._blur_field(gen, cfg.n_units, width)
            elif cfg.kind == "tiles":
                r = cfg.shared_rank
                u = self._blur_field(gen, 1, r)                       # [1][hw][r], same for all tiles
                a = self._randn(gen, r, width) / math.sqrt(r)
                own = self._blur_field(gen, cfg.n_units, width)
                f = math.sqrt(0.5) * (u @ a) + math.sqrt(0.5) * own
            elif cfg.kind == "video":
                fresh = self._blur_field(gen, cfg.n_units, width)
                f = torch.empty_like(fresh)
                rho = cfg.rho
                for t in range(cfg.n_units):
                    if t == 0 or (cfg.scene_cut and t % cfg.scene_cut == 0):
                        f[t] = fresh[t]
                    else:
                        f[t] = rho * f[t - 1] + math.sqrt(1.0 - rho * rho) * fresh[t]
            else:
                raise ValueError(cfg.kind)
            out.append(f.reshape(cfg.n_vision, width))
        self._base = tuple(out)
        return self._base

    def _orthogonal(self, gen, width: int) -> torch.Tensor:
        a = self._randn(gen, width, width)
        qm, rm = torch.linalg.qr(a)
        return qm * torch.sign(torch.diagonal(rm)).unsqueeze(0)

    # -- per-layer tensors -----------------------------------------------------------
    def layer(self, layer: int):
        cfg = self.cfg
        gen = self._gen(layer)
        res = []
        for base, heads in zip(self._base_fields(), (cfg.n_q_heads, cfg.n_kv_heads, cfg.n_kv_heads)):
            width = heads * cfg.head_dim
            x = base
            if cfg.mix_layers:
                x = x @ self._orthogonal(gen, width)
            x = x + cfg.noise_std * self._randn(gen, cfg.n_vision, width)
            text = self._randn(gen, cfg.n_text, width)
            full = torch.cat([x, text], dim=0).reshape(cfg.n_tokens, heads, cfg.head_dim)
            res.append(full.to(cfg.torch_dtype).contiguous())
        return tuple(res)


def reduced(cfg: WorkloadConfig, n_layers: int = 1, n_units: Optional[int] = None,
            n_text: Optional[int] = None) -> WorkloadConfig:
    """Same shapes per token, fewer layers / tiles / frames: for tests the oracle finishes quickly."""
    return cfg.scaled(n_layers=n_layers,
                      n_units=cfg.n_units if n_units is None else n_units,
                      n_text=cfg.n_text if n_text is None else n_text)
