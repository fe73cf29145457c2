"""Seeded synthetic workloads shaped like the paper's generations.

This module only *makes inputs*: token counts, (t, h, w) coordinates, Gaussian
Q/K/V with channel outliers, frame tables and budget parameters.  It holds none
of the method's arithmetic (no RoPE, no scoring, no budget apportionment, no
attention), so both the CPU oracle's tests and the CUDA path's tests may import
it without sharing any computation.

Shapes follow the paper's setup (Sec. 4.1: a text prompt of a few hundred
tokens, one conditioning image, then latent frames of equal token count) at the
granularity the benchmark configurations fix: frames of 24x42 = 1008 tokens,
128 text tokens, 24 query heads / 8 KV heads of dimension 128.

Coordinates follow MM-RoPE's scaling of latent coordinates by (4, 8, 8)
(Sec. 3.1): text token i sits at (i, i, i); a visual token of frame f, row r,
column c sits at (n_text + 4 f, 8 r, 8 c), the conditioning image being f = 0,
history frames f = 1..F and the frame being generated f = F + 1.  The fourth
position column is an opaque tag (a global token id) that compaction must carry
through unchanged.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Tuple

import numpy as np

# decay kinds (values mirror the C-ABI enum and the oracle's enum; they are
# interface constants, not arithmetic)
GEOMETRIC = 0
CLOSED_HALF = 1
LINEAR = 2
HALFLIFE = 3

F32 = "f32"
BF16 = "bf16"


@dataclass(frozen=True)
class Budget:
    kind: int
    param: float
    total: int
    keep_full: int = 0


@dataclass(frozen=True)
class Config:
    name: str
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str
    n_text: int
    grid: Tuple[int, int]          # (rows, cols) of one latent frame
    n_frames: int                  # history frames F
    budget: Budget
    outliers: bool = False         # K/V channel outliers (scale 4 on 2% of channels)
    rope_base: float = 10000.0
    n_layers: int = 1
    seed: int = 0

    @property
    def frame_tokens(self) -> int:
        return self.grid[0] * self.grid[1]

    @property
    def n_anchor(self) -> int:
        return self.n_text + self.frame_tokens

    @property
    def n_q(self) -> int:
        return self.frame_tokens

    @property
    def n_src(self) -> int:
        return self.n_frames * self.frame_tokens

    @property
    def max_pos(self) -> Tuple[int, int, int]:
        """Exclusive upper bounds of the three coordinates this workload uses."""
        t = self.n_text + 4 * (self.n_frames + 1) + 1
        h = max(self.n_text, 8 * (self.grid[0] - 1) + 1)
        w = max(self.n_text, 8 * (self.grid[1] - 1) + 1)
        return (max(t, self.n_text), h, w)


def _lumos(name: str, n_frames: int, budget: Budget, **kw) -> Config:
    return Config(name=name, n_q_heads=24, n_kv_heads=8, head_dim=128, dtype=BF16,
                  n_text=128, grid=(24, 42), n_frames=n_frames, budget=budget,
                  outliers=True, **kw)


CONFIGS: Dict[str, Config] = {
    # configs[0]: tiny fp32 correctness case; closed-form half-life-1 allocation (Eq. 7)
    "tiny": Config(name="tiny", n_q_heads=4, n_kv_heads=2, head_dim=64, dtype=F32,
                   n_text=32, grid=(8, 8), n_frames=6,
                   budget=Budget(CLOSED_HALF, 0.5, 128)),
    # configs[1]: 12 history frames, 25% of history, linear decay
    "lumos12": _lumos("lumos12", 12, Budget(LINEAR, 0.0, (12 * 1008) // 4)),
    # configs[2]: 24 history frames, 6048 retained, half-life 4
    "lumos24": _lumos("lumos24", 24, Budget(HALFLIFE, 4.0, 6048)),
    # configs[3]: 47 history frames, newest 2 kept whole, 6048 over the rest at half-life 4
    "lumos47": _lumos("lumos47", 47, Budget(HALFLIFE, 4.0, 2 * 1008 + 6048, keep_full=2)),
    # configs[4]: 28 stacked layers of the lumos shape, sweep driven by the caller
    "stack28": _lumos("stack28", 47, Budget(HALFLIFE, 4.0, (47 * 1008) // 4), n_layers=28),
}


def small_bf16(n_frames: int = 5, grid: Tuple[int, int] = (9, 15), n_text: int = 37,
               total: int = 300, kind: int = HALFLIFE, param: float = 2.0,
               keep_full: int = 1, seed: int = 3) -> Config:
    """A lumos-shaped case small enough for the oracle, with ragged tile tails."""
    return Config(name=f"small_bf16_{n_frames}x{grid[0]}x{grid[1]}", n_q_heads=24, n_kv_heads=8,
                  head_dim=128, dtype=BF16, n_text=n_text, grid=grid, n_frames=n_frames,
                  budget=Budget(kind, param, total, keep_full), outliers=True, seed=seed)


# ---------------------------------------------------------------------------
# storage rounding (data formatting only)
# ---------------------------------------------------------------------------
def round_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even), returned as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Upper 16 bits of float32 values that are already exactly representable in bfloat16."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return (u >> 16).astype(np.uint16).reshape(x.shape)


def bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Inverse of :func:`bf16_bits`."""
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


def to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float32)
    return round_bf16(x) if dtype == BF16 else x


# ---------------------------------------------------------------------------
# positions
# ---------------------------------------------------------------------------
def text_positions(n_text: int, tag0: int = 0) -> np.ndarray:
    i = np.arange(n_text, dtype=np.int32)
    return np.stack([i, i, i, i + tag0], axis=1).astype(np.int32)


def frame_positions(cfg: Config, f: int, tag0: int) -> np.ndarray:
    """Positions of the visual tokens of frame index f (0 = conditioning image)."""
    rows, cols = cfg.grid
    r, c = np.meshgrid(np.arange(rows, dtype=np.int32), np.arange(cols, dtype=np.int32), indexing="ij")
    n = rows * cols
    out = np.empty((n, 4), dtype=np.int32)
    out[:, 0] = cfg.n_text + 4 * f
    out[:, 1] = 8 * r.reshape(-1)
    out[:, 2] = 8 * c.reshape(-1)
    out[:, 3] = tag0 + np.arange(n, dtype=np.int32)
    return out


@dataclass
class Layer:
    """One layer's tensors, float32 arrays already rounded to the storage dtype."""
    cfg: Config
    q: np.ndarray            # [n_q][Hq][d]
    q_pos: np.ndarray        # [n_q][4] int32
    anchor_k: np.ndarray     # [A][Hkv][d]
    anchor_v: np.ndarray
    anchor_pos: np.ndarray   # [A][4]
    hist_k: np.ndarray       # [F*N][Hkv][d], frames oldest -> newest
    hist_v: np.ndarray
    hist_pos: np.ndarray     # [F*N][4]
    frame_count: np.ndarray  # [F] int32
    cur_k: np.ndarray = field(default=None)   # [n_q][Hkv][d] K/V of the frame being generated
    cur_v: np.ndarray = field(default=None)


def positions(cfg: Config):
    n = cfg.frame_tokens
    a_pos = np.concatenate([text_positions(cfg.n_text), frame_positions(cfg, 0, cfg.n_text)], axis=0)
    h_pos = np.concatenate([frame_positions(cfg, f, cfg.n_anchor + (f - 1) * n)
                            for f in range(1, cfg.n_frames + 1)], axis=0) if cfg.n_frames else \
        np.zeros((0, 4), np.int32)
    q_pos = frame_positions(cfg, cfg.n_frames + 1, cfg.n_anchor + cfg.n_frames * n)
    return a_pos, h_pos, q_pos


def _outlier_bias(rng: np.random.Generator, cfg: Config) -> np.ndarray:
    """A [Hkv][d] bias: +-4 on a fixed random 2% of the (kv head, channel) slots, else 0."""
    slots = cfg.n_kv_heads * cfg.head_dim
    k = max(1, int(round(0.02 * slots)))
    pick = rng.choice(slots, size=k, replace=False)
    bias = np.zeros(slots, dtype=np.float32)
    bias[pick] = 4.0 * rng.choice(np.array([-1.0, 1.0], dtype=np.float32), size=k)
    return bias.reshape(cfg.n_kv_heads, cfg.head_dim)


def _gauss(rng: np.random.Generator, shape, bias=None) -> np.ndarray:
    x = rng.standard_normal(size=shape, dtype=np.float32)
    if bias is not None:
        x += bias
    return x


def make_layer(cfg: Config, layer: int = 0, with_current: bool = False) -> Layer:
    """Draw one layer's Q / K / V.  Streams are keyed by (seed, layer) so layers differ."""
    rng = np.random.Generator(np.random.Philox(key=[cfg.seed, layer]))
    hq, hkv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    a_pos, h_pos, q_pos = positions(cfg)
    kb = _outlier_bias(rng, cfg) if cfg.outliers else None
    vb = _outlier_bias(rng, cfg) if cfg.outliers else None
    st = lambda x: to_storage(x, cfg.dtype)
    q = st(_gauss(rng, (cfg.n_q, hq, d)))
    ak = st(_gauss(rng, (cfg.n_anchor, hkv, d), kb))
    av = st(_gauss(rng, (cfg.n_anchor, hkv, d), vb))
    hk = st(_gauss(rng, (cfg.n_src, hkv, d), kb))
    hv = st(_gauss(rng, (cfg.n_src, hkv, d), vb))
    lay = Layer(cfg=cfg, q=q, q_pos=q_pos, anchor_k=ak, anchor_v=av, anchor_pos=a_pos,
                hist_k=hk, hist_v=hv, hist_pos=h_pos,
                frame_count=np.full(cfg.n_frames, cfg.frame_tokens, dtype=np.int32))
    if with_current:
        lay.cur_k = st(_gauss(rng, (cfg.n_q, hkv, d), kb))
        lay.cur_v = st(_gauss(rng, (cfg.n_q, hkv, d), vb))
    return lay


def with_budget(cfg: Config, **kw) -> Config:
    return replace(cfg, budget=replace(cfg.budget, **kw))


def tie_scores(rng: np.random.Generator, n: int, levels: int = 7) -> np.ndarray:
    """Scores drawn from a few discrete levels (with +0/-0 mixed in) to force ties."""
    s = rng.integers(-(levels // 2), levels // 2 + 1, size=n).astype(np.float32) * np.float32(0.25)
    neg0 = rng.random(n) < 0.5
    s[(s == 0) & neg0] = np.float32(-0.0)
    return s
