"""Seeded synthetic inputs shared by the tests, the benchmark and the CPU oracle.

This module holds shapes, random draws and bf16 rounding only -- none of the
method's arithmetic (no trace, no layout, no block math).  Both the CUDA path
and the oracle receive exactly these arrays, so neither has to trust the other
for its inputs.

Value recipe: matrices and biases ~ N(0, 0.02^2); the two RMSNorm gain vectors
are 1 + N(0, 0.02^2); activations and the timestep embedding ~ N(0, 1).
Everything is drawn in float32 with numpy's PCG64 generator, rounded to bf16
(round-to-nearest-even) and handed out both as the uint16 bit patterns (for
device upload) and as bf16-exact float64 (for the oracle).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
import numpy as np

__all__ = [
    "Template", "TEMPLATES", "template", "bf16_bits", "bits_to_f64",
    "WEIGHT_ORDER", "weight_shapes", "make_block_weights", "make_activations",
    "ACTIVATION_SEED", "sample_rows",
]

ACTIVATION_SEED = 1_000_000


@dataclass(frozen=True)
class Template:
    """Shape description of one request template (a DiT block or a stack of blocks)."""
    name: str
    batch: int
    s_text: int
    grid_t: int
    grid_h: int
    grid_w: int
    hidden: int
    heads: int
    head_dim: int
    ffn: int
    temb_dim: int = 512
    rope_dim_t: int = 0
    rope_dim_h: int = 0
    rope_dim_w: int = 0
    rope_base: float = 10000.0
    ln_eps: float = 1e-6
    rms_eps: float = 1e-6
    n_blocks: int = 1

    def __post_init__(self):
        if self.rope_dim_t == 0 and self.rope_dim_h == 0 and self.rope_dim_w == 0:
            dh = self.head_dim
            object.__setattr__(self, "rope_dim_t", dh // 4)
            object.__setattr__(self, "rope_dim_h", 3 * dh // 8)
            object.__setattr__(self, "rope_dim_w", 3 * dh // 8)

    @property
    def seq(self) -> int:
        return self.s_text + self.grid_t * self.grid_h * self.grid_w

    def with_(self, **kw) -> "Template":
        return replace(self, **kw)


TEMPLATES = {
    # hidden 512, 8 heads x 64, 32 text + 4x8x8 video tokens
    "tiny": Template("tiny", 1, 32, 4, 8, 8, 512, 8, 64, 2048),
    # CogVideoX-5B-shaped block: 226 text + 13x30x45 video tokens
    "cogvideox": Template("cogvideox", 1, 226, 13, 30, 45, 3072, 48, 64, 12288),
    # Flux-style 1024x1024 image block: 512 text + 64x64 image tokens, head_dim 128
    "flux": Template("flux", 1, 512, 1, 64, 64, 3072, 24, 128, 12288),
    # 1080p x 49 frame shaped block: 226 text + 13x68x120 video tokens
    "longvideo": Template("longvideo", 1, 226, 13, 68, 120, 3072, 48, 64, 12288),
    # full denoising step: 42 stacked CogVideoX-shaped blocks
    "step": Template("step", 1, 226, 13, 30, 45, 3072, 48, 64, 12288, n_blocks=42),
}


def template(name: str, **overrides) -> Template:
    t = TEMPLATES[name]
    return t.with_(**overrides) if overrides else t


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 array -> uint16 bf16 bit patterns, round-to-nearest-even."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float64 (exact)."""
    u = bits.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


# Fixed draw order of one block's parameters.
WEIGHT_ORDER = ("w_mod", "b_mod", "w_qkv", "b_qkv", "g_q", "g_k",
                "w_o", "b_o", "w_1", "b_1", "w_2", "b_2")


def weight_shapes(t: Template) -> dict:
    D, F, Dt, dh = t.hidden, t.ffn, t.temb_dim, t.head_dim
    return {
        "w_mod": (6 * D, Dt), "b_mod": (6 * D,),
        "w_qkv": (3 * D, D), "b_qkv": (3 * D,),
        "g_q": (dh,), "g_k": (dh,),
        "w_o": (D, D), "b_o": (D,),
        "w_1": (F, D), "b_1": (F,),
        "w_2": (D, F), "b_2": (D,),
    }


def make_block_weights(t: Template, seed: int) -> dict:
    """bf16 bit patterns of one block's parameters, drawn in WEIGHT_ORDER from `seed`."""
    rng = np.random.Generator(np.random.PCG64(seed))
    out = {}
    for name, shape in weight_shapes(t).items():
        z = rng.standard_normal(shape, dtype=np.float32) * np.float32(0.02)
        if name in ("g_q", "g_k"):
            z = np.float32(1.0) + z
        out[name] = bf16_bits(z)
    return out


def make_activations(t: Template, seed: int = ACTIVATION_SEED) -> tuple:
    """(x [B,S,D], temb [B,Dt]) as bf16 bit patterns, ~N(0,1)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    x = bf16_bits(rng.standard_normal((t.batch, t.seq, t.hidden), dtype=np.float32))
    temb = bf16_bits(rng.standard_normal((t.batch, t.temb_dim), dtype=np.float32))
    return x, temb


def sample_rows(t: Template, boundaries=(), n_random: int = 192, seed: int = 7) -> np.ndarray:
    """Sorted, unique token rows for sampled parity: the first and last row, both
    sides of the text/video boundary, both sides of every row index listed in
    `boundaries` (the caller passes its chunk starts), plus `n_random` seeded rows."""
    S = t.seq
    rows = {0, S - 1, max(t.s_text - 1, 0), min(t.s_text, S - 1)}
    for r in boundaries:
        r = int(r)
        if 0 < r < S:
            rows.update((r - 1, r))
    rng = np.random.Generator(np.random.PCG64(seed))
    rows.update(int(v) for v in rng.integers(0, S, size=n_random))
    return np.array(sorted(rows), dtype=np.int64)
