"""Seeded random-init weights and synthetic media items.

Every tensor is drawn from numpy's PCG64 generator and rounded ONCE to bfloat16
(round-to-nearest-even); the same rounded values go to the CPU oracle (as float32 arrays
that hold bf16-exact numbers) and to the GPU (as bf16), so a comparison measures internal
rounding only, never input quantisation."""
from __future__ import annotations
import math
import numpy as np
from . import configs as C


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float32 array whose values are the nearest bfloat16 (ties to even)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    out = ((u + r) & np.uint32(0xFFFF0000)).view(np.float32)
    return out


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of an array that already holds bf16-exact float32 values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16)


def sinusoid_table(n_pos: int, d: int) -> np.ndarray:
    """Fixed sinusoid position table of the audio encoder: first half sines, second half cosines,
    wavelengths in geometric progression from 2*pi to 10000*2*pi."""
    half = d // 2
    r = np.exp(-np.arange(half, dtype=np.float64) * (math.log(10000.0) / (half - 1)))
    ang = np.arange(n_pos, dtype=np.float64)[:, None] * r[None, :]
    return np.concatenate([np.sin(ang), np.cos(ang)], axis=1)


def make_weights(cfg: dict, seed: int | None = None, profile: str = "plain") -> dict:
    """Random-init weights: matrices, tables, CLS, biases and norm offsets ~ N(0, 0.02^2); norm
    gains = 1 + N(0, 0.02^2).  profile="sharp" doubles the query and key rows of every qkv
    matrix (and bias) so that softmax is far from uniform and position / scaling mistakes show.
    Returns name -> float32 array of bf16-exact values."""
    if seed is None:
        seed = 1000 + C.CONFIG_INDEX.get(cfg["name"], 9)
    rng = np.random.Generator(np.random.PCG64(seed))
    d = cfg["d_model"]
    w = {}
    for name, shape in C.weight_shapes(cfg).items():
        a = rng.standard_normal(shape, dtype=np.float32) * np.float32(0.02)
        if name.endswith("norm1.g") or name.endswith("norm2.g") or name.endswith("norm.g"):
            a = a + np.float32(1.0)
        if name == "pos" and cfg["family"] == C.FAMILY_AUDIO_CONV:
            a = sinusoid_table(cfg["max_pos"], d).astype(np.float32)
        if profile == "sharp" and (name.endswith("qkv.w") or name.endswith("qkv.b")):
            a[: 2 * d] *= np.float32(2.0)
        w[name] = round_to_bf16(a)
    return w


def draw_item_shapes(cfg: dict, n_items: int, seed: int) -> list:
    """(frames, height, width) per item, following each workload's size distribution."""
    rng = np.random.Generator(np.random.PCG64(seed))
    name = cfg["name"]
    shapes = []
    for _ in range(n_items):
        if name == "c0":
            shapes.append((1, 224, 224))
        elif name == "c1":
            shapes.append((1, 336, 336))
        elif name == "c2":   # height and width uniform over multiples of 28 in [224, 1344]
            a, b = rng.integers(8, 49, size=2)
            shapes.append((1, 28 * int(a), 28 * int(b)))
        elif name == "c3":   # 448x448 clips with 16, 32 or 64 frames
            shapes.append((int(rng.choice([16, 32, 64])), 448, 448))
        elif name == "c4":
            shapes.append((3000, 128, 1))
        else:
            raise ValueError(name)
    return shapes


def make_items(cfg: dict, shapes, seed: int) -> list:
    """One float32 array of bf16-exact values per item.  Images [C,H,W]; clips [F,C,H,W], pixels
    uniform in [0,1); audio [n_frames, n_mel] log-mel values ~ N(0,1)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    items = []
    for (f, h, w) in shapes:
        if cfg["family"] == C.FAMILY_AUDIO_CONV:
            a = rng.standard_normal((f, h), dtype=np.float32)
        elif cfg["temporal_patch"] > 1:
            a = rng.random((f, cfg["in_channels"], h, w), dtype=np.float32)
        else:
            a = rng.random((cfg["in_channels"], h, w), dtype=np.float32)
        items.append(round_to_bf16(a))
    return items
