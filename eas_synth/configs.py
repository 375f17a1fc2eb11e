"""Architecture tables for the five encoder workloads (plain data, no arithmetic).

The encoder families follow Table 3 of the paper (CLIP-style ViT for images, a
dynamic-resolution ViT for video, a Whisper-style encoder for audio); Section 2.1 defines
Encode as encoder plus connector.  The numbers are the benchmark configurations c0..c4."""
from __future__ import annotations
import copy

FAMILY_VIT_LEARNED, FAMILY_VIT_ROPE_MERGER, FAMILY_AUDIO_CONV = 0, 1, 2
NORM_LAYERNORM, NORM_RMSNORM = 0, 1
MLP_GELU, MLP_SWIGLU = 0, 1
POS_TABLE, POS_ROPE_2D = 0, 1
HEAD_NONE, HEAD_MLP_PROJECTOR, HEAD_MERGER_2X2 = 0, 1, 2

CONFIGS = {
    # tiny ViT: 224x224 RGB, patch 16 -> 196 tokens, final LayerNorm, no head
    "c0": dict(name="c0", family=FAMILY_VIT_LEARNED, n_layers=2, d_model=256, n_heads=4, d_mlp=1024,
               norm=NORM_LAYERNORM, norm_eps=1e-5, mlp=MLP_GELU, in_channels=3, patch=16,
               temporal_patch=1, has_cls=0, embed_norm=0, final_norm=1, pos=POS_TABLE, max_pos=196,
               rope_theta=0.0, head=HEAD_NONE, d_head_hidden=0, d_out=256),
    # ViT-L/14-style: 336x336 -> 576 patches + CLS, LayerNorm after embedding, MLP projector to 4096
    "c1": dict(name="c1", family=FAMILY_VIT_LEARNED, n_layers=24, d_model=1024, n_heads=16, d_mlp=4096,
               norm=NORM_LAYERNORM, norm_eps=1e-5, mlp=MLP_GELU, in_channels=3, patch=14,
               temporal_patch=1, has_cls=1, embed_norm=1, final_norm=0, pos=POS_TABLE, max_pos=577,
               rope_theta=0.0, head=HEAD_MLP_PROJECTOR, d_head_hidden=4096, d_out=4096),
    # native-resolution ViT: RMSNorm, SwiGLU, 2-D RoPE, 2x2 patch merger to 3584
    "c2": dict(name="c2", family=FAMILY_VIT_ROPE_MERGER, n_layers=32, d_model=1280, n_heads=16, d_mlp=5120,
               norm=NORM_RMSNORM, norm_eps=1e-6, mlp=MLP_SWIGLU, in_channels=3, patch=14,
               temporal_patch=1, has_cls=0, embed_norm=0, final_norm=0, pos=POS_ROPE_2D, max_pos=0,
               rope_theta=10000.0, head=HEAD_MERGER_2X2, d_head_hidden=5120, d_out=3584),
    # video: the c2 encoder with 14x14x2 spatio-temporal patches
    "c3": dict(name="c3", family=FAMILY_VIT_ROPE_MERGER, n_layers=32, d_model=1280, n_heads=16, d_mlp=5120,
               norm=NORM_RMSNORM, norm_eps=1e-6, mlp=MLP_SWIGLU, in_channels=3, patch=14,
               temporal_patch=2, has_cls=0, embed_norm=0, final_norm=0, pos=POS_ROPE_2D, max_pos=0,
               rope_theta=10000.0, head=HEAD_MERGER_2X2, d_head_hidden=5120, d_out=3584),
    # Whisper-large-style audio: 128 mel bins, two k=3 convolutions (stride 1, 2), sinusoid table
    "c4": dict(name="c4", family=FAMILY_AUDIO_CONV, n_layers=32, d_model=1280, n_heads=20, d_mlp=5120,
               norm=NORM_LAYERNORM, norm_eps=1e-5, mlp=MLP_GELU, in_channels=128, patch=1,
               temporal_patch=1, has_cls=0, embed_norm=0, final_norm=1, pos=POS_TABLE, max_pos=1500,
               rope_theta=0.0, head=HEAD_NONE, d_head_hidden=0, d_out=1280),
}
CONFIG_INDEX = {"c0": 0, "c1": 1, "c2": 2, "c3": 3, "c4": 4}


def get_config(name: str, **overrides) -> dict:
    """A copy of configuration `name` with fields overridden (e.g. n_layers=2 for a shallow test)."""
    cfg = copy.deepcopy(CONFIGS[name])
    cfg.update(overrides)
    return cfg


def embed_k(cfg: dict) -> int:
    """Length of one flattened patch (channel, [frame,] row, column)."""
    return cfg["in_channels"] * cfg["temporal_patch"] * cfg["patch"] * cfg["patch"]


def weight_shapes(cfg: dict) -> dict:
    """Name -> shape of every weight tensor.  Linear weights are [out_features, in_features]."""
    d, I, L = cfg["d_model"], cfg["d_mlp"], cfg["n_layers"]
    ln = cfg["norm"] == NORM_LAYERNORM
    s = {}
    if cfg["family"] == FAMILY_AUDIO_CONV:
        s["conv1.w"] = (d, 3, cfg["in_channels"]); s["conv1.b"] = (d,)
        s["conv2.w"] = (d, 3, d); s["conv2.b"] = (d,)
    else:
        s["embed.w"] = (d, embed_k(cfg)); s["embed.b"] = (d,)
    if cfg["has_cls"]:
        s["cls"] = (d,)
    if cfg["pos"] == POS_TABLE:
        s["pos"] = (cfg["max_pos"], d)
    if cfg["embed_norm"]:
        s["embed_norm.g"] = (d,)
        if ln: s["embed_norm.b"] = (d,)
    for i in range(L):
        p = f"blk{i}."
        s[p + "norm1.g"] = (d,)
        if ln: s[p + "norm1.b"] = (d,)
        s[p + "qkv.w"] = (3 * d, d); s[p + "qkv.b"] = (3 * d,)
        s[p + "proj.w"] = (d, d); s[p + "proj.b"] = (d,)
        s[p + "norm2.g"] = (d,)
        if ln: s[p + "norm2.b"] = (d,)
        if cfg["mlp"] == MLP_SWIGLU:
            s[p + "gate.w"] = (I, d); s[p + "gate.b"] = (I,)
            s[p + "up.w"] = (I, d); s[p + "up.b"] = (I,)
        else:
            s[p + "fc1.w"] = (I, d); s[p + "fc1.b"] = (I,)
        s[p + "fc2.w"] = (d, I); s[p + "fc2.b"] = (d,)
    if cfg["final_norm"]:
        s["final_norm.g"] = (d,)
        if ln: s["final_norm.b"] = (d,)
    if cfg["head"] == HEAD_MLP_PROJECTOR:
        s["head.fc1.w"] = (cfg["d_head_hidden"], d); s["head.fc1.b"] = (cfg["d_head_hidden"],)
        s["head.fc2.w"] = (cfg["d_out"], cfg["d_head_hidden"]); s["head.fc2.b"] = (cfg["d_out"],)
    elif cfg["head"] == HEAD_MERGER_2X2:
        s["head.norm.g"] = (d,)
        s["head.fc1.w"] = (cfg["d_head_hidden"], 4 * d); s["head.fc1.b"] = (cfg["d_head_hidden"],)
        s["head.fc2.w"] = (cfg["d_out"], cfg["d_head_hidden"]); s["head.fc2.b"] = (cfg["d_out"],)
    return s


def tokens_per_item(cfg: dict, shape) -> int:
    """Encoder tokens of one item.  shape = (frames, height, width); audio: (n_frames, n_mel, 1)."""
    f, h, w = (int(v) for v in shape)
    if cfg["family"] == FAMILY_AUDIO_CONV:
        return (f + 1) // 2         # k=3, stride 2, padding 1: floor((f - 1) / 2) + 1 output frames
    P = cfg["patch"]
    return (f // cfg["temporal_patch"]) * (h // P) * (w // P) + (1 if cfg["has_cls"] else 0)


def out_tokens_per_item(cfg: dict, shape) -> int:
    s = tokens_per_item(cfg, shape)
    if cfg["head"] == HEAD_MLP_PROJECTOR and cfg["has_cls"]:
        return s - 1
    if cfg["head"] == HEAD_MERGER_2X2:
        return s // 4
    return s
