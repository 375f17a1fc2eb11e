"""CPU fp64 oracle of the Encode stage forward pass.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition that the CUDA encoder is checked against.  Only the
tests, the smoke check and the benchmark's cpu-baseline leg may import it; the product path never
does.  It shares no code with the CUDA path.

What it follows.  The paper defines Encode as "modality encoder plus connector" producing
modality embeddings (Section 2.1), run as one forward pass per micro-batch (Section 3.2) with
the encoder family per modality given in Table 3 (CLIP-style ViT, dynamic-resolution ViT,
Whisper-style audio encoder).  The paper fixes nothing below that level; each operation here is
its textbook definition written out in float64, and every reading the sources leave open is listed
next to the function that takes it.

Structure.  One outer loop PER ITEM: an item is encoded from its own pixels/frames only, so
no token of another item can be read and an item's output is bit-identical however it is packed.
Library primitives used as steps: float64 matmul, exp, erf, sqrt, sin, cos.

Parity pins (tests/test_oracle_*.py): closed-form activation values, softmax and RoPE invariants,
library cross-checks (conv2d/conv3d/conv1d, layer_norm, rms_norm, scaled_dot_product_attention),
structural zero-weight tests, an independent pure-Python brute force on a tiny encoder.  The full
depth composite of c1..c4 has no external reference beyond those pins: for the composite, parity is
unpinned beyond the per-stage and structural pins.
"""
from __future__ import annotations
import math
import numpy as np
import torch

F64 = torch.float64

# enumerations of the architecture record (same integers as eas_synth.configs, restated here so
# that the oracle reads a plain dict and depends on nothing else)
FAMILY_VIT_LEARNED, FAMILY_VIT_ROPE_MERGER, FAMILY_AUDIO_CONV = 0, 1, 2
NORM_LAYERNORM, NORM_RMSNORM = 0, 1
MLP_GELU, MLP_SWIGLU = 0, 1
POS_TABLE, POS_ROPE_2D = 0, 1
HEAD_NONE, HEAD_MLP_PROJECTOR, HEAD_MERGER_2X2 = 0, 1, 2


def _t(a) -> torch.Tensor:
    """Promote an array of bf16-exact float32 values to float64 (exact)."""
    if isinstance(a, torch.Tensor):
        return a.to(F64)
    return torch.from_numpy(np.ascontiguousarray(a)).to(F64)


# --------------------------------------------------------------------------- elementary operations

def linear(x: torch.Tensor, W: torch.Tensor, b: torch.Tensor | None) -> torch.Tensor:
    """y[t,o] = sum_i x[t,i] W[o,i] + b[o]   (W is [out_features, in_features])."""
    y = x @ W.T
    return y if b is None else y + b


def layer_norm(x, g, b, eps):
    """(x - mean) / sqrt(biased variance + eps) * g + b over the last axis."""
    d = x.shape[-1]
    mu = x.sum(dim=-1, keepdim=True) / d
    var = ((x - mu) ** 2).sum(dim=-1, keepdim=True) / d
    return (x - mu) / torch.sqrt(var + eps) * g + b


def rms_norm(x, g, eps):
    """x / sqrt(mean(x^2) + eps) * g over the last axis."""
    d = x.shape[-1]
    ms = (x * x).sum(dim=-1, keepdim=True) / d
    return x / torch.sqrt(ms + eps) * g


def gelu(x):
    """Exact GELU: x * Phi(x) = x/2 * (1 + erf(x / sqrt 2)).  Reading: every "GELU" is this form."""
    return 0.5 * x * (1.0 + torch.erf(x / math.sqrt(2.0)))


def silu(x):
    """x * sigmoid(x) = x / (1 + exp(-x))."""
    return x / (1.0 + torch.exp(-x))


def softmax_rows(s):
    """Row softmax with the row maximum subtracted first."""
    m = s.max(dim=-1, keepdim=True).values
    e = torch.exp(s - m)
    return e / e.sum(dim=-1, keepdim=True)


def attention_one_item(q, k, v, row_chunk: int = 2048):
    """Non-causal softmax attention of ONE item.  q, k, v: [S, H, hd].  For every head,
    s[t,u] = q[t].k[u] / sqrt(hd), p = softmax over all keys u of the same item, o[t] = sum_u p[t,u] v[u].
    Query rows are independent, so long items are processed a slab of rows at a time (this changes
    no sum).  Returns [S, H*hd] with heads concatenated in order."""
    S, H, hd = q.shape
    scale = 1.0 / math.sqrt(hd)
    o = torch.empty(S, H, hd, dtype=F64)
    for h in range(H):
        kh, vh = k[:, h, :], v[:, h, :]
        for r0 in range(0, S, row_chunk):
            s = (q[r0:r0 + row_chunk, h, :] @ kh.T) * scale
            o[r0:r0 + row_chunk, h, :] = softmax_rows(s) @ vh
    return o.reshape(S, H * hd)


def rope_2d(x, hpos, wpos, theta):
    """2-D rotary embedding of x [S, H, hd] by token grid position (hpos[S], wpos[S]).

    Reading taken (the sources only say "2D RoPE"): with P = hd/2 pairs (j, j+P), j in [0,P), and
    frequencies w_i = theta^(-i/(P/2)), i in [0,P/2): pair j < P/2 turns by the angle hpos*w_j, pair
    j >= P/2 by wpos*w_{j-P/2};  (x_j, x_{j+P}) <- (x_j cos - x_{j+P} sin, x_{j+P} cos + x_j sin)."""
    S, H, hd = x.shape
    P = hd // 2
    nf = P // 2
    freq = torch.tensor([theta ** (-(i / nf)) for i in range(nf)], dtype=F64)
    ang = torch.cat([hpos.to(F64)[:, None] * freq[None, :], wpos.to(F64)[:, None] * freq[None, :]], dim=1)  # [S,P]
    c, s = torch.cos(ang)[:, None, :], torch.sin(ang)[:, None, :]
    a, b = x[..., :P], x[..., P:]
    return torch.cat([a * c - b * s, b * c + a * s], dim=-1)


# --------------------------------------------------------------------------- embedding front ends

def patch_rows_raster(img, P):
    """Image [C,H,W] -> [gh*gw, C*P*P]; token (r,c) has index r*gw + c; a row lists (channel, py, px)."""
    C, H, W = img.shape
    gh, gw = H // P, W // P
    x = img.reshape(C, gh, P, gw, P).permute(1, 3, 0, 2, 4)       # gh, gw, C, py, px
    return x.reshape(gh * gw, C * P * P)


def merge_order_positions(gt, gh, gw):
    """Token order of the native-resolution ViT (reading: merge-group-major, so that the 2x2 merger
    is a reshape).  index = t*gh*gw + ((hb*(gw/2) + wb)*4 + hi*2 + wi), grid row h = 2hb+hi, column
    w = 2wb+wi.  Returns (tpos, hpos, wpos), each int64 [gt*gh*gw]."""
    t, hb, wb, hi, wi = torch.meshgrid(torch.arange(gt), torch.arange(gh // 2), torch.arange(gw // 2),
                                       torch.arange(2), torch.arange(2), indexing="ij")
    return t.reshape(-1), (2 * hb + hi).reshape(-1), (2 * wb + wi).reshape(-1)


def patch_rows_merge_order(clip, P, pt):
    """Clip [F,C,H,W] (an image is F = pt = 1) -> [S, C*pt*P*P] in merge-group-major token order; a
    row lists (channel, frame-in-patch, py, px)."""
    F_, C, H, W = clip.shape
    gt, gh, gw = F_ // pt, H // P, W // P
    x = clip.reshape(gt, pt, C, gh // 2, 2, P, gw // 2, 2, P)
    #            0   1   2   3      4  5   6      7  8
    x = x.permute(0, 3, 6, 4, 7, 2, 1, 5, 8)        # t, hb, wb, hi, wi, C, pt, py, px
    return x.reshape(gt * gh * gw, C * pt * P * P)


def conv1d_k3(x, W, b, stride):
    """x [n, Cin], W [Cout, 3, Cin] (tap-major, then channel): y[t,o] = b[o] + sum_k sum_c W[o,k,c]
    x[stride*t + k - 1, c], rows outside [0,n) read as zero; t in [0, floor((n-1)/stride)] ."""
    n, cin = x.shape
    n_out = (n + 2 - 3) // stride + 1
    xp = torch.zeros(n + 2, cin, dtype=F64)
    xp[1:n + 1] = x
    y = torch.zeros(n_out, W.shape[0], dtype=F64) + b
    for k in range(3):
        rows = xp[k: k + stride * (n_out - 1) + 1: stride]        # x[stride*t + k - 1]
        y = y + rows @ W[:, k, :].T
    return y


# --------------------------------------------------------------------------- the encoder

class _W:
    """Weights by name, promoted to float64 on use."""
    def __init__(self, weights):
        self.w = weights

    def __call__(self, name):
        return _t(self.w[name])

    def get(self, name):
        return _t(self.w[name]) if name in self.w else None


def _norm(cfg, W, prefix, x):
    if cfg["norm"] == NORM_LAYERNORM:
        return layer_norm(x, W(prefix + ".g"), W(prefix + ".b"), cfg["norm_eps"])
    return rms_norm(x, W(prefix + ".g"), cfg["norm_eps"])


def embed_item(cfg, W, item):
    """Item -> (x [S, d], hpos, wpos).  Front end per family:
    learned-position ViT: raster patches, linear, optional CLS row first, + position table rows,
      optional LayerNorm after the embedding;
    RoPE ViT: merge-order patches (2 frames per patch for clips), linear, no table, no CLS;
    audio: conv1d(k3,s1) + GELU, conv1d(k3,s2) + GELU (reading: GELU after both), + sinusoid table."""
    fam = cfg["family"]
    hpos = wpos = None
    if fam == FAMILY_VIT_LEARNED:
        rows = patch_rows_raster(_t(item), cfg["patch"])
        x = linear(rows, W("embed.w"), W("embed.b"))
        if cfg["has_cls"]:
            x = torch.cat([W("cls")[None, :], x], dim=0)
        x = x + W("pos")[: x.shape[0]]
        if cfg["embed_norm"]:
            x = _norm(cfg, W, "embed_norm", x)
    elif fam == FAMILY_VIT_ROPE_MERGER:
        clip = _t(item)
        if clip.dim() == 3:
            clip = clip[None]
        P, pt = cfg["patch"], cfg["temporal_patch"]
        rows = patch_rows_merge_order(clip, P, pt)
        x = linear(rows, W("embed.w"), W("embed.b"))
        _, hpos, wpos = merge_order_positions(clip.shape[0] // pt, clip.shape[2] // P, clip.shape[3] // P)
    elif fam == FAMILY_AUDIO_CONV:
        mel = _t(item)                                             # [n_frames, n_mel]
        h1 = gelu(conv1d_k3(mel, W("conv1.w"), W("conv1.b"), 1))
        h2 = gelu(conv1d_k3(h1, W("conv2.w"), W("conv2.b"), 2))
        x = h2 + W("pos")[: h2.shape[0]]
    else:
        raise ValueError("unknown family")
    return x, hpos, wpos


def block(cfg, W, i, x, hpos, wpos, rnd=None):
    """Pre-norm transformer block: x <- x + proj(Attn(qkv(Norm1 x))); x <- x + MLP(Norm2 x).
    qkv rows are ordered all-Q, all-K, all-V; head h owns columns h*hd..h*hd+hd of each third."""
    rnd = rnd or (lambda name, v: v)
    d, H = cfg["d_model"], cfg["n_heads"]
    hd = d // H
    p = f"blk{i}."
    n = rnd("norm", _norm(cfg, W, p + "norm1", x))
    qkv = linear(n, W(p + "qkv.w"), W(p + "qkv.b"))
    S = x.shape[0]
    q = qkv[:, :d].reshape(S, H, hd)
    k = qkv[:, d:2 * d].reshape(S, H, hd)
    v = qkv[:, 2 * d:].reshape(S, H, hd)
    if cfg["pos"] == POS_ROPE_2D:
        q = rope_2d(q, hpos, wpos, cfg["rope_theta"])
        k = rope_2d(k, hpos, wpos, cfg["rope_theta"])
    q, k, v = rnd("qkv", q), rnd("qkv", k), rnd("qkv", v)
    o = rnd("attn_out", attention_one_item(q, k, v))
    x = x + linear(o, W(p + "proj.w"), W(p + "proj.b"))
    n = rnd("norm", _norm(cfg, W, p + "norm2", x))
    if cfg["mlp"] == MLP_SWIGLU:
        a = silu(linear(n, W(p + "gate.w"), W(p + "gate.b"))) * linear(n, W(p + "up.w"), W(p + "up.b"))
    else:
        a = gelu(linear(n, W(p + "fc1.w"), W(p + "fc1.b")))
    a = rnd("mlp_act", a)
    return x + linear(a, W(p + "fc2.w"), W(p + "fc2.b"))


def head(cfg, W, x, rnd=None):
    """Connector.  none: optional final norm.  MLP projector: drop the CLS row, Linear + GELU + Linear.
    2x2 merger (reading): RMSNorm per token, concatenate each 4 consecutive tokens (one 2x2 group in
    merge order), Linear + GELU + Linear."""
    rnd = rnd or (lambda name, v: v)
    if cfg["final_norm"]:
        x = _norm(cfg, W, "final_norm", x)
    if cfg["head"] == HEAD_NONE:
        return x
    if cfg["head"] == HEAD_MLP_PROJECTOR:
        if cfg["has_cls"]:
            x = x[1:]
        x = rnd("norm", x)
        hmid = rnd("mlp_act", gelu(linear(x, W("head.fc1.w"), W("head.fc1.b"))))
        return linear(hmid, W("head.fc2.w"), W("head.fc2.b"))
    if cfg["head"] == HEAD_MERGER_2X2:
        n = rnd("norm", rms_norm(x, W("head.norm.g"), cfg["norm_eps"]))
        g = n.reshape(n.shape[0] // 4, 4 * n.shape[1])
        hmid = rnd("mlp_act", gelu(linear(g, W("head.fc1.w"), W("head.fc1.b"))))
        return linear(hmid, W("head.fc2.w"), W("head.fc2.b"))
    raise ValueError("unknown head")


def encode_item(cfg, weights, item, taps=None, rnd=None):
    """One media item -> its embedding block [out_tokens, d_out], float64.
    taps: optional dict filled with the residual stream after the embedding ("embed") and after each
    block ("blk{i}")."""
    W = _W(weights)
    x, hpos, wpos = embed_item(cfg, W, item)
    if taps is not None:
        taps["embed"] = x.clone()
    for i in range(cfg["n_layers"]):
        x = block(cfg, W, i, x, hpos, wpos, rnd)
        if taps is not None:
            taps[f"blk{i}"] = x.clone()
    return head(cfg, W, x, rnd)


def encode_microbatch(cfg, weights, items, rnd=None):
    """Micro-batch -> (embeddings [sum out_tokens, d_out] float64 ndarray, cu_seqlens of ENCODER tokens,
    cu_out of output rows).  Items are encoded one at a time and stacked in order."""
    outs, cu, cu_out = [], [0], [0]
    for item in items:
        taps = {}
        y = encode_item(cfg, weights, item, taps=taps, rnd=rnd)
        outs.append(y)
        cu.append(cu[-1] + taps["embed"].shape[0])
        cu_out.append(cu_out[-1] + y.shape[0])
    return torch.cat(outs, dim=0).numpy(), np.asarray(cu, dtype=np.int32), np.asarray(cu_out, dtype=np.int32)


# --------------------------------------------------------------------------- diagnostic (never the reference)

def bf16_rounder(points=("norm", "qkv", "attn_out", "mlp_act")):
    """Returns a hook that rounds to bfloat16 at the named points, to PREDICT the error of a
    bf16-operand GPU pipeline before it exists.  A diagnostic; the reference is always unrounded."""
    def rnd(name, v):
        if name in points:
            return v.to(torch.bfloat16).to(F64)
        return v
    return rnd
