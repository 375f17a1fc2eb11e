"""Pins for the CPU fp64 oracle: closed forms, invariants, library cross-checks, brute force.
Each test is chosen so that a plausible mistake in one place of the oracle (a dropped term, a wrong
sign or index, a transposed operand, a wrong token order) fails it."""
import math
import os
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import eas_synth as S
from eas_synth import configs as C
from oracle import encoder_oracle as O
from tests import bruteforce_encoder as BF

F64 = torch.float64
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(*shape, seed=0):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(*shape, generator=g, dtype=F64)


# ---------------------------------------------------------------- activations: closed-form values

def test_activation_closed_forms():
    fn = {"gelu": O.gelu, "silu": O.silu}
    n = 0
    for line in open(os.path.join(GOLDEN, "activation_values.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, x, val = line.split()
        got = fn[name](torch.tensor([float(x)], dtype=F64)).item()
        assert abs(got - float(val)) < 2e-10, (name, x, got, val)
        n += 1
    assert n == 8


def test_gelu_identities():
    x = _rand(1000) * 3
    g = O.gelu(x)
    # GELU(x) - GELU(-x) = x  (Phi(x) + Phi(-x) = 1)
    assert torch.allclose(g - O.gelu(-x), x, atol=1e-14)
    # the exact form is not the tanh approximation (max gap about 4.7e-4 near |x| = 2.2)
    tanh_form = 0.5 * x * (1 + torch.tanh(math.sqrt(2 / math.pi) * (x + 0.044715 * x ** 3)))
    assert 1e-4 < (g - tanh_form).abs().max() < 1e-3
    assert torch.allclose(g, F.gelu(x), atol=1e-15)
    assert torch.allclose(O.silu(x), F.silu(x), atol=1e-15)


# ---------------------------------------------------------------- norms

def test_layernorm_rmsnorm_against_library_and_moments():
    x = _rand(7, 48) * 3 + 1.5
    g, b = _rand(48, seed=1), _rand(48, seed=2)
    assert torch.allclose(O.layer_norm(x, g, b, 1e-5), F.layer_norm(x, (48,), g, b, 1e-5), atol=1e-13)
    assert torch.allclose(O.rms_norm(x, g, 1e-6), F.rms_norm(x, (48,), g, 1e-6), atol=1e-13)
    y = O.layer_norm(x, torch.ones(48, dtype=F64), torch.zeros(48, dtype=F64), 0.0)
    assert y.mean(-1).abs().max() < 1e-14
    assert (y.var(-1, unbiased=False) - 1).abs().max() < 1e-13
    z = O.rms_norm(x, torch.ones(48, dtype=F64), 0.0)
    assert ((z * z).mean(-1) - 1).abs().max() < 1e-13


# ---------------------------------------------------------------- softmax / attention

def test_softmax_rows_sum_to_one_and_degenerate_cases():
    s = _rand(33, 57) * 8
    p = O.softmax_rows(s)
    assert (p.sum(-1) - 1).abs().max() < 1e-14
    assert (p >= 0).all()
    # huge scores do not overflow (row maximum is subtracted)
    p2 = O.softmax_rows(s + 1e4)
    assert torch.allclose(p, p2, atol=1e-12)
    # a single-token item attends to itself only: o = v
    q, k, v = _rand(1, 2, 8, seed=3), _rand(1, 2, 8, seed=4), _rand(1, 2, 8, seed=5)
    assert torch.allclose(O.attention_one_item(q, k, v), v.reshape(1, 16), atol=1e-15)
    # all keys equal -> uniform weights -> o = mean of v
    q, v = _rand(6, 2, 8, seed=6), _rand(6, 2, 8, seed=7)
    k = _rand(1, 2, 8, seed=8).expand(6, 2, 8)
    o = O.attention_one_item(q, k, v)
    assert torch.allclose(o, v.mean(0).reshape(1, 16).expand(6, 16), atol=1e-14)


def test_attention_against_library_with_block_diagonal_mask():
    lens = [5, 1, 9, 16]
    H, hd = 3, 8
    T = sum(lens)
    q, k, v = _rand(T, H, hd, seed=10) * 2, _rand(T, H, hd, seed=11) * 2, _rand(T, H, hd, seed=12)
    mask = torch.zeros(T, T, dtype=torch.bool)
    outs, a = [], 0
    for L in lens:
        mask[a:a + L, a:a + L] = True
        outs.append(O.attention_one_item(q[a:a + L], k[a:a + L], v[a:a + L]))
        a += L
    ref = F.scaled_dot_product_attention(q.permute(1, 0, 2)[None], k.permute(1, 0, 2)[None],
                                         v.permute(1, 0, 2)[None], attn_mask=mask)[0]
    ref = ref.permute(1, 0, 2).reshape(T, H * hd)
    assert torch.allclose(torch.cat(outs), ref, atol=1e-13)
    # processing query rows in slabs changes no sum (only the library matmul's rounding order)
    o_small = O.attention_one_item(q[:16], k[:16], v[:16], row_chunk=5)
    assert torch.allclose(o_small, O.attention_one_item(q[:16], k[:16], v[:16], row_chunk=2048), atol=1e-14)


# ---------------------------------------------------------------- RoPE

def test_rope_norm_identity_and_relative_property():
    Sx, H, hd = 12, 2, 16
    x = _rand(Sx, H, hd, seed=20)
    hp, wp = torch.randint(0, 90, (Sx,)), torch.randint(0, 90, (Sx,))
    y = O.rope_2d(x, hp, wp, 10000.0)
    assert torch.allclose(y.norm(dim=-1), x.norm(dim=-1), atol=1e-13)
    # every pair (j, j+hd/2) keeps its own norm
    P = hd // 2
    assert torch.allclose(y[..., :P] ** 2 + y[..., P:] ** 2, x[..., :P] ** 2 + x[..., P:] ** 2, atol=1e-13)
    z = torch.zeros(Sx, dtype=torch.int64)
    assert torch.equal(O.rope_2d(x, z, z, 10000.0), x)
    # scores depend on position differences only: shift every (h, w) by a constant
    kx = _rand(Sx, H, hd, seed=21)
    s0 = torch.einsum("thd,uhd->htu", O.rope_2d(x, hp, wp, 1e4), O.rope_2d(kx, hp, wp, 1e4))
    s1 = torch.einsum("thd,uhd->htu", O.rope_2d(x, hp + 7, wp + 3, 1e4), O.rope_2d(kx, hp + 7, wp + 3, 1e4))
    assert torch.allclose(s0, s1, atol=1e-11)
    # a row shift alone must change the rotation (catches an axis that is ignored)
    assert not torch.allclose(O.rope_2d(x, hp + 1, wp, 1e4), y)
    assert not torch.allclose(O.rope_2d(x, hp, wp + 1, 1e4), y)


def test_rope_explicit_small_case():
    # hd = 8: pairs (0,4) (1,5) use the row with frequencies 1, theta^-1/2; (2,6) (3,7) the column
    x = torch.arange(1, 9, dtype=F64).reshape(1, 1, 8)
    y = O.rope_2d(x, torch.tensor([2]), torch.tensor([3]), 100.0)[0, 0]
    angs = [2 * 1.0, 2 * 0.1, 3 * 1.0, 3 * 0.1]
    for j, a in enumerate(angs):
        assert abs(y[j] - (x[0, 0, j] * math.cos(a) - x[0, 0, j + 4] * math.sin(a))) < 1e-14
        assert abs(y[j + 4] - (x[0, 0, j + 4] * math.cos(a) + x[0, 0, j] * math.sin(a))) < 1e-14


# ---------------------------------------------------------------- patch / conv front ends

def test_raster_patch_embedding_is_a_strided_convolution():
    Cc, H, Wd, P, d = 3, 28, 42, 14, 10
    img, W, b = _rand(Cc, H, Wd, seed=30), _rand(d, Cc * P * P, seed=31), _rand(d, seed=32)
    got = O.linear(O.patch_rows_raster(img, P), W, b)
    ref = F.conv2d(img[None], W.reshape(d, Cc, P, P), b, stride=P)[0]      # [d, gh, gw]
    assert torch.allclose(got, ref.permute(1, 2, 0).reshape(-1, d), atol=1e-12)


def test_merge_order_patch_embedding_is_a_strided_conv3d_in_group_major_order():
    Fr, Cc, H, Wd, P, pt, d = 4, 3, 8, 12, 2, 2, 6
    clip, W, b = _rand(Fr, Cc, H, Wd, seed=33), _rand(d, Cc * pt * P * P, seed=34), _rand(d, seed=35)
    got = O.linear(O.patch_rows_merge_order(clip, P, pt), W, b)
    ref = F.conv3d(clip.permute(1, 0, 2, 3)[None], W.reshape(d, Cc, pt, P, P), b, stride=(pt, P, P))[0]  # d,gt,gh,gw
    tpos, hpos, wpos = O.merge_order_positions(Fr // pt, H // P, Wd // P)
    for idx in range(got.shape[0]):
        assert torch.allclose(got[idx], ref[:, tpos[idx], hpos[idx], wpos[idx]], atol=1e-12)
    # order: groups in raster order, 4 tokens of a 2x2 group consecutive
    gw = Wd // P
    for idx in range(got.shape[0]):
        r = idx % (len(hpos) // (Fr // pt))
        grp, within = divmod(r, 4)
        hb, wb = divmod(grp, gw // 2)
        assert (int(hpos[idx]), int(wpos[idx])) == (2 * hb + within // 2, 2 * wb + within % 2)


@pytest.mark.parametrize("stride", [1, 2])
def test_conv1d_k3_against_library(stride):
    n, cin, cout = 14, 5, 7
    x, W, b = _rand(n, cin, seed=36), _rand(cout, 3, cin, seed=37), _rand(cout, seed=38)
    got = O.conv1d_k3(x, W, b, stride)
    ref = F.conv1d(x.T[None], W.permute(0, 2, 1), b, stride=stride, padding=1)[0].T
    assert got.shape == ref.shape
    assert torch.allclose(got, ref, atol=1e-12)


def test_audio_token_count():
    x, W, b = _rand(3000, 2, seed=39), _rand(3, 3, 2, seed=40), _rand(3, seed=41)
    assert O.conv1d_k3(O.conv1d_k3(x, W[:, :, :], b, 1)[:, :2], W, b, 2).shape[0] == 1500


def test_sinusoid_table():
    t = S.sinusoid_table(1500, 1280)
    assert np.all(t[0, :640] == 0) and np.all(t[0, 640:] == 1)
    for p in (1, 7, 1499):
        assert abs(t[p, 0] - math.sin(p)) < 1e-12 and abs(t[p, 640] - math.cos(p)) < 1e-12
        assert abs(t[p, 639] - math.sin(p / 10000.0)) < 1e-12


# ---------------------------------------------------------------- whole-encoder structure

def _tiny_cfg(family):
    if family == 0:
        return dict(name="t0", family=0, n_layers=2, d_model=8, n_heads=2, d_mlp=12, norm=0, norm_eps=1e-5, mlp=0,
                    in_channels=2, patch=2, temporal_patch=1, has_cls=1, embed_norm=1, final_norm=1, pos=0,
                    max_pos=9, rope_theta=0.0, head=1, d_head_hidden=6, d_out=5)
    if family == 1:
        return dict(name="t1", family=1, n_layers=2, d_model=16, n_heads=2, d_mlp=12, norm=1, norm_eps=1e-6, mlp=1,
                    in_channels=2, patch=2, temporal_patch=2, has_cls=0, embed_norm=0, final_norm=0, pos=1,
                    max_pos=0, rope_theta=100.0, head=2, d_head_hidden=10, d_out=6)
    return dict(name="t2", family=2, n_layers=2, d_model=8, n_heads=2, d_mlp=12, norm=0, norm_eps=1e-5, mlp=0,
                in_channels=3, patch=1, temporal_patch=1, has_cls=0, embed_norm=0, final_norm=1, pos=0,
                max_pos=8, rope_theta=0.0, head=0, d_head_hidden=0, d_out=8)


def _tiny_items(cfg, seed):
    rng = np.random.Generator(np.random.PCG64(seed))
    if cfg["family"] == 0:      # 3 and 5(+CLS) ... images of 2x6 and 2x10 pixels, patch 2 -> 3 and 5 patches
        return [rng.random((2, 2, 6)), rng.random((2, 2, 10))]
    if cfg["family"] == 1:      # clips: 2 frames 4x4 (4 tokens) and 4 frames 4x8 (16 tokens)
        return [rng.random((2, 2, 4, 4)), rng.random((4, 2, 4, 8))]
    return [rng.standard_normal((6, 3)), rng.standard_normal((10, 3))]


@pytest.mark.parametrize("family", [0, 1, 2])
def test_tiny_encoder_against_pure_python_brute_force(family):
    cfg = _tiny_cfg(family)
    w = S.make_weights(cfg, seed=77 + family, profile="sharp")
    # larger weights so that every term matters at 1e-9
    w = {k: (v * 10 if (k.endswith(".w") or k == "pos" or k == "cls") else v).astype(np.float64) for k, v in w.items()}
    items = _tiny_items(cfg, 5 + family)
    wl = {k: v.tolist() for k, v in w.items()}
    for it in items:
        got = O.encode_item(cfg, w, it).numpy()
        ref = np.asarray(BF.encode_item(cfg, wl, it.tolist()))
        assert got.shape == ref.shape
        assert np.abs(got - ref).max() < 1e-11 * max(1.0, np.abs(ref).max())
        assert np.abs(ref).max() > 1e-3


@pytest.mark.parametrize("family", [0, 1, 2])
def test_layer_loop_reads_each_layers_own_weights(family):
    """Two layers with different weights: exchanging blk0.* and blk1.* must change the output (a loop that read one
    layer's weights twice, or the layers in the wrong order, would not notice), and exchanging twice restores it.
    The brute-force test above pins the right order; this one pins that the order matters at all."""
    cfg = _tiny_cfg(family)
    assert cfg["n_layers"] == 2
    w = S.make_weights(cfg, seed=31 + family, profile="sharp")
    w = {k: (v * 10 if k.endswith(".w") else v).astype(np.float64) for k, v in w.items()}
    swapped = {}
    for k, v in w.items():
        if k.startswith("blk0."):
            swapped["blk1." + k[5:]] = v
        elif k.startswith("blk1."):
            swapped["blk0." + k[5:]] = v
        else:
            swapped[k] = v
    assert any(not np.array_equal(w[k], swapped[k]) for k in w if k.startswith("blk"))
    item = _tiny_items(cfg, 21)[1]
    a = O.encode_item(cfg, w, item).numpy()
    b = O.encode_item(cfg, swapped, item).numpy()
    assert np.abs(a - b).max() > 1e-3 * np.abs(a).max()
    # the taps after block 0 must already differ (block 0 reads blk0.*, not blk1.*)
    ta, tb = {}, {}
    O.encode_item(cfg, w, item, taps=ta)
    O.encode_item(cfg, swapped, item, taps=tb)
    assert (ta["blk0"] - tb["blk0"]).abs().max() > 1e-6
    # one layer of the swapped weights == running only blk1 of the original: block 0 of `swapped` IS blk1 of `w`
    cfg1 = dict(cfg, n_layers=1)
    w_only1 = {k: v for k, v in swapped.items() if not k.startswith("blk1.")}
    t1 = {}
    O.encode_item(cfg1, w_only1, item, taps=t1)
    assert torch.equal(t1["blk0"], tb["blk0"])


@pytest.mark.parametrize("family", [0, 1, 2])
def test_packing_invariance_is_bit_exact(family):
    cfg = _tiny_cfg(family)
    w = S.make_weights(cfg, seed=3)
    items = _tiny_items(cfg, 9)
    alone = [O.encode_item(cfg, w, it).numpy() for it in items]
    packed, cu, cu_out = O.encode_microbatch(cfg, w, items[::-1] + items)
    assert np.array_equal(packed[cu_out[2]:cu_out[3]], alone[0])
    assert np.array_equal(packed[cu_out[0]:cu_out[1]], alone[1])
    assert np.array_equal(packed[cu_out[3]:cu_out[4]], alone[1])
    assert cu[-1] == 2 * sum(S.tokens_per_item(cfg, _shape(cfg, it)) for it in items)


def _shape(cfg, it):
    if cfg["family"] == 2:
        return (it.shape[0], it.shape[1], 1)
    if it.ndim == 4:
        return (it.shape[0], it.shape[2], it.shape[3])
    return (1, it.shape[1], it.shape[2])


def test_zero_block_weights_leave_head_of_embedding():
    cfg = S.get_config("c0", n_layers=2)
    w = S.make_weights(cfg, seed=5)
    item = S.make_items(cfg, [(1, 224, 224)], seed=6)[0]
    Wp = O._W(w)
    x0, _, _ = O.embed_item(cfg, Wp, item)
    expect = O.head(cfg, Wp, x0)
    # proj and fc2 (weights and biases) zero: both residual branches vanish
    w2 = dict(w)
    for i in range(2):
        for n in ("proj.w", "proj.b", "fc2.w", "fc2.b"):
            w2[f"blk{i}.{n}"] = np.zeros_like(w[f"blk{i}.{n}"])
    assert torch.allclose(O.encode_item(cfg, w2, item), expect, atol=1e-13)
    # only fc2 zero: the attention branch must change the result (residual wiring is live)
    w3 = dict(w)
    for i in range(2):
        for n in ("fc2.w", "fc2.b"):
            w3[f"blk{i}.{n}"] = np.zeros_like(w[f"blk{i}.{n}"])
    assert (O.encode_item(cfg, w3, item) - expect).abs().max() > 1e-4


def test_token_permutation_equivariance_without_positions():
    cfg = _tiny_cfg(0)
    cfg.update(has_cls=0, head=0, d_out=8, final_norm=1)
    w = S.make_weights(cfg, seed=8)
    w["pos"] = np.zeros_like(w["pos"])
    img = np.random.Generator(np.random.PCG64(1)).random((2, 2, 12))
    perm = [3, 0, 5, 1, 4, 2]
    img_p = np.concatenate([img[:, :, 2 * p:2 * p + 2] for p in perm], axis=2)
    a = O.encode_item(cfg, w, img).numpy()
    b = O.encode_item(cfg, w, img_p).numpy()
    assert np.allclose(b, a[perm], atol=1e-13)
    assert not np.allclose(b, a, atol=1e-6)


def test_merger_is_gather_over_2x2_neighbourhoods():
    cfg = _tiny_cfg(1)
    w = S.make_weights(cfg, seed=12)
    clip = np.random.Generator(np.random.PCG64(2)).random((2, 2, 8, 12))   # gt=1, gh=4, gw=6
    taps = {}
    out = O.encode_item(cfg, w, clip, taps=taps).numpy()
    x = taps[f"blk{cfg['n_layers'] - 1}"]          # residual stream after the last block
    n = O.rms_norm(x, O._t(w["head.norm.g"]), cfg["norm_eps"])
    _, hpos, wpos = O.merge_order_positions(1, 4, 6)
    index_of = {(int(h), int(c)): i for i, (h, c) in enumerate(zip(hpos, wpos))}
    rows = []
    for hb in range(2):
        for wb in range(3):
            rows.append(torch.cat([n[index_of[(2 * hb + hi, 2 * wb + wi)]] for hi in range(2) for wi in range(2)]))
    g = torch.stack(rows)
    ref = O.linear(O.gelu(O.linear(g, O._t(w["head.fc1.w"]), O._t(w["head.fc1.b"]))),
                   O._t(w["head.fc2.w"]), O._t(w["head.fc2.b"]))
    assert np.allclose(out, ref.numpy(), atol=1e-13)
    assert out.shape == (6, cfg["d_out"])


def test_c0_shapes_and_cu_seqlens():
    cfg = S.get_config("c0")
    w = S.make_weights(cfg)
    items = S.make_items(cfg, S.draw_item_shapes(cfg, 2, 3002), seed=2002)
    out, cu, cu_out = O.encode_microbatch(cfg, w, items)
    assert out.shape == (392, 256) and list(cu) == [0, 196, 392] and list(cu_out) == [0, 196, 392]
    assert np.isfinite(out).all()
    # final LayerNorm: every row has mean ~ beta-mean and unit-ish scale
    assert 0.5 < out.std() < 1.5
