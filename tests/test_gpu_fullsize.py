"""Parity at the benchmark's sizes and at full depth.  The oracle costs 0.4-30 TFLOP of fp64 per item, so
full-size micro-batches are checked on sampled items (an item's output does not depend on its neighbours, which
the bit-equality tests below establish on the GPU side), and the largest shapes at reduced depth."""
import numpy as np
import pytest
import torch

import eas_synth as S
from oracle import encoder_oracle as O
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _make(cfg, profile="plain"):
    import paper_2609_31551_b200 as P
    w = S.make_weights(cfg, profile=profile)
    return w, P.Encoder(cfg, P.weights_to_device(w))


def _out_slices(cfg, items):
    rows = [S.out_tokens_per_item(cfg, G.item_shape(cfg, it)) for it in items]
    cu = np.concatenate([[0], np.cumsum(rows)])
    return [slice(int(a), int(b)) for a, b in zip(cu[:-1], cu[1:])]


def test_c1_bench_configuration_sampled_items():
    """c1 at micro-batch 32, full depth, all SMs: the configuration bench.py times."""
    cfg = S.get_config("c1")
    w, enc = _make(cfg)
    shapes = S.draw_item_shapes(cfg, 32, 3105)
    items = S.make_items(cfg, shapes, seed=2105)
    got, out_dev = G.run_gpu(enc, cfg, items)
    sl = _out_slices(cfg, items)
    for i in (0, 17, 31):
        ref = O.encode_item(cfg, w, items[i]).numpy()
        rel, mabs = G.assert_parity(got[sl[i]], ref, f"c1 mb32 item {i}")
        G.record_margin(f"c1 mb32 full depth, item {i}", "plain", 2105, rel, mabs)
        print(f"c1 mb32 item {i}: row-rel {rel:.3e} max-abs {mabs:.3e}")
    # an item encoded alone gives the same bytes as inside the micro-batch, for any SM budget
    _, alone = G.run_gpu(enc, cfg, [items[17]], sm_budget=37)
    assert torch.equal(alone, out_dev[sl[17]])


@pytest.mark.parametrize("name,shapes,seed", [("c1", [(1, 336, 336)] * 2, 2121),
                                               ("c2", [(1, 224, 224), (1, 448, 336)], 2221)])
def test_full_depth_with_folded_normalisation(name, shapes, seed):
    """Full depth with eas_encoder_set_norm_fold on: LayerNorm (c1) and RMSNorm with rotary positions (c2)."""
    cfg = S.get_config(name)
    w, enc = _make(cfg, "sharp")
    enc.set_norm_fold(True)
    items = S.make_items(cfg, shapes, seed=seed)
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    got, _ = G.run_gpu(enc, cfg, items)
    rel, mabs = G.assert_parity(got, ref, f"{name} folded")
    G.record_margin(f"{name} full depth, folded normalisation", "sharp", seed, rel, mabs)


@pytest.mark.parametrize("profile,seed", [("sharp", 2101), ("sharp", 2111), ("plain", 2112)])
def test_c1_full_depth_two_images(profile, seed):
    cfg = S.get_config("c1")
    w, enc = _make(cfg, profile)
    items = S.make_items(cfg, [(1, 336, 336)] * 2, seed=seed)
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    got, _ = G.run_gpu(enc, cfg, items)
    rel, mabs = G.assert_parity(got, ref, f"c1 {profile}")
    G.record_margin("c1 mb2 full depth", profile, seed, rel, mabs)
    print(f"c1 {profile} full depth seed {seed}:", rel, mabs)
    # the same pass with fp32 output (EAS_OUT_FP32): what remains of the error without the output rounding
    import paper_2609_31551_b200 as P
    enc32 = P.Encoder(dict(cfg, out_dtype=1), enc._weights)
    got32, dev32 = G.run_gpu(enc32, cfg, items)
    assert dev32.dtype == torch.float32
    rel32, mabs32 = G.assert_parity(got32, ref, f"c1 {profile} fp32 out")
    G.record_margin("c1 mb2 full depth, fp32 output", profile, seed, rel32, mabs32)
    assert mabs32 <= mabs


@pytest.mark.parametrize("profile,seed", [("plain", 2203), ("sharp", 2203), ("plain", 2213)])
def test_c2_full_depth_packed_native_resolution(profile, seed):
    cfg = S.get_config("c2")
    w, enc = _make(cfg, profile)
    shapes = [(1, 224, 224), (1, 448, 336), (1, 1344, 224)]       # 256, 768, 1536 tokens
    items = S.make_items(cfg, shapes, seed=seed)
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    got, out_dev = G.run_gpu(enc, cfg, items)
    rel, mabs = G.assert_parity(got, ref, f"c2 {profile}")
    G.record_margin("c2 three packed images, full depth", profile, seed, rel, mabs)
    print(f"c2 {profile} full depth seed {seed}:", rel, mabs)
    sl = _out_slices(cfg, items)
    _, alone = G.run_gpu(enc, cfg, [items[1]], sm_budget=74)
    assert torch.equal(alone, out_dev[sl[1]])


def test_c2_largest_image_two_layers():
    cfg = S.get_config("c2", n_layers=2)
    w, enc = _make(cfg, "sharp")
    items = S.make_items(cfg, [(1, 1344, 1344)], seed=2299)       # 9216 tokens
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    got, _ = G.run_gpu(enc, cfg, items)
    rel, mabs = G.assert_parity(got, ref, "c2 largest")
    G.record_margin("c2 1344x1344 (9216 tokens), 2 layers", "sharp", 2299, rel, mabs)
    print("c2 1344x1344, 2 layers:", rel, mabs)


def test_c3_full_depth_short_clip_and_long_clip_two_layers():
    cfg = S.get_config("c3")
    w, enc = _make(cfg)
    items = S.make_items(cfg, [(4, 448, 448)], seed=2301)         # 2048 tokens, full depth
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    got, _ = G.run_gpu(enc, cfg, items)
    rel, mabs = G.assert_parity(got, ref, "c3 full depth")
    G.record_margin("c3 4-frame clip (2048 tokens), full depth", "plain", 2301, rel, mabs)
    print("c3 4-frame clip full depth:", rel, mabs)
    cfg2 = S.get_config("c3", n_layers=2)
    w2, enc2 = _make(cfg2, "sharp")
    items2 = S.make_items(cfg2, [(16, 448, 448)], seed=2302)      # 8192 tokens
    ref2, _, _ = O.encode_microbatch(cfg2, w2, items2)
    got2, _ = G.run_gpu(enc2, cfg2, items2)
    rel, mabs = G.assert_parity(got2, ref2, "c3 16 frames")
    G.record_margin("c3 16-frame clip (8192 tokens), 2 layers", "sharp", 2302, rel, mabs)
    print("c3 16-frame clip, 2 layers:", rel, mabs)


def test_c3_full_depth_sharp_profile_short_clip():
    cfg = S.get_config("c3")
    w, enc = _make(cfg, "sharp")
    items = S.make_items(cfg, [(4, 448, 448)], seed=2311)         # 2048 tokens, full depth
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    got, _ = G.run_gpu(enc, cfg, items)
    rel, mabs = G.assert_parity(got, ref, "c3 sharp full depth")
    G.record_margin("c3 4-frame clip (2048 tokens), full depth", "sharp", 2311, rel, mabs)
    print("c3 sharp 4-frame clip full depth:", rel, mabs)


def test_c3_maximum_clip_against_the_oracle_one_layer():
    """The longest sequence of any workload (64 frames = 32768 tokens, attention over the whole clip), one layer,
    every output row against the oracle."""
    cfg = S.get_config("c3", n_layers=1)
    w, enc = _make(cfg, "sharp")
    items = S.make_items(cfg, [(64, 448, 448)], seed=2304)
    got, _ = G.run_gpu(enc, cfg, items)
    ref = O.encode_item(cfg, w, items[0]).numpy()
    rel, mabs = G.assert_parity(got, ref, "c3 64-frame clip, 1 layer")
    G.record_margin("c3 64-frame clip (32768 tokens), 1 layer", "sharp", 2304, rel, mabs)
    print("c3 64-frame clip, 1 layer:", rel, mabs)


def test_c3_maximum_clip_is_finite_and_packing_invariant():
    """64-frame clip = 32768 tokens (the longest sequence of any workload), one layer, GPU-side properties."""
    cfg = S.get_config("c3", n_layers=1)
    w, enc = _make(cfg)
    items = S.make_items(cfg, [(2, 448, 448), (64, 448, 448)], seed=2303)
    got, out_dev = G.run_gpu(enc, cfg, items)
    assert np.isfinite(got).all()
    _, alone = G.run_gpu(enc, cfg, [items[1]], sm_budget=111)
    assert torch.equal(alone, out_dev[256:])
    # rows of the short clip against the oracle (it shares the batch with the 32768-token clip)
    ref = O.encode_item(cfg, w, items[0]).numpy()
    G.assert_parity(got[:256], ref, "c3 short clip next to the longest")


@pytest.mark.parametrize("profile,seed", [("plain", 2401), ("sharp", 2411)])
def test_c4_full_depth(profile, seed):
    cfg = S.get_config("c4")
    w, enc = _make(cfg, profile)
    items = S.make_items(cfg, [(3000, 128, 1), (1000, 128, 1)], seed=seed)
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    got, out_dev = G.run_gpu(enc, cfg, items)
    rel, mabs = G.assert_parity(got, ref, f"c4 {profile}")
    G.record_margin("c4 mb2 (3000 + 1000 frames), full depth", profile, seed, rel, mabs)
    print(f"c4 {profile} full depth:", rel, mabs)
    for budget in (37, 74, 111):
        _, b = G.run_gpu(enc, cfg, items, sm_budget=budget)
        assert torch.equal(b, out_dev), budget


def test_degenerate_micro_batches():
    """One item; the smallest legal items; many tiny items (64) in one micro-batch."""
    cfg = S.get_config("c2", n_layers=2)
    w, enc = _make(cfg)
    tiny = S.make_items(cfg, [(1, 28, 28)], seed=1)               # 4 tokens -> 1 output row
    ref, _, _ = O.encode_microbatch(cfg, w, tiny)
    got, _ = G.run_gpu(enc, cfg, tiny)
    G.assert_parity(got, ref, "single 2x2-patch image")
    many = S.make_items(cfg, [(1, 28, 28 * (1 + i % 3)) for i in range(64)], seed=2)
    ref, _, _ = O.encode_microbatch(cfg, w, many)
    got, _ = G.run_gpu(enc, cfg, many)
    G.assert_parity(got, ref, "64 tiny images")
    most = S.make_items(cfg, [(1, 28 * (1 + i % 2), 28 * (1 + i % 5)) for i in range(128)], seed=4)   # EAS_MAX_ITEMS
    ref, _, _ = O.encode_microbatch(cfg, w, most)
    got, _ = G.run_gpu(enc, cfg, most)
    G.assert_parity(got, ref, "128 items, the most a call takes")
    import paper_2609_31551_b200 as P
    with pytest.raises(P.EasError) as e:
        G.run_gpu(enc, cfg, S.make_items(cfg, [(1, 28, 28)] * 129, seed=5))
    assert e.value.status == 1 and "n_items" in str(e.value)
    cfg4 = S.get_config("c4", n_layers=1)
    w4, enc4 = _make(cfg4)
    odd = S.make_items(cfg4, [(7, 128, 1), (1, 128, 1), (1001, 128, 1), (6, 128, 1), (129, 128, 1)], seed=6)
    ref, _, _ = O.encode_microbatch(cfg4, w4, odd)                # odd frame counts: ceil(n / 2) tokens each
    assert ref.shape[0] == 4 + 1 + 501 + 3 + 65
    got, _ = G.run_gpu(enc4, cfg4, odd)
    G.assert_parity(got, ref, "audio clips with odd frame counts")
    a = S.make_items(cfg4, [(2, 128, 1)] * 3, seed=3)             # 1 token per clip
    ref, _, _ = O.encode_microbatch(cfg4, w4, a)
    got, _ = G.run_gpu(enc4, cfg4, a)
    G.assert_parity(got, ref, "one-token audio clips")


@pytest.mark.parametrize("name,over,shapes", [
    ("c0", {}, [(1, 224, 224)] * 2),                                       # final LayerNorm writes the output
    ("c1", dict(n_layers=2), [(1, 336, 336)] * 2),                         # the projector's second GEMM writes it
    ("c2", dict(n_layers=2), [(1, 56, 84), (1, 224, 224)]),                # the merger's second GEMM
])
def test_fp32_output_is_the_unrounded_result(name, over, shapes):
    """EAS_OUT_FP32: the same forward pass with the last kernel storing fp32.  Rounding that output to bf16 must give
    the bf16 build's bytes exactly, and the fp32 rows sit closer to the oracle (no 2^-9 output rounding)."""
    import paper_2609_31551_b200 as P
    cfg = S.get_config(name, **over)
    w = S.make_weights(cfg)
    dw = P.weights_to_device(w)
    enc16 = P.Encoder(cfg, dw)
    enc32 = P.Encoder(dict(cfg, out_dtype=1), dw)
    items = S.make_items(cfg, shapes, seed=77)
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    got16, dev16 = G.run_gpu(enc16, cfg, items)
    got32, dev32 = G.run_gpu(enc32, cfg, items)
    assert dev32.dtype == torch.float32 and dev16.dtype == torch.bfloat16
    assert torch.equal(dev32.to(torch.bfloat16), dev16)
    r16, a16 = G.assert_parity(got16, ref, name + " bf16 out")
    r32, a32 = G.assert_parity(got32, ref, name + " fp32 out")
    assert r32 <= r16 * 1.001 and a32 <= a16 * 1.001
    G.record_margin(f"{name} {over or 'full depth'} fp32 output", "plain", 77, r32, a32, bf16_row_rel=r16, bf16_max_abs=a16)
