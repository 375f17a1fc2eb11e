"""Whole-encoder parity: the CUDA path through the C ABI against the fp64 oracle, element by element
on the same seeded inputs, for all five workload families; plus the determinism properties."""
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
    enc = P.Encoder(cfg, P.weights_to_device(w))
    return w, enc


CASES = {
    # name: (config overrides, item shapes)
    "c0_full": ("c0", {}, [(1, 224, 224)] * 4),
    "c1_2layers": ("c1", dict(n_layers=2), [(1, 336, 336)] * 3),
    "c2_2layers": ("c2", dict(n_layers=2), [(1, 56, 84), (1, 224, 224), (1, 28, 28), (1, 140, 364)]),
    "c3_2layers": ("c3", dict(n_layers=2), [(4, 56, 56), (2, 112, 84)]),
    "c4_2layers": ("c4", dict(n_layers=2, max_pos=1500), [(200, 128, 1), (600, 128, 1), (2, 128, 1)]),
}


@pytest.mark.parametrize("case", list(CASES))
@pytest.mark.parametrize("profile", ["plain", "sharp"])
def test_encoder_parity_small(case, profile):
    name, over, shapes = CASES[case]
    cfg = S.get_config(name, **over)
    w, enc = _make(cfg, profile)
    items = S.make_items(cfg, shapes, seed=2000 + len(shapes))
    ref, cu, _ = O.encode_microbatch(cfg, w, items)
    got, _ = G.run_gpu(enc, cfg, items)
    rel, mabs = G.assert_parity(got, ref, case)
    print(f"{case}/{profile}: row-rel {rel:.3e} max-abs {mabs:.3e}")


@pytest.mark.parametrize("case", ["c0_full", "c1_2layers", "c2_2layers", "c3_2layers", "c4_2layers"])
def test_folded_normalisation_parity_and_determinism(case):
    """eas_encoder_set_norm_fold: the blocks' normalisations applied inside the GEMMs around them (no normalisation
    kernel inside a block).  Same tolerance against the oracle as the default path, the same bytes for every SM
    budget and for an item alone or packed, fewer launches, and switching it off restores the default path's bytes."""
    name, over, shapes = CASES[case]
    cfg = S.get_config(name, **over)
    w, enc = _make(cfg, "sharp")
    items = S.make_items(cfg, shapes, seed=2050 + len(shapes))
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    plain, plain_dev = G.run_gpu(enc, cfg, items)
    n_plain = enc.last_launch_count()
    enc.set_norm_fold(True)
    got, dev = G.run_gpu(enc, cfg, items)
    rel, mabs = G.assert_parity(got, ref, case + " folded")
    G.record_margin(f"{case}, folded normalisation", "sharp", 2050 + len(shapes), rel, mabs)
    assert enc.last_launch_count() == n_plain - 2 * cfg["n_layers"] + 1
    assert np.abs(got - plain).max() <= G.ABS_TOL          # two roundings of the same values
    for budget in (3, 37, 111):
        _, again = G.run_gpu(enc, cfg, items, sm_budget=budget)
        assert torch.equal(dev, again), budget
    sl0 = S.out_tokens_per_item(cfg, G.item_shape(cfg, items[0]))
    _, alone = G.run_gpu(enc, cfg, [items[0]])
    assert torch.equal(alone, dev[:sl0])
    enc.set_norm_fold(False)
    _, back = G.run_gpu(enc, cfg, items)
    assert torch.equal(back, plain_dev)


def test_c0_bit_stability_and_packing_invariance():
    cfg = S.get_config("c0")
    w, enc = _make(cfg)
    items = S.make_items(cfg, [(1, 224, 224)] * 4, seed=2002)
    _, a = G.run_gpu(enc, cfg, items)
    _, b = G.run_gpu(enc, cfg, items)
    assert torch.equal(a, b)                                  # same input twice -> same bytes
    for budget in (37, 74, 111):
        _, c = G.run_gpu(enc, cfg, items, sm_budget=budget)
        assert torch.equal(a, c), budget                      # any sm_budget -> same bytes
    _, alone = G.run_gpu(enc, cfg, [items[2]])
    assert torch.equal(a[2 * 196:3 * 196], alone)             # item alone == item packed


def test_invalid_arguments_are_rejected_before_launch():
    import paper_2609_31551_b200 as P
    cfg = S.get_config("c0")
    w, enc = _make(cfg)
    items = S.make_items(cfg, [(1, 224, 224)], seed=1)
    data, offs = P.pack_items(items)
    with pytest.raises(P.EasError) as e:
        enc.encode_microbatch(data, [(1, 224, 224)], offs, [0, 195])
    assert e.value.status == 1
    with pytest.raises(P.EasError) as e:
        enc.encode_microbatch(data, [(1, 224, 230)], offs, [0, 196])
    assert e.value.status == 1
    with pytest.raises(P.EasError) as e:
        enc.encode_microbatch(data, [(1, 224, 224)], offs, [0, 196], sm_budget=100000)
    assert e.value.status == 1
    small = torch.empty(1024, dtype=torch.uint8, device="cuda")
    with pytest.raises(P.EasError) as e:
        enc.encode_microbatch(data, [(1, 224, 224)], offs, [0, 196], workspace=small)
    assert e.value.status == 3
    # a device cu_seqlens that differs from the host copy is reported by the device check
    bad = torch.tensor([0, 100], dtype=torch.int32, device="cuda")
    enc.encode_microbatch(data, [(1, 224, 224)], offs, [0, 196], cu_seqlens_dev=bad)
    with pytest.raises(P.EasError) as e:
        enc.status()
    assert e.value.status == 7


def test_split_k_is_deterministic_budget_independent_and_optional():
    """Latency path: small micro-batches split the K loop of the residual GEMMs (eas_encoder_set_split_k, off by default).  The result must not depend
    on sm_budget or on the run, must stay within the oracle tolerance, and with the mode off an item's embeddings are
    bit-identical whatever it is packed with."""
    cfg = S.get_config("c1", n_layers=3)
    w, enc = _make(cfg)
    shapes = [(1, 336, 336)] * 2                                  # 1154 tokens: fc2 (K = 4096) splits, proj does not
    items = S.make_items(cfg, shapes, seed=2100)
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    enc.set_split_k(True)
    got, a = G.run_gpu(enc, cfg, items)
    G.assert_parity(got, ref, "split K")
    _, b = G.run_gpu(enc, cfg, items)
    assert torch.equal(a, b)
    for budget in (20, 37, 111):
        _, c = G.run_gpu(enc, cfg, items, sm_budget=budget)
        assert torch.equal(a, c), budget
    enc.set_split_k(False)
    got_off, off = G.run_gpu(enc, cfg, items)
    G.assert_parity(got_off, ref, "split K off")
    assert not torch.equal(a, off)                                # the mode did something (another summation order)
    assert float((a.float() - off.float()).abs().max()) < 0.05
    rows = off.shape[0] // 2
    _, alone = G.run_gpu(enc, cfg, [items[1]])
    assert torch.equal(off[rows:], alone)                         # off: item alone == item packed
    big = items + S.make_items(cfg, [(1, 336, 336)] * 4, seed=2101)    # 3462 tokens: no split either way
    _, packed = G.run_gpu(enc, cfg, big)
    assert torch.equal(packed[rows:2 * rows], alone)
    enc.set_split_k(True)
    _, packed_on = G.run_gpu(enc, cfg, big)
    assert torch.equal(packed_on, packed)


@pytest.mark.parametrize("case", ["c1_2layers", "c2_2layers", "c3_2layers", "c4_2layers"])
def test_split_k_parity_all_families(case):
    """The small cases of every family with split K on (RMSNorm and LayerNorm, SwiGLU and GELU MLPs, d = 1024 and 1280)."""
    name, over, shapes = CASES[case]
    cfg = S.get_config(name, **over)
    w, enc = _make(cfg, "sharp")
    enc.set_split_k(True)
    items = S.make_items(cfg, shapes, seed=2300 + len(shapes))
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    got, dev = G.run_gpu(enc, cfg, items)
    G.assert_parity(got, ref, case + " split K")
    _, again = G.run_gpu(enc, cfg, items, sm_budget=37)
    assert torch.equal(dev, again)


EMBED_CASES = {
    "c0": [(1, 224, 224), (1, 32, 48)],
    "c1": [(1, 336, 336)] * 2,
    "c2": [(1, 56, 84), (1, 364, 140), (1, 28, 28), (1, 224, 1344)],
    "c3": [(4, 56, 56), (2, 112, 84), (6, 28, 28)],
}


@pytest.mark.parametrize("name", list(EMBED_CASES))
def test_fused_patch_embedding_alone(name):
    """An encoder without transformer blocks is the embedding (patch gather fused into the GEMM, bias, position
    rows, CLS) followed by the connector: the gather's index arithmetic for images, clips, raster and
    merge-group-major patch order, several items of different sizes and a ragged last tile, against the oracle."""
    over = dict(n_layers=0)
    if name in ("c0", "c1"):
        over["max_pos"] = 600
    cfg = S.get_config(name, **over)
    if name == "c0":
        cfg = dict(cfg, out_dtype=1)           # final LayerNorm in fp32: nothing but the embedding's own rounding is left
    w, enc = _make(cfg)
    shapes = EMBED_CASES[name]
    items = S.make_items(cfg, shapes, seed=4100)
    ref, _, _ = O.encode_microbatch(cfg, w, items)
    got, dev = G.run_gpu(enc, cfg, items)
    rel, mabs = G.assert_parity(got, ref, f"{name} embedding only")
    if name == "c0":
        assert rel < 2e-3, rel                 # bf16 operands with fp32 accumulation: far inside the tolerance
    for budget in (1, 5, 37):
        _, b = G.run_gpu(enc, cfg, items, sm_budget=budget)
        assert torch.equal(b, dev), budget


def test_fused_patch_embedding_with_odd_item_offsets():
    """Item offsets that are odd element counts break the 4-byte alignment of pixel pairs: the gather then loads
    single elements.  Same values, same accumulation order: the result must be the same bytes."""
    import paper_2609_31551_b200 as P
    cfg = S.get_config("c2", n_layers=1)
    w, enc = _make(cfg)
    shapes = [(1, 56, 84), (1, 28, 140)]
    items = S.make_items(cfg, shapes, seed=4200)
    _, want = G.run_gpu(enc, cfg, items)
    flat = [torch.from_numpy(np.ascontiguousarray(it).reshape(-1)).to(torch.bfloat16) for it in items]
    offsets = [1, 1 + flat[0].numel() + 2]     # 1 and an odd number: both items start on odd elements
    buf = torch.zeros(offsets[1] + flat[1].numel() + 8, dtype=torch.bfloat16)
    for f, o in zip(flat, offsets):
        buf[o:o + f.numel()] = f
    cu = G.cu_seqlens_of(cfg, items)
    out = enc.encode_microbatch(buf.cuda(), shapes, offsets, cu)
    enc.status()
    assert torch.equal(out, want)
