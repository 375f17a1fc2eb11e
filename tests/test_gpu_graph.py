"""The launch-overhead path (eas_encoder_set_graph_mode): captured forward passes replayed as CUDA graphs.

Small micro-batches are bound by kernel-launch overhead (Section 3.2), so the library can capture the launches of
a micro-batch once and replay them.  The kernels and their arguments are those of the ordinary path: the results
must be bit-identical, for the capturing call, for every replay, and after the input VALUES change behind the same
pointers.  A different shape, pointer or SM budget is a different micro-batch and gets its own capture."""
import numpy as np
import pytest
import torch

import eas_synth as S
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def _setup(cfg_name, shapes, seed):
    import paper_2609_31551_b200 as P
    cfg = S.get_config(cfg_name)
    enc = P.Encoder(cfg, P.weights_to_device(S.make_weights(cfg)))
    items = S.make_items(cfg, shapes, seed=seed)
    data, offsets = P.pack_items(items)
    cu = G.cu_seqlens_of(cfg, items)
    return P, cfg, enc, items, data, offsets, cu


@pytest.mark.parametrize("cfg_name,shapes", [("c0", [(1, 224, 224)] * 2), ("c2", [(1, 224, 280), (1, 336, 224)]),
                                             ("c4", [(3000, 128, 1)])])
def test_graph_replay_is_bit_identical(cfg_name, shapes):
    P, cfg, enc, items, data, offsets, cu = _setup(cfg_name, shapes, seed=21)
    cu_dev = torch.from_numpy(cu).cuda()
    ref = enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev)
    enc.status()
    launches = enc.last_launch_count()
    ws = torch.empty(enc.workspace_bytes(int(cu[-1]), len(shapes)) + 1024, dtype=torch.uint8, device="cuda")
    out = torch.zeros_like(ref)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    enc.set_graph_mode(True)
    with torch.cuda.stream(side):
        for it in range(3):                                   # capture + launch, then two replays
            out.zero_()
            enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, out=out, workspace=ws, stream=side)
            enc.status(side)
            assert torch.equal(out, ref), f"call {it} in graph mode differs from the ordinary path"
            assert enc.last_launch_count() == launches
        st = enc.graph_stats()
        assert st == {"hits": 2, "captures": 1, "cached": 1}
        # new values behind the same pointers: the replay must read them
        items2 = S.make_items(cfg, shapes, seed=22)
        data2, _ = P.pack_items(items2)
        data.copy_(data2)
        enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, out=out, workspace=ws, stream=side)
        enc.status(side)
        assert enc.graph_stats()["hits"] == 3
    enc.set_graph_mode(False)
    assert enc.graph_stats()["cached"] == 0
    ref2 = enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev)
    enc.status()
    assert torch.equal(out, ref2)
    assert not torch.equal(ref, ref2)


def test_graph_mode_follows_the_normalisation_mode():
    """A captured forward pass belongs to the normalisation mode it was captured in: switching
    eas_encoder_set_norm_fold between calls must not replay the other mode's launches."""
    P, cfg, enc, items, data, offsets, cu = _setup("c0", [(1, 224, 224)] * 2, seed=31)
    shapes = [(1, 224, 224)] * 2
    cu_dev = torch.from_numpy(cu).cuda()
    plain = enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev).clone()
    enc.set_norm_fold(True)
    folded = enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev).clone()
    n_folded = enc.last_launch_count()
    enc.set_norm_fold(False)
    enc.status()
    assert not torch.equal(plain, folded)                      # two roundings of the same values
    ws = torch.empty(enc.workspace_bytes(int(cu[-1]), 2) + 1024, dtype=torch.uint8, device="cuda")
    out = torch.zeros_like(plain)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    enc.set_graph_mode(True)
    with torch.cuda.stream(side):
        for fold, want in ((False, plain), (True, folded), (False, plain), (True, folded)):
            enc.set_norm_fold(fold)
            out.zero_()
            enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, out=out, workspace=ws, stream=side)
            enc.status(side)
            assert torch.equal(out, want), fold
            if fold:
                assert enc.last_launch_count() == n_folded
    assert enc.graph_stats() == {"hits": 2, "captures": 2, "cached": 2}
    enc.set_graph_mode(False)


def test_graph_cache_keys_on_shape_budget_and_pointers():
    P, cfg, enc, items, data, offsets, cu = _setup("c0", [(1, 224, 224)] * 3, seed=5)
    cu_dev = torch.from_numpy(cu).cuda()
    shapes = [(1, 224, 224)] * 3
    ws = torch.empty(enc.workspace_bytes(int(cu[-1]), 3) + 1024, dtype=torch.uint8, device="cuda")
    out_a = torch.empty((int(cu[-1]), cfg["d_out"]), dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty_like(out_a)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    enc.set_graph_mode(True)
    with torch.cuda.stream(side):
        enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, out=out_a, workspace=ws, stream=side)
        enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, out=out_b, workspace=ws, stream=side)   # other output
        enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, out=out_a, workspace=ws, stream=side,
                              sm_budget=37)                                                                          # other budget
        cu2 = cu[:3].copy()
        enc.encode_microbatch(data, shapes[:2], offsets[:2], cu2, cu_seqlens_dev=cu_dev[:3], out=out_b[: int(cu2[-1])],
                              workspace=ws, stream=side)                                                             # other shape
        enc.status(side)
        assert enc.graph_stats() == {"hits": 0, "captures": 4, "cached": 4}
        enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, out=out_a, workspace=ws, stream=side)
        enc.status(side)
        assert enc.graph_stats()["hits"] == 1
    enc.set_graph_mode(False)
    ref = enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev)
    enc.status()
    assert torch.equal(out_a, ref)


def test_graph_mode_on_the_default_stream_runs_uncaptured():
    P, cfg, enc, items, data, offsets, cu = _setup("c0", [(1, 224, 224)], seed=6)
    enc.set_graph_mode(True)
    a = enc.encode_microbatch(data, [(1, 224, 224)], offsets, cu)
    enc.status()
    assert enc.graph_stats() == {"hits": 0, "captures": 0, "cached": 0}
    enc.set_graph_mode(False)
    b = enc.encode_microbatch(data, [(1, 224, 224)], offsets, cu)
    enc.status()
    assert torch.equal(a, b)


def test_invalid_input_in_graph_mode_reports_the_ordinary_error_and_leaves_the_stream_usable():
    P, cfg, enc, items, data, offsets, cu = _setup("c0", [(1, 224, 224)], seed=7)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    enc.set_graph_mode(True)
    bad_cu = cu.copy()
    bad_cu[-1] += 1                                           # token count that does not match the shape
    with torch.cuda.stream(side):
        with pytest.raises(P.EasError):
            enc.encode_microbatch(data, [(1, 224, 224)], offsets, bad_cu, stream=side)
        good = enc.encode_microbatch(data, [(1, 224, 224)], offsets, cu, stream=side)
        enc.status(side)
    assert np.isfinite(good.float().cpu().numpy()).all()
    assert enc.graph_stats()["captures"] == 1


def test_graph_replay_with_split_k_is_bit_identical():
    """The two halves of the latency path together: split K (partial sums added by the following normalisation) inside
    captured and replayed forward passes, and through the allocation-free entry point."""
    shapes = [(1, 336, 336)]
    P, cfg, enc, items, data, offsets, cu = _setup("c1", shapes, seed=23)
    cu_dev = torch.from_numpy(cu).cuda()
    plain = enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev)
    enc.status()
    enc.set_split_k(True)
    ref = enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev)
    enc.status()
    # another summation order: a few bf16 last-place differences after 24 layers, nothing more
    assert not torch.equal(ref, plain)
    assert float((ref.float() - plain.float()).abs().max()) <= 2.0 ** -6 * float(plain.float().abs().max())
    ws = torch.empty(enc.workspace_bytes(int(cu[-1]), 1) + 1024, dtype=torch.uint8, device="cuda")
    out = torch.zeros_like(ref)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    enc.set_graph_mode(True)
    with torch.cuda.stream(side):
        for it in range(3):
            out.zero_()
            enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev, out=out, workspace=ws, stream=side)
            enc.status(side)
            assert torch.equal(out, ref), f"call {it}"
        assert enc.graph_stats()["hits"] == 2
    enc.set_graph_mode(False)
    out.zero_()
    enc.encode_microbatch_static(data, shapes, offsets, cu, cu_dev, out)
    enc.status()
    assert torch.equal(out, ref)
