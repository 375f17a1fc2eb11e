"""The allocation-free entry point (eas_encode_microbatch_static) against the ordinary one and the oracle.

Some callers of the encoder cannot allocate device memory: a worker that shares its GPU with a neighbour
that already owns the rest of HBM, or a serving loop where an allocation may stall the device.  For them the
library carries its own scratch array.  These tests call that entry point through the C ABI twice in a row (the
array keeps the first call's contents, so the second call shows that nothing stale is read).  Both entry points
run the same kernels in the same order, so their results must be the same BYTES, not merely close; and each
result is also held against the CPU oracle with the tolerance of the other parity tests.  One case per encoder
family, so that every scratch region (patch operand, row maps, rotary table, padded mel / convolution rows) is
covered.  A micro-batch too large for the built-in scratch must be refused with a clear error.
Collected last on purpose."""
import numpy as np
import pytest
import torch

import eas_synth as S
from oracle import encoder_oracle as O
from tests import gpu_util as G

pytestmark = pytest.mark.gpu

CASES = {
    # family: (config, overrides, [first micro-batch, second micro-batch])
    "vit_table": ("c0", {}, [[(1, 224, 224)] * 3, [(1, 224, 224)] * 2]),
    "vit_rope_merger": ("c2", dict(n_layers=2), [[(1, 224, 224), (1, 56, 84)], [(1, 28, 28), (1, 140, 364), (1, 56, 56)]]),
    "audio_conv": ("c4", dict(n_layers=1), [[(200, 128, 1), (7, 128, 1)], [(2, 128, 1), (600, 128, 1), (64, 128, 1)]]),
}


@pytest.mark.parametrize("family", list(CASES))
def test_static_scratch_entry_point_matches_and_repeats(family):
    import paper_2609_31551_b200 as P
    name, over, batches = CASES[family]
    cfg = S.get_config(name, **over)
    w = S.make_weights(cfg)
    enc = P.Encoder(cfg, P.weights_to_device(w))
    runs = []
    for k, shapes in enumerate(batches):            # two different micro-batches, back to back on the same scratch
        items = S.make_items(cfg, shapes, seed=11 + k)
        data, offsets = P.pack_items(items)
        cu = G.cu_seqlens_of(cfg, items)
        cu_dev = torch.from_numpy(cu).cuda()
        assert enc.workspace_bytes(int(cu[-1]), len(shapes)) < (32 << 20) - 1024
        want = enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev)
        enc.status()
        out = torch.full_like(want, float("nan"))
        enc.encode_microbatch_static(data, shapes, offsets, cu, cu_dev, out)
        enc.status()
        runs.append((items, out, want))
    for items, out, want in runs:
        assert torch.equal(out, want), "static-scratch entry point differs from the workspace entry point"
        ref, _, _ = O.encode_microbatch(cfg, w, items)
        G.assert_parity(out.double().cpu().numpy(), ref, f"static-scratch entry point vs oracle ({family})")


def test_static_scratch_rejects_a_micro_batch_that_does_not_fit():
    import paper_2609_31551_b200 as P
    cfg = S.get_config("c0")
    w = S.make_weights(cfg)
    enc = P.Encoder(cfg, P.weights_to_device(w))
    n = 64                                         # 64 images need far more than the built-in scratch
    shapes = [(1, 224, 224)] * n
    cu = np.arange(n + 1, dtype=np.int32) * 196
    assert enc.workspace_bytes(int(cu[-1]), n) > (32 << 20)
    data = torch.zeros(n * 3 * 224 * 224, dtype=torch.bfloat16, device="cuda")
    offsets = [i * 3 * 224 * 224 for i in range(n)]
    out = torch.empty((n * 196, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(P.EasError) as e:
        enc.encode_microbatch_static(data, shapes, offsets, cu, torch.from_numpy(cu).cuda(), out)
    assert e.value.status == 3 and "built-in scratch" in str(e.value)
