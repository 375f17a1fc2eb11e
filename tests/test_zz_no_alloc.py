"""The allocation-free entry point (eas_encode_microbatch_static) against the ordinary one.

Some callers of the encoder cannot allocate device memory: a worker that shares its GPU with a neighbour
that already owns the rest of HBM, or a serving loop where an allocation may stall the device.  For them the
library carries its own scratch array.  This test calls that entry point through the C ABI twice in a row (the
array keeps the first call's contents, so the second call shows that nothing stale is read) and compares both
results with eas_encode_microbatch on a caller-allocated workspace.  It also checks that a micro-batch too large
for the built-in scratch is refused with a clear error.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import eas_synth as S
from tests import gpu_util as G

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_and_repeats():
    import paper_2609_31551_b200 as P
    cfg = S.get_config("c0")
    w = S.make_weights(cfg)
    enc = P.Encoder(cfg, P.weights_to_device(w))
    outs = []
    for seed, n in ((11, 3), (12, 2)):            # two different micro-batches, back to back
        shapes = [(1, 224, 224)] * n
        items = S.make_items(cfg, shapes, seed=seed)
        data, offsets = P.pack_items(items)
        cu = G.cu_seqlens_of(cfg, items)
        cu_dev = torch.from_numpy(cu).cuda()
        ref = enc.encode_microbatch(data, shapes, offsets, cu, cu_seqlens_dev=cu_dev)
        enc.status()
        out = torch.zeros_like(ref)
        enc.encode_microbatch_static(data, shapes, offsets, cu, cu_dev, out)
        enc.status()
        outs.append((out, ref))
    for out, ref in outs:
        got, want = out.double().cpu().numpy(), ref.double().cpu().numpy()
        assert np.isfinite(got).all()
        G.assert_parity(got, want, "static-scratch entry point vs workspace entry point")


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
