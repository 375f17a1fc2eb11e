"""The host-side mechanisms driving the real encoder on a small configuration: capacity profiling, SM table from a
latency sweep, and a simulated arrival trace through batcher -> SM lookup -> encode -> router/envelopes."""
import numpy as np
import pytest
import torch

import eas_synth as S

pytestmark = pytest.mark.gpu


def test_profiling_and_simulated_serving_on_c0():
    from paper_2609_31551_b200 import serve_sim as SS
    w = SS.EncodeWorker("c0")
    ce, b_sat, curve = SS.profile_encode_capacity(w, max_batch=32)
    assert ce > 0 and 1 <= b_sat <= 32
    assert [b for b, _ in curve] == [2 ** i for i in range(len(curve))]          # doubling
    table, sm_counts, lat, excl = SS.build_sm_table(w, 148, [1, 2, 4, 8])
    assert sm_counts == sorted(sm_counts) and table.n_levels == 5
    # (the measured latencies of this tiny model are launch-bound and noisy, so only the table's structure is checked)
    assert all(0 <= table.max_batch[i] <= 8 for i in range(5))
    from paper_2609_31551_b200 import serving as SV
    assert all(SV.sm_table_lookup(table, b) in sm_counts for b in (1, 2, 4, 8, 9))
    res = SS.simulate(w, rate=2000.0, n_requests=400, batch_bound=8, offload=0.7, table=table)
    assert res["requests"] == 400 and 1.0 <= res["mean_batch"] <= 8.0
    assert abs(res["remote_fraction"] - 0.7) < 0.01                               # the router holds the ratio
    assert res["transfers"] <= 3 * res["dispatches"]                              # at most one envelope per destination
    assert res["encode_latency_p99_s"] < 1.0 + 0.5                                # the age cap bounds the wait


def test_grouped_item_order_writes_each_request_into_its_envelope():
    """Section 3.3: with the requests listed in eas_envelope_order's order, the forward pass itself writes every
    request's embeddings into its destination's contiguous envelope, bit-identical to encoding in arrival order."""
    import paper_2609_31551_b200 as P
    from paper_2609_31551_b200 import serving as SV
    cfg = S.get_config("c2")
    enc = P.Encoder(cfg, P.weights_to_device(S.make_weights(cfg)))
    shapes = [(1, 224, 280), (1, 336, 224), (1, 224, 224), (1, 280, 280), (1, 224, 336)]
    dest = [1, 0, 2, 0, 1]
    items = S.make_items(cfg, shapes, seed=31)
    data, offsets = P.pack_items(items)
    tok = [S.tokens_per_item(cfg, s) for s in shapes]
    rows = [S.out_tokens_per_item(cfg, s) for s in shapes]
    cu = np.concatenate([[0], np.cumsum(tok)]).astype(np.int32)
    ref = enc.encode_microbatch(data, shapes, offsets, cu)
    enc.status()
    order, first = SV.envelope_order(dest, rows, 3)
    offs, totals = SV.envelope_plan(dest, rows, 3)
    g_shapes = [shapes[i] for i in order]
    g_offsets = [offsets[i] for i in order]             # the items stay where they are in `data`: only the listing changes
    g_cu = np.concatenate([[0], np.cumsum([tok[i] for i in order])]).astype(np.int32)
    out = enc.encode_microbatch(data, g_shapes, g_offsets, g_cu)
    enc.status()
    ref_start = np.concatenate([[0], np.cumsum(rows)])
    for i in range(len(shapes)):
        lo = first[dest[i]] + offs[i]
        assert torch.equal(out[lo: lo + rows[i]], ref[ref_start[i]: ref_start[i] + rows[i]]), f"request {i}"
    assert sum(totals) == out.shape[0]


def test_coresidency_measurement_runs_and_reports_sane_numbers():
    """Encoder on a share of the SMs beside a GEMM stream on the rest (Section 3.4): structural checks only, the
    figures themselves are machine-dependent."""
    from paper_2609_31551_b200 import coresidency as CR
    rows = CR.measure("c0", 4, levels=(0.5,), reps=3, neighbour_shape=(2048, 2048, 2048))
    assert len(rows) == 1
    r = rows[0]
    assert r["sm_encode"] + r["sm_neighbour"] == torch.cuda.get_device_properties(0).multi_processor_count
    for k in ("encode_ms_exclusive", "encode_ms_alone", "encode_ms_beside_neighbour", "neighbour_tflops_alone",
              "neighbour_tflops_beside_encoder"):
        assert np.isfinite(r[k]) and r[k] > 0
    assert 0.5 < r["inflation"] < 20
    g = CR.measure("c0", 4, levels=(0.5,), reps=3, neighbour_shape=(2048, 2048, 2048), partition="green")[0]
    assert g["partition"] == "green" and g["sm_encode"] >= 74 and g["sm_neighbour"] > 0
    assert np.isfinite(g["inflation"]) and 0.5 < g["inflation"] < 20


def test_sm_partition_splits_the_device_and_the_encoder_runs_on_its_side():
    """Section 3.4: two disjoint SM sets with a stream each.  The encoder on side 0 gives the bits of an ordinary call
    (the result does not depend on which or how many SMs run it), with a neighbour busy on side 1 meanwhile."""
    import paper_2609_31551_b200 as P
    total = torch.cuda.get_device_properties(0).multi_processor_count
    part = P.SmPartition(44)
    n0, n1 = part.sm_count(0), part.sm_count(1)
    assert n0 >= 44 and n1 > 0 and n0 + n1 <= total
    assert part.sm_count(2) == 0
    cfg = S.get_config("c0")
    enc = P.Encoder(cfg, P.weights_to_device(S.make_weights(cfg)))
    shapes = [(1, 224, 224)] * 3
    items = S.make_items(cfg, shapes, seed=41)
    data, offsets = P.pack_items(items)
    cu = np.concatenate([[0], np.cumsum([S.tokens_per_item(cfg, s) for s in shapes])]).astype(np.int32)
    ref = enc.encode_microbatch(data, shapes, offsets, cu)
    enc.status()
    torch.cuda.synchronize()
    a = (torch.randn(2048, 2048, device="cuda") * 0.05).bfloat16()
    bias = torch.zeros(2048, dtype=torch.bfloat16, device="cuda")
    s0, s1 = part.stream(0), part.stream(1)
    nb_out = None
    for _ in range(8):                                     # the neighbour: GEMMs on side 1's SMs
        nb_out, nb_status = P.kernel_gemm(a, a, bias, sm_budget=n1, stream=s1)
    with torch.cuda.stream(s0):
        out = enc.encode_microbatch(data, shapes, offsets, cu, sm_budget=n0, stream=s0)
        enc.status(s0)
        # a grid larger than the side still runs there (its CTAs queue for the side's SMs)
        out_big = enc.encode_microbatch(data, shapes, offsets, cu, sm_budget=total, stream=s0)
        enc.status(s0)
    torch.cuda.synchronize()
    assert torch.equal(out, ref) and torch.equal(out_big, ref)
    assert int(nb_status[0]) == 0
    want = (a.double() @ a.double().T)[:4, :4].cpu().numpy()
    assert np.allclose(nb_out[:4, :4].double().cpu().numpy(), want, rtol=2e-2, atol=2e-2)
    part.close()
    with pytest.raises(P.EasError):
        P.SmPartition(0)
    with pytest.raises(P.EasError):
        P.SmPartition(total)
