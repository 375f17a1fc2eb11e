"""The host-side mechanisms driving the real encoder on a small configuration: capacity profiling, SM table from a
latency sweep, and a simulated arrival trace through batcher -> SM lookup -> encode -> router/envelopes."""
import numpy as np
import pytest

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
