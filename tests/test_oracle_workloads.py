"""The oracle run over the tiny synthetic stack (config 1) and structure checks of the larger workloads."""
import numpy as np

from oracle import milora_oracle as O
from oracle import reference_run as R
from synth import get_workload, tensor_seed
from synth.workloads import decode_sweep_workload


def test_workload_structure():
    c2 = get_workload("c2")
    assert c2.n_requests == 64 and c2.dims(6) == (11008, 4096) and c2.rank == 16
    c3 = get_workload("c3")
    assert c3.n_requests == 32 and c3.prompt_len.min() >= 128 and c3.prompt_len.max() <= 2048
    assert c3.request_tenant.min() >= 0 and c3.request_tenant.max() < 32
    c4 = get_workload("c4")
    distinct = len(np.unique(c4.request_tenant))
    assert 60 <= distinct <= 160                       # about 110 expected under Zipf(1.1) over 1000
    assert np.bincount(c4.request_tenant).max() / 256 > 0.08
    c5 = get_workload("c5")
    assert len(c5.prefill_ids) == 8 and len(c5.decode_ids) == 192 and c5.d_kv == 1024
    assert decode_sweep_workload(16).n_tenants == 16
    # seeds: distinct tensors get distinct seeds, same ids the same seed
    assert tensor_seed(0, 1, 2, 3) == tensor_seed(0, 1, 2, 3) != tensor_seed(0, 1, 3, 2)
    A1, _ = c2.adapter(3, 0, 4)
    A2, _ = c2.adapter(3, 0, 4)
    assert A1.shape == (4096, 16) and bool((A1 == A2).all())


def test_config1_full_stack_invariants():
    """Config 1 end to end in the oracle: routes from prompts, prefill apply, then 4 decode steps
    that reuse the table; the factored output equals x (W + s A B) on selected modules and x W elsewhere."""
    w = get_workload("c1")
    table, margins = R.full_route_table(w)
    assert table.shape == (4, 2) and table.min() >= 0 and table.max() < 7 and margins.min() >= 0
    frozen = table.copy()
    T = int(w.prompt_len.sum())
    token_slot = np.repeat(np.arange(4), 16)
    for layer in range(w.n_layers):
        for m in range(7):
            x = w.module_input(layer, m, T, tag=0)
            W = R.to_f64(w.base_weight(layer, m))
            yb = O.base_projection(R.to_f64(x), W)
            y = R.apply_site(w, layer, m, x, yb, token_slot, table[:, layer])
            for t in range(0, T, 5):
                slot = token_slot[t]
                if table[slot, layer] == m:
                    A, B = w.adapter(int(w.request_tenant[slot]), layer, m)
                    Wm = O.merged_weight(W, R.to_f64(A), R.to_f64(B), w.scale)
                    np.testing.assert_allclose(y[t], R.to_f64(x)[t] @ Wm, rtol=1e-11, atol=1e-12)
                else:
                    assert np.array_equal(y[t], yb[t])
    # decode: one token per request per step, the table is only read
    for step in range(w.decode_steps):
        for layer in range(w.n_layers):
            m = int(table[0, layer])
            x = w.module_input(layer, m, 4, tag=100 + step)
            yb = w.base_output(layer, m, 4, tag=100 + step)
            y = R.apply_site(w, layer, m, x, yb, np.arange(4), table[:, layer])
            changed = [not np.array_equal(y[t], R.to_f64(yb)[t]) for t in range(4)]
            assert changed == [bool(table[t, layer] == m) for t in range(4)]
        assert np.array_equal(table, frozen)
    # grouping of the prefill batch: each prompt is one contiguous run in its bucket
    g = R.group_layer(w, token_slot, table[:, 0])
    assert g["n_excluded"] == 0 and len(g["perm"]) == T
    assert sorted(g["perm"].tolist()) == list(range(T))
