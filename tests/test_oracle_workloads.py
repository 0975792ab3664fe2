"""The oracle run over the tiny synthetic stack (config 1) and structure checks of the larger workloads."""
import numpy as np
import torch

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


class _HandWorkload:
    """Just enough of a workload for reference_run.route_requests, with hand-built tensors that differ per
    tenant, layer and request, so that a mix-up of any index changes the logits."""
    n_tenants, n_layers, d = 3, 2, 6
    request_tenant = np.array([2, 0, 1, 2], dtype=np.int32)

    def _t(self, *ids, shape):
        base = sum((i + 1) * f for i, f in zip(ids, (0.37, 0.11, 0.05)))
        n = int(np.prod(shape))
        return torch.tensor(np.sin(base + 0.7 * np.arange(n)).reshape(shape), dtype=torch.float64)

    def hidden(self, layer, request):
        return self._t(layer, request, 5, shape=(3 + request, self.d))

    def router(self, tenant, layer):
        return self._t(tenant, layer, 1, shape=(self.d, 7))

    def w_sa(self, tenant, layer):
        return self._t(tenant, layer, 2, shape=(self.d,))

    def router_bias(self, tenant, layer):
        return self._t(tenant, layer, 3, shape=(7,))

    def rational_coef(self, tenant, layer):
        c = self._t(tenant, layer, 4, shape=(12,)) * 0.3
        return c[:7].clone(), c[7:].clone()


def test_route_requests_hands_the_right_tensors_to_the_oracle():
    """The variant branches of reference_run.route_requests (self-attention pooling, rational activation, bias,
    top-k table) against direct calls of the oracle with the tensors picked by hand for each request's tenant and
    the layer; picking another tenant's or layer's tensor changes the logits, so the comparison has power."""
    w = _HandWorkload()
    layer, ids, k = 1, [3, 0, 2], 3
    table = np.full((4, 2), -1, dtype=np.int32)
    topk = np.full((4, 2, k), -1, dtype=np.int32)
    logits, margins = R.route_requests(w, layer, ids, table, pooler=O.POOL_SELFATTN, activation=O.ACT_RATIONAL,
                                       with_bias=True, k=k, topk_table=topk)
    for p, i in enumerate(ids):
        t = int(w.request_tenant[i])
        a, b = w.rational_coef(t, layer)
        want = O.route_prompt(w.hidden(layer, i).numpy(), w.router(t, layer).numpy(), pooler=O.POOL_SELFATTN,
                              activation=O.ACT_RATIONAL, k=k, w_sa=w.w_sa(t, layer).numpy(), coef_a=a.numpy(),
                              coef_b=b.numpy(), bias=w.router_bias(t, layer).numpy())
        assert np.array_equal(logits[p], want["logits"]) and margins[p] == want["margin"]
        assert table[i, layer] == want["route"] and topk[i, layer].tolist() == list(want["topk"])
        assert topk[i, layer, 0] == table[i, layer]
        # each ingredient matters: another tenant's query column, coefficients or bias, or another layer's router
        other = (t + 1) % 3
        for kw in ({"w_sa": w.w_sa(other, layer).numpy()}, {"coef_a": w.rational_coef(other, layer)[0].numpy()},
                   {"bias": w.router_bias(other, layer).numpy()}):
            args = dict(w_sa=w.w_sa(t, layer).numpy(), coef_a=a.numpy(), coef_b=b.numpy(), bias=w.router_bias(t, layer).numpy())
            args.update(kw)
            wrong = O.route_prompt(w.hidden(layer, i).numpy(), w.router(t, layer).numpy(), pooler=O.POOL_SELFATTN,
                                   activation=O.ACT_RATIONAL, k=k, **args)
            assert not np.allclose(wrong["logits"], logits[p])
        wrong = O.route_prompt(w.hidden(layer, i).numpy(), w.router(t, 0).numpy(), pooler=O.POOL_SELFATTN,
                               activation=O.ACT_RATIONAL, k=k, w_sa=w.w_sa(t, layer).numpy(), coef_a=a.numpy(),
                               coef_b=b.numpy(), bias=w.router_bias(t, layer).numpy())
        assert not np.allclose(wrong["logits"], logits[p])
    # rows of requests that were not routed, and the other layer, stay untouched
    assert table[1, layer] == -1 and (table[:, 0] == -1).all() and (topk[:, 0] == -1).all()
    # the plain branch: no bias, mean pooling, tanh, top-1 (no top-k table)
    table2 = np.full((4, 2), -1, dtype=np.int32)
    lo2, _ = R.route_requests(w, 0, [1], table2)
    want = O.route_prompt(w.hidden(0, 1).numpy(), w.router(0, 0).numpy())
    assert np.array_equal(lo2[0], want["logits"]) and table2[1, 0] == want["route"]
    # a caller-supplied hidden-state function replaces the workload's own
    lo3, _ = R.route_requests(w, 0, [1], table2, hidden=lambda i: w.hidden(1, 2))
    assert np.array_equal(lo3[0], O.route_prompt(w.hidden(1, 2).numpy(), w.router(0, 0).numpy())["logits"])
