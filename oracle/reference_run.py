"""Runs the oracle over a synthetic workload (glue between `synth` and `milora_oracle`).

TEST INFRASTRUCTURE ONLY.  Tensors come from `synth` (torch), are widened to float64
and handed to the oracle functions; nothing here adds arithmetic of its own.
"""
from __future__ import annotations

import numpy as np
import torch

from . import milora_oracle as O


def to_f64(t) -> np.ndarray:
    if isinstance(t, torch.Tensor):
        return t.detach().to("cpu").to(torch.float64).numpy()
    return np.asarray(t, dtype=np.float64)


def route_requests(w, layer: int, ids, route_table: np.ndarray, *, pooler=O.POOL_MEAN,
                   activation=O.ACT_TANH, with_bias=False, k: int = 1, hidden=None, topk_table=None):
    """Route the prompts of requests `ids` at `layer` (request i uses slot i).

    hidden: optional callable request -> H tensor (default: the workload's own H^l).
    Returns (logits (P,7), margins (P,)).  Writes route_table[slot, layer] and, when given,
    topk_table[slot, layer, :k].
    """
    P = len(ids)
    logits = np.zeros((P, O.N_MOD))
    margins = np.zeros(P)
    for p, i in enumerate(ids):
        i = int(i)
        tenant = int(w.request_tenant[i])
        H = to_f64(hidden(i) if hidden is not None else w.hidden(layer, i))
        kw = {}
        if pooler == O.POOL_SELFATTN:
            kw["w_sa"] = to_f64(w.w_sa(tenant, layer))
        if activation == O.ACT_RATIONAL:
            a, b = w.rational_coef(tenant, layer)
            kw["coef_a"], kw["coef_b"] = to_f64(a), to_f64(b)
        if with_bias:
            kw["bias"] = to_f64(w.router_bias(tenant, layer))
        out = O.route_prompt(H, to_f64(w.router(tenant, layer)), pooler=pooler, activation=activation, k=k, **kw)
        route_table[i, layer] = out["route"]
        if topk_table is not None:
            topk_table[i, layer, :k] = out["topk"]
        logits[p] = out["logits"]
        margins[p] = out["margin"]
    return logits, margins


def full_route_table(w, ids=None, **kw):
    """Route table (n_requests, n_layers) int32 for the whole workload; -1 where not routed."""
    ids = np.arange(w.n_requests) if ids is None else ids
    table = np.full((w.n_requests, w.n_layers), -1, dtype=np.int32)
    margins = np.zeros((len(ids), w.n_layers))
    for layer in range(w.n_layers):
        _, m = route_requests(w, layer, ids, table, **kw)
        margins[:, layer] = m
    return table, margins


def adapters_of(w, layer: int):
    """callable (tenant, module) -> (A, B, s) in float64 for the workload's adapters at `layer`."""
    cache = {}

    def get(tenant, module):
        key = (int(tenant), int(module))
        if key not in cache:
            A, B = w.adapter(key[0], layer, key[1])
            cache[key] = (to_f64(A), to_f64(B), float(w.scale))
        return cache[key]

    return get


def apply_site(w, layer: int, module: int, x, y_base, token_slot, route_sel, rows=None, gate=None):
    """Oracle output of one module call site.  With `rows`, x / y_base hold only those rows."""
    slot_tenant = w.request_tenant
    ad = adapters_of(w, layer)
    if rows is None:
        return O.apply_module(to_f64(y_base), to_f64(x), token_slot, slot_tenant, route_sel, module, ad, gate=gate)
    return O.apply_module_sampled(to_f64(y_base), to_f64(x), rows, token_slot, slot_tenant, route_sel, module, ad,
                                  gate=gate)


def group_layer(w, token_slot, route_col, max_tenants=None):
    return O.group_tokens(token_slot, w.request_tenant, route_col, lambda t, m: True,
                          max_tenants if max_tenants is not None else w.n_tenants)
