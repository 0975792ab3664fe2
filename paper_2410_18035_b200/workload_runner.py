"""Loads a synthetic workload into a library context and drives the hot path through the binding.

Glue for the tests, the smoke check and the benchmark: tensors come from `synth`, every step of the
path is a call into libmilora.so.  Nothing is computed here.
"""
from __future__ import annotations

import numpy as np
import torch

from .binding import ACT_TANH, N_MOD, POOL_MEAN, Milora


class LoadedWorkload:
    """A `synth.Workload` registered into a `Milora` context on one device.

    layers: which workload layers are registered (context layer index = position in `layers`).
    Request i of the workload uses slot i.
    """

    def __init__(self, w, device="cuda", layers=None, tenants=None, pool=POOL_MEAN, act=ACT_TANH, with_bias=False,
                 max_requests=None, register_adapters=True, top_k=1, gate=0):
        self.w = w
        self.device = torch.device(device)
        self.layers = list(range(w.n_layers)) if layers is None else list(layers)
        self.tenants = [int(t) for t in (w.active_tenants() if tenants is None else tenants)]
        self.pool, self.act, self.with_bias = pool, act, with_bias
        self.ml = Milora(len(self.layers), w.d_model, w.d_ff, w.d_kv, w.dtype, w.rank, w.n_tenants,
                         max_requests or w.n_requests, top_k=top_k, gate=gate)
        for tenant in self.tenants:
            for li, layer in enumerate(self.layers):
                self.register_router(tenant, li, layer)
                if register_adapters:
                    for m in range(N_MOD):
                        A, B = w.adapter(tenant, layer, m, self.device)
                        self.ml.register_adapter(tenant, li, m, A, B, w.scale)
        torch.cuda.synchronize(self.device)
        for i in range(w.n_requests):
            self.ml.request_open(i, int(w.request_tenant[i]))

    def register_router(self, tenant, li, layer):
        w = self.w
        kw = {}
        if self.with_bias:
            kw["bias"] = w.router_bias(tenant, layer, self.device)
        if self.pool == 3:
            kw["Wsa"] = w.w_sa(tenant, layer, self.device)
        if self.act == 4:
            a, b = w.rational_coef(tenant, layer)
            kw["coef_a"], kw["coef_b"] = a.tolist(), b.tolist()
        self.ml.register_router(tenant, li, w.router(tenant, layer, self.device), pool=self.pool, act=self.act, **kw)

    # ---- batch descriptors ---------------------------------------------------------------
    def seq_arrays(self, prefill_ids, decode_ids):
        """cu_seqlens / seq_slot of a step whose rows are the prompts of `prefill_ids` followed by one row
        per request of `decode_ids`."""
        lens = [int(self.w.prompt_len[i]) for i in prefill_ids] + [1] * len(decode_ids)
        cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        slots = np.array(list(prefill_ids) + list(decode_ids), dtype=np.int32)
        return (torch.from_numpy(cu).to(self.device), torch.from_numpy(slots).to(self.device), int(cu[-1]))

    def route(self, li, prefill_ids, H=None, logits=None, probs=None):
        """Route the prompts of `prefill_ids` at context layer li; H defaults to the workload's H^l."""
        w = self.w
        if H is None:
            H = w.hidden_batch(self.layers[li], prefill_ids, self.device)
        cu = torch.from_numpy(w.cu_seqlens(prefill_ids)).to(self.device)
        slots = torch.tensor(list(prefill_ids), dtype=torch.int32, device=self.device)
        self.ml.route(li, H, cu, slots, logits, probs)
        return H

    def close(self):
        self.ml.close()
