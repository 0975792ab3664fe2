"""Seeded synthetic inputs shaped like LLaMA-class multi-tenant LoRA serving batches.

Every tensor is addressable on its own: its seed is a hash of (master seed, tensor kind,
tenant, layer, module, ...), so one adapter, one router or one prompt's hidden states can
be regenerated without generating anything else.  Values are drawn as fp32 normals,
scaled, and rounded to the workload's dtype; the rounded values are the inputs both the
CPU oracle and the CUDA library see.

Distributions (std unless stated):
  base weights W_m       N(0, 0.02)
  LoRA A (d1 x r)        N(0, variance 1/d_model)
  LoRA B (r x d2)        N(0, 0.01)
  router W_r (d x 7)     N(0, 0.02), no bias
  hidden states H, module inputs x, base outputs y_base   N(0, 1)
Batch structure (prompt lengths, tenant of each request) comes from numpy's PCG64 with
the same master seed.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

MODULES = ("q", "k", "v", "o", "gate", "up", "down")
N_MOD = 7

_KINDS = {"adapter_A": 1, "adapter_B": 2, "router_W": 3, "base_W": 4, "hidden": 5,
          "x": 6, "y_base": 7, "w_sa": 8, "router_bias": 9, "coef": 10}


def module_dims(d_model: int, d_ff: int, d_kv: int, module: int) -> tuple[int, int]:
    name = MODULES[module]
    if name in ("q", "o"):
        return d_model, d_model
    if name in ("k", "v"):
        return d_model, d_kv
    if name in ("gate", "up"):
        return d_model, d_ff
    return d_ff, d_model


def _mix64(z: int) -> int:
    z = (z + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
    return z ^ (z >> 31)


def tensor_seed(master: int, *ids: int) -> int:
    """Hash a master seed and a tuple of small integers into a 63-bit generator seed."""
    h = _mix64(master & 0xFFFFFFFFFFFFFFFF)
    for v in ids:
        h = _mix64(h ^ ((int(v) + 0x1000) & 0xFFFFFFFFFFFFFFFF))
    return h & 0x7FFFFFFFFFFFFFFF


def _torch_dtype(name: str):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


@dataclass
class Workload:
    name: str
    dtype: str                      # "f32" | "bf16"
    n_layers: int
    d_model: int
    d_ff: int
    d_kv: int
    rank: int
    scale: float
    n_tenants: int
    seed: int
    request_tenant: np.ndarray      # (n_requests,) tenant of request i; request i uses slot i
    prompt_len: np.ndarray          # (n_requests,) prompt length of request i
    prefill_ids: np.ndarray         # requests whose prompt tokens are in the step (routed + prefill apply)
    decode_ids: np.ndarray          # requests that contribute one decode token to the step
    decode_steps: int = 1
    has_base_weights: bool = False
    note: str = ""
    # Device whose random-number generator draws every tensor ("cpu" or "cuda").  A tensor is drawn there and
    # then moved to the device that was asked for, so all users of one workload see the same values.
    gen_device: str = "cpu"
    _cache: dict = field(default_factory=dict, repr=False)

    # ---- structure -------------------------------------------------------
    @property
    def n_requests(self) -> int:
        return int(self.request_tenant.shape[0])

    @property
    def torch_dtype(self):
        return _torch_dtype(self.dtype)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    def dims(self, module: int) -> tuple[int, int]:
        return module_dims(self.d_model, self.d_ff, self.d_kv, module)

    def active_tenants(self) -> np.ndarray:
        return np.unique(self.request_tenant)

    def cu_seqlens(self, ids) -> np.ndarray:
        lens = self.prompt_len[np.asarray(ids, dtype=np.int64)]
        return np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)

    # ---- tensors ---------------------------------------------------------
    def _normal(self, shape, std: float, kind: str, ids, device, dtype=None):
        g = torch.Generator(device=self.gen_device)
        g.manual_seed(tensor_seed(self.seed, _KINDS[kind], *ids))
        t = torch.randn(shape, generator=g, device=self.gen_device, dtype=torch.float32)
        if std != 1.0:
            t.mul_(std)
        return t.to(dtype if dtype is not None else self.torch_dtype).to(device)

    def adapter(self, tenant: int, layer: int, module: int, device="cpu"):
        """(A, B): A is d1 x r, B is r x d2 (the orientation of Eq. 1 of the paper)."""
        d1, d2 = self.dims(module)
        A = self._normal((d1, self.rank), self.d_model ** -0.5, "adapter_A", (tenant, layer, module), device)
        B = self._normal((self.rank, d2), 0.01, "adapter_B", (tenant, layer, module), device)
        return A, B

    def router(self, tenant: int, layer: int, device="cpu"):
        """W_r, d x 7."""
        return self._normal((self.d_model, N_MOD), 0.02, "router_W", (tenant, layer), device)

    def router_bias(self, tenant: int, layer: int, device="cpu"):
        return self._normal((N_MOD,), 0.02, "router_bias", (tenant, layer), device, dtype=torch.float32)

    def w_sa(self, tenant: int, layer: int, device="cpu"):
        """Query column of the self-attention pooler, (d,)."""
        return self._normal((self.d_model,), self.d_model ** -0.5, "w_sa", (tenant, layer), device)

    def rational_coef(self, tenant: int, layer: int, n_a: int = 7, n_b: int = 5):
        """Small seeded coefficients a_0..a_m, b_1..b_n for the rational activation (fp32, host)."""
        c = self._normal((n_a + n_b,), 0.3, "coef", (tenant, layer), "cpu", dtype=torch.float32)
        return c[:n_a].clone(), c[n_a:].clone()

    def base_weight(self, layer: int, module: int, device="cpu"):
        d1, d2 = self.dims(module)
        return self._normal((d1, d2), 0.02, "base_W", (layer, module), device)

    def hidden(self, layer: int, request: int, device="cpu"):
        """H^l of one request's prompt, (n_p, d)."""
        n_p = int(self.prompt_len[request])
        return self._normal((n_p, self.d_model), 1.0, "hidden", (layer, request), device)

    def hidden_batch(self, layer: int, ids, device="cpu"):
        parts = [self.hidden(layer, int(i), device) for i in ids]
        if not parts:
            return torch.zeros((0, self.d_model), dtype=self.torch_dtype, device=device)
        return torch.cat(parts, dim=0)

    def module_input(self, layer: int, module: int, n_tokens: int, tag: int, device="cpu"):
        d1, _ = self.dims(module)
        return self._normal((n_tokens, d1), 1.0, "x", (layer, module, tag), device)

    def base_output(self, layer: int, module: int, n_tokens: int, tag: int, device="cpu"):
        _, d2 = self.dims(module)
        return self._normal((n_tokens, d2), 1.0, "y_base", (layer, module, tag), device)


def _zipf_tenants(rng: np.random.Generator, n: int, n_tenants: int, alpha: float) -> np.ndarray:
    """Inverse-CDF draws from p_k proportional to k^-alpha over ranks 1..n_tenants (tenant id = rank - 1)."""
    w = np.arange(1, n_tenants + 1, dtype=np.float64) ** (-alpha)
    cdf = np.cumsum(w / w.sum())
    u = rng.random(n)
    return np.minimum(np.searchsorted(cdf, u, side="left"), n_tenants - 1).astype(np.int32)


def _c1(seed):
    n = 4
    return Workload("c1_tiny_f32", "f32", 2, 256, 688, 256, 8, 2.0, 4, seed,
                    np.arange(n, dtype=np.int32), np.full(n, 16, dtype=np.int32),
                    np.arange(n), np.arange(n), decode_steps=4, has_base_weights=True,
                    note="tiny fp32 stack with base weights; 4 prompts x 16 tokens, 4 decode steps")


def _c2(seed):
    n = 64
    return Workload("c2_llama2_7b_layer_bf16", "bf16", 1, 4096, 11008, 4096, 16, 2.0, 64, seed,
                    np.arange(n, dtype=np.int32), np.full(n, 512, dtype=np.int32),
                    np.arange(n), np.arange(n),
                    note="LLaMA-2-7B one layer; 64 requests on 64 distinct tenants; 512-token prompts")


def _c3(seed):
    rng = np.random.default_rng(seed + 3)
    n = 32
    lens = rng.integers(128, 2049, size=n).astype(np.int32)
    ten = rng.integers(0, 32, size=n).astype(np.int32)
    return Workload("c3_llama2_7b_prefill_bf16", "bf16", 32, 4096, 11008, 4096, 16, 2.0, 32, seed,
                    ten, lens, np.arange(n), np.zeros(0, dtype=np.int64),
                    note="LLaMA-2-7B 32 layers; prefill of 32 prompts, lengths U[128,2048], tenants U[0,32)")


def _c4(seed):
    rng = np.random.default_rng(seed + 4)
    n = 256
    ten = _zipf_tenants(rng, n, 1000, 1.1)
    return Workload("c4_llama2_13b_zipf_bf16", "bf16", 40, 5120, 13824, 5120, 32, 2.0, 1000, seed,
                    ten, np.full(n, 256, dtype=np.int32), np.arange(n), np.arange(n),
                    note="LLaMA-2-13B 40 layers; 256 decode requests, tenants Zipf(1.1) over 1000; 256-token prompts")


def _c5(seed, n_prefill=8, n_decode=192):
    rng = np.random.default_rng(seed + 5)
    n = n_prefill + n_decode
    lens = np.concatenate([rng.integers(256, 4097, size=n_prefill),
                           np.full(n_decode, 256)]).astype(np.int32)
    ten = rng.integers(0, 128, size=n).astype(np.int32)
    return Workload("c5_llama3_8b_mixed_bf16", "bf16", 32, 4096, 14336, 1024, 16, 2.0, 128, seed,
                    ten, lens, np.arange(n_prefill), np.arange(n_prefill, n),
                    note="LLaMA-3-8B GQA 32 layers; mixed step: 8 prefill prompts U[256,4096] + 192 decode tokens")


CONFIGS = {"c1": _c1, "c2": _c2, "c3": _c3, "c4": _c4, "c5": _c5}


def get_workload(name: str, seed: int = 0, **kw) -> Workload:
    return CONFIGS[name](seed, **kw)


def decode_sweep_workload(batch: int, seed: int = 0) -> Workload:
    """LLaMA-3-8B shapes, decode only, `batch` requests on `batch` distinct tenants (batch-size sweep)."""
    n = batch
    return Workload(f"c5_sweep_b{batch}", "bf16", 32, 4096, 14336, 1024, 16, 2.0, max(n, 1), seed,
                    np.arange(n, dtype=np.int32), np.full(n, 256, dtype=np.int32),
                    np.arange(n), np.arange(n), note="decode-only batch sweep, tenants = batch size")


def scaled_workload(base: Workload, **overrides) -> Workload:
    """A copy of `base` with some fields replaced (smaller layer counts or batches for tests)."""
    import dataclasses
    d = {f.name: getattr(base, f.name) for f in dataclasses.fields(base) if f.name != "_cache"}
    d.update(overrides)
    return Workload(**d)


def shard_by_tenant(request_tenant, world_size: int):
    """Requests of each rank when tenants are placed round-robin (tenant % world_size): every adapter lives on
    exactly one rank and a request follows its tenant, so no rank ever needs another rank's data."""
    t = np.asarray(request_tenant)
    return [np.nonzero(t % world_size == r)[0] for r in range(world_size)]
