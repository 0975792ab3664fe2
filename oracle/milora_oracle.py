"""fp64 CPU oracle of the MiLoRA serving hot path (numpy).

TEST INFRASTRUCTURE ONLY - never imported by the CUDA library or its binding.

Everything here follows the paper's definitions in the paper's order and
notation, with no blocking, fusion or reordering:

* Section 3.1, Eq. 1    LoRA-augmented projection  x' = x W_m + x W_m^A W_m^B + b_m
* Section 3.3, Eq. 2    h^l = Pooler(H^l)           (last / average / max / self-attention)
* Appendix C            the self-attention pooler
* Section 3.4, Eq. 7    the rational activation
* Section 3.3, Eq. 3    R^l(h^l) = Top-k(Softmax(g(h^l) W_r^l))
* Section 3.3           the routing decision is taken once per prompt and
                        reused for every generated token
* Section 4.5           adapters stay unmerged (multi-tenant serving), so a
                        batch mixes tenants; tokens are bucketed by
                        (module, tenant) before the adapters are applied

All inputs are converted to float64 on entry; bf16/fp32 inputs are exactly
representable, so the oracle sees precisely the values the GPU sees.

Pins (tests marked "not gpu"): brute-force merged weights W + s A B, closed
forms (unit vectors, rank 1, zero B, linearity), pooler special cases, the
parameter-count identities printed in Section 4.3 / Table 1, textbook
activations at tabulated points, stable-sort brute force for grouping.
The paper prints no worked numeric example of a route or of an output, so
absolute output values are "parity unpinned" against the paper itself; they are
pinned by the definitions and invariants above.
"""
from __future__ import annotations

import math

import numpy as np

# Section 3.1: the seven linear modules of a LLaMA-style layer, N_mod = 7.
MODULES = ("q", "k", "v", "o", "gate", "up", "down")
N_MOD = len(MODULES)

POOL_MEAN, POOL_LAST, POOL_MAX, POOL_SELFATTN = 0, 1, 2, 3
ACT_TANH, ACT_IDENTITY, ACT_RELU, ACT_GELU, ACT_RATIONAL = 0, 1, 2, 3, 4


def _f64(a):
    return np.asarray(a, dtype=np.float64)


# --------------------------------------------------------------------------
# Shapes (Section 3.1; Fig. 1 left)
# --------------------------------------------------------------------------
def module_dims(d_model: int, d_ff: int, d_kv: int, module: int) -> tuple[int, int]:
    """(d1, d2) of W_m for module index 0..6 = q,k,v,o,gate,up,down."""
    name = MODULES[module]
    if name in ("q", "o"):
        return d_model, d_model
    if name in ("k", "v"):
        return d_model, d_kv
    if name in ("gate", "up"):
        return d_model, d_ff
    return d_ff, d_model  # down


def lora_param_count(d_model: int, d_ff: int, d_kv: int, r: int, n_layers: int,
                     modules=range(N_MOD)) -> int:
    """Parameters of rank-r LoRA pairs (W^A: d1 x r, W^B: r x d2) on `modules` of every layer."""
    per_layer = 0
    for m in modules:
        d1, d2 = module_dims(d_model, d_ff, d_kv, m)
        per_layer += r * (d1 + d2)
    return per_layer * n_layers


def router_param_count(d_model: int, n_layers: int, bias: bool = False) -> int:
    """Parameters of the per-layer routers W_r^l in R^{d x N_mod} (Eq. 3)."""
    return n_layers * (d_model * N_MOD + (N_MOD if bias else 0))


def max_activated_param_count(d_model: int, d_ff: int, d_kv: int, r: int, n_layers: int, k: int) -> int:
    """Upper bound of parameters in use for one prompt: the k largest LoRA modules
    of every layer plus all routers (Section 4.3, 'at most ... activated')."""
    sizes = sorted((r * sum(module_dims(d_model, d_ff, d_kv, m)) for m in range(N_MOD)), reverse=True)
    return n_layers * sum(sizes[:k]) + router_param_count(d_model, n_layers)


# --------------------------------------------------------------------------
# Poolers (Section 3.3, Eq. 2; Appendix C)
# --------------------------------------------------------------------------
def pool_last(H):
    """(a) last-token pooling: the last prompt token's hidden state."""
    H = _f64(H)
    return H[-1, :].copy()


def pool_mean(H):
    """(b) average pooling over the n_p prompt tokens."""
    H = _f64(H)
    n_p = H.shape[0]
    return H.sum(axis=0) / n_p


def pool_max(H):
    """(c) max pooling over the n_p prompt tokens, per hidden dimension."""
    H = _f64(H)
    return H.max(axis=0)


def pool_self_attention(H, w_sa):
    """(d) Appendix C: U = H W_sa, A = Softmax(U) over the tokens, p = A^T H.

    W_sa is a single query column (d x 1); no 1/sqrt(d) scaling is printed.
    """
    H = _f64(H)
    w_sa = _f64(w_sa).reshape(-1)
    U = H @ w_sa                       # (n_p,)
    A = softmax(U)                     # over the sequence dimension
    return A @ H                       # (d,)


def pool(H, kind: int, w_sa=None):
    if kind == POOL_MEAN:
        return pool_mean(H)
    if kind == POOL_LAST:
        return pool_last(H)
    if kind == POOL_MAX:
        return pool_max(H)
    if kind == POOL_SELFATTN:
        return pool_self_attention(H, w_sa)
    raise ValueError(f"unknown pooler {kind}")


# --------------------------------------------------------------------------
# Activations g (Section 3.3; Section 3.4, Eq. 7)
# --------------------------------------------------------------------------
_erf = np.vectorize(math.erf, otypes=[np.float64])


def act_gelu(x):
    """Exact GeLU: x * Phi(x) with the erf form of the normal CDF."""
    x = _f64(x)
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def act_rational(x, a, b):
    """Eq. 7: Ra(x) = sum_{j=0..m} a_j x^j / (1 + |sum_{i=1..n} b_i x^i|).

    `a` holds a_0..a_m, `b` holds b_1..b_n.  The absolute value is taken of the
    whole denominator polynomial.
    """
    x = _f64(x)
    a = _f64(a).reshape(-1)
    b = _f64(b).reshape(-1)
    num = np.zeros_like(x)
    for j in range(a.size):
        num = num + a[j] * x ** j
    den_poly = np.zeros_like(x)
    for i in range(1, b.size + 1):
        den_poly = den_poly + b[i - 1] * x ** i
    return num / (1.0 + np.abs(den_poly))


def activate(h, kind: int, coef_a=None, coef_b=None):
    h = _f64(h)
    if kind == ACT_TANH:
        return np.tanh(h)
    if kind == ACT_IDENTITY:
        return h.copy()
    if kind == ACT_RELU:
        return np.maximum(h, 0.0)
    if kind == ACT_GELU:
        return act_gelu(h)
    if kind == ACT_RATIONAL:
        return act_rational(h, coef_a, coef_b if coef_b is not None else [])
    raise ValueError(f"unknown activation {kind}")


# --------------------------------------------------------------------------
# Router (Section 3.3, Eq. 3)
# --------------------------------------------------------------------------
def softmax(z):
    """Softmax over the last axis (max-subtracted; mathematically the plain definition)."""
    z = _f64(z)
    e = np.exp(z - z.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def router_logits(g, W_r, bias=None):
    """g(h^l) W_r^l with W_r^l in R^{d x N_mod}; the paper prints no bias (optional here)."""
    g = _f64(g)
    W_r = _f64(W_r)
    z = g @ W_r
    if bias is not None:
        z = z + _f64(bias)
    return z


def top_k(p, k: int):
    """Indices of the k largest entries, largest first; equal entries go to the lower index."""
    p = _f64(p)
    order = np.argsort(-p, kind="stable")
    return order[:k].astype(np.int32)


def route_prompt(H, W_r, *, bias=None, pooler=POOL_MEAN, w_sa=None, activation=ACT_TANH,
                 coef_a=None, coef_b=None, k: int = 1):
    """One router evaluation for one prompt at one layer (Eq. 2 then Eq. 3).

    Returns a dict with
      h       pooled vector                       (d,)
      logits  g(h) W_r (+ bias)                   (N_mod,)
      probs   Softmax(logits)                     (N_mod,)
      topk    the k selected module indices       (k,)  int32
      route   topk[0]
      margin  largest logit minus second largest  (>= 0)
    Selection is made on the softmax probabilities; softmax is strictly
    increasing in each logit, so this is also the order of the logits.
    """
    h = pool(H, pooler, w_sa)
    g = activate(h, activation, coef_a, coef_b)
    z = router_logits(g, W_r, bias)
    p = softmax(z)
    sel = top_k(p, k)
    zs = np.sort(z)[::-1]
    return {"h": h, "logits": z, "probs": p, "topk": sel, "route": int(sel[0]),
            "margin": float(zs[0] - zs[1])}


def route_batch(H, cu_seqlens, seq_slot, slot_tenant, routers, layer: int, route_table, **kw):
    """Route every prompt of a ragged batch at one layer.

    H           (T_total, d) rows of all prompts back to back
    cu_seqlens  (P+1,) row offsets
    seq_slot    (P,)  request slot of each prompt
    slot_tenant (R,)  tenant of each slot
    routers     callable (tenant, layer) -> dict(W_r=..., bias=..., pooler=..., ...)
    route_table (R, L) int32, row `slot`, column `layer` is written.
    Returns (logits (P, N_mod), margins (P,)).
    """
    H = _f64(H)
    P = len(seq_slot)
    logits = np.zeros((P, N_MOD))
    margins = np.zeros(P)
    for p in range(P):
        lo, hi = int(cu_seqlens[p]), int(cu_seqlens[p + 1])
        slot = int(seq_slot[p])
        tenant = int(slot_tenant[slot])
        rp = dict(routers(tenant, layer))
        W_r = rp.pop("W_r")
        out = route_prompt(H[lo:hi], W_r, **rp, **kw)
        route_table[slot, layer] = out["route"]
        logits[p] = out["logits"]
        margins[p] = out["margin"]
    return logits, margins


# --------------------------------------------------------------------------
# Token grouping by (module, tenant)  (multi-tenant serving, Section 4.5)
# --------------------------------------------------------------------------
def group_tokens(token_slot, slot_tenant, route_col, has_adapter, max_tenants: int):
    """Bucket the tokens of one step for one layer.

    token_slot  (T,) request slot of every token
    slot_tenant (R,) tenant of each slot (-1: slot closed)
    route_col   (R,) routed module of each slot at this layer (-1: not routed), or (R, k) for
                Top-k routing (Eq. 3; the k sweep of Section 4.5): the k selected modules
    has_adapter callable (tenant, module) -> bool
    A token belongs to one bucket per selected module on which its tenant has an adapter.
    Tokens whose slot is closed, unrouted or without any such adapter are excluded.

    Returns dict:
      perm        (n_active,) token indices of the (token, module) pairs ordered by
                  (module, tenant, token index); a token appears once per selected module
      seg_key     (S,) module * max_tenants + tenant of every non-empty bucket, ascending
      seg_offset  (S+1,) bucket boundaries in perm
      mod_offset  (N_mod+1,) bucket-index boundaries per module
      n_excluded  number of excluded tokens
    """
    T = len(token_slot)
    route_sel = np.asarray(route_col)
    if route_sel.ndim == 1:
        route_sel = route_sel[:, None]
    pairs = []                                   # (key, token) in token order
    n_excluded = 0
    for t in range(T):
        slot = int(token_slot[t])
        tenant = int(slot_tenant[slot])
        found = False
        if tenant >= 0:
            for module in (int(v) for v in route_sel[slot]):
                if module < 0 or not has_adapter(tenant, module):
                    continue
                pairs.append((module * max_tenants + tenant, t))
                found = True
        if not found:
            n_excluded += 1
    pairs.sort(key=lambda kt: kt[0])             # Python's sort is stable
    perm = np.array([t for _, t in pairs], dtype=np.int32)
    seg_key, seg_offset = [], [0]
    for i, (key, _) in enumerate(pairs):
        if i == 0 or key != pairs[i - 1][0]:
            if i > 0:
                seg_offset.append(i)
            seg_key.append(int(key))
    if pairs:
        seg_offset.append(len(pairs))
    seg_key = np.array(seg_key, dtype=np.int32)
    seg_offset = np.array(seg_offset, dtype=np.int32)
    mod_offset = np.zeros(N_MOD + 1, dtype=np.int32)
    for m in range(N_MOD):
        mod_offset[m + 1] = mod_offset[m] + int(np.sum(seg_key // max_tenants == m))
    return {"perm": perm, "seg_key": seg_key, "seg_offset": seg_offset,
            "mod_offset": mod_offset, "n_excluded": n_excluded}


# --------------------------------------------------------------------------
# LoRA-augmented projection (Section 3.1, Eq. 1)
# --------------------------------------------------------------------------
def lora_delta(x, A, B, s: float):
    """s * (x W^A) W^B with W^A: d1 x r, W^B: r x d2.  Eq. 1 prints no scale; s is the
    usual LoRA scaling factor supplied per adapter (s = 1 gives Eq. 1 verbatim)."""
    x = _f64(x)
    v = x @ _f64(A)
    return float(s) * (v @ _f64(B))


def base_projection(x, W, b=None):
    """x W_m + b_m (the backbone's own linear module)."""
    y = _f64(x) @ _f64(W)
    if b is not None:
        y = y + _f64(b)
    return y


def lora_projection(x, W, A, B, s: float, b=None):
    """Eq. 1: x' = x W_m + s x W_m^A W_m^B + b_m."""
    return base_projection(x, W, b) + lora_delta(x, A, B, s)


def merged_weight(W, A, B, s: float):
    """W_m + s W_m^A W_m^B, materialised (d1 x d2).  Used only to cross-check Eq. 1."""
    return _f64(W) + float(s) * (_f64(A) @ _f64(B))


def _selection_weight(route_sel, gate, slot: int, module: int):
    """None if `module` is not among the slot's selected modules, else the weight of its LoRA term:
    1 (hard selection) or gate[slot][j] for the position j at which it was selected."""
    sel = [int(v) for v in route_sel[slot]]
    if module not in sel:
        return None
    if gate is None:
        return 1.0
    return float(np.asarray(gate, dtype=np.float64).reshape(len(route_sel), -1)[slot][sel.index(module)])


def apply_module(y_base, x, token_slot, slot_tenant, route_sel, module: int, adapters, gate=None):
    """Outputs of module `module` for a mixed batch.

    y_base     (T, d2) the backbone's x W_m + b_m (an input here)
    x          (T, d1)
    route_sel  (R,) int, or (R, k) int for top-k routing: the module(s) selected
               for each slot at this layer
    adapters   callable (tenant, module) -> (A, B, s) or None
    gate       optional (R,) / (R, k) weights, gate[slot][j] for the j-th selected module
               (the paper only selects, so None = weight 1 is the default reading; a
               probability-weighted mixture passes the router's softmax values here)
    A token receives s (x A) B iff its slot's selection contains `module` and the
    tenant has an adapter there; every other row is returned unchanged.
    """
    y = _f64(y_base).copy()
    x = _f64(x)
    route_sel = np.asarray(route_sel)
    if route_sel.ndim == 1:
        route_sel = route_sel[:, None]
    for t in range(y.shape[0]):
        slot = int(token_slot[t])
        tenant = int(slot_tenant[slot])
        wgt = None if tenant < 0 else _selection_weight(route_sel, gate, slot, module)
        if wgt is None:
            continue
        ad = adapters(tenant, module)
        if ad is None:
            continue
        A, B, s = ad
        y[t] = y[t] + wgt * lora_delta(x[t:t + 1], A, B, s)[0]
    return y


def apply_module_sampled(y_base_rows, x_rows, rows, token_slot, slot_tenant, route_sel, module, adapters, gate=None):
    """Same as apply_module, restricted to the token indices `rows` (for full-size
    workloads where only sampled outputs are checked).  y_base_rows / x_rows hold
    just those rows, in the order of `rows`."""
    y = _f64(y_base_rows).copy()
    x = _f64(x_rows)
    route_sel = np.asarray(route_sel)
    if route_sel.ndim == 1:
        route_sel = route_sel[:, None]
    for i, t in enumerate(rows):
        slot = int(token_slot[int(t)])
        tenant = int(slot_tenant[slot])
        wgt = None if tenant < 0 else _selection_weight(route_sel, gate, slot, module)
        if wgt is None:
            continue
        ad = adapters(tenant, module)
        if ad is None:
            continue
        A, B, s = ad
        y[i] = y[i] + wgt * lora_delta(x[i:i + 1], A, B, s)[0]
    return y


# --------------------------------------------------------------------------
# Error metric used by the parity tests
# --------------------------------------------------------------------------
def max_rel_err(y, y_ref) -> float:
    """max_i |y_i - yref_i| / max(|yref_i|, rms(yref)); 0 for empty or all-zero references
    that are matched exactly."""
    y = _f64(y)
    y_ref = _f64(y_ref)
    if y_ref.size == 0:
        return 0.0
    rms = math.sqrt(float(np.mean(y_ref * y_ref)))
    den = np.maximum(np.abs(y_ref), rms)
    diff = np.abs(y - y_ref)
    if rms == 0.0:
        return 0.0 if float(diff.max()) == 0.0 else float("inf")
    return float((diff / den).max())
