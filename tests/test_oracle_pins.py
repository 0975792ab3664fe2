"""Pins for the fp64 oracle: closed forms, brute force, special cases, printed values.

None of these retype the oracle's formulas with the same library calls; they use
pure-Python loops, hand-computed numbers, invariants, and the counts the paper prints.
"""
import math
import os
import random

import numpy as np
import pytest

from oracle import milora_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ shapes
def _golden_counts():
    out = {}
    with open(os.path.join(GOLDEN, "param_counts.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, val = line.split()[:2]
            out[name] = float(val)
    return out


def test_param_counts_match_paper_tables():
    """Table 1 / Section 4.3 print 80.0M, 80.9M and 16.4M for LLaMA-2 7B at rank 32.
    They pin: the seven module shapes, the bias-free d x 7 router, and top-1 selection."""
    g = _golden_counts()
    d, d_ff, L, r = 4096, 11008, 32, 32
    lora = O.lora_param_count(d, d_ff, d, r, L)
    tunable = lora + O.router_param_count(d, L)
    activated = O.max_activated_param_count(d, d_ff, d, r, L, k=1)
    assert lora == 79_953_920
    assert tunable == 80_871_424
    assert activated == 16_384_000
    assert round(lora / 1e6, 1) == g["lora_all_modules_r32"]
    assert round(tunable / 1e6, 1) == g["milora_tunable_r32"]
    assert round(activated / 1e6, 1) == g["milora_max_activated_r32"]
    # a router with a bias, or k = 2, would not print as 80.9M / 16.4M
    assert round(O.max_activated_param_count(d, d_ff, d, r, L, k=2) / 1e6, 1) != g["milora_max_activated_r32"]


def test_module_dims_table():
    dims = [O.module_dims(4096, 14336, 1024, m) for m in range(7)]
    assert dims == [(4096, 4096), (4096, 1024), (4096, 1024), (4096, 4096),
                    (4096, 14336), (4096, 14336), (14336, 4096)]
    assert O.MODULES == ("q", "k", "v", "o", "gate", "up", "down") and O.N_MOD == 7


# ------------------------------------------------------------------ Eq. 1
def _rand(rng, *shape):
    return rng.standard_normal(shape)


def _loops_matmul(a, b):
    n, k = len(a), len(a[0])
    m = len(b[0])
    assert len(b) == k
    return [[math.fsum(a[i][t] * b[t][j] for t in range(k)) for j in range(m)] for i in range(n)]


@pytest.mark.parametrize("d1,d2,r,s", [(5, 3, 2, 2.0), (4, 7, 1, 0.5), (6, 6, 3, 1.0)])
def test_lora_projection_equals_merged_weight_bruteforce(d1, d2, r, s):
    """x (W + s A B) computed with Python loops equals the factored form of Eq. 1."""
    rng = np.random.default_rng(d1 * 100 + d2)
    x, W, A, B, b = _rand(rng, 3, d1), _rand(rng, d1, d2), _rand(rng, d1, r), _rand(rng, r, d2), _rand(rng, d2)
    AB = _loops_matmul(A.tolist(), B.tolist())
    Wm = [[W[i][j] + s * AB[i][j] for j in range(d2)] for i in range(d1)]
    ref = _loops_matmul(x.tolist(), Wm)
    ref = [[ref[i][j] + b[j] for j in range(d2)] for i in range(3)]
    got = O.lora_projection(x, W, A, B, s, b)
    np.testing.assert_allclose(got, np.array(ref), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(O.merged_weight(W, A, B, s), np.array(Wm), rtol=1e-12, atol=1e-13)
    # and the delta alone is x (s A B)
    dref = _loops_matmul(x.tolist(), [[s * v for v in row] for row in AB])
    np.testing.assert_allclose(O.lora_delta(x, A, B, s), np.array(dref), rtol=1e-12, atol=1e-13)


def test_lora_delta_closed_forms():
    rng = np.random.default_rng(7)
    d1, d2, r, s = 6, 4, 3, 2.0
    A, B = _rand(rng, d1, r), _rand(rng, r, d2)
    # unit vector picks row i of A
    for i in range(d1):
        e = np.zeros((1, d1)); e[0, i] = 1.0
        want = [s * math.fsum(A[i, k] * B[k, j] for k in range(r)) for j in range(d2)]
        np.testing.assert_allclose(O.lora_delta(e, A, B, s)[0], want, rtol=1e-13, atol=1e-15)
    # rank 1: s (x.a) b
    a, b = _rand(rng, d1, 1), _rand(rng, 1, d2)
    x = _rand(rng, 2, d1)
    for t in range(2):
        dot = math.fsum(x[t, i] * a[i, 0] for i in range(d1))
        np.testing.assert_allclose(O.lora_delta(x, a, b, s)[t], [s * dot * b[0, j] for j in range(d2)], rtol=1e-13)
    # B = 0 gives no change; linear in s and in x
    assert np.all(O.lora_delta(x, A, np.zeros_like(B), s) == 0.0)
    np.testing.assert_allclose(O.lora_delta(x, A, B, 3.0), 3.0 * O.lora_delta(x, A, B, 1.0), rtol=1e-13)
    x2 = _rand(rng, 2, d1)
    np.testing.assert_allclose(O.lora_delta(x + 2 * x2, A, B, s),
                               O.lora_delta(x, A, B, s) + 2 * O.lora_delta(x2, A, B, s), rtol=1e-12, atol=1e-14)
    # s = 1 and no LoRA term reduce to the plain linear module
    W = _rand(rng, d1, d2)
    np.testing.assert_allclose(O.lora_projection(x, W, A, np.zeros_like(B), 1.0), x @ W, rtol=1e-14)


def test_lora_hand_example():
    # x = [1, 2]; A = [[1],[1]] -> xA = 3; B = [[1, -1, 2]]; s = 2 -> delta = [6, -6, 12]
    # W = [[1,0,0],[0,1,0]] -> xW = [1,2,0]; b = [0,0,1]
    got = O.lora_projection([[1.0, 2.0]], [[1, 0, 0], [0, 1, 0]], [[1.0], [1.0]], [[1.0, -1.0, 2.0]], 2.0, [0, 0, 1.0])
    assert got.tolist() == [[7.0, -4.0, 13.0]]


def test_operand_orientation_is_checked_by_shapes():
    rng = np.random.default_rng(3)
    x, A, B = _rand(rng, 2, 5), _rand(rng, 5, 2), _rand(rng, 2, 3)
    with pytest.raises(ValueError):
        O.lora_delta(x, A.T, B, 1.0)
    with pytest.raises(ValueError):
        O.lora_delta(x, A, B.T, 1.0)


# ------------------------------------------------------------------ poolers (Eq. 2, Appendix C)
def test_poolers_hand_example():
    H = [[1.0, 0.0, 2.0], [3.0, 1.0, 0.0]]
    assert O.pool_mean(H).tolist() == [2.0, 0.5, 1.0]
    assert O.pool_last(H).tolist() == [3.0, 1.0, 0.0]
    assert O.pool_max(H).tolist() == [3.0, 1.0, 2.0]
    # w chosen so that U = H w = [0, ln 3]  ->  attention weights [1/4, 3/4]
    w = [math.log(3.0) / 3.0, 0.0, -math.log(3.0) / 6.0]
    np.testing.assert_allclose(O.pool_self_attention(H, w), [2.5, 0.75, 0.5], rtol=1e-14)


def test_poolers_special_cases():
    rng = np.random.default_rng(11)
    w = _rand(rng, 8)
    one = _rand(rng, 1, 8)
    for kind in (O.POOL_MEAN, O.POOL_LAST, O.POOL_MAX, O.POOL_SELFATTN):
        np.testing.assert_allclose(O.pool(one, kind, w), one[0], rtol=1e-15)
    same = np.repeat(one, 5, axis=0)
    for kind in (O.POOL_MEAN, O.POOL_LAST, O.POOL_MAX, O.POOL_SELFATTN):
        np.testing.assert_allclose(O.pool(same, kind, w), one[0], rtol=1e-14)
    H = _rand(rng, 6, 8)
    np.testing.assert_allclose(O.pool_self_attention(H, np.zeros(8)), O.pool_mean(H), rtol=1e-14)
    perm = rng.permutation(6)
    for kind in (O.POOL_MEAN, O.POOL_MAX, O.POOL_SELFATTN):
        np.testing.assert_allclose(O.pool(H[perm], kind, w), O.pool(H, kind, w), rtol=1e-13)
    assert not np.allclose(O.pool_last(H[::-1]), O.pool_last(H))
    # mean via python loops
    want = [math.fsum(H[t, i] for t in range(6)) / 6 for i in range(8)]
    np.testing.assert_allclose(O.pool_mean(H), want, rtol=1e-14)
    # self-attention weights favour the token with the largest score: a huge score isolates it
    big = np.zeros(8); big[0] = 1000.0
    Hs = H.copy(); Hs[:, 0] = 0.0; Hs[2, 0] = 1.0
    np.testing.assert_allclose(O.pool_self_attention(Hs, big), Hs[2], rtol=1e-12)


# ------------------------------------------------------------------ activations (Eq. 7)
def test_activations_tabulated_points():
    x = np.array([-2.0, -1.0, 0.0, 1.0, 2.0])
    np.testing.assert_allclose(O.activate(x, O.ACT_TANH),
                               [-0.9640275800758169, -0.7615941559557649, 0.0, 0.7615941559557649, 0.9640275800758169],
                               rtol=1e-15)
    assert O.activate(x, O.ACT_RELU).tolist() == [0.0, 0.0, 0.0, 1.0, 2.0]
    assert O.activate(x, O.ACT_IDENTITY).tolist() == x.tolist()
    # x * Phi(x) with the standard normal CDF values Phi(1) = 0.8413447460685429, Phi(2) = 0.9772498680518208
    np.testing.assert_allclose(O.activate(x, O.ACT_GELU),
                               [-2 * (1 - 0.9772498680518208), -(1 - 0.8413447460685429), 0.0,
                                0.8413447460685429, 2 * 0.9772498680518208], rtol=1e-13, atol=1e-16)


def test_rational_activation_closed_forms():
    x = np.array([-2.0, -0.5, 0.0, 0.5, 2.0])
    # a = (0, 1), b = () is the identity
    np.testing.assert_allclose(O.act_rational(x, [0.0, 1.0], []), x, rtol=1e-15)
    # b = 0: a polynomial (Horner form computed by hand below)
    a = [0.5, -1.0, 0.25, 2.0, 0.0, 0.0, 1.0]
    horner = ((((((a[6] * x + a[5]) * x + a[4]) * x + a[3]) * x + a[2]) * x + a[1]) * x + a[0])
    np.testing.assert_allclose(O.act_rational(x, a, [0.0] * 5), horner, rtol=1e-13)
    # hand numbers: a = (1, 2), b = (-3): x=2 -> 5 / (1+|-6|) = 5/7 ; x=-2 -> -3 / (1+|6|) = -3/7
    got = O.act_rational(np.array([2.0, -2.0]), [1.0, 2.0], [-3.0])
    np.testing.assert_allclose(got, [5.0 / 7.0, -3.0 / 7.0], rtol=1e-15)
    # the absolute value covers the whole denominator sum, not each term:
    # b = (1, -1) at x = 2: |2 - 4| = 2 -> den 3 (term-wise absolute values would give 7)
    np.testing.assert_allclose(O.act_rational(np.array([2.0]), [3.0], [1.0, -1.0]), [1.0], rtol=1e-15)
    # orders m = 6, n = 5 as in Section 4.3
    rng = np.random.default_rng(5)
    a6, b5 = rng.standard_normal(7) * 0.1, rng.standard_normal(5) * 0.1
    xs = 0.7
    num = sum(a6[j] * xs ** j for j in range(7))
    den = 1 + abs(sum(b5[i - 1] * xs ** i for i in range(1, 6)))
    np.testing.assert_allclose(O.activate(np.array([xs]), O.ACT_RATIONAL, a6, b5), [num / den], rtol=1e-14)


# ------------------------------------------------------------------ router (Eq. 3)
def test_softmax_properties():
    rng = np.random.default_rng(0)
    z = _rand(rng, 7) * 3
    p = O.softmax(z)
    assert abs(p.sum() - 1.0) < 1e-15 and np.all(p > 0)
    np.testing.assert_allclose(O.softmax(z + 123.0), p, rtol=1e-12)
    assert int(np.argmax(p)) == int(np.argmax(z))
    # two-class softmax is the logistic function
    np.testing.assert_allclose(O.softmax([0.0, math.log(3.0)]), [0.25, 0.75], rtol=1e-15)


def test_router_logits_hand_example_and_orientation():
    # g = [1, 2]; W_r (2 x 7): row0 = 0..6, row1 = 10,9,..,4  -> z_j = j + 2 (10 - j) = 20 - j
    W = np.array([list(range(7)), [10 - j for j in range(7)]], dtype=float)
    z = O.router_logits([1.0, 2.0], W)
    assert z.tolist() == [20.0 - j for j in range(7)]
    assert O.router_logits([1.0, 2.0], W, bias=np.arange(7.0) * 2).tolist() == [20.0 + j for j in range(7)]
    with pytest.raises(ValueError):
        O.router_logits([1.0, 2.0], W.T)


def test_top_k_order_and_ties():
    p = [0.1, 0.3, 0.3, 0.05, 0.2, 0.05, 0.0]
    assert O.top_k(p, 1).tolist() == [1]
    assert O.top_k(p, 3).tolist() == [1, 2, 4]
    assert O.top_k(p, 7).tolist() == [1, 2, 4, 0, 3, 5, 6]
    assert O.top_k([0.0] * 7, 1).tolist() == [0]


def test_route_prompt_pipeline():
    """A router whose column j equals a fixed direction u selects j when tanh(mean H) aligns with u."""
    rng = np.random.default_rng(2)
    d, n_p = 16, 5
    H = _rand(rng, n_p, d)
    g = np.tanh(H.mean(axis=0))
    for j in range(7):
        W = 0.01 * _rand(rng, d, 7)
        W[:, j] += g                      # logit j gains |g|^2
        out = O.route_prompt(H, W)
        assert out["route"] == j and out["topk"].tolist() == [j]
        assert out["margin"] > 0
        assert abs(out["probs"].sum() - 1) < 1e-14
        # the activation matters: with the identity the pooled vector is mean(H) itself
        out_id = O.route_prompt(H, W, activation=O.ACT_IDENTITY)
        np.testing.assert_allclose(out_id["logits"], H.mean(axis=0) @ W, rtol=1e-13)
        np.testing.assert_allclose(out["logits"], g @ W, rtol=1e-13)
    # bias decides between otherwise equal logits
    out = O.route_prompt(H, np.zeros((d, 7)), bias=[0, 0, 0, 0, 0, 1.0, 0])
    assert out["route"] == 5
    out = O.route_prompt(H, np.zeros((d, 7)))
    assert out["route"] == 0 and out["margin"] == 0.0   # all tied: lowest index


def test_route_batch_indexing():
    """Slots, tenants and layers are indexed independently; a mix-up of any two is caught."""
    rng = np.random.default_rng(4)
    d, L, R = 8, 3, 6
    lens = [3, 1, 4]
    cu = np.concatenate([[0], np.cumsum(lens)])
    H = _rand(rng, int(cu[-1]), d)
    seq_slot = [4, 0, 2]
    slot_tenant = [2, -1, 0, -1, 1, -1]
    Ws = {(t, l): _rand(rng, d, 7) for t in range(3) for l in range(L)}
    table = np.full((R, L), -1, dtype=np.int32)
    logits, margins = O.route_batch(H, cu, seq_slot, slot_tenant, lambda t, l: {"W_r": Ws[(t, l)]}, 1, table)
    for p, slot in enumerate(seq_slot):
        Hp = H[cu[p]:cu[p + 1]]
        z = np.tanh(Hp.mean(axis=0)) @ Ws[(slot_tenant[slot], 1)]
        np.testing.assert_allclose(logits[p], z, rtol=1e-13)
        assert table[slot, 1] == int(np.argmax(z))
        zs = np.sort(z)
        assert abs(margins[p] - (zs[-1] - zs[-2])) < 1e-14
    assert np.all(table[:, 0] == -1) and np.all(table[:, 2] == -1)
    assert np.all(table[[1, 3, 5], 1] == -1)


# ------------------------------------------------------------------ grouping
def test_group_tokens_hand_example():
    # slots: 0 -> tenant 1 routed to module 2; 1 -> tenant 0 module 2; 2 -> tenant 1 module 0;
    #        3 -> closed; 4 -> tenant 2 module 5 but no adapter there
    slot_tenant = [1, 0, 1, -1, 2]
    route_col = [2, 2, 0, 3, 5]
    token_slot = [0, 1, 2, 0, 3, 4, 1, 2, 0]
    has = lambda tenant, module: not (tenant == 2 and module == 5)
    g = O.group_tokens(token_slot, slot_tenant, route_col, has, max_tenants=10)
    # keys: module*10 + tenant : slot0 -> 21, slot1 -> 20, slot2 -> 1
    assert g["perm"].tolist() == [2, 7, 1, 6, 0, 3, 8]
    assert g["seg_key"].tolist() == [1, 20, 21]
    assert g["seg_offset"].tolist() == [0, 2, 4, 7]
    assert g["mod_offset"].tolist() == [0, 1, 1, 3, 3, 3, 3, 3]
    assert g["n_excluded"] == 2


def test_group_tokens_matches_library_sort_and_invariants():
    rng = random.Random(9)
    R, T, max_tenants = 12, 200, 5
    slot_tenant = [rng.choice([-1, 0, 1, 2, 3, 4]) for _ in range(R)]
    route_col = [rng.randrange(-1, 7) for _ in range(R)]
    token_slot = [rng.randrange(R) for _ in range(T)]
    missing = {(1, 3), (4, 0)}
    g = O.group_tokens(token_slot, slot_tenant, route_col, lambda t, m: (t, m) not in missing, max_tenants)
    keys = []
    for t in range(T):
        s = token_slot[t]
        ok = slot_tenant[s] >= 0 and route_col[s] >= 0 and (slot_tenant[s], route_col[s]) not in missing
        keys.append(route_col[s] * max_tenants + slot_tenant[s] if ok else -1)
    keys = np.array(keys)
    act = np.nonzero(keys >= 0)[0]
    order = act[np.lexsort((act, keys[act]))]          # library routine: sort by key, then token index
    assert g["perm"].tolist() == order.tolist()
    assert g["n_excluded"] + len(g["perm"]) == T
    assert sorted(g["perm"].tolist()) == act.tolist()
    assert list(g["seg_key"]) == sorted(set(keys[act].tolist()))
    for s in range(len(g["seg_key"])):
        seg = g["perm"][g["seg_offset"][s]:g["seg_offset"][s + 1]]
        assert len(seg) > 0 and np.all(keys[seg] == g["seg_key"][s]) and np.all(np.diff(seg) > 0)
    assert g["mod_offset"][-1] == len(g["seg_key"])
    for m in range(7):
        ks = g["seg_key"][g["mod_offset"][m]:g["mod_offset"][m + 1]]
        assert np.all(ks // max_tenants == m)


def test_group_tokens_empty_and_all_excluded():
    g = O.group_tokens([], [0], [0], lambda t, m: True, 4)
    assert g["perm"].size == 0 and g["seg_key"].size == 0 and g["n_excluded"] == 0
    assert g["mod_offset"].tolist() == [0] * 8
    g = O.group_tokens([0, 0], [-1], [0], lambda t, m: True, 4)
    assert g["perm"].size == 0 and g["n_excluded"] == 2


# ------------------------------------------------------------------ selection + reuse
def _tiny_stack(rng, d=8, d_ff=12, r=2, tenants=3):
    ad = {}
    for t in range(tenants):
        for m in range(7):
            d1, d2 = O.module_dims(d, d_ff, d, m)
            ad[(t, m)] = (_rand(rng, d1, r), _rand(rng, r, d2), 2.0)
    return ad


def test_group_tokens_top_k_hand_example_and_library_sort():
    """Eq. 3 with k > 1: a token sits in one bucket per selected module that has an adapter."""
    # slot 0: tenant 1 selects modules (2, 0); slot 1: tenant 0 selects (2, 5) but has no adapter on 5;
    # slot 2: closed; slot 3: tenant 2 selects (6, -1)
    slot_tenant = [1, 0, -1, 2]
    sel = np.array([[2, 0], [2, 5], [1, 3], [6, -1]])
    token_slot = [0, 1, 2, 3, 0]
    has = lambda tenant, module: not (tenant == 0 and module == 5)
    g = O.group_tokens(token_slot, slot_tenant, sel, has, max_tenants=10)
    # keys: slot0 -> 21 and 1; slot1 -> 20; slot3 -> 62
    assert g["seg_key"].tolist() == [1, 20, 21, 62]
    assert g["perm"].tolist() == [0, 4, 1, 0, 4, 3]
    assert g["seg_offset"].tolist() == [0, 2, 3, 5, 6]
    assert g["mod_offset"].tolist() == [0, 1, 1, 3, 3, 3, 3, 4]
    assert g["n_excluded"] == 1
    # a 2-D selection with one column is the top-1 case
    col = np.array([2, 2, 1, 6])
    g1 = O.group_tokens(token_slot, slot_tenant, col, has, 10)
    g2 = O.group_tokens(token_slot, slot_tenant, col[:, None], has, 10)
    for key in ("perm", "seg_key", "seg_offset", "mod_offset"):
        assert np.array_equal(g1[key], g2[key])
    # random case against a library sort of the explicit (key, token) pairs
    rng = random.Random(31)
    R, T, k, max_tenants = 9, 150, 3, 4
    slot_tenant = [rng.choice([-1, 0, 1, 2, 3]) for _ in range(R)]
    sel = np.array([rng.sample(range(7), k) for _ in range(R)])
    sel[2, 1] = -1
    token_slot = [rng.randrange(R) for _ in range(T)]
    missing = {(1, 3), (2, 0), (3, 6)}
    g = O.group_tokens(token_slot, slot_tenant, sel, lambda t, m: (t, m) not in missing, max_tenants)
    keys, toks = [], []
    for t in range(T):
        s_ = token_slot[t]
        for m in sel[s_]:
            if slot_tenant[s_] >= 0 and m >= 0 and (slot_tenant[s_], int(m)) not in missing:
                keys.append(int(m) * max_tenants + slot_tenant[s_]); toks.append(t)
    keys, toks = np.array(keys), np.array(toks)
    order = np.lexsort((toks, keys))
    assert g["perm"].tolist() == toks[order].tolist()
    assert g["n_excluded"] == T - len(set(toks.tolist()))
    assert list(g["seg_key"]) == sorted(set(keys.tolist()))
    counts = np.bincount(g["perm"], minlength=T)
    assert counts.max() <= k


def test_gate_weights_scale_the_lora_term():
    """Weights of one reproduce hard selection; any weight scales that module's term linearly."""
    rng = np.random.default_rng(33)
    d, d_ff = 8, 12
    ad = _tiny_stack(rng, d, d_ff, tenants=2)
    slot_tenant = [0, 1]
    sel = np.array([[4, 1], [1, 6]])
    gate = np.array([[0.7, 0.2], [0.5, 0.25]])
    token_slot = [0, 1, 1]
    get = lambda t, mm: ad.get((t, mm))
    for m in (1, 4, 6, 0):
        d1, d2 = O.module_dims(d, d_ff, d, m)
        x, yb = _rand(rng, 3, d1), _rand(rng, 3, d2)
        hard = O.apply_module(yb, x, token_slot, slot_tenant, sel, m, get)
        ones = O.apply_module(yb, x, token_slot, slot_tenant, sel, m, get, gate=np.ones((2, 2)))
        assert np.array_equal(hard, ones)
        soft = O.apply_module(yb, x, token_slot, slot_tenant, sel, m, get, gate=gate)
        for t, slot in enumerate(token_slot):
            if m in sel[slot]:
                wgt = gate[slot][list(sel[slot]).index(m)]
                A, B, s_ = ad[(slot_tenant[slot], m)]
                np.testing.assert_allclose(soft[t], yb[t] + wgt * s_ * (x[t] @ A) @ B, rtol=1e-13)
                np.testing.assert_allclose(soft[t] - yb[t], wgt * (hard[t] - yb[t]), rtol=1e-10, atol=1e-14)
            else:
                assert np.array_equal(soft[t], yb[t])
        rows = [2, 0]
        samp = O.apply_module_sampled(yb[rows], x[rows], rows, token_slot, slot_tenant, sel, m, get, gate=gate)
        assert np.array_equal(samp, soft[rows])


def test_apply_module_selection_invariants():
    rng = np.random.default_rng(21)
    d, d_ff = 8, 12
    ad = _tiny_stack(rng, d, d_ff)
    slot_tenant = [0, 1, 2, -1]
    route = np.array([4, 6, 4, 4])
    token_slot = [0, 1, 2, 3, 0, 2]
    for m in range(7):
        d1, d2 = O.module_dims(d, d_ff, d, m)
        x, yb = _rand(rng, 6, d1), _rand(rng, 6, d2)
        y = O.apply_module(yb, x, token_slot, slot_tenant, route, m, lambda t, mm: ad.get((t, mm)))
        for t, slot in enumerate(token_slot):
            if slot_tenant[slot] >= 0 and route[slot] == m:
                A, B, s = ad[(slot_tenant[slot], m)]
                np.testing.assert_allclose(y[t], yb[t] + s * (x[t] @ A) @ B, rtol=1e-13)
                assert not np.array_equal(y[t], yb[t])
            else:
                assert np.array_equal(y[t], yb[t])      # bit-identical, not merely close
    # sampled variant agrees with the full one
    m = 4
    d1, d2 = O.module_dims(d, d_ff, d, m)
    x, yb = _rand(rng, 6, d1), _rand(rng, 6, d2)
    full = O.apply_module(yb, x, token_slot, slot_tenant, route, m, lambda t, mm: ad.get((t, mm)))
    rows = [5, 0, 3]
    samp = O.apply_module_sampled(yb[rows], x[rows], rows, token_slot, slot_tenant, route, m,
                                  lambda t, mm: ad.get((t, mm)))
    assert np.array_equal(samp, full[rows])


def test_all_experts_active_reduces_to_plain_lora():
    """Section 4.5 (k sweep): with every expert selected the method is vanilla LoRA on all 7 modules."""
    rng = np.random.default_rng(22)
    d, d_ff = 8, 12
    ad = _tiny_stack(rng, d, d_ff, tenants=1)
    route_all = np.tile(np.arange(7), (1, 1))          # slot 0 selects all seven
    for m in range(7):
        d1, d2 = O.module_dims(d, d_ff, d, m)
        x, W = _rand(rng, 3, d1), _rand(rng, d1, d2)
        yb = O.base_projection(x, W)
        y = O.apply_module(yb, x, [0, 0, 0], [0], route_all, m, lambda t, mm: ad.get((t, mm)))
        A, B, s = ad[(0, m)]
        np.testing.assert_allclose(y, x @ O.merged_weight(W, A, B, s), rtol=1e-12, atol=1e-13)


def test_route_is_fixed_by_the_prompt_alone():
    """Section 3.3: the decision is computed from the prompt's hidden states and then reused.
    A variant that pooled generated tokens as well must be able to change the decision,
    otherwise this test would have no power."""
    rng = np.random.default_rng(23)
    d = 16
    W = _rand(rng, d, 7)
    flips = 0
    for trial in range(50):
        H = _rand(rng, 4, d)
        route0 = O.route_prompt(H, W)["route"]
        table = np.full((1, 1), -1, dtype=np.int32)
        O.route_batch(H, [0, 4], [0], [0], lambda t, l: {"W_r": W}, 0, table)
        assert table[0, 0] == route0
        gen = _rand(rng, 4, d) * 3
        snapshot = table.copy()
        # decode steps only read the table: each generated token gets its term on the module the PROMPT selected,
        # whatever its own hidden state would have selected, and applying never writes the table
        A, B = _rand(rng, d, 2), _rand(rng, 2, d)
        for step in range(4):
            x = gen[step:step + 1]
            y_base = _rand(rng, 1, d)
            for module in range(O.N_MOD):
                y = O.apply_module(y_base, x, [0], [0], table[:, 0], module, lambda t, m: (A, B, 2.0))
                assert np.array_equal(y != y_base, np.full_like(y_base, module == route0, dtype=bool))
            assert np.array_equal(table, snapshot)
        if O.route_prompt(np.vstack([H, gen]), W)["route"] != route0:
            flips += 1
    assert flips > 0


def test_max_rel_err_metric():
    ref = np.array([1.0, -2.0, 0.0, 4.0])
    rms = math.sqrt((1 + 4 + 0 + 16) / 4)
    y = ref + np.array([0.1, 0.0, 0.2, -0.4])
    want = max(0.1 / rms, 0.2 / rms, 0.4 / 4.0)
    assert abs(O.max_rel_err(y, ref) - want) < 1e-15
    assert O.max_rel_err(ref, ref) == 0.0
    assert O.max_rel_err(np.zeros(0), np.zeros(0)) == 0.0
