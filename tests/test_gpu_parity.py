"""GPU parity: every step of the hot path, through the C ABI, element by element against the fp64 oracle."""
import numpy as np
import pytest
import torch

from oracle import milora_oracle as O
from oracle import reference_run as R
from synth import get_workload
from synth.workloads import scaled_workload

from parity_utils import assert_apply_close, assert_groups_equal, compare_routes, read_group_block

pytestmark = pytest.mark.gpu


def _loaded(w, **kw):
    from paper_2410_18035_b200.workload_runner import LoadedWorkload
    return LoadedWorkload(w, "cuda", **kw)


def _route_all_layers(lw, ids, **okw):
    """Route on the GPU and with the oracle; returns (gpu table, oracle table, excused mismatches)."""
    w = lw.w
    table_o = np.full((w.n_requests, len(lw.layers)), -1, dtype=np.int32)
    excused = 0
    P = len(ids)
    logits = torch.zeros((P, 7), dtype=torch.float32, device="cuda")
    probs = torch.zeros((P, 7), dtype=torch.float32, device="cuda")
    for li, layer in enumerate(lw.layers):
        lw.route(li, ids, logits=logits, probs=probs)
        tmp = np.full((w.n_requests, w.n_layers), -1, dtype=np.int32)
        lo, margins = R.route_requests(w, layer, ids, tmp, **okw)
        table_o[:, li] = tmp[:, layer]
        table_g = lw.ml.route_table_read(0, w.n_requests).numpy()
        excused += compare_routes(table_g[list(ids), li], table_o[list(ids), li], margins)
        # logits: fp32 accumulation over d terms against fp64
        lg = logits.cpu().numpy().astype(np.float64)
        scale = max(1e-3, float(np.abs(lo).max()))
        assert np.abs(lg - lo).max() <= 2e-4 * scale, "router logits"
        np.testing.assert_allclose(probs.cpu().numpy(), O.softmax(lo), atol=2e-4)
    table_g = lw.ml.route_table_read(0, w.n_requests).numpy()
    return table_g, table_o, excused


def _step_parity(lw, li, prefill_ids, decode_ids, table, tag, use_multi=False, gate=None, decode_path="auto",
                 shared=None):
    """group + apply (prefill and decode lists) on one step; compares grouping and all 7 module outputs.
    table is [R, L] (top-1) or [R, L, k]; gate, when given, holds the [R, L, k] weights of the selected modules.
    decode_path picks the kernel set of milora_apply_decode (bf16 contexts).  shared: lists of modules that are
    given one input matrix; the prefill rows then go through milora_apply_prefill_shared (use_multi: through
    milora_apply_prefill_multi with equal X pointers)."""
    w, ml = lw.w, lw.ml
    ml.set_decode_path(decode_path)
    layer = lw.layers[li]
    cu, slots, T = lw.seq_arrays(prefill_ids, decode_ids)
    n_seq = slots.numel()
    ws = ml.alloc_group_ws(1, n_seq, T)
    ml.group(li, 1, cu, slots, n_seq, T, ws)
    cu_h = cu.cpu().numpy()
    token_slot = np.repeat(slots.cpu().numpy(), np.diff(cu_h))
    g_o = R.group_layer(w, token_slot, table[:, li])
    g_o["max_tenants"] = w.n_tenants
    g_g = read_group_block(ml, ws[0], n_seq, T)
    assert_groups_equal(g_g, g_o, cu_h)
    groups = ml.groups(ws[0], n_seq, T)
    Xs, Ys, Ybs = [], [], []
    for m in range(7):
        X = w.module_input(layer, m, T, tag, "cuda")
        if w.has_base_weights:
            Yb = (X.float() @ w.base_weight(layer, m, "cuda").float()).to(w.torch_dtype)
        else:
            Yb = w.base_output(layer, m, T, tag, "cuda")
        Xs.append(X); Ybs.append(Yb); Ys.append(Yb.clone())
    for mods in shared or []:
        for m in mods[1:]:
            Xs[m] = Xs[mods[0]]
    if shared and not use_multi:
        rest = [m for m in range(7) if not any(m in mods for mods in shared)]
        for mods in shared:
            ml.apply_prefill_shared(li, list(mods), Xs[mods[0]], [Ys[m] for m in mods], groups)
        for m in rest:
            ml.apply_prefill(li, m, Xs[m], Ys[m], groups)
        ml.apply_decode_multi(li, list(range(7)), Xs, Ys, groups)
    elif use_multi:
        ml.apply_prefill_multi(li, list(range(7)), Xs, Ys, groups)
        ml.apply_decode_multi(li, list(range(7)), Xs, Ys, groups)
    else:
        for m in range(7):
            ml.apply_prefill(li, m, Xs[m], Ys[m], groups)
            ml.apply_decode(li, m, Xs[m], Ys[m], groups)
    torch.cuda.synchronize()
    worst = 0.0
    for m in range(7):
        y_o = R.apply_site(w, layer, m, Xs[m].cpu(), Ybs[m].cpu(), token_slot, table[:, li],
                           gate=None if gate is None else gate[:, li])
        worst = max(worst, assert_apply_close(Ys[m], y_o, Ybs[m], w.dtype, what=f"{w.name} layer {layer} module {m}"))
    assert ml.poll_error() == 0
    return worst


def test_config1_full_path_fp32():
    """Config 1: route from the prompts, prefill apply, then 4 decode steps that only read the table."""
    w = get_workload("c1")
    lw = _loaded(w)
    ids = list(range(w.n_requests))
    table_g, table_o, excused = _route_all_layers(lw, ids)
    assert excused == 0 and np.array_equal(table_g, table_o)
    for li in range(len(lw.layers)):
        _step_parity(lw, li, ids, [], table_o, tag=0)
    before = lw.ml.route_table_read().numpy().copy()
    for step in range(w.decode_steps):
        for li in range(len(lw.layers)):
            _step_parity(lw, li, [], ids, table_o, tag=100 + step, use_multi=(step % 2 == 1))
    assert np.array_equal(lw.ml.route_table_read().numpy(), before), "decode steps must not touch the route table"
    lw.close()


def test_config1_base_projection_identity():
    """On the routed module the result equals x (W + s A B) computed by the oracle from the weights."""
    w = get_workload("c1")
    lw = _loaded(w)
    ids = list(range(4))
    _, table_o, _ = _route_all_layers(lw, ids)
    li = 0
    cu, slots, T = lw.seq_arrays(ids, [])
    ws = lw.ml.alloc_group_ws(1, 4, T)
    lw.ml.group(li, 1, cu, slots, 4, T, ws)
    groups = lw.ml.groups(ws[0], 4, T)
    token_slot = np.repeat(np.arange(4), 16)
    for m in range(7):
        X = w.module_input(0, m, T, 5, "cuda")
        W = w.base_weight(0, m, "cuda")
        Y = (X @ W).contiguous()
        lw.ml.apply_prefill(li, m, X, Y, groups)
        lw.ml.apply_decode(li, m, X, Y, groups)
        yg = R.to_f64(Y)
        for t in range(T):
            slot = token_slot[t]
            Wm = R.to_f64(W)
            if table_o[slot, 0] == m:
                A, B = w.adapter(int(w.request_tenant[slot]), 0, m)
                Wm = O.merged_weight(Wm, R.to_f64(A), R.to_f64(B), w.scale)
            ref = R.to_f64(X[t].cpu()) @ Wm
            assert O.max_rel_err(yg[t], ref) <= 1e-4
    lw.close()


RAGGED = [1, 33, 130, 257, 31, 32, 7, 129]


@pytest.mark.parametrize("dtype,d,d_ff,d_kv,r", [("f32", 256, 688, 256, 8), ("bf16", 512, 1376, 128, 16),
                                                 ("bf16", 256, 688, 256, 40), ("bf16", 1024, 2816, 256, 16),
                                                 ("bf16", 512, 1408, 512, 32), ("bf16", 512, 1408, 128, 64),
                                                 ("bf16", 256, 768, 256, 40)])
@pytest.mark.parametrize("decode_path", ["cluster", "split", "stream"])
def test_ragged_mixed_batch(dtype, d, d_ff, d_kv, r, decode_path):
    """Sequences of 1..257 rows (both work lists, ragged tile tails) mixed with decode rows; tenants repeat so
    that several sequences share a bucket; one slot is closed and one tenant has no adapters."""
    base = get_workload("c1")
    n = len(RAGGED) + 6
    lens = np.array(RAGGED + [16] * 6, dtype=np.int32)
    tenants = np.array([0, 1, 2, 0, 1, 3, 2, 0, 0, 1, 1, 2, 3, 0], dtype=np.int32)
    w = scaled_workload(base, name=f"ragged_{dtype}", dtype=dtype, d_model=d, d_ff=d_ff, d_kv=d_kv, rank=r,
                        n_tenants=5, request_tenant=tenants, prompt_len=lens, prefill_ids=np.arange(len(RAGGED)),
                        decode_ids=np.arange(len(RAGGED), n), has_base_weights=False, n_layers=2)
    lw = _loaded(w, tenants=[0, 1, 2, 3])
    ids = list(range(n))
    table_g, table_o, excused = _route_all_layers(lw, ids)
    assert excused <= 1
    table = table_g.copy()        # use the GPU's decisions downstream so that an excused near tie cannot cascade
    prefill, decode = list(range(len(RAGGED))), list(range(len(RAGGED), n))
    for li in range(2):
        _step_parity(lw, li, prefill, decode, table, tag=7, decode_path=decode_path)
        _step_parity(lw, li, prefill[::-1], decode, table, tag=8, use_multi=True, decode_path=decode_path)
    # close a slot: its rows become excluded and stay bit-identical
    lw.ml.request_close(3)
    w.request_tenant = w.request_tenant.copy()
    w.request_tenant[3] = -1
    _step_parity(lw, 0, prefill, decode, table, tag=9, decode_path=decode_path)
    lw.close()


@pytest.mark.parametrize("dtype,d,d_ff,d_kv,r,k,gate", [("f32", 256, 688, 256, 8, 3, 0), ("bf16", 512, 1408, 128, 16, 3, 0),
                                                        ("bf16", 512, 1408, 512, 32, 2, 1), ("f32", 256, 688, 256, 8, 7, 1),
                                                        ("bf16", 256, 688, 256, 40, 3, 1), ("bf16", 2048, 1408, 256, 16, 3, 0),
                                                        ("bf16", 512, 1408, 512, 64, 5, 1)])
def test_top_k_routing_grouping_and_apply(dtype, d, d_ff, d_kv, r, k, gate):
    """Eq. 3 with k > 1 (Section 4.5 sweeps k): the route table holds the k best modules in order, every token
    is bucketed once per selected module and receives each selected module's LoRA term, optionally weighted by
    the router probability."""
    base = get_workload("c1")
    n = len(RAGGED) + 6
    lens = np.array(RAGGED + [16] * 6, dtype=np.int32)
    tenants = np.array([0, 1, 2, 0, 1, 3, 2, 0, 0, 1, 1, 2, 3, 0], dtype=np.int32)
    w = scaled_workload(base, name=f"topk_{dtype}", dtype=dtype, d_model=d, d_ff=d_ff, d_kv=d_kv, rank=r,
                        n_tenants=5, request_tenant=tenants, prompt_len=lens, prefill_ids=np.arange(len(RAGGED)),
                        decode_ids=np.arange(len(RAGGED), n), has_base_weights=False, n_layers=2)
    lw = _loaded(w, tenants=[0, 1, 2, 3], top_k=k, gate=gate)
    ids = list(range(n))
    P = len(ids)
    logits = torch.zeros((P, 7), dtype=torch.float32, device="cuda")
    probs_o = np.zeros((w.n_requests, 2, 7))
    excused = 0
    for li in range(2):
        lw.route(li, ids, logits=logits)
        tmp = np.full((w.n_requests, w.n_layers), -1, dtype=np.int32)
        topk_o = np.full((w.n_requests, w.n_layers, k), -1, dtype=np.int32)
        lo, _ = R.route_requests(w, li, ids, tmp, k=k, topk_table=topk_o)
        probs_o[ids, li] = O.softmax(lo)
        table_g = lw.ml.route_table_read(0, w.n_requests).numpy().reshape(w.n_requests, 2, k)
        for p, i in enumerate(ids):
            assert len(set(table_g[i, li].tolist())) == k
            if not np.array_equal(table_g[i, li], topk_o[i, li]):
                zs = np.sort(lo[p])[::-1]
                gaps = zs[:k] - zs[1:k + 1] if k < 7 else zs[:6] - zs[1:7]
                assert gaps.min() < 1e-3, f"top-k mismatch at request {i}: {table_g[i, li]} vs {topk_o[i, li]}"
                excused += 1
    assert excused <= 2
    table = lw.ml.route_table_read(0, w.n_requests).numpy().reshape(w.n_requests, 2, k).copy()
    gates_g = lw.ml.gate_table_read(0, w.n_requests).numpy()
    gates_o = np.take_along_axis(probs_o, table.astype(np.int64), axis=2)
    np.testing.assert_allclose(gates_g, gates_o, atol=2e-4)
    gate_arg = gates_o if gate else None
    prefill, decode = list(range(len(RAGGED))), list(range(len(RAGGED), n))
    for li in range(2):
        _step_parity(lw, li, prefill, decode, table, tag=11, gate=gate_arg, decode_path="cluster")
        _step_parity(lw, li, prefill[::-1], decode, table, tag=12, use_multi=True, gate=gate_arg, decode_path="split")
        # q, k, v read one matrix and gate, up another (Section 3.1 lists the seven modules of a block): one X tile
        # feeds the shrink of every selected module of the group
        _step_parity(lw, li, prefill, decode, table, tag=13, gate=gate_arg, shared=[(0, 1, 2), (4, 5)])
        _step_parity(lw, li, prefill[::-1], decode, table, tag=14, use_multi=True, gate=gate_arg,
                     shared=[(0, 1, 2), (4, 5)])
        # more siblings than one pass takes: five modules on one matrix
        _step_parity(lw, li, prefill, decode, table, tag=15, use_multi=True, gate=gate_arg, shared=[(5, 0, 4, 2, 1)])
    # modules that do not have the same input width cannot share an input matrix
    if dtype == "bf16":
        import ctypes as C
        from paper_2410_18035_b200 import MiloraError
        cu_s, slots_s, T_s = lw.seq_arrays(prefill, [])
        ws_s = lw.ml.alloc_group_ws(1, len(prefill), T_s)
        lw.ml.group(0, 1, cu_s, slots_s, len(prefill), T_s, ws_s)
        g_s = lw.ml.groups(ws_s[0], len(prefill), T_s)
        Xq = w.module_input(lw.layers[0], 0, T_s, 16, "cuda")
        Yq, Yd = w.base_output(lw.layers[0], 0, T_s, 16, "cuda"), w.base_output(lw.layers[0], 6, T_s, 16, "cuda")
        mods = (C.c_int * 2)(0, 6)
        ys = (C.c_void_p * 2)(Yq.data_ptr(), Yd.data_ptr())
        st = lw.ml.lib.milora_apply_prefill_shared(lw.ml.h, 0, 2, mods, C.c_void_p(Xq.data_ptr()), ys, C.byref(g_s), None)
        assert st == 1, "q and down read matrices of different widths: MILORA_E_ARG"
    # restoring a table by hand: duplicates inside a cell are refused
    from paper_2410_18035_b200 import MiloraError
    if k >= 2:
        bad = table[:1].copy()
        bad[0, 0, 1] = bad[0, 0, 0]
        with pytest.raises(MiloraError):
            lw.ml.route_table_write(0, bad)
    lw.ml.route_table_write(0, table)
    assert np.array_equal(lw.ml.route_table_read(0, w.n_requests).numpy().reshape(table.shape), table)
    lw.close()


def _assert_fused_close(Y, y_o, y_base_o, what, twice_rounded_rows=None):
    """Fused projection against the oracle's x W + b + delta: full-output metric, and per element an error
    budget of the delta tolerance plus the rounding of the stored bf16 output and of the fp32 accumulation.  The
    output is rounded once (half an ulp), except on the rows of `twice_rounded_rows` (decode rows: the projection
    is stored, then the gathered kernel adds the LoRA term to the stored value: two roundings)."""
    from parity_utils import TOL, half_ulp
    yg, yr = R.to_f64(Y), np.asarray(y_o, dtype=np.float64)
    assert O.max_rel_err(yg, yr) <= TOL["bf16"], what
    delta = yr - y_base_o
    rms = np.sqrt(np.mean(delta[np.any(delta != 0, axis=1)] ** 2)) if np.any(delta != 0) else 0.0
    roundings = np.full((yr.shape[0], 1), 1.01)
    if twice_rounded_rows is not None:
        roundings[np.asarray(twice_rounded_rows)] = 2.02
    allowed = TOL["bf16"] * np.where(delta != 0, np.maximum(np.abs(delta), rms), 0.0) + roundings * half_ulp(yr, "bf16") + 2e-5
    worst = float((np.abs(yg - yr) / allowed).max())
    assert worst <= 1.0, f"{what}: error is {worst:.3f}x the allowed bound"


@pytest.mark.parametrize("d,d_ff,d_kv,r,k", [(512, 1536, 256, 16, 1), (256, 768, 256, 32, 1), (512, 1536, 512, 8, 3)])
def test_fused_projection_matches_oracle(d, d_ff, d_kv, r, k):
    """milora_linear_prefill: y = x W + b + s (x A) B on the routed prompt rows in one kernel (Eq. 1), ragged
    sequences that straddle the 128-row blocks of the GEMM, then the decode rows through milora_apply_decode."""
    base = get_workload("c1")
    n = len(RAGGED) + 6
    lens = np.array(RAGGED + [1] * 6, dtype=np.int32)
    tenants = np.array([0, 1, 2, 0, 1, 3, 2, 0, 0, 1, 1, 2, 3, 0], dtype=np.int32)
    w = scaled_workload(base, name="fused", dtype="bf16", d_model=d, d_ff=d_ff, d_kv=d_kv, rank=r, n_tenants=5,
                        request_tenant=tenants, prompt_len=lens, prefill_ids=np.arange(len(RAGGED)),
                        decode_ids=np.arange(len(RAGGED), n), has_base_weights=False, n_layers=1)
    lw = _loaded(w, tenants=[0, 1, 2, 3], top_k=k)
    ml = lw.ml
    ids = list(range(n))
    lw.route(0, ids)
    table = ml.route_table_read(0, w.n_requests).numpy().reshape(w.n_requests, 1, k)
    prefill, decode = list(range(len(RAGGED)))[::-1], list(range(len(RAGGED), n))
    cu, slots, T = lw.seq_arrays(prefill, decode)
    n_seq = slots.numel()
    ws = ml.alloc_group_ws(1, n_seq, T)
    ml.group(0, 1, cu, slots, n_seq, T, ws)
    groups = ml.groups(ws[0], n_seq, T)
    token_slot = np.repeat(slots.cpu().numpy(), np.diff(cu.cpu().numpy()))
    for m in range(7):
        X = w.module_input(0, m, T, 21, "cuda")
        W = w.base_weight(0, m, "cuda")
        bias = (w.base_output(0, m, 1, 22, "cuda")[0] * 0.1).contiguous() if m % 2 else None
        Y = torch.full((T, W.shape[1]), float("nan"), dtype=torch.bfloat16, device="cuda")
        ml.linear_prefill(0, m, X, W.t().contiguous(), Y, groups, bias=bias)
        ml.apply_decode(0, m, X, Y, groups)
        torch.cuda.synchronize()
        yb = O.base_projection(R.to_f64(X), R.to_f64(W), None if bias is None else R.to_f64(bias))
        y_o = R.apply_site(w, 0, m, X.cpu(), yb, token_slot, table[:, 0])
        short = np.nonzero(np.diff(cu.cpu().numpy())[np.searchsorted(cu.cpu().numpy(), np.arange(T), side="right") - 1] < 32)[0]
        _assert_fused_close(Y, y_o, yb, f"fused projection module {m}", twice_rounded_rows=short)
    assert ml.poll_error() == 0
    lw.close()


def test_fused_projection_refuses_what_it_cannot_run():
    """Shapes and dtypes outside the tensor-core kernel's limits are refused before anything is launched."""
    from paper_2410_18035_b200 import Milora, MiloraError
    def call(ml, module, T, dtype):
        d1, d2 = ml.module_dims(module)
        X = torch.zeros((T, d1), dtype=dtype, device="cuda")
        Wt = torch.zeros((d2, d1), dtype=dtype, device="cuda")
        Y = torch.full((T, d2), 7.0, dtype=dtype, device="cuda")
        slots = torch.zeros(1, dtype=torch.int32, device="cuda")
        cu = torch.tensor([0, T], dtype=torch.int32, device="cuda")
        ws = ml.alloc_group_ws(1, 1, T)
        ml.request_open(0, 0) if not getattr(ml, "_opened", False) else None
        ml._opened = True
        ml.group(0, 1, cu, slots, 1, T, ws)
        ml.linear_prefill(0, module, X, Wt, Y, ml.groups(ws[0], 1, T))
        torch.cuda.synchronize()
        return Y
    ml = Milora(1, 256, 768, 256, "f32", 8, 2, 2)                 # fp32 context
    with pytest.raises(MiloraError) as e:
        call(ml, 0, 256, torch.float32)
    assert e.value.status == 2
    ml.close()
    ml = Milora(1, 512, 1408, 128, "bf16", 16, 2, 2)              # d_ff and d_kv are not multiples of 256
    for module in (1, 4):
        with pytest.raises(MiloraError) as e:
            call(ml, module, 256, torch.bfloat16)
        assert e.value.status == 2
    with pytest.raises(MiloraError) as e:                         # fewer rows than one tile
        call(ml, 0, 64, torch.bfloat16)
    assert e.value.status == 2
    # a step without any routed adapter is a plain projection: x = 0 gives y = 0 on every row
    Y = call(ml, 0, 300, torch.bfloat16)
    assert float(Y.float().abs().max()) == 0.0
    assert ml.poll_error() == 0
    ml.close()
    ml = Milora(1, 512, 1536, 256, "bf16", 64, 2, 2)              # rank limit of the fused kernel
    with pytest.raises(MiloraError) as e:
        call(ml, 0, 256, torch.bfloat16)
    assert e.value.status == 2
    ml.close()


@pytest.mark.parametrize("decode_path", ["cluster", "split", "stream"])
def test_back_to_back_launches_equal_serialised_ones_bit_for_bit(decode_path):
    """Every kernel may start while the one before it is still draining (programmatic dependent launch) and takes
    its work from device-side lists.  The results must not depend on that: the whole step enqueued back to back,
    twice, and once with a device synchronisation after every call give bit-identical routes, logits and outputs."""
    base = get_workload("c1")
    lens = np.array([700, 130, 257, 64, 33, 512, 31, 7] + [1] * 24, dtype=np.int32)
    n = len(lens)
    tenants = (np.arange(n) % 5).astype(np.int32)
    w = scaled_workload(base, name="pdl", dtype="bf16", d_model=1024, d_ff=2816, d_kv=256, rank=16, n_tenants=5,
                        request_tenant=tenants, prompt_len=lens, prefill_ids=np.arange(8), decode_ids=np.arange(8, n),
                        has_base_weights=False, n_layers=1)
    w.gen_device = "cuda"
    lw = _loaded(w)
    ml = lw.ml
    ml.set_decode_path(decode_path)     # the two-launch set hands its units out through a counter: same requirement
    prefill, decode = list(range(8)), list(range(8, n))
    lw.route(0, decode)                                   # the running requests were routed earlier
    H = w.hidden_batch(0, prefill, "cuda")
    cu_p = torch.from_numpy(w.cu_seqlens(prefill)).cuda()
    slots_p = torch.tensor(prefill, dtype=torch.int32, device="cuda")
    cu, slots, T = lw.seq_arrays(prefill, decode)
    n_seq = slots.numel()
    Xs = [w.module_input(0, m, T, 1, "cuda") for m in range(7)]
    Ybs = [w.base_output(0, m, T, 1, "cuda") for m in range(7)]
    mods = list(range(7))

    def step(sync):
        wait = torch.cuda.synchronize if sync else (lambda: None)
        logits = torch.zeros((len(prefill), 7), dtype=torch.float32, device="cuda")
        ws = ml.alloc_group_ws(1, n_seq, T)
        Ys = [y.clone() for y in Ybs]
        torch.cuda.synchronize()
        ml.route(0, H, cu_p, slots_p, logits); wait()
        ml.group(0, 1, cu, slots, n_seq, T, ws); wait()
        g = ml.groups(ws[0], n_seq, T)
        ml.apply_prefill_multi(0, mods, Xs, Ys, g); wait()
        ml.apply_decode_multi(0, mods, Xs, Ys, g); wait()
        torch.cuda.synchronize()
        return ml.route_table_read(0, n).numpy().copy(), logits.cpu(), ws.cpu(), [y.cpu() for y in Ys]

    ref = step(sync=True)
    for _ in range(2):
        got = step(sync=False)
        assert np.array_equal(got[0], ref[0])
        assert torch.equal(got[1], ref[1])
        lay = ml.group_layout(n_seq, T)
        hdr = ref[2][0, lay.header:lay.header + 5].tolist()
        used = [(lay.header, 16), (lay.seg_key, hdr[0]), (lay.seg_offset, hdr[0] + 1), (lay.perm, hdr[2]),
                (lay.tiles, 16 * hdr[3]), (lay.gather, 16 * hdr[4])]
        for off, cnt in used:
            assert torch.equal(got[2][0, off:off + cnt], ref[2][0, off:off + cnt])
        for m in range(7):
            assert torch.equal(got[3][m], ref[3][m]), f"module {m}: output depends on launch overlap"
    assert (ref[3][0] != Ybs[0].cpu()).any()
    assert ml.poll_error() == 0
    lw.close()


def test_tenant_without_adapter_is_excluded():
    base = get_workload("c1")
    w = scaled_workload(base, n_tenants=6)
    lw = _loaded(w, register_adapters=False)
    # tenant 0..3 get routers only; register adapters for tenants 0 and 2 on every module
    for tenant in (0, 2):
        for li in range(2):
            for m in range(7):
                A, B = w.adapter(tenant, li, m, "cuda")
                lw.ml.register_adapter(tenant, li, m, A, B, w.scale)
    ids = list(range(4))
    table_g, table_o, _ = _route_all_layers(lw, ids)
    cu, slots, T = lw.seq_arrays(ids, [])
    ws = lw.ml.alloc_group_ws(1, 4, T)
    lw.ml.group(0, 1, cu, slots, 4, T, ws)
    g = read_group_block(lw.ml, ws[0], 4, T)
    assert g["n_excluded"] == 32 and g["n_active"] == 32
    token_slot = np.repeat(np.arange(4), 16)
    g_o = O.group_tokens(token_slot, w.request_tenant, table_o[:, 0], lambda t, m: t in (0, 2), w.n_tenants)
    assert np.array_equal(g["perm"], g_o["perm"]) and np.array_equal(g["seg_key"], g_o["seg_key"])
    lw.close()


def test_tenant_churn_reuses_the_pool():
    """A server that drops tenants and admits others (at other ranks too) must not grow: the copies of a dropped
    tenant go back to the pool and later registrations are served from there; after the churn a tenant's adapters
    still give the oracle's result."""
    base = get_workload("c1")
    w = scaled_workload(base, name="churn", dtype="bf16", d_model=256, d_ff=768, d_kv=256, rank=16, n_tenants=4,
                        request_tenant=np.array([0, 1, 2, 3], dtype=np.int32), has_base_weights=False, n_layers=1)
    lw = _loaded(w)
    ml = lw.ml
    full = ml.resident_bytes()
    assert full > 0
    for i in range(4):
        ml.request_close(i)
    seen = []
    for rnd in range(6):
        for tenant in range(4):
            ml.unregister_tenant(tenant)
        assert ml.resident_bytes() == 0
        rank = (16, 8, 16, 4, 12, 16)[rnd]
        for tenant in range(4):
            lw.register_router(tenant, 0, 0)
            for m in range(7):
                A, B = w.adapter(tenant, 0, m, "cuda")
                ml.register_adapter(tenant, 0, m, A[:, :rank].contiguous(), B[:rank].contiguous(), w.scale)
        seen.append(ml.resident_bytes())
    assert seen[-1] == full and max(seen) <= full, f"pool use after churn {seen} against {full} at the start"
    torch.cuda.synchronize()
    for i in range(4):
        ml.request_open(i, i)
    ids = [0, 1, 2, 3]
    table_g, table_o, _ = _route_all_layers(lw, ids)
    _step_parity(lw, 0, ids, [], table_g, tag=31)
    lw.close()


def test_group_edge_cases_and_device_flags():
    w = get_workload("c1")
    lw = _loaded(w)
    ml = lw.ml
    ids = list(range(4))
    _route_all_layers(lw, ids)
    # empty step
    ws = ml.alloc_group_ws(1, 0, 0)
    ws.fill_(-7)
    empty = torch.zeros(1, dtype=torch.int32, device="cuda")
    ml.group(0, 1, empty, empty, 0, 0, ws)
    g = read_group_block(ml, ws[0], 0, 0)
    assert (g["n_seg"], g["n_excluded"], g["n_active"], g["n_tiles"], g["n_gather"]) == (0, 0, 0, 0, 0)
    assert g["mod_offset"].tolist() == [0] * 8
    # an out-of-range slot id inside the device array is skipped and flagged, nothing faults
    slots = torch.tensor([0, 99, 1], dtype=torch.int32, device="cuda")
    ws = ml.alloc_group_ws(1, 3, 3)
    ml.group(0, 1, None, slots, 3, 3, ws)
    g = read_group_block(ml, ws[0], 3, 3)
    assert g["n_active"] == 2 and g["n_excluded"] == 1
    assert ml.poll_error() & 1
    assert ml.poll_error() == 0
    # zero-length sequences are ignored
    cu = torch.tensor([0, 0, 5, 5], dtype=torch.int32, device="cuda")
    slots = torch.tensor([0, 1, 2], dtype=torch.int32, device="cuda")
    ws = ml.alloc_group_ws(1, 3, 5)
    ml.group(0, 1, cu, slots, 3, 5, ws)
    g = read_group_block(ml, ws[0], 3, 5)
    assert g["n_seg"] == 1 and g["n_active"] == 5 and g["perm"].tolist() == [0, 1, 2, 3, 4]
    lw.close()


def test_router_flags_bad_row_ranges_without_touching_memory():
    """cu_seqlens lives in device memory, so the host cannot check it: a range that runs past the rows of H, a
    reversed one and a negative one are treated as empty prompts (their requests stay "not routed") and raise the
    bad-row flag; the well-formed prompts of the same call are routed as usual.  H is allocated large enough that
    no access could leave it even without the check."""
    w = get_workload("c1")
    lw = _loaded(w, register_adapters=False)
    ml = lw.ml
    ids = [0, 1, 2, 3]
    Hbig = torch.zeros((4096, w.d_model), dtype=torch.float32, device="cuda")
    H = Hbig[1024:]                                          # rows before and after the 64 real ones exist
    H[:64] = w.hidden_batch(0, ids, "cuda")
    slots = torch.tensor(ids, dtype=torch.int32, device="cuda")
    for cu_bad, bad in (([0, 16, 32, 48, 400], [3]),        # the last prompt claims rows beyond T_total = 64
                        ([0, 16, 8, 48, 64], [1]),           # reversed range (and prompt 2 overlaps prompt 0: still in range)
                        ([-16, 16, 32, 48, 64], [0])):       # negative start
        ml.route_table_write(0, np.full((w.n_requests, len(lw.layers)), -1, dtype=np.int32))
        cu = torch.tensor(cu_bad, dtype=torch.int32, device="cuda")
        ml._check(ml.lib.milora_route(ml.h, 0, H.data_ptr(), cu.data_ptr(), slots.data_ptr(), 4, 64, None, None, None),
                  "milora_route")
        torch.cuda.synchronize()
        assert ml.poll_error() & 2
        col = ml.route_table_read(0, 4).numpy()[:, 0]
        assert all(col[i] == -1 for i in bad)
        good = [i for i in ids if i not in bad and cu_bad[i + 1] - cu_bad[i] == 16 and cu_bad[i] == 16 * i]
        tmp = np.full((w.n_requests, w.n_layers), -1, dtype=np.int32)
        R.route_requests(w, 0, good, tmp)
        assert all(col[i] == tmp[i, 0] for i in good) and len(good) >= 2
    assert ml.poll_error() == 0
    lw.close()


@pytest.mark.parametrize("decode_path", ["cluster", "split", "stream"])
def test_decode_kernel_sets_edge_cases(decode_path):
    """Every decode kernel set: a batch without any short sequence (empty gathered list) leaves every row
    bit-identical; the same decode batch applied five times in a row (the two-launch set hands its unit counters
    from one call to the next) gives bit-identical results each time, equal to the oracle's; a set other than
    the named ones is refused."""
    from paper_2410_18035_b200 import MiloraError
    base = get_workload("c1")
    lens = np.array([40, 64] + [1] * 9, dtype=np.int32)
    n = len(lens)
    tenants = (np.arange(n) % 3).astype(np.int32)
    d_ff = 1408 if decode_path == "stream" else 1376      # the persistent kernel wants multiples of 128
    w = scaled_workload(base, name="decode_edges", dtype="bf16", d_model=512, d_ff=d_ff, d_kv=128, rank=24, n_tenants=3,
                        request_tenant=tenants, prompt_len=lens, prefill_ids=np.arange(2), decode_ids=np.arange(2, n),
                        has_base_weights=False, n_layers=1)
    lw = _loaded(w)
    ml = lw.ml
    with pytest.raises(MiloraError):
        ml.set_decode_path(4)
    ml.set_decode_path(decode_path)
    ids = list(range(n))
    lw.route(0, ids)
    table = ml.route_table_read(0, n).numpy()[:, 0].copy()
    # 1. prompts only: nothing for the decode kernels to do
    cu, slots, T = lw.seq_arrays([0, 1], [])
    ws = ml.alloc_group_ws(1, 2, T)
    ml.group(0, 1, cu, slots, 2, T, ws)
    groups = ml.groups(ws[0], 2, T)
    for m in range(7):
        X = w.module_input(0, m, T, 3, "cuda")
        Yb = w.base_output(0, m, T, 3, "cuda")
        Y = Yb.clone()
        ml.apply_decode(0, m, X, Y, groups)
        torch.cuda.synchronize()
        assert torch.equal(Y, Yb)
    # 2. the decode rows, five calls in a row on fresh copies of y
    dec = list(range(2, n))
    cu, slots, T = lw.seq_arrays([], dec)
    ws = ml.alloc_group_ws(1, len(dec), T)
    ml.group(0, 1, cu, slots, len(dec), T, ws)
    groups = ml.groups(ws[0], len(dec), T)
    token_slot = slots.cpu().numpy()
    Xs = [w.module_input(0, m, T, 4, "cuda") for m in range(7)]
    Ybs = [w.base_output(0, m, T, 4, "cuda") for m in range(7)]
    first = None
    for rep in range(5):
        Ys = [y.clone() for y in Ybs]
        ml.apply_decode_multi(0, list(range(7)), Xs, Ys, groups)
        torch.cuda.synchronize()
        if first is None:
            first = Ys
            for m in range(7):
                y_o = R.apply_site(w, 0, m, Xs[m].cpu(), Ybs[m].cpu(), token_slot, table)
                assert_apply_close(Ys[m], y_o, Ybs[m], "bf16", what=f"decode edges module {m}")
        else:
            for m in range(7):
                assert torch.equal(Ys[m], first[m]), f"call {rep}, module {m}: result changed between calls"
    assert ml.poll_error() == 0
    lw.close()


@pytest.mark.parametrize("d,d_ff,d_kv,r,n_dec,unit_stages", [(512, 1408, 128, 16, 37, 0), (1024, 2816, 256, 32, 70, 1),
                                                             (512, 1536, 512, 48, 9, 3), (256, 688, 256, 8, 12, 0)])
def test_decode_layers_one_launch(d, d_ff, d_kv, r, n_dec, unit_stages):
    """milora_apply_decode_layers: three layers with their own routes, adapters and outputs in ONE call, against
    the oracle layer by layer; tenants repeat (jobs of up to four rows, several jobs per adapter), one layer skips
    two modules (NULL pair: those outputs stay bit-identical), and repeated calls give bit-identical results (the
    kernel's job states and unit counter clean themselves up).  The last shape does not fit the persistent kernel
    and takes the per-layer calls behind the same entry point."""
    base = get_workload("c1")
    L = 3
    lens = np.full(n_dec, 8, dtype=np.int32)
    tenants = (np.arange(n_dec) * 7 % 5).astype(np.int32)
    w = scaled_workload(base, name="decode_layers", dtype="bf16", d_model=d, d_ff=d_ff, d_kv=d_kv, rank=r, n_tenants=5,
                        request_tenant=tenants, prompt_len=lens, prefill_ids=np.arange(0), decode_ids=np.arange(n_dec),
                        has_base_weights=False, n_layers=L)
    lw = _loaded(w)
    ml = lw.ml
    ml.set_decode_unit_stages(unit_stages)
    ids = list(range(n_dec))
    for li in range(L):
        for i0 in range(0, n_dec, 32):
            lw.route(li, ids[i0:i0 + 32])
    table = ml.route_table_read(0, n_dec).numpy().copy()
    cu, slots, T = lw.seq_arrays([], ids)
    ws = ml.alloc_group_ws(L, n_dec, T)
    ml.group(0, L, cu, slots, n_dec, T, ws)
    token_slot = slots.cpu().numpy()
    Xs = [[w.module_input(li, m, T, 20 + li, "cuda") for m in range(7)] for li in range(L)]
    Ybs = [[w.base_output(li, m, T, 20 + li, "cuda") for m in range(7)] for li in range(L)]
    skipped = {1: (2, 5)}
    first = None
    for rep in range(3):
        Ys = [[y.clone() for y in row] for row in Ybs]
        entries = []
        for li in range(L):
            sites = {m: (Xs[li][m], Ys[li][m]) for m in range(7) if m not in skipped.get(li, ())}
            entries.append((li, ml.groups(ws[li], n_dec, T), sites))
        ml.apply_decode_layers(ml.decode_layers(entries))
        torch.cuda.synchronize()
        if first is None:
            first = Ys
            for li in range(L):
                for m in range(7):
                    if m in skipped.get(li, ()):
                        assert torch.equal(Ys[li][m], Ybs[li][m])
                        continue
                    y_o = R.apply_site(w, li, m, Xs[li][m].cpu(), Ybs[li][m].cpu(), token_slot, table[:, li])
                    assert_apply_close(Ys[li][m], y_o, Ybs[li][m], "bf16", what=f"decode layers: layer {li} module {m}")
        else:
            for li in range(L):
                for m in range(7):
                    assert torch.equal(Ys[li][m], first[li][m]), f"call {rep}, layer {li}, module {m}"
    assert any((first[li][m] != Ybs[li][m]).any() for li in range(L) for m in range(7))
    assert ml.poll_error() == 0
    lw.close()


@pytest.mark.parametrize("pool,act,bias", [(O.POOL_MAX, O.ACT_RELU, False), (O.POOL_LAST, O.ACT_GELU, True),
                                            (O.POOL_SELFATTN, O.ACT_RATIONAL, False),
                                            (O.POOL_MEAN, O.ACT_IDENTITY, True), (O.POOL_SELFATTN, O.ACT_TANH, True)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_router_variants(pool, act, bias, dtype):
    """All poolers of Eq. 2 / Appendix C and activations incl. Eq. 7, on ragged prompts."""
    base = get_workload("c1")
    lens = np.array([1, 5, 64, 65, 200, 333], dtype=np.int32)
    w = scaled_workload(base, name="router_variants", dtype=dtype, d_model=512, d_ff=1376, d_kv=512, n_tenants=3,
                        request_tenant=np.array([0, 1, 2, 0, 1, 2], dtype=np.int32), prompt_len=lens,
                        prefill_ids=np.arange(6), decode_ids=np.zeros(0, dtype=np.int64), has_base_weights=False)
    lw = _loaded(w, pool=pool, act=act, with_bias=bias, register_adapters=False)
    _, _, excused = _route_all_layers(lw, list(range(6)), pooler=pool, activation=act, with_bias=bias)
    assert excused <= 1
    lw.close()


def test_host_validation_reports_errors_before_launch():
    from paper_2410_18035_b200 import Milora, MiloraError
    with pytest.raises(MiloraError) as e:
        Milora(1, 250, 688, 256, "bf16", 8, 4, 4)            # 250 is not a multiple of 8
    assert e.value.status == 2
    with pytest.raises(MiloraError) as e:
        Milora(1, 256, 688, 256, "f32", 300, 4, 4)
    assert e.value.status == 5
    ml = Milora(2, 256, 688, 256, "f32", 8, 4, 4)
    A = torch.zeros((256, 16), device="cuda"); B = torch.zeros((16, 256), device="cuda")
    with pytest.raises(MiloraError) as e:
        ml.register_adapter(0, 0, 0, A, B, 1.0)               # rank 16 > max_rank 8
    assert e.value.status == 5
    with pytest.raises(MiloraError) as e:
        ml.request_open(9, 0)
    assert e.value.status == 1
    ml.request_open(1, 2)
    with pytest.raises(MiloraError) as e:
        ml.request_open(1, 2)
    assert e.value.status == 6
    with pytest.raises(MiloraError) as e:
        ml.unregister_tenant(2)
    assert e.value.status == 6
    ml.request_close(1)
    ml.unregister_tenant(2)
    with pytest.raises(MiloraError) as e:
        ml.route_table_write(0, [[7, 0]])
    assert e.value.status == 1
    ml.route_table_write(2, [[3, -1]])
    assert ml.route_table_read(2, 1).tolist() == [[3, -1]]
    ml.close()
    # invalid k or weighting mode; with k selected modules per sequence a grouping call takes 4096 / k sequences
    for kw in ({"top_k": 8}, {"top_k": -1}, {"gate": 5}):
        with pytest.raises(MiloraError) as e:
            Milora(1, 256, 688, 256, "f32", 8, 4, 4, **kw)
        assert e.value.status == 1
    ml = Milora(1, 256, 688, 256, "f32", 8, 4, 4, top_k=3)
    with pytest.raises(MiloraError) as e:
        ml.group_layout(2000, 2000)
    assert e.value.status == 5
    assert ml.group_layout(1365, 1365).total > 0
    slots = torch.zeros(2000, dtype=torch.int32, device="cuda")
    ws = torch.zeros((1, 1 << 20), dtype=torch.int32, device="cuda")
    with pytest.raises(MiloraError) as e:
        ml.group(0, 1, None, slots, 2000, 2000, ws)
    assert e.value.status == 5
    ml.close()


def test_step_from_host_buffers_matches_oracle():
    """milora_step_host: inputs in pinned host memory, outputs back in host memory, one call per step."""
    base = get_workload("c1")
    lens = np.array([130, 40, 7, 64, 1, 1, 1], dtype=np.int32)
    w = scaled_workload(base, name="host_step", dtype="bf16", d_model=512, d_ff=1408, d_kv=128, rank=16, n_tenants=3,
                        request_tenant=np.array([0, 1, 2, 0, 1, 2, 0], dtype=np.int32), prompt_len=lens,
                        prefill_ids=np.arange(4), decode_ids=np.arange(4, 7), has_base_weights=False, n_layers=1)
    lw = _loaded(w)
    ml = lw.ml
    prefill, decode = [0, 1, 2, 3], [4, 5, 6]
    # the decode requests were routed earlier from their own prompts
    lw.route(0, decode)
    cu, slots, T = lw.seq_arrays(prefill, decode)
    pin = lambda t: t.cpu().pin_memory()
    cu_p = pin(torch.from_numpy(w.cu_seqlens(prefill)))
    slot_p = pin(torch.tensor(prefill, dtype=torch.int32))
    H = pin(w.hidden_batch(0, prefill))
    Xs = {m: pin(w.module_input(0, m, T, 3)) for m in range(7)}
    Ybs = {m: w.base_output(0, m, T, 3) for m in range(7)}
    Ys = {m: pin(Ybs[m].clone()) for m in range(7)}
    step = ml.make_host_step(0, cu_p, slot_p, H, pin(cu), pin(slots), T, Xs, Ys)
    # the workspace starts as NaN patterns: only the rows of routed sequences are sent to the device, and only those
    # rows may come back, so no other row of Y_host can pick up what the workspace held
    ws = torch.full((ml.step_host_workspace(step) + 256,), 255, dtype=torch.uint8, device="cuda")
    ws = ws[(-ws.data_ptr()) % 256:]
    ml.step_host(step, ws)
    torch.cuda.synchronize()
    assert ml.poll_error() == 0
    for m in range(7):
        assert not bool(torch.isnan(Ys[m].float()).any()), f"module {m}: an unsent row came back from the workspace"
    table = ml.route_table_read(0, w.n_requests).numpy()
    tmp = np.full((w.n_requests, 1), -1, dtype=np.int32)
    _, margins = R.route_requests(w, 0, prefill, tmp)
    compare_routes(table[prefill, 0], tmp[prefill, 0], margins)
    token_slot = np.repeat(slots.cpu().numpy(), np.diff(cu.cpu().numpy()))
    for m in range(7):
        y_o = R.apply_site(w, 0, m, Xs[m], Ybs[m], token_slot, table[:, 0])
        assert_apply_close(Ys[m], y_o, Ybs[m], "bf16", what=f"host step module {m}")
    # a workspace that is too small is refused before anything is enqueued
    from paper_2410_18035_b200 import MiloraError
    with pytest.raises(MiloraError) as e:
        ml.step_host(step, ws[:1024])
    assert e.value.status == 1
    lw.close()
