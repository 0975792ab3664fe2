"""Parity at the benchmark's full sizes (LLaMA-2-7B layer, bf16) in the launch configuration bench.py times,
and at the shapes of the larger configs with fewer layers / tenants.

The oracle cannot redo 32k tokens x 7 modules in seconds, so outputs are checked on sampled rows that it
computes one by one (first, last and random rows of every prompt, every decode row); rows that no adapter
touches are compared bit for bit on the whole tensors; routes and groupings are checked in full.
"""
import numpy as np
import pytest
import torch

from oracle import milora_oracle as O
from oracle import reference_run as R
from synth import get_workload
from synth.workloads import scaled_workload

from parity_utils import TOL, assert_apply_close, assert_groups_equal, compare_routes, read_group_block

pytestmark = pytest.mark.gpu


def _loaded(w, **kw):
    from paper_2410_18035_b200.workload_runner import LoadedWorkload
    return LoadedWorkload(w, "cuda", **kw)


def _sample_rows(cu, rng, per_seq=6):
    rows = []
    for lo, hi in zip(cu[:-1], cu[1:]):
        if hi <= lo:
            continue
        pick = {int(lo), int(hi - 1)}
        for r in (int(lo) + 127, int(lo) + 128, int(hi) - 129):     # tile boundaries of the dense path
            if lo <= r < hi:
                pick.add(r)
        pick.update(int(v) for v in rng.integers(lo, hi, size=per_seq))
        rows += sorted(pick)
    return np.array(sorted(set(rows)), dtype=np.int64)


def _apply_and_check(lw, li, groups, cu_h, token_slot, table_col, T, tag, rng, multi=True, decode_path="auto"):
    """Multi-site prefill apply and decode apply of one layer on a grouped step; outputs against the oracle on
    sampled rows, untouched rows bit for bit on the whole tensors."""
    w, ml = lw.w, lw.ml
    ml.set_decode_path(decode_path)
    layer = lw.layers[li]
    Xs = [w.module_input(layer, m, T, tag, "cuda") for m in range(7)]
    Ybs = [w.base_output(layer, m, T, tag, "cuda") for m in range(7)]
    Ys = [y.clone() for y in Ybs]
    mods = list(range(7))
    if multi:
        ml.apply_prefill_multi(li, mods, Xs, Ys, groups)
        ml.apply_decode_multi(li, mods, Xs, Ys, groups)
    else:
        for m in mods:
            ml.apply_prefill(li, m, Xs[m], Ys[m], groups)
            ml.apply_decode(li, m, Xs[m], Ys[m], groups)
    torch.cuda.synchronize()
    assert ml.poll_error() == 0
    _check_outputs(w, layer, Xs, Ybs, Ys, cu_h, token_slot, table_col, rng)


def _check_outputs(w, layer, Xs, Ybs, Ys, cu_h, token_slot, table_col, rng):
    rows = _sample_rows(cu_h, rng)
    slot_module = np.asarray(table_col)
    for m in range(7):
        active = torch.from_numpy(slot_module[token_slot] == m).cuda()
        # rows whose request routes elsewhere: bit-identical over the whole tensor
        assert torch.equal(Ys[m][~active], Ybs[m][~active]), f"module {m}: an unrouted row changed"
        # every routed row must have changed somewhere
        if active.any():
            changed = (Ys[m][active] != Ybs[m][active]).any(dim=1)
            assert bool(changed.all()), f"module {m}: a routed row was not updated"
        sel = rows[slot_module[token_slot[rows]] == m]
        if sel.size == 0:
            continue
        idx = torch.from_numpy(sel).cuda()
        y_o = R.apply_site(w, layer, m, Xs[m][idx].cpu(), Ybs[m][idx].cpu(), token_slot, table_col, rows=sel)
        assert_apply_close(Ys[m][idx], y_o, Ybs[m][idx], w.dtype, what=f"{w.name} layer {layer} module {m}")


def _check_step(lw, li, prefill_ids, decode_ids, table_col, tag, rng, multi=True, decode_path="auto"):
    """One step in the bench's configuration: group, multi-site prefill apply, multi-site decode apply
    (decode_path: which kernel set milora_apply_decode uses)."""
    w, ml = lw.w, lw.ml
    cu, slots, T = lw.seq_arrays(prefill_ids, decode_ids)
    n_seq = slots.numel()
    ws = ml.alloc_group_ws(1, n_seq, T)
    ml.group(li, 1, cu, slots, n_seq, T, ws)
    cu_h = cu.cpu().numpy()
    token_slot = np.repeat(slots.cpu().numpy(), np.diff(cu_h))
    g_o = R.group_layer(w, token_slot, table_col)
    g_o["max_tenants"] = w.n_tenants
    assert_groups_equal(read_group_block(ml, ws[0], n_seq, T), g_o, cu_h)
    _apply_and_check(lw, li, ml.groups(ws[0], n_seq, T), cu_h, token_slot, table_col, T, tag, rng, multi, decode_path)


def _spread(n_layers):
    """First, last and two layers inside the stack."""
    return sorted({0, n_layers // 3, (2 * n_layers) // 3, n_layers - 1})


def _full_stack(lw, prefill_ids, decode_ids, rng, max_excused, decode_path="auto"):
    """Every layer of the workload: routes against the oracle in full, one grouping call for all layers compared
    block by block, the step applied on four layers spread over the stack, and (when the step has decode rows) the
    decode rows of ALL layers in one milora_apply_decode_layers call, checked on the same four layers against the
    oracle and on every layer for rows that must stay untouched.  Returns the number of excused near-tie routes."""
    w, ml = lw.w, lw.ml
    L = len(lw.layers)
    ids = sorted(set(int(i) for i in prefill_ids) | set(int(i) for i in decode_ids))
    table = np.full((w.n_requests, L), -1, dtype=np.int32)
    excused = 0
    for li in range(L):
        for i0 in range(0, len(ids), 64):
            lw.route(li, ids[i0:i0 + 64])
        tmp = np.full((w.n_requests, w.n_layers), -1, dtype=np.int32)
        _, margins = R.route_requests(w, lw.layers[li], ids, tmp)
        col = ml.route_table_read(0, w.n_requests).numpy()[:, li]
        excused += compare_routes(col[ids], tmp[ids, lw.layers[li]], margins)
        table[:, li] = col          # the GPU's decisions downstream, so that an excused near tie cannot cascade
    assert excused <= max_excused, f"{excused} near-tie route mismatches over {L} layers"
    cu, slots, T = lw.seq_arrays(prefill_ids, decode_ids)
    n_seq = slots.numel()
    ws = ml.alloc_group_ws(L, n_seq, T)
    ml.group(0, L, cu, slots, n_seq, T, ws)
    cu_h = cu.cpu().numpy()
    token_slot = np.repeat(slots.cpu().numpy(), np.diff(cu_h))
    for li in range(L):
        g_o = R.group_layer(w, token_slot, table[:, li])
        g_o["max_tenants"] = w.n_tenants
        assert_groups_equal(read_group_block(ml, ws[li], n_seq, T), g_o, cu_h)
    for li in _spread(L):
        _apply_and_check(lw, li, ml.groups(ws[li], n_seq, T), cu_h, token_slot, table[:, li], T, 50 + li, rng,
                         decode_path=decode_path)
    if len(decode_ids):
        # the decode rows alone, every layer in one launch, every layer its own outputs
        ml.set_decode_path("auto")
        cu_d, slots_d, T_d = lw.seq_arrays([], decode_ids)
        n_d = slots_d.numel()
        ws_d = ml.alloc_group_ws(L, n_d, T_d)
        ml.group(0, L, cu_d, slots_d, n_d, T_d, ws_d)
        slot_d = slots_d.cpu().numpy()
        Xs = [w.module_input(lw.layers[0], m, T_d, 90, "cuda") for m in range(7)]          # inputs shared by the layers
        Ybs = [w.base_output(lw.layers[0], m, T_d, 90, "cuda") for m in range(7)]
        Ys = [[y.clone() for y in Ybs] for _ in range(L)]
        entries = [(li, ml.groups(ws_d[li], n_d, T_d), {m: (Xs[m], Ys[li][m]) for m in range(7)}) for li in range(L)]
        ml.apply_decode_layers(ml.decode_layers(entries))
        torch.cuda.synchronize()
        assert ml.poll_error() == 0
        cu_dh = cu_d.cpu().numpy()
        for li in range(L):
            if li in _spread(L):
                # the adapters differ per layer; x and y_base are those of tag 90 for every layer
                rows = np.arange(T_d)
                for m in range(7):
                    sel = rows[table[slot_d, li] == m]
                    if sel.size == 0:
                        continue
                    idx = torch.from_numpy(sel).cuda()
                    y_o = R.apply_site(w, lw.layers[li], m, Xs[m][idx].cpu(), Ybs[m][idx].cpu(), slot_d, table[:, li], rows=sel)
                    assert_apply_close(Ys[li][m][idx], y_o, Ybs[m][idx], w.dtype, what=f"{w.name} one call, layer {li} module {m}")
            for m in range(7):
                active = torch.from_numpy(table[slot_d, li] == m).cuda()
                assert torch.equal(Ys[li][m][~active], Ybs[m][~active]), f"layer {li} module {m}: an unrouted row changed"
                if active.any():
                    assert bool((Ys[li][m][active] != Ybs[m][active]).any(dim=1).all()), f"layer {li} module {m}: a routed row was not updated"
    return excused


def _route_and_check(lw, li, ids):
    w = lw.w
    lw.route(li, ids)
    tmp = np.full((w.n_requests, w.n_layers), -1, dtype=np.int32)
    _, margins = R.route_requests(w, lw.layers[li], ids, tmp)
    table_g = lw.ml.route_table_read(0, w.n_requests).numpy()[:, li]
    excused = compare_routes(table_g[list(ids)], tmp[list(ids), lw.layers[li]], margins)
    return table_g.copy(), excused


def test_config2_full_size_bench_configuration():
    """LLaMA-2-7B one layer: 64 prompts x 512 tokens routed, 32,768 prompt rows + 64 decode rows applied."""
    w = get_workload("c2")
    w.gen_device = "cuda"
    lw = _loaded(w, layers=[0])
    ids = list(range(64))
    table, excused = _route_and_check(lw, 0, ids)
    assert excused <= 3, f"{excused} near-tie route mismatches (oracle top-2 logit gap < 1e-3)"
    rng = np.random.default_rng(0)
    _check_step(lw, 0, ids, [], table, tag=0, rng=rng)          # prefill rows (dense tiles)
    _check_step(lw, 0, [], ids, table, tag=1, rng=rng)          # decode rows (gathered)
    _check_step(lw, 0, [], ids, table, tag=4, rng=rng, decode_path="split")
    _check_step(lw, 0, [], ids, table, tag=5, rng=rng, decode_path="stream")
    _check_step(lw, 0, ids[:8], ids[8:], table, tag=2, rng=rng, multi=False)   # mixed, per-site calls
    _check_step(lw, 0, ids, ids, table, tag=3, rng=rng)         # all prompts and all decode rows as one batch
    lw.close()


def test_config3_full_stack_ragged_prefill():
    """LLaMA-2-7B, all 32 layers registered: 32 prompts with lengths U[128, 2048] and repeated tenants; routes and
    groupings on every layer, the segmented apply on four layers spread over the stack."""
    w = get_workload("c3")
    w.gen_device = "cuda"
    lw = _loaded(w)
    ids = list(range(w.n_requests))
    _full_stack(lw, ids, [], np.random.default_rng(1), max_excused=32)
    lw.close()


def test_config4_full_stack_zipf_decode():
    """LLaMA-2-13B shapes, all 40 layers registered, rank 32, 256 decode requests whose tenants follow Zipf(1.1) over
    1000 ids (every drawn tenant gets backing: about 110 tenants x 40 layers x 7 adapters), 256-token prompts:
    routes (40 x 256) and groupings on every layer, the gathered apply on four layers with the library's own choice
    (the persistent kernel), on one layer each with the other two kernel sets,
    and the whole stack in one milora_apply_decode_layers call."""
    w = get_workload("c4")
    w.gen_device = "cuda"
    free, _ = torch.cuda.mem_get_info()
    per_tenant = w.n_layers * sum(2 * 2 * w.rank * sum(w.dims(m)) for m in range(7))      # row-major + images, bf16
    n_active = len(w.active_tenants())
    assert per_tenant * n_active < 0.8 * free, f"{n_active} tenants x {per_tenant >> 20} MB do not fit this device"
    lw = _loaded(w)
    ids = list(range(w.n_requests))
    assert lw.ml.decode_path_for(len(ids), len(ids)) == 3       # a batch of this size takes the persistent kernel
    _full_stack(lw, [], ids, np.random.default_rng(2), max_excused=120, decode_path="auto")
    rng = np.random.default_rng(22)
    table = lw.ml.route_table_read(0, w.n_requests).numpy()
    _check_step(lw, 0, [], ids, table[:, 0], tag=1, rng=rng, decode_path="cluster")
    _check_step(lw, 39, [], ids, table[:, 39], tag=2, rng=rng, decode_path="split")
    lw.close()


def test_config5_full_stack_mixed_step():
    """LLaMA-3-8B GQA shapes, all 32 layers registered: 8 prompts U[256, 4096] plus 192 decode rows in one step."""
    w = get_workload("c5")
    w.gen_device = "cuda"
    lw = _loaded(w)
    _full_stack(lw, [int(i) for i in w.prefill_ids], [int(i) for i in w.decode_ids], np.random.default_rng(3),
                max_excused=80)
    lw.close()


def test_decode_batch_sweep_small_batches():
    """Batch sizes 1, 2, 4 and 256 of the decode sweep (tenants = batch size)."""
    from synth.workloads import decode_sweep_workload
    rng = np.random.default_rng(4)
    for b in (1, 2, 4, 256):
        w = scaled_workload(decode_sweep_workload(b), n_layers=1, prompt_len=np.full(b, 64, dtype=np.int32))
        w.gen_device = "cuda"
        lw = _loaded(w)
        ids = list(range(b))
        for i0 in range(0, b, 64):
            lw.route(0, ids[i0:i0 + 64])
        table = lw.ml.route_table_read(0, w.n_requests).numpy()[:, 0].copy()
        _check_step(lw, 0, [], ids, table, tag=b, rng=rng)
        _check_step(lw, 0, [], ids, table, tag=b + 1, rng=rng, decode_path="stream")
        lw.close()


def test_config2_fused_projection_full_size():
    """milora_linear_prefill at the benchmark's size (32,768 prompt rows of the LLaMA-2-7B layer; q: 4096 -> 4096 and
    down: 11008 -> 4096), weights drawn as bench.py draws them.  The oracle recomputes sampled rows one by one
    (x W in fp64 plus the LoRA term); every row must differ from the plain projection exactly where its request
    selects the module."""
    from parity_utils import half_ulp
    w = get_workload("c2")
    w.gen_device = "cuda"
    lw = _loaded(w, layers=[0])
    ml = lw.ml
    ids = list(range(64))
    table, _ = _route_and_check(lw, 0, ids)
    cu, slots, T = lw.seq_arrays(ids, [])
    ws = ml.alloc_group_ws(1, 64, T)
    ml.group(0, 1, cu, slots, 64, T, ws)
    groups = ml.groups(ws[0], 64, T)
    cu_h = cu.cpu().numpy()
    token_slot = np.repeat(slots.cpu().numpy(), np.diff(cu_h))
    rng = np.random.default_rng(5)
    rows = _sample_rows(cu_h, rng, per_seq=2)
    idx = torch.from_numpy(rows).cuda()
    for m in (0, 6):
        d1, d2 = w.dims(m)
        g = torch.Generator(device="cuda")
        g.manual_seed(1234 + m)
        Wt = (torch.randn((d2, d1), generator=g, device="cuda", dtype=torch.float32) * 0.02).to(torch.bfloat16)
        X = w.module_input(0, m, T, 0, "cuda")
        Y = torch.full((T, d2), float("nan"), dtype=torch.bfloat16, device="cuda")
        ml.linear_prefill(0, m, X, Wt, Y, groups)
        torch.cuda.synchronize()
        assert ml.poll_error() == 0
        assert not bool(torch.isnan(Y.float()).any()), "a tile of the output was not written"
        yb = O.base_projection(R.to_f64(X[idx]), R.to_f64(Wt).T)
        y_o = R.apply_site(w, 0, m, X[idx].cpu(), yb, token_slot, table, rows=rows)
        yg = R.to_f64(Y[idx])
        assert O.max_rel_err(yg, y_o) <= TOL["bf16"]
        delta = y_o - yb
        routed = table[token_slot[rows]] == m
        assert np.array_equal(np.any(delta != 0, axis=1), routed)
        rms = np.sqrt(np.mean(delta[routed] ** 2)) if routed.any() else 0.0
        allowed = TOL["bf16"] * np.where(delta != 0, np.maximum(np.abs(delta), rms), 0.0) + 1.01 * half_ulp(y_o, "bf16") + 1e-4
        worst = float((np.abs(yg - y_o) / allowed).max())
        assert worst <= 1.0, f"fused projection module {m}: error is {worst:.3f}x the allowed bound"
        # the LoRA term is really there: on routed rows the output differs from the plain projection
        plain = (X[idx].float() @ Wt.float().t()).to(torch.bfloat16)
        differs = (plain != Y[idx]).float().mean(dim=1).cpu().numpy()
        assert (differs[routed] > 0.5).all() and (differs[~routed] < 0.02).all()
        del Wt, X, Y
    lw.close()


def test_config2_top3_shared_input_full_size():
    """Section 3.3 with k = 3 at config 2's sizes: q, k, v read one matrix and gate, up another.  The shared-input
    call must give, bit for bit, what one call per module gives, and on sampled rows the oracle's value."""
    w = get_workload("c2")
    w.gen_device = "cuda"
    lw = _loaded(w, layers=[0], top_k=3)
    ml = lw.ml
    ids = list(range(64))
    lw.route(0, ids)
    table = ml.route_table_read(0, w.n_requests).numpy().reshape(w.n_requests, 1, 3)[:, 0].copy()
    assert all(len(set(row.tolist())) == 3 for row in table[ids])
    cu, slots, T = lw.seq_arrays(ids, [])
    ws = ml.alloc_group_ws(1, len(ids), T)
    ml.group(0, 1, cu, slots, len(ids), T, ws)
    groups = ml.groups(ws[0], len(ids), T)
    cu_h = cu.cpu().numpy()
    token_slot = np.repeat(slots.cpu().numpy(), np.diff(cu_h))
    shared = [(0, 1, 2), (4, 5)]
    # the sharing must really occur: prompts that select at least two modules of a group
    n_sharing = sum(int(np.isin(table[i], mods).sum() >= 2) for i in ids for mods in shared)
    assert n_sharing >= 8, "the routed table gives the shared-input kernel nothing to share"
    Xs = {mods: w.module_input(0, mods[0], T, 21, "cuda") for mods in shared}
    rng = np.random.default_rng(5)
    rows = _sample_rows(cu_h, rng, per_seq=3)
    for mods in shared:
        X = Xs[mods]
        Ybs = [w.base_output(0, m, T, 21, "cuda") for m in mods]
        Y_shared = [y.clone() for y in Ybs]
        Y_single = [y.clone() for y in Ybs]
        ml.apply_prefill_shared(0, list(mods), X, Y_shared, groups)
        for m, Y in zip(mods, Y_single):
            ml.apply_prefill(0, m, X, Y, groups)
        torch.cuda.synchronize()
        assert ml.poll_error() == 0
        for m, Yb, Ys, Y1 in zip(mods, Ybs, Y_shared, Y_single):
            assert torch.equal(Ys, Y1), f"module {m}: shared-input call differs from the single call"
            active = torch.from_numpy((table[token_slot] == m).any(axis=1)).cuda()
            assert torch.equal(Ys[~active], Yb[~active]), f"module {m}: an unrouted row changed"
            sel = rows[(table[token_slot[rows]] == m).any(axis=1)]
            if sel.size == 0:
                continue
            idx = torch.from_numpy(sel).cuda()
            y_o = R.apply_site(w, 0, m, X[idx].cpu(), Yb[idx].cpu(), token_slot, table, rows=sel)
            assert_apply_close(Ys[idx], y_o, Yb[idx], w.dtype, what=f"c2 top-3 shared input, module {m}")
    lw.close()
