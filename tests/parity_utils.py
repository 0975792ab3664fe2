"""Shared helpers of the GPU parity tests: tolerances and element-wise comparisons against the oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import milora_oracle as O
from oracle import reference_run as R

# Tolerances: max relative error 1e-4 (fp32) and 2e-2 (bf16); route mismatches are excused only where
# the oracle's two largest logits differ by less than 1e-3.
TOL = {"f32": 1e-4, "bf16": 2e-2}
MARGIN_EXCUSE = 1e-3


def compare_routes(gpu_col, oracle_col, margins):
    """Returns the number of excused near-tie mismatches; asserts that every other entry is identical."""
    gpu_col = np.asarray(gpu_col)
    oracle_col = np.asarray(oracle_col)
    bad = np.nonzero(gpu_col != oracle_col)[0]
    for i in bad:
        assert margins[i] < MARGIN_EXCUSE, (
            f"route mismatch at {i}: gpu {gpu_col[i]} oracle {oracle_col[i]} with top-2 logit gap {margins[i]:.3e}")
    return len(bad)


def half_ulp(y_ref: np.ndarray, dtype: str) -> np.ndarray:
    """Upper bound of the rounding error of storing y in `dtype` (round to nearest)."""
    bits = 8 if dtype == "bf16" else 24
    return np.abs(y_ref) * 2.0 ** (-bits)


def assert_apply_close(y_gpu, y_oracle, y_base, dtype: str, active_rows=None, what=""):
    """y_gpu (torch) against the oracle's float64 output.

    1. full-output metric: max |y - yref| / max(|yref|, rms(yref)) <= tol
    2. delta metric: the error must fit in tol * max(|delta_ref|, rms(delta_ref)) plus the unavoidable
       rounding of the stored output (half an ulp of y in the storage dtype, and of the accumulation)
    3. rows the oracle leaves unchanged are bit-identical to y_base
    """
    tol = TOL[dtype]
    yg = R.to_f64(y_gpu)
    yb = R.to_f64(y_base)
    yr = np.asarray(y_oracle, dtype=np.float64)
    assert yg.shape == yr.shape
    if yr.size == 0:
        return 0.0
    err_full = O.max_rel_err(yg, yr)
    assert err_full <= tol, f"{what}: full-output max rel err {err_full:.3e} > {tol}"
    delta_ref = yr - yb
    changed = np.any(delta_ref != 0.0, axis=1)
    if active_rows is not None:
        assert np.array_equal(np.nonzero(changed)[0], np.sort(np.asarray(active_rows))), f"{what}: active rows differ"
    untouched = ~changed
    assert np.array_equal(yg[untouched], yb[untouched]), f"{what}: a row without a routed adapter was modified"
    if changed.any():
        d = delta_ref[changed]
        rms = np.sqrt(np.mean(d * d))
        # the stored y is rounded once (half an ulp); 1 % on top for the fp32 sums behind it
        allowed = tol * np.maximum(np.abs(d), rms) + 1.01 * half_ulp(yr[changed], dtype)
        err = np.abs(yg[changed] - yr[changed])
        worst = float((err / allowed).max())
        assert worst <= 1.0, f"{what}: delta error is {worst:.3f}x the allowed bound"
    return err_full


def read_group_block(ml, ws_layer: torch.Tensor, n_seq: int, T: int):
    """Decode one layer's group block (host copies of every array)."""
    lay = ml.group_layout(n_seq, T)
    ws = ws_layer.cpu().numpy()
    hdr = ws[lay.header:lay.header + 16]
    n_seg, n_excl, n_active, n_tiles, n_gather = (int(v) for v in hdr[:5])
    out = {
        "n_seg": n_seg, "n_excluded": n_excl, "n_active": n_active, "n_tiles": n_tiles, "n_gather": n_gather,
        "mod_offset": ws[lay.mod_offset:lay.mod_offset + 8].copy(),
        "mod_tile_offset": ws[lay.mod_tile_offset:lay.mod_tile_offset + 8].copy(),
        "mod_gather_offset": ws[lay.mod_gather_offset:lay.mod_gather_offset + 8].copy(),
        "seg_key": ws[lay.seg_key:lay.seg_key + n_seg].copy(),
        "seg_offset": ws[lay.seg_offset:lay.seg_offset + n_seg + 1].copy(),
        "perm": ws[lay.perm:lay.perm + n_active].copy(),
        "layout": lay,
    }
    # job records are 16 int32 each: two / four 64-bit pointers first, then the integer fields
    tiles = ws[lay.tiles:lay.tiles + 16 * n_tiles].reshape(-1, 16)
    gather = ws[lay.gather:lay.gather + 16 * n_gather].reshape(-1, 16)
    # (seg, start, count, module) per dense tile
    out["tiles"] = np.stack([tiles[:, 12], tiles[:, 13], tiles[:, 11], tiles[:, 10]], axis=1) if n_tiles else np.zeros((0, 4), int)
    out["tile_rank"] = tiles[:, 8].copy()
    # (count, module, rows[4]) per gather job, and the per-row weights (fp32 bit patterns in ints 12..15)
    out["gather"] = [(int(g[7]), int(g[6]), [int(v) for v in g[8:12]]) for g in gather]
    out["gather_gate"] = gather[:, 12:16].copy().view(np.float32) if n_gather else np.zeros((0, 4), np.float32)
    out["gather_rank"] = gather[:, 4].copy()
    return out


def assert_groups_equal(g_gpu, g_oracle, cu, long_seq=32, tile_rows=128, gather_rows=4):
    """perm / seg_key / seg_offset / mod_offset / n_excluded are compared bit for bit; the work lists must
    cover every active (row, module) pair exactly once, dense tiles with consecutive rows of long sequences only."""
    assert g_gpu["n_excluded"] == g_oracle["n_excluded"]
    assert g_gpu["n_seg"] == len(g_oracle["seg_key"])
    assert np.array_equal(g_gpu["perm"], g_oracle["perm"])
    assert np.array_equal(g_gpu["seg_key"], g_oracle["seg_key"])
    if g_gpu["n_seg"]:
        assert np.array_equal(g_gpu["seg_offset"], g_oracle["seg_offset"])
    assert np.array_equal(g_gpu["mod_offset"], g_oracle["mod_offset"])
    # work lists
    cu = np.asarray(cu)
    seq_of_row = np.repeat(np.arange(len(cu) - 1), np.diff(cu))
    seq_len = np.diff(cu)
    max_tenants = g_oracle["max_tenants"]
    covered = []
    seg_of_pair = {}
    for s in range(g_gpu["n_seg"]):
        module = int(g_gpu["seg_key"][s]) // max_tenants
        for q in range(g_gpu["seg_offset"][s], g_gpu["seg_offset"][s + 1]):
            seg_of_pair[(int(g_gpu["perm"][q]), module)] = s
    for seg, start, count, module in g_gpu["tiles"]:
        assert 1 <= count <= tile_rows
        rows = list(range(start, start + count))
        assert len({seq_of_row[r] for r in rows}) == 1 and seq_len[seq_of_row[start]] >= long_seq
        assert all(seg_of_pair[(r, int(module))] == seg for r in rows)
        assert module == g_gpu["seg_key"][seg] // max_tenants
        covered += [(r, int(module)) for r in rows]
    for count, module, job_rows in g_gpu["gather"]:
        assert 1 <= count <= gather_rows
        rows = job_rows[:count]
        assert all(r == -1 for r in job_rows[count:])
        assert len({seg_of_pair[(r, module)] for r in rows}) == 1, "rows of a gather job share one bucket"
        assert all(seq_len[seq_of_row[r]] < long_seq for r in rows)
        covered += [(r, module) for r in rows]
    assert sorted(covered) == sorted(seg_of_pair.keys()), "work lists do not cover the active pairs exactly once"
    assert len(covered) == len(g_gpu["perm"])
    for m in range(7):
        t0, t1 = g_gpu["mod_tile_offset"][m], g_gpu["mod_tile_offset"][m + 1]
        assert all(row[3] == m for row in g_gpu["tiles"][t0:t1])
        q0, q1 = g_gpu["mod_gather_offset"][m], g_gpu["mod_gather_offset"][m + 1]
        assert all(job[1] == m for job in g_gpu["gather"][q0:q1])
    assert g_gpu["mod_tile_offset"][7] == g_gpu["n_tiles"] and g_gpu["mod_gather_offset"][7] == g_gpu["n_gather"]
