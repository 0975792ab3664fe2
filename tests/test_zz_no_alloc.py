"""milora_route_static against milora_route and against the oracle, and that it allocates nothing.

Some callers of this library cannot allocate device memory while they serve: an inference engine whose
memory pool has taken the whole GPU, code running while the allocator is frozen, or a latency path that
cannot afford the device-wide synchronisation a cudaMalloc/cudaFree implies.  milora_route may grow a
scratch buffer; milora_route_static keeps its scratch in a fixed array inside the library instead.  Both
must write the same route table, logits and probabilities, and both are compared with the fp64 oracle (the
two entry points share their kernels, so agreeing with each other alone would not show a fault in what they
share).  The fixed array is shared by all calls and keeps the previous call's contents, so the comparison is
made on two calls in a row, with different prompts, and the second call must not be disturbed by what the first
one left behind.  The static call is also made first on a fresh context, with a batch larger than any before,
and the device's free memory must be the same before and after it.

This file sorts last on purpose: a run that stops at the first failure has then run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import milora_oracle as O
from oracle import reference_run as R
from synth import get_workload
from synth.workloads import scaled_workload

from parity_utils import compare_routes

pytestmark = pytest.mark.gpu

TOL = 1e-4   # same relative tolerance as the fp32 parity tests (the two entry points share one kernel)


def _route_both(lw, li, ids, H):
    w = lw.w
    cu = torch.from_numpy(w.cu_seqlens(ids)).cuda()
    slots = torch.tensor(list(ids), dtype=torch.int32, device="cuda")
    P = len(ids)
    out = {}
    for name, fn in (("dynamic", lw.ml.route), ("static", lw.ml.route_static)):
        # forget earlier decisions so that each entry point has to write the rows itself
        lw.ml.route_table_write(0, np.full((w.n_requests, len(lw.layers)), -1, dtype=np.int32))
        logits = torch.full((P, 7), float("nan"), device="cuda")
        probs = torch.full((P, 7), float("nan"), device="cuda")
        fn(li, H, cu, slots, logits, probs)
        torch.cuda.synchronize()
        out[name] = (lw.ml.route_table_read(0, w.n_requests).numpy().copy(), logits.cpu().numpy(), probs.cpu().numpy())
    return out


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_route_static_matches_route_on_two_calls_in_a_row(dtype):
    from paper_2410_18035_b200.workload_runner import LoadedWorkload
    base = get_workload("c1")
    lens = np.array([300, 64, 1, 129, 17, 257], dtype=np.int32)
    w = scaled_workload(base, name="no_alloc", dtype=dtype, d_model=512, d_ff=1376, d_kv=512, n_tenants=3,
                        request_tenant=np.array([0, 1, 2, 0, 1, 2], dtype=np.int32), prompt_len=lens,
                        prefill_ids=np.arange(6), decode_ids=np.zeros(0, dtype=np.int64), has_base_weights=False)
    lw = LoadedWorkload(w, "cuda", register_adapters=False)
    calls = [(0, [0, 1, 2, 3, 4, 5]), (1, [5, 2, 0])]      # second call: other layer, fewer and other prompts
    for li, ids in calls:
        H = w.hidden_batch(lw.layers[li], ids, "cuda")
        got = _route_both(lw, li, ids, H)
        table_d, logits_d, probs_d = got["dynamic"]
        table_s, logits_s, probs_s = got["static"]
        assert np.array_equal(table_s, table_d)
        assert (table_s[ids, li] >= 0).all() and np.isfinite(logits_s).all()
        scale = max(1e-3, float(np.abs(logits_d).max()))
        assert np.abs(logits_s - logits_d).max() <= TOL * scale
        assert np.abs(probs_s - probs_d).max() <= TOL
        # and against the oracle: routes bit-exact (near ties excused and counted), logits to fp32 accumulation
        tmp = np.full((w.n_requests, w.n_layers), -1, dtype=np.int32)
        lo, margins = R.route_requests(w, lw.layers[li], ids, tmp)
        assert compare_routes(table_s[ids, li], tmp[ids, lw.layers[li]], margins) <= 1
        assert np.abs(logits_s - lo).max() <= 2e-4 * max(1e-3, float(np.abs(lo).max()))
        np.testing.assert_allclose(probs_s, O.softmax(lo), atol=2e-4)
    assert lw.ml.poll_error() == 0
    lw.close()


def test_route_static_allocates_nothing():
    """The static call first on a fresh context, with a batch larger than any this context has seen: the free
    memory of the device is the same before and after (every tensor of the test exists before the first reading)."""
    from paper_2410_18035_b200.workload_runner import LoadedWorkload
    base = get_workload("c1")
    lens = np.array([900, 700, 64, 1], dtype=np.int32)
    w = scaled_workload(base, name="no_alloc_fresh", dtype="bf16", d_model=1024, d_ff=2816, d_kv=256, n_tenants=2,
                        request_tenant=np.array([0, 1, 0, 1], dtype=np.int32), prompt_len=lens, prefill_ids=np.arange(4),
                        decode_ids=np.zeros(0, dtype=np.int64), has_base_weights=False, n_layers=1)
    lw = LoadedWorkload(w, "cuda", register_adapters=False)
    ids = [0, 1, 2, 3]
    H = w.hidden_batch(0, ids, "cuda")
    cu = torch.from_numpy(w.cu_seqlens(ids)).cuda()
    slots = torch.tensor(ids, dtype=torch.int32, device="cuda")
    logits = torch.zeros((4, 7), device="cuda")
    probs = torch.zeros((4, 7), device="cuda")
    lw.ml.route_static(0, H[:64], cu[:2].clone().fill_(0), slots[:1], logits[:1], probs[:1])   # set-up call (looks the array up)
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    lw.ml.route_static(0, H, cu, slots, logits, probs)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "milora_route_static changed the device's free memory"
    tmp = np.full((w.n_requests, w.n_layers), -1, dtype=np.int32)
    lo, margins = R.route_requests(w, 0, ids, tmp)
    table = lw.ml.route_table_read(0, w.n_requests).numpy()
    assert compare_routes(table[ids, 0], tmp[ids, 0], margins) == 0
    assert np.abs(logits.cpu().numpy() - lo).max() <= 2e-4 * max(1e-3, float(np.abs(lo).max()))
    assert lw.ml.poll_error() == 0
    lw.close()


def test_route_static_rejects_batches_beyond_its_fixed_scratch():
    from paper_2410_18035_b200 import Milora, MiloraError
    ml = Milora(1, 4096, 11008, 4096, "bf16", 16, 2, 2)
    # (T/64 + P) * (d + 2) floats must fit in 4 Mi floats: 70,000 rows of width 4096 do not
    T = 70_000
    H = torch.empty((T, 4096), dtype=torch.bfloat16, device="cuda")
    cu = torch.tensor([0, T], dtype=torch.int32, device="cuda")
    slots = torch.zeros(1, dtype=torch.int32, device="cuda")
    with pytest.raises(MiloraError) as e:
        ml.route_static(0, H, cu, slots)
    assert e.value.status == 5
    ml.close()
