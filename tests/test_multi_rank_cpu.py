"""The N > 1 path on CPU ranks (gloo, world size 2): requests are sharded by tenant, every rank works on its own
shard with no data-path collective, and the only communication is the barrier and the MAX of the step times."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import reference_run as R
    from synth import get_workload
    from synth.workloads import shard_by_tenant

    w = get_workload("c1")
    mine = shard_by_tenant(w.request_tenant, world)[rank]
    table = np.full((w.n_requests, w.n_layers), -1, dtype=np.int32)
    for layer in range(w.n_layers):
        R.route_requests(w, layer, mine, table)
    # timing protocol of the benchmark: barrier, then the slowest rank defines the step time
    dist.barrier()
    t = torch.tensor([1.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    # gather the shards' route rows (a test-side check only; the data path itself never communicates)
    rows = [torch.zeros((w.n_requests, w.n_layers), dtype=torch.int32) for _ in range(world)]
    dist.all_gather(rows, torch.from_numpy(table))
    if rank == 0:
        np.save(os.path.join(out_dir, "gathered.npy"), np.stack([r.numpy() for r in rows]))
        np.save(os.path.join(out_dir, "tmax.npy"), t.numpy())
    dist.destroy_process_group()


def test_tenant_sharding_over_two_gloo_ranks(tmp_path):
    from oracle import reference_run as R
    from synth import get_workload
    from synth.workloads import shard_by_tenant

    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    gathered = np.load(tmp_path / "gathered.npy")
    w = get_workload("c1")
    full, _ = R.full_route_table(w)
    shards = shard_by_tenant(w.request_tenant, world)
    # the shards partition the requests, every tenant sits on exactly one rank
    assert sorted(np.concatenate(shards).tolist()) == list(range(w.n_requests))
    for r in range(world):
        assert set(w.request_tenant[shards[r]] % world) <= {r}
        assert np.array_equal(gathered[r][shards[r]], full[shards[r]])          # same decisions as one process
        other = np.setdiff1d(np.arange(w.n_requests), shards[r])
        assert np.all(gathered[r][other] == -1)                                # and nothing outside the shard
    assert np.load(tmp_path / "tmax.npy")[0] == 2.0                            # MAX over ranks


def test_shard_by_tenant_structure():
    from synth import get_workload
    from synth.workloads import shard_by_tenant
    w = get_workload("c4")
    for world in (1, 2, 4, 8):
        shards = shard_by_tenant(w.request_tenant, world)
        assert sum(len(s) for s in shards) == w.n_requests
        tenants = [set(w.request_tenant[s].tolist()) for s in shards]
        for a in range(world):
            for b in range(a + 1, world):
                assert not (tenants[a] & tenants[b])


def _c4_routes(w, layer):
    """A seeded stand-in for layer `layer`'s route column of config 4 (grouping depends on routes and tenants only;
    routing 256 prompts of 256 x 5120 with the oracle is not needed to test the sharding)."""
    return np.random.default_rng(1000 + layer).integers(0, 7, size=w.n_requests).astype(np.int32)


def _rank_group_c4(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import milora_oracle as O
    from synth import get_workload
    from synth.workloads import shard_by_tenant

    w = get_workload("c4")
    mine = shard_by_tenant(w.request_tenant, world)[rank]
    out = {}
    for layer in (0, 17, 39):
        routes = _c4_routes(w, layer)
        # this rank's decode step: one row per request of its shard, in request order
        g = O.group_tokens(mine, w.request_tenant, routes, lambda t, m: True, w.n_tenants)
        out[f"perm{layer}"] = mine[g["perm"]]                 # as request ids, comparable across ranks
        out[f"key{layer}"] = g["seg_key"]
        out[f"off{layer}"] = g["seg_offset"]
    dist.barrier()
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), **out)
    dist.destroy_process_group()


def test_one_c4_batch_sharded_by_tenant_groups_like_one_process(tmp_path):
    """One decode batch of config 4 (256 requests, Zipf tenants) split over two ranks by tenant: every (module, tenant)
    bucket of the single-process grouping lands on exactly one rank, whole and in the same row order, for layers at
    both ends and in the middle of the stack; no rank sees a request of the other."""
    from oracle import milora_oracle as O
    from synth import get_workload
    from synth.workloads import shard_by_tenant

    world = 2
    mp.spawn(_rank_group_c4, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    w = get_workload("c4")
    shards = shard_by_tenant(w.request_tenant, world)
    ranks = [np.load(tmp_path / f"rank{r}.npz") for r in range(world)]
    everyone = np.arange(w.n_requests)
    for layer in (0, 17, 39):
        routes = _c4_routes(w, layer)
        g = O.group_tokens(everyone, w.request_tenant, routes, lambda t, m: True, w.n_tenants)
        full = {int(k): g["perm"][g["seg_offset"][s]:g["seg_offset"][s + 1]].tolist() for s, k in enumerate(g["seg_key"])}
        seen = {}
        for r in range(world):
            keys, off, perm = ranks[r][f"key{layer}"], ranks[r][f"off{layer}"], ranks[r][f"perm{layer}"]
            assert set(perm.tolist()) == set(shards[r].tolist())
            assert np.all(np.diff(keys) > 0)                                   # canonical order: module, then tenant
            for s, k in enumerate(keys):
                assert int(k) not in seen, "a bucket is split over two ranks"
                seen[int(k)] = perm[off[s]:off[s + 1]].tolist()
                assert (int(k) % w.n_tenants) % world == r                     # the tenant's home rank
        assert seen == full
