"""Population sharding: the host-side logic on two gloo ranks on CPU (the oracle stands in for the kernels)."""
import os
import subprocess
import sys
import textwrap

import pytest

from paper_2511_16652_b200 import sharding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("N,world,anti", [(10, 3, False), (32, 4, True), (6, 4, True), (7, 2, False), (2, 3, True)])
def test_member_ranges_partition_the_population(N, world, anti):
    covered = []
    for r in range(world):
        base, cnt = sharding.member_range(N, world, r, anti)
        if anti:
            assert base % 2 == 0 and cnt % 2 == 0
        covered += list(range(base, base + cnt))
    assert covered == list(range(N))
    sizes = [sharding.member_range(N, world, r, anti)[1] for r in range(world)]
    assert max(sizes) - min(sizes) <= (2 if anti else 1)


def test_two_rank_step_equals_single_process(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(textwrap.dedent(f"""
        import sys, json
        sys.path.insert(0, {ROOT!r}); sys.path.insert(0, {os.path.join(ROOT, 'tests')!r})
        import numpy as np, torch, torch.distributed as dist
        import oracle, workloads
        from paper_2511_16652_b200 import sharding
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        N, T, m, n, r, seed, sigma, alpha = 10, 2, 6, 8, 2, 4, 0.3, 0.2
        W, X = workloads.linear_layer(1, m, n, N * T, bf16=False)
        X = workloads.pair_shared_rows(X, T)
        target = workloads.rng(1, 3).standard_normal(m)
        base, cnt = sharding.member_range(N, world, rank, antithetic=True)
        members = np.arange(base, base + cnt)
        Y = oracle.perturbed_linear(X[base * T:(base + cnt) * T], W, members, T, r, 0, seed, oracle.ANTITHETIC, sigma)
        local = -((Y - target) ** 2).sum(axis=1).reshape(cnt, T).mean(axis=1)
        full = sharding.all_gather_fitness(torch.from_numpy(local), N, antithetic=True).numpy()
        shaped = oracle.fitness_shape(full.astype(np.float32), oracle.SHAPE_CENTERED_RANK)
        Wn, _ = oracle.es_update(W, shaped, r, 0, seed, oracle.ANTITHETIC, alpha)
        # single-process answer, computed on every rank
        Y1 = oracle.perturbed_linear(X, W, np.arange(N), T, r, 0, seed, oracle.ANTITHETIC, sigma)
        f1 = -((Y1 - target) ** 2).sum(axis=1).reshape(N, T).mean(axis=1)
        W1, _ = oracle.es_update(W, oracle.fitness_shape(f1.astype(np.float32), oracle.SHAPE_CENTERED_RANK), r, 0, seed,
                                 oracle.ANTITHETIC, alpha)
        ok = bool(np.array_equal(full, f1) and np.array_equal(Wn, W1))
        flags = [None] * world
        dist.all_gather_object(flags, ok)
        if rank == 0:
            print(json.dumps({{"ok": all(flags), "ranges": [sharding.member_range(N, world, q, True) for q in range(world)]}}))
        dist.destroy_process_group()
    """))
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29741", str(script)],
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-3000:]
    import json
    res = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert res["ok"], res
    assert res["ranges"] == [[0, 4], [4, 6]]


def test_three_rank_packed_sign_exchange(tmp_path):
    """Base-3 packed exchange of pair signs on three gloo ranks with uneven ranges (the oracle's pack / unpack stand in
    for the kernels): every rank ends with the full sign vector."""
    script = tmp_path / "worker_pack.py"
    script.write_text(textwrap.dedent(f"""
        import sys, json
        sys.path.insert(0, {ROOT!r})
        import numpy as np, torch, torch.distributed as dist
        import oracle, workloads
        from paper_2511_16652_b200 import sharding
        dist.init_process_group("gloo")
        rank, world = dist.get_rank(), dist.get_world_size()
        N = 46                                            # 23 pairs over 3 ranks: 7, 8, 8 pairs -> 2 bytes each
        raw = workloads.rng(5, 1).integers(-3, 4, size=N).astype(np.int32)
        signs = oracle.fitness_shape_i8(raw)
        base, cnt = sharding.member_range(N, world, rank, antithetic=True)
        local = torch.from_numpy(signs[base // 2:(base + cnt) // 2].copy())
        pack = lambda t: torch.from_numpy(oracle.pack3(t.numpy()))
        unpack = lambda b, c: torch.from_numpy(oracle.unpack3(b.numpy(), c))
        full = sharding.all_gather_packed_signs(local, N, pack, unpack).numpy()
        ok = bool(np.array_equal(full, signs))
        flags = [None] * world
        dist.all_gather_object(flags, ok)
        if rank == 0:
            print(json.dumps({{"ok": all(flags), "pairs": [sharding.member_range(N, world, q, True)[1] // 2 for q in range(world)]}}))
        dist.destroy_process_group()
    """))
    out = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=3",
                          "--master-addr", "127.0.0.1", "--master-port", "29743", str(script)],
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-3000:]
    import json
    res = json.loads([l for l in out.stdout.splitlines() if l.startswith("{")][-1])
    assert res["ok"], res
    assert sorted(res["pairs"]) == [7, 8, 8]
