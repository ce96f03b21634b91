"""World-size-2 check of the multi-GPU host logic on CPU (gloo): ranks own disjoint rollout groups, agree on the
global per-model counts, and the all-reduced dW equals the single-process result.  The per-rank compute is the
fp64 oracle (test infrastructure), so the test exercises exactly the exchange code the benchmark uses."""
import os

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import unity_oracle as orc
from paper_2605_26646_b200 import sharding


def make_problem():
    rng = np.random.default_rng(5)
    G, per_group, H, V, K = 6, 3, 8, 24, 2
    S = G * per_group
    inv_group = np.repeat(np.arange(G), per_group)
    inv_role = rng.integers(0, 3, S)
    role_model = np.array([0, 1, 0])
    lens = rng.integers(1, 5, S)
    cu = np.concatenate([[0], np.cumsum(lens)])
    N = int(cu[-1])
    return dict(G=G, K=K, inv_group=inv_group, inv_role=inv_role, role_model=role_model, cu=cu,
                hidden=rng.normal(size=(N, H)), W=[rng.normal(size=(V, H)) * 0.3 for _ in range(K)],
                target=rng.integers(0, V, N), mask=(rng.random(N) < 0.8).astype(np.uint8),
                old=rng.normal(size=N) * 0.1 - 3, ref=rng.normal(size=N) * 0.1 - 3, adv=rng.normal(size=N))


def run_oracle(p, keep_inv, norm):
    """Oracle on the invocations in keep_inv (others lose their tokens through the mask)."""
    tok_inv = orc.token_invocation(p["cu"])
    mask = p["mask"] * keep_inv[tok_inv]
    return orc.ppo_loss_fwd_bwd(p["hidden"], p["W"], p["cu"], p["inv_role"], p["role_model"], p["target"], mask,
                                p["old"], p["ref"], p["adv"], kl_coef=0.1, norm=norm), mask


def worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    p = make_problem()
    mine = sharding.shard_groups(p["G"], rank, world)
    keep_inv = np.isin(p["inv_group"], list(mine)).astype(np.uint8)
    tok_inv = orc.token_invocation(p["cu"])
    _, tok_model = orc.token_role_model(p["cu"], p["inv_role"], p["role_model"])
    mask = p["mask"] * keep_inv[tok_inv]
    counts = sharding.local_counts(torch.from_numpy(tok_model), torch.from_numpy(mask), p["K"])
    norm = sharding.global_norm(counts)
    res, _ = run_oracle(p, keep_inv, norm)
    dW = [torch.from_numpy(x.copy()) for x in res["dW"]]
    sharding.allreduce_grads(dW)
    loss = torch.from_numpy(res["loss"].copy())
    dist.all_reduce(loss)
    if rank == 0:
        torch.save(dict(norm=norm, dW=dW, loss=loss), out)
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reproduce_the_single_process_update(tmp_path):
    out = str(tmp_path / "r0.pt")
    port = 29500 + (os.getpid() % 2000)
    mp.spawn(worker, args=(2, port, out), nprocs=2, join=True)
    got = torch.load(out)
    p = make_problem()
    full, mask = run_oracle(p, np.ones(len(p["inv_group"]), np.uint8), None)
    assert got["norm"] == [float(x) for x in full["M"]]
    assert np.allclose(got["loss"].numpy(), full["loss"], atol=1e-13)
    for k in range(p["K"]):
        assert np.allclose(got["dW"][k].numpy(), full["dW"][k], atol=1e-13)


def test_group_shards_partition_the_groups():
    for n, world in [(64, 8), (7, 2), (3, 4)]:
        owned = [g for r in range(world) for g in sharding.shard_groups(n, r, world)]
        assert owned == list(range(n))
