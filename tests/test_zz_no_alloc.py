"""unity_role_advantage_noalloc against unity_role_advantage and against the fp64 oracle.

The allocation-free entry point serves hosts that cannot create a context (no cudaMalloc allowed: all device
memory belongs to the host framework's allocator, or an allocation's device-wide sync is unaffordable).  It must
give what the regular call gives, and both must match the oracle.  Two calls in a row, the second on a smaller and
different batch, also check that nothing left in the shared static scratch by one call leaks into the next; the free
device memory reported by the driver must not move across a call.  Collected last on purpose."""
import numpy as np
import pytest
import torch

import parity_harness as pu
from paper_2605_26646_b200 import binding as ub
from paper_2605_26646_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def both_ways(ctx, w):
    d = pu.DeviceInputs(w)
    ref = pu.gpu_advantage(ctx, w, d)
    out = {k: torch.full_like(v, 7.0) for k, v in ref.items()}
    flag = torch.full((1,), 5, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream
    ub.unity_role_advantage_noalloc(0, stream, w.n_traj, w.n_roles, w.n_groups, d.inv_role, d.inv_group, d.inv_traj,
                                    d.r_node, d.r_turn, d.r_traj, w.lam.tolist(), w.adv_eps, w.adv_ddof, d.cu_seqlens,
                                    d.tok_mask, out["adv_inv"], out["adv_tok"], out["seg_mean"], out["seg_std"], flag)
    torch.cuda.synchronize()
    oracle = pu.oracle_advantage(w)
    for k in ref:
        assert (out[k] - ref[k]).abs().max().item() <= pu.TOL_ADV, k
        assert np.abs(out[k].cpu().numpy() - oracle[k]).max() <= pu.TOL_ADV, k       # parity is defined against the oracle
    return int(flag.item())


def test_noalloc_matches_regular_entry_point_on_two_calls_in_a_row():
    ctx = ub.Context(0, 1 << 22)
    assert both_ways(ctx, wl.make_structure("stress")) == 0            # 8192 invocations, 131072 tokens
    small = wl.make_structure("search", cut_rows=500, cut_max_len=40)   # fewer invocations, other rewards
    small.lam = torch.tensor([[1.0, 0.5, 2.0], [0.0, 1.0, 1.0], [1.5, 1.0, 0.25]])
    assert both_ways(ctx, small) == 0
    # an out-of-range role id is reported through the device flag and the invocation is left out
    bad = wl.make_structure("tiny")
    bad.inv_role[3] = 9
    d = pu.DeviceInputs(bad)
    adv_inv = torch.empty(bad.n_inv, device="cuda")
    adv_tok = torch.empty(bad.n_tok, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    ub.unity_role_advantage_noalloc(0, torch.cuda.current_stream().cuda_stream, bad.n_traj, bad.n_roles, bad.n_groups,
                                    d.inv_role, d.inv_group, d.inv_traj, d.r_node, d.r_turn, d.r_traj, None, 1e-6, 0,
                                    d.cu_seqlens, d.tok_mask, adv_inv, adv_tok, None, None, flag)
    torch.cuda.synchronize()
    assert flag.item() != 0 and adv_inv[3].item() == 0.0
    ctx.close()


def test_noalloc_call_leaves_free_device_memory_unchanged_and_covers_long_invocations():
    """1024 invocations of 160 tokens take the one-warp-per-invocation broadcast; after a first call (which may load
    the library's device code) a second call must not change the free memory the driver reports."""
    n_inv, seq, R, G = 1024, 160, 2, 64
    w = wl.make_structure("tiny")
    rng = np.random.default_rng(5)
    w.n_inv, w.n_roles, w.n_groups, w.n_traj, w.n_tok = n_inv, R, G, n_inv, n_inv * seq
    w.inv_role = torch.from_numpy(rng.integers(0, R, n_inv).astype(np.int32))
    w.inv_group = torch.from_numpy(rng.integers(0, G, n_inv).astype(np.int32))      # groups interleaved
    w.inv_traj = torch.arange(n_inv, dtype=torch.int32)
    w.r_node = torch.from_numpy(rng.normal(size=n_inv).astype(np.float32))
    w.r_turn, w.r_traj, w.lam = torch.zeros(n_inv), torch.zeros(n_inv), torch.ones(R, 3)
    w.cu_seqlens = torch.arange(n_inv + 1, dtype=torch.int64) * seq
    w.tok_mask = torch.from_numpy((rng.random(w.n_tok) < 0.8).astype(np.uint8))
    d = pu.DeviceInputs(w)
    adv_inv, adv_tok = torch.empty(n_inv, device="cuda"), torch.empty(w.n_tok, device="cuda")
    stream = torch.cuda.current_stream().cuda_stream

    def call():
        ub.unity_role_advantage_noalloc(0, stream, w.n_traj, R, G, d.inv_role, d.inv_group, d.inv_traj, d.r_node,
                                        d.r_turn, d.r_traj, None, 1e-6, 0, d.cu_seqlens, d.tok_mask, adv_inv, adv_tok)
        torch.cuda.synchronize()

    call()
    free_before = torch.cuda.mem_get_info()[0]
    call()
    assert torch.cuda.mem_get_info()[0] == free_before
    o = pu.oracle_advantage(w)
    assert np.abs(adv_tok.cpu().numpy() - o["adv_tok"]).max() <= pu.TOL_ADV


def test_noalloc_rejects_sizes_beyond_its_static_scratch():
    n = ub.UNITY_NOALLOC_MAX_INV + 1
    z32 = torch.zeros(n, dtype=torch.int32, device="cuda")
    zf = torch.zeros(n, device="cuda")
    cu = torch.zeros(n + 1, dtype=torch.int64, device="cuda")
    with pytest.raises(ub.UnityError) as e:
        ub.unity_role_advantage_noalloc(0, 0, 1, 1, 1, z32, z32, z32, zf, None, None, None, 1e-6, 0, cu, None, zf,
                                        torch.empty(0, device="cuda"))
    assert e.value.code == -2 and "UNITY_NOALLOC_MAX_INV" in str(e.value)
    with pytest.raises(ub.UnityError) as e:              # more (group, role) segments than the static table holds
        ub.unity_role_advantage_noalloc(0, 0, 1, 64, ub.UNITY_NOALLOC_MAX_SEG // 64 + 1, z32[:8], z32[:8], z32[:8],
                                        zf[:8], None, None, None, 1e-6, 0, cu[:9], None, zf[:8],
                                        torch.empty(0, device="cuda"))
    assert e.value.code == -2 and "UNITY_NOALLOC_MAX_SEG" in str(e.value)
