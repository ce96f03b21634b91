"""GPU parity of the ready-batch construction and the delayed-reward alignment (integer work: bit-exact)."""
import numpy as np
import pytest
import torch

import oracle.unity_oracle as orc
from paper_2605_26646_b200 import binding as ub
from paper_2605_26646_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def run_plan(ctx, w, done, role_model, K, seed, n_parts, pad_to):
    order = torch.full((w.n_inv,), 7, dtype=torch.int32, device="cuda")
    out_cu = torch.full((w.n_inv + 1,), 7, dtype=torch.int64, device="cuda")
    model_offsets = torch.full((K + 1,), 7, dtype=torch.int32, device="cuda")
    part_offsets = torch.full((K * n_parts + 1,), 7, dtype=torch.int32, device="cuda")
    totals = torch.full((2,), 7, dtype=torch.int64, device="cuda")
    ctx.ready_batch_plan(w.cu_seqlens.cuda(), w.inv_role.cuda(), w.inv_traj.cuda(), done.cuda(), role_model, K, seed,
                         n_parts, pad_to, order, out_cu, model_offsets, part_offsets, totals)
    ctx.check_status()
    return order, out_cu, model_offsets, part_offsets, totals


@pytest.mark.parametrize("name,n_parts,pad_to,seed", [("tiny", 1, 1, 1), ("rag_qa", 8, 1, 20260528),
                                                      ("search", 4, 16, (1 << 63) + 5), ("code", 3, 128, 7),
                                                      ("stress", 16, 8, 99)])
def test_ready_batch_plan_and_gather_match_the_oracle(name, n_parts, pad_to, seed):
    w = wl.make_structure(name)
    done = (wl.uniform(31, 1, w.n_traj) < 0.8).to(torch.uint8)
    role_model = w.role_model.tolist()
    ctx = ub.Context(0, 1 << 22)
    order, out_cu, model_offsets, part_offsets, totals = run_plan(ctx, w, done, role_model, w.K, seed, n_parts, pad_to)
    o = orc.ready_batch_plan(w.cu_seqlens.numpy(), w.inv_role.numpy(), w.inv_traj.numpy(), done.numpy(), role_model,
                             w.K, seed, n_parts=n_parts, pad_to=pad_to)
    n_kept = o["n_kept"]
    assert totals.tolist() == [n_kept, o["n_tok"]]
    assert np.array_equal(order.cpu().numpy()[:n_kept], o["order"]) and torch.all(order[n_kept:] == -1)
    assert np.array_equal(out_cu.cpu().numpy()[:n_kept + 1], o["out_cu"]) and torch.all(out_cu[n_kept:] == o["n_tok"])
    assert np.array_equal(model_offsets.cpu().numpy(), o["model_offsets"])
    assert np.array_equal(part_offsets.cpu().numpy(), o["part_offsets"])

    # token-level tensors of three widths: int32 ids, u8 mask, bf16 rows
    n_out = int(o["n_tok"])
    src_cu = w.cu_seqlens.cuda()
    tgt = w.target.cuda()
    dst = torch.full((n_out + 3,), 7, dtype=torch.int32, device="cuda")
    ctx.ready_batch_gather(order, src_cu, out_cu, totals, tgt, dst, pad_value=-100)
    want = orc.ready_batch_gather(w.target.numpy(), w.cu_seqlens.numpy(), o["order"], o["out_cu"], -100)
    assert np.array_equal(dst.cpu().numpy()[:n_out], want) and torch.all(dst[n_out:] == 7)
    msk = w.tok_mask.cuda()
    dstm = torch.full((n_out,), 7, dtype=torch.uint8, device="cuda")
    ctx.ready_batch_gather(order, src_cu, out_cu, totals, msk, dstm, pad_value=0)
    assert np.array_equal(dstm.cpu().numpy(), orc.ready_batch_gather(w.tok_mask.numpy(), w.cu_seqlens.numpy(),
                                                                     o["order"], o["out_cu"], 0))
    if w.n_tok <= 200000:
        Hs = 72                                                    # rows of 144 bytes: 16-byte copy units
        rows = (torch.arange(w.n_tok * Hs, dtype=torch.float32) % 251).to(torch.bfloat16).view(w.n_tok, Hs)
        dsth = torch.full((n_out, Hs), 7, dtype=torch.bfloat16, device="cuda")
        ctx.ready_batch_gather(order, src_cu, out_cu, totals, rows.cuda(), dsth, pad_value=0)
        wanth = orc.ready_batch_gather(rows.float().numpy(), w.cu_seqlens.numpy(), o["order"], o["out_cu"], 0.0)
        assert np.array_equal(dsth.float().cpu().numpy(), wanth)
    ctx.check_status()
    ctx.close()


def test_ready_batch_edge_cases():
    w = wl.make_structure("tiny")
    ctx = ub.Context(0, 1 << 20)
    # nothing complete: empty batch, every model and partition empty
    done = torch.zeros(w.n_traj, dtype=torch.uint8)
    order, out_cu, mo, po, totals = run_plan(ctx, w, done, [0, 0], 1, 3, 4, 8)
    assert totals.tolist() == [0, 0] and torch.all(order == -1) and torch.all(out_cu == 0)
    assert mo.tolist() == [0, 0] and po.tolist() == [0] * 5
    # a role that is not trained (-1) is dropped without an error; a model without data is empty
    done = torch.ones(w.n_traj, dtype=torch.uint8)
    order, out_cu, mo, po, totals = run_plan(ctx, w, done, [-1, 1], 2, 3, 2, 1)
    o = orc.ready_batch_plan(w.cu_seqlens.numpy(), w.inv_role.numpy(), w.inv_traj.numpy(), done.numpy(), [-1, 1], 2, 3,
                             n_parts=2, pad_to=1)
    assert totals[0].item() == o["n_kept"] == int((w.inv_role == 1).sum())
    assert np.array_equal(order.cpu().numpy()[:o["n_kept"]], o["order"])
    assert np.array_equal(po.cpu().numpy(), o["part_offsets"]) and mo.tolist() == o["model_offsets"].tolist()
    # bad ids: dropped and flagged, nothing else disturbed
    bad_role = w.inv_role.clone()
    bad_role[3] = 9
    order2 = torch.empty(w.n_inv, dtype=torch.int32, device="cuda")
    out_cu2 = torch.empty(w.n_inv + 1, dtype=torch.int64, device="cuda")
    mo2 = torch.empty(2, dtype=torch.int32, device="cuda")
    po2 = torch.empty(2, dtype=torch.int32, device="cuda")
    tot2 = torch.empty(2, dtype=torch.int64, device="cuda")
    ctx.ready_batch_plan(w.cu_seqlens.cuda(), bad_role.cuda(), w.inv_traj.cuda(), done.cuda(), [0, 0], 1, 3, 1, 1,
                         order2, out_cu2, mo2, po2, tot2)
    with pytest.raises(ub.UnityError) as e:
        ctx.check_status()
    assert e.value.code == -7
    assert tot2[0].item() == w.n_inv - 1 and 3 not in order2.tolist()
    # argument errors
    with pytest.raises(ub.UnityError):
        ctx.ready_batch_plan(w.cu_seqlens.cuda(), w.inv_role.cuda(), w.inv_traj.cuda(), done.cuda(), [0, 2], 2, 3, 1, 1,
                             order2, out_cu2, mo2, po2, tot2)
    with pytest.raises(ub.UnityError):
        ctx.ready_batch_plan(w.cu_seqlens.cuda(), w.inv_role.cuda(), w.inv_traj.cuda(), done.cuda(), [0, 0], 1, 3, 0, 1,
                             order2, out_cu2, mo2, po2, tot2)
    ctx.close()


@pytest.mark.parametrize("name,masked", [("tiny", True), ("code", True), ("search", False)])
def test_align_rewards_full_size(name, masked):
    w = wl.make_structure(name)
    r = wl.normal(32, 1, w.n_inv)
    mask = w.tok_mask if masked else None
    ctx = ub.Context(0, 1 << 20)
    out = torch.full((w.n_tok,), 7.0, device="cuda")
    ctx.align_rewards(w.cu_seqlens.cuda(), None if mask is None else mask.cuda(), r.cuda(), out)
    ctx.check_status()
    want = orc.align_rewards(r.numpy(), w.cu_seqlens.numpy(), None if mask is None else mask.numpy())
    assert np.array_equal(out.cpu().numpy().astype(np.float64), want)
    ctx.close()


def test_align_rewards_unaligned_views_and_all_masked_sequences():
    w = wl.make_structure("rag_qa")
    r = wl.normal(33, 1, w.n_inv)
    mask = w.tok_mask.clone()
    lo, hi = int(w.cu_seqlens[5]), int(w.cu_seqlens[6])
    mask[lo:hi] = 0                                            # a sequence without any unmasked token drops its reward
    ctx = ub.Context(0, 1 << 20)
    m_dev = torch.cat([torch.zeros(1, dtype=torch.uint8), mask]).cuda()[1:]          # pointers off by one element
    out = torch.full((w.n_tok + 1,), 7.0, device="cuda")[1:]
    ctx.align_rewards(w.cu_seqlens.cuda(), m_dev, r.cuda(), out)
    ctx.check_status()
    want = orc.align_rewards(r.numpy(), w.cu_seqlens.numpy(), mask.numpy())
    assert np.array_equal(out.cpu().numpy().astype(np.float64), want) and np.all(want[lo:hi] == 0)
    # the aligned path on the same data
    out2 = torch.full((w.n_tok,), 7.0, device="cuda")
    ctx.align_rewards(w.cu_seqlens.cuda(), mask.cuda(), r.cuda(), out2)
    ctx.check_status()
    assert np.array_equal(out2.cpu().numpy().astype(np.float64), want)
    ctx.close()


def test_ready_batch_many_partitions_sixteen_models_and_zero_length_invocations():
    # more partitions than invocations per model (most are empty), the largest model count, invocations of length 0
    w = wl.make_structure("search", cut_rows=2000, cut_max_len=40)      # most invocations keep no tokens at all
    R, K = ub.UNITY_MAX_ROLES, ub.UNITY_MAX_MODELS
    s = torch.arange(w.n_inv)
    inv_role = ((w.inv_role.long() + 3 * (s % 22)) % R).to(torch.int32)
    role_model = [(v * 7) % K if v % 5 else -1 for v in range(R)]      # every fifth role is not trained
    done = (wl.uniform(34, 1, w.n_traj) < 0.6).to(torch.uint8)
    n_parts, pad_to, seed = 300, 32, 123456789
    ctx = ub.Context(0, 1 << 22)
    order = torch.full((w.n_inv,), 7, dtype=torch.int32, device="cuda")
    out_cu = torch.full((w.n_inv + 1,), 7, dtype=torch.int64, device="cuda")
    mo = torch.full((K + 1,), 7, dtype=torch.int32, device="cuda")
    po = torch.full((K * n_parts + 1,), 7, dtype=torch.int32, device="cuda")
    totals = torch.full((2,), 7, dtype=torch.int64, device="cuda")
    ctx.ready_batch_plan(w.cu_seqlens.cuda(), inv_role.cuda(), w.inv_traj.cuda(), done.cuda(), role_model, K, seed,
                         n_parts, pad_to, order, out_cu, mo, po, totals)
    ctx.check_status()
    o = orc.ready_batch_plan(w.cu_seqlens.numpy(), inv_role.numpy(), w.inv_traj.numpy(), done.numpy(), role_model, K,
                             seed, n_parts=n_parts, pad_to=pad_to)
    n_kept = o["n_kept"]
    assert totals.tolist() == [n_kept, o["n_tok"]] and n_kept > 0
    assert np.array_equal(order.cpu().numpy()[:n_kept], o["order"])
    assert np.array_equal(out_cu.cpu().numpy()[:n_kept + 1], o["out_cu"])
    assert np.array_equal(mo.cpu().numpy(), o["model_offsets"])
    assert np.array_equal(po.cpu().numpy(), o["part_offsets"])
    ctx.close()
