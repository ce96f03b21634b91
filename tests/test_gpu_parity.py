"""GPU parity: libunity (through its C ABI) against the fp64 oracle, element by element, on the same
seeded inputs.  Sizes span several row tiles, vocabulary tiles and chunks, with ragged tails."""
import numpy as np
import pytest
import torch

import parity_harness as pu
from paper_2605_26646_b200 import binding as ub
from paper_2605_26646_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def check_forward(g, o, mask):
    for key in ("logp", "entropy", "lse"):
        if key in g and key in o:
            got = g[key].cpu().numpy()
            assert np.abs(got - o[key]).max() <= pu.TOL_LOGP, key
            assert np.all(got[~mask] == 0), key + " must be 0 on masked rows"


def check_ppo(g, o, w, atol_loss=1e-6):
    mask = w.tok_mask.numpy() != 0
    check_forward(g, o, mask)
    loss = g["loss"].cpu().numpy()
    assert np.all(np.abs(loss - o["loss"]) <= pu.TOL_LOSS * np.abs(o["loss"]) + atol_loss), (loss, o["loss"])
    tl = g["tok_loss"].cpu().numpy()
    assert np.abs(tl - o["tok_loss"]).max() <= pu.TOL_LOGP
    assert np.all(tl[~mask] == 0)
    dH = g["dHidden"].float().cpu().numpy()
    assert np.all(dH[~mask] == 0), "dHidden must be 0 on masked rows"
    if np.linalg.norm(o["dHidden"]) > 0:
        assert pu.rel_fro(dH, o["dHidden"]) <= pu.TOL_GRAD
        # the same tolerance row by row: a wrong tile, store segment or ragged tail cannot hide in the whole-tensor norm
        slack = pu.dh_row_allowance(w, o, g["logp"].cpu().numpy(), **o["inputs"]) if "inputs" in o else None
        assert pu.worst_row_rel(dH, o["dHidden"], slack) <= pu.TOL_GRAD
    else:
        assert np.abs(dH).max() == 0
    for k in range(w.K):
        got = g["dW"][k].cpu().numpy()
        if o["dW"][k] is None:
            continue
        if np.linalg.norm(o["dW"][k]) > 0:
            assert pu.rel_fro(got, o["dW"][k]) <= pu.TOL_GRAD, f"dW[{k}]"
            # ... and per block of 256 vocabulary rows (one output tile of the dW GEMM)
            assert pu.worst_block_rel_fro(got, o["dW"][k]) <= pu.TOL_GRAD, f"dW[{k}] per block"
        else:
            assert np.abs(got).max() == 0
    om = np.concatenate([o["metrics_model"], o["metrics_role"]])
    gm = g["metrics"].cpu().numpy()
    assert np.array_equal(gm[:, 0], om[:, 0])                       # valid counts are exact
    assert np.abs(gm - om).max() <= 1e-3 * max(1.0, np.abs(om[:, 1:]).max())


def run_all_stages(w, ctas=None, options=(), **ppo_kw):
    d = pu.DeviceInputs(w)
    ctx = pu.make_ctx(w, stash=(ub.OPT_LOGIT_STASH, 1) in list(options))
    try:
        if ctas is not None:                       # CTAs per output tile for the four GEMM classes
            for option, value in enumerate(ctas):
                ctx.set_option(option, value)
        for option, value in options:
            ctx.set_option(option, value)
        ga, oa = pu.gpu_advantage(ctx, w, d), pu.oracle_advantage(w)
        assert np.abs(ga["adv_inv"].cpu().numpy() - oa["adv_inv"]).max() <= pu.TOL_ADV
        assert np.abs(ga["adv_tok"].cpu().numpy() - oa["adv_tok"]).max() <= pu.TOL_ADV
        gl, ol = pu.gpu_logprob(ctx, w, d), pu.oracle_logprob(w)
        check_forward(gl, ol, w.tok_mask.numpy() != 0)
        cur = torch.from_numpy(ol["logp"].astype(np.float32))
        old, ref = cur + w.noise_old, cur + w.noise_ref
        adv = torch.from_numpy(oa["adv_tok"].astype(np.float32))
        gp = pu.gpu_ppo(ctx, w, d, old.cuda(), ref.cuda(), adv.cuda(), **ppo_kw)
        op = pu.oracle_ppo(w, old.numpy(), ref.numpy(), adv.numpy(), **ppo_kw)
        check_ppo(gp, op, w)
    finally:
        ctx.close()


# ------------------------------------------------------------------------------------ stage 1

@pytest.mark.parametrize("name", list(wl.CONFIGS))
def test_advantage_full_size(name):
    w = wl.make_structure(name)
    d = pu.DeviceInputs(w)
    ctx = ub.Context(0, 1 << 22)
    g, o = pu.gpu_advantage(ctx, w, d), pu.oracle_advantage(w)
    assert np.abs(g["adv_inv"].cpu().numpy() - o["adv_inv"]).max() <= pu.TOL_ADV
    assert np.abs(g["adv_tok"].cpu().numpy() - o["adv_tok"]).max() <= pu.TOL_ADV
    assert np.abs(g["seg_mean"].cpu().numpy() - o["seg_mean"]).max() <= pu.TOL_ADV
    assert np.abs(g["seg_std"].cpu().numpy() - o["seg_std"]).max() <= pu.TOL_ADV
    if name == "stress":                       # constant segments give exactly zero
        seg = (w.inv_group.long() * w.n_roles + w.inv_role.long()).numpy()
        const = o["seg_std"][seg] == 0
        assert const.any() and np.all(g["adv_inv"].cpu().numpy()[const] == 0)
    ctx.close()


@pytest.mark.parametrize("ddof,eps,one_group", [(1, 1e-6, False), (0, 0.0, False), (0, 1e-6, True)])
def test_advantage_variants(ddof, eps, one_group):
    w = wl.make_structure("search", cut_rows=500, cut_max_len=40)
    if one_group:                              # role-wise whitening over the whole batch
        w.inv_group.zero_()
        w.n_groups = 1
    w.lam = torch.tensor([[1.0, 0.5, 2.0], [0.0, 1.0, 1.0], [1.5, 1.0, 0.25]])
    w.r_node = wl.normal(5, 77, w.n_inv)
    d = pu.DeviceInputs(w)
    ctx = ub.Context(0, 1 << 22)
    g, o = pu.gpu_advantage(ctx, w, d, ddof=ddof, eps=eps), pu.oracle_advantage(w, ddof=ddof, eps=eps)
    assert np.abs(g["adv_inv"].cpu().numpy() - o["adv_inv"]).max() <= pu.TOL_ADV
    assert np.abs(g["adv_tok"].cpu().numpy() - o["adv_tok"]).max() <= pu.TOL_ADV
    ctx.close()


def shuffled_structure(name, seed=11, **kw):
    """A configuration's invocations in a seeded random order (rollout groups interleaved, as a buffer filled in
    arrival order holds them); token data follows its invocation."""
    w = wl.make_structure(name, **kw)
    perm = torch.from_numpy(np.random.default_rng(seed).permutation(w.n_inv))
    lens = (w.cu_seqlens[1:] - w.cu_seqlens[:-1])[perm]
    starts = w.cu_seqlens[:-1][perm]
    tok_src = torch.cat([torch.arange(int(a), int(a) + int(n)) for a, n in zip(starts, lens)]) if w.n_tok else None
    for key in ("inv_role", "inv_group", "inv_traj", "r_node", "r_turn"):
        setattr(w, key, getattr(w, key)[perm].contiguous())
    w.cu_seqlens = torch.cat([torch.zeros(1, dtype=torch.int64), torch.cumsum(lens, 0)])
    if tok_src is not None:
        w.tok_mask = w.tok_mask[tok_src].contiguous()
    return w


@pytest.mark.parametrize("name", ["search", "stress"])
def test_advantage_with_invocations_in_shuffled_order(name):
    w = shuffled_structure(name)
    assert (w.inv_group[1:] < w.inv_group[:-1]).any()              # groups really are interleaved
    d = pu.DeviceInputs(w)
    ctx = ub.Context(0, 1 << 22)
    g, o = pu.gpu_advantage(ctx, w, d), pu.oracle_advantage(w)
    for key in ("adv_inv", "adv_tok", "seg_mean", "seg_std"):
        assert np.abs(g[key].cpu().numpy() - o[key]).max() <= pu.TOL_ADV, key
    again = pu.gpu_advantage(ctx, w, d)                              # order-free integer sums: bitwise reproducible
    assert all(torch.equal(g[k], again[k]) for k in g)
    ctx.close()


@pytest.mark.parametrize("case", ["offset", "tiny", "huge", "one_segment", "pairs"])
def test_advantage_statistics_on_awkward_rewards(case):
    """Rewards with a large common offset, very small and very large magnitudes, one segment holding the whole batch
    (16384 members per role) and segments of two: the per-segment integer grid must keep the oracle's result."""
    n_inv, R = 65536, 4
    G = {"one_segment": 1, "pairs": n_inv // (2 * R)}.get(case, 2048)
    rng = np.random.default_rng(3)
    w = wl.make_structure("tiny")
    w.n_inv, w.n_roles, w.n_groups, w.n_traj = n_inv, R, G, n_inv
    w.inv_role = torch.from_numpy(rng.integers(0, R, n_inv).astype(np.int32))
    w.inv_group = torch.from_numpy(rng.integers(0, G, n_inv).astype(np.int32))
    w.inv_traj = torch.arange(n_inv, dtype=torch.int32)
    base = rng.normal(size=n_inv).astype(np.float32)
    r = {"offset": 1000.0 + 0.01 * base, "tiny": 1e-30 * base, "huge": 1e30 * base}.get(case, base)
    w.r_node = torch.from_numpy(np.asarray(r, np.float32))
    w.r_turn = torch.zeros(n_inv)
    w.r_traj = torch.zeros(n_inv)
    w.lam = torch.ones(R, 3)
    w.cu_seqlens = torch.arange(n_inv + 1, dtype=torch.int64) * 2
    w.n_tok = 2 * n_inv
    w.tok_mask = torch.ones(w.n_tok, dtype=torch.uint8)
    d = pu.DeviceInputs(w)
    ctx = ub.Context(0, ub.unity_advantage_workspace_bytes(n_inv, G, R))
    eps = 0.0 if case in ("tiny", "huge") else 1e-6          # eps = 1e-6 would swamp a sigma of 1e-30
    g, o = pu.gpu_advantage(ctx, w, d, eps=eps), pu.oracle_advantage(w, eps=eps)
    assert np.abs(g["adv_inv"].cpu().numpy() - o["adv_inv"]).max() <= pu.TOL_ADV
    assert np.abs(g["adv_tok"].cpu().numpy() - o["adv_tok"]).max() <= pu.TOL_ADV
    scale = max(1.0, float(np.abs(o["seg_mean"]).max()))
    assert np.abs(g["seg_mean"].cpu().numpy() - o["seg_mean"]).max() <= 1e-6 * scale
    assert np.abs(g["seg_std"].cpu().numpy() - o["seg_std"]).max() <= 1e-6 * max(1e-30, float(o["seg_std"].max()))
    ctx.close()


def test_advantage_workspace_query_and_too_small_workspace():
    w = wl.make_structure("stress")
    d = pu.DeviceInputs(w)
    need = ub.unity_advantage_workspace_bytes(w.n_inv, w.n_groups, w.n_roles)
    assert 8 * w.n_inv + 32 * w.n_groups * w.n_roles <= need <= 8 * w.n_inv + 32 * w.n_groups * w.n_roles + 2048
    ctx = ub.Context(0, need)
    g, o = pu.gpu_advantage(ctx, w, d), pu.oracle_advantage(w)
    assert np.abs(g["adv_tok"].cpu().numpy() - o["adv_tok"]).max() <= pu.TOL_ADV
    ctx.close()
    ctx = ub.Context(0, need - 512)
    with pytest.raises(ub.UnityError) as e:
        pu.gpu_advantage(ctx, w, d)
    assert e.value.code == -4 and "unity_advantage_workspace_bytes" in str(e.value)
    ctx.close()


def test_advantage_null_inputs_unaligned_views_and_empty_batch():
    import oracle.unity_oracle as orc
    w = wl.make_structure("rag_qa")
    d = pu.DeviceInputs(w)
    ctx = ub.Context(0, 1 << 22)
    # no turn reward, no mask, default lambda
    adv_inv = torch.empty(w.n_inv, device="cuda")
    big = torch.empty(w.n_tok + 3, device="cuda")
    adv_tok = big[1:1 + w.n_tok]              # 4-byte aligned only: exercises the scalar store path
    ctx.role_advantage(w.n_traj, w.n_roles, w.n_groups, d.inv_role, d.inv_group, d.inv_traj, d.r_node, None, d.r_traj,
                       None, 1e-6, 0, d.cu_seqlens, None, adv_inv, adv_tok)
    ctx.check_status()
    o = orc.role_advantage(w.inv_role.numpy(), w.inv_group.numpy(), w.inv_traj.numpy(), w.r_node.numpy(), None,
                           w.r_traj.numpy(), None, w.n_roles, w.n_groups, w.cu_seqlens.numpy(), None)
    assert np.abs(adv_tok.cpu().numpy() - o["adv_tok"]).max() <= pu.TOL_ADV
    # invocations without any token
    cu0 = torch.zeros(w.n_inv + 1, dtype=torch.int64, device="cuda")
    ctx.role_advantage(w.n_traj, w.n_roles, w.n_groups, d.inv_role, d.inv_group, d.inv_traj, d.r_node, None, d.r_traj,
                       None, 1e-6, 0, cu0, None, adv_inv, torch.empty(0, device="cuda"))
    ctx.check_status()
    assert np.abs(adv_inv.cpu().numpy() - o["adv_inv"]).max() <= pu.TOL_ADV
    ctx.close()


def test_bad_indices_are_flagged_not_fatal():
    w = wl.make_structure("tiny")
    w.inv_role[3] = 9                          # role id out of range
    d = pu.DeviceInputs(w)
    ctx = ub.Context(0, 1 << 22)
    adv_inv = torch.empty(w.n_inv, device="cuda")
    adv_tok = torch.empty(w.n_tok, device="cuda")
    ctx.role_advantage(w.n_traj, w.n_roles, w.n_groups, d.inv_role, d.inv_group, d.inv_traj, d.r_node, d.r_turn,
                       d.r_traj, None, 1e-6, 0, d.cu_seqlens, d.tok_mask, adv_inv, adv_tok)
    with pytest.raises(ub.UnityError) as e:
        ctx.check_status()
    assert e.value.code == -7
    assert adv_inv[3].item() == 0.0
    ctx.check_status()                         # the status word was cleared
    ctx.close()


@pytest.mark.parametrize("name,rules", [("code", [(2, 0), (2, 1)]), ("search", [(1, 0), (2, 0), (1, 0)])])
def test_reward_assembly_full_size(name, rules):
    import oracle.unity_oracle as orc
    w = wl.make_structure(name)                # code: coder / reflector deltas; search: planner, searcher, answerer
    max_turns = int(w.inv_turn.max()) + 1
    score = wl.uniform(21, 3, w.n_traj * max_turns).float().view(w.n_traj, max_turns)
    n_scores = (torch.zeros(w.n_traj, dtype=torch.int64).scatter_reduce(0, w.inv_traj.long(), w.inv_turn.long() + 1,
                                                                        "amax")).to(torch.int32)
    inv_end = wl.bernoulli(21, 4, w.n_inv, 0.1).to(torch.uint8)
    ctx = ub.Context(0, 1 << 20)
    out = torch.full((w.n_inv,), 7.0, device="cuda")
    ctx.reward_assembly(w.inv_role.cuda(), w.inv_traj.cuda(), w.inv_turn.cuda(), score.cuda(), n_scores.cuda(),
                        inv_end.cuda(), rules, out)
    ctx.check_status()
    ref = orc.reward_assembly(w.inv_role.numpy(), w.inv_traj.numpy(), w.inv_turn.numpy(), score.numpy(),
                              n_scores.numpy(), rules, inv_end.numpy())
    assert np.abs(out.cpu().numpy() - ref).max() <= 1e-6
    assert np.abs(ref).max() > 0 and (ref == 0).any()
    ctx.close()


@pytest.mark.parametrize("name,gamma,lam,masked", [("tiny", 1.0, 0.95, True), ("search", 0.99, 0.9, True),
                                                   ("code", 0.97, 1.0, True), ("stress", 0.9, 0.0, False)])
def test_gae_full_size(name, gamma, lam, masked):
    import oracle.unity_oracle as orc
    w = wl.make_structure(name)                # sequence lengths 0 .. 2048, padded spans, zero-length sequences
    r = wl.normal(11, 5, w.n_tok)
    v = wl.normal(11, 6, w.n_tok)
    mask = w.tok_mask if masked else None
    ctx = ub.Context(0, 1 << 20)
    adv = torch.full((w.n_tok,), 7.0, device="cuda")
    ret = torch.full((w.n_tok,), 7.0, device="cuda")
    ctx.gae(w.cu_seqlens.cuda(), r.cuda(), v.cuda(), None if mask is None else mask.cuda(), gamma, lam, adv, ret)
    ctx.check_status()
    # the oracle evaluates the double sum literally: check the first 400 sequences (all of them for small configs)
    n_seq = min(w.n_inv, 400)
    n_chk = int(w.cu_seqlens[n_seq])
    oa, orr = orc.gae(r.numpy()[:n_chk], v.numpy()[:n_chk], w.cu_seqlens.numpy()[:n_seq + 1], gamma, lam,
                      None if mask is None else mask.numpy()[:n_chk])
    scale = max(1.0, float(np.abs(oa).max()))
    assert np.abs(adv.cpu().numpy()[:n_chk] - oa).max() <= 1e-5 * scale
    assert np.abs(ret.cpu().numpy()[:n_chk] - orr).max() <= 1e-5 * scale
    # beyond the checked prefix: masked tokens are zero and returns - advantages reproduces the values
    a_all, r_all = adv.cpu(), ret.cpu()
    keep = torch.ones(w.n_tok, dtype=torch.bool) if mask is None else mask != 0
    assert torch.all(a_all[~keep] == 0) and torch.all(r_all[~keep] == 0)
    assert torch.allclose((r_all - a_all)[keep], v[keep], atol=1e-5 * scale)
    ctx.close()


@pytest.mark.parametrize("name,clip_v,with_norm,masked", [("tiny", 0.2, False, True), ("search", 0.3, True, True),
                                                          ("code", 1e30, False, True), ("rag_qa", 0.1, False, False)])
def test_value_loss_full_size(name, clip_v, with_norm, masked):
    import oracle.unity_oracle as orc
    w = wl.make_structure(name)
    v = wl.normal(12, 1, w.n_tok)
    ov = v + 0.25 * wl.normal(12, 2, w.n_tok)
    ret = v + wl.normal(12, 3, w.n_tok)
    mask = w.tok_mask if masked else None
    norm = [float(1000 + 37 * k) for k in range(w.K)] if with_norm else None
    ctx = ub.Context(0, 1 << 20)
    loss = torch.full((w.K,), 7.0, device="cuda")
    frac = torch.full((w.K,), 7.0, device="cuda")
    tok = torch.full((w.n_tok,), 7.0, device="cuda")
    dv = torch.full((w.n_tok,), 7.0, device="cuda")
    ctx.value_loss_fwd_bwd(w.cu_seqlens.cuda(), w.inv_role.cuda(), w.role_model.tolist(), w.K,
                           None if mask is None else mask.cuda(), v.cuda(), ov.cuda(), ret.cuda(), clip_v, norm, loss,
                           frac, tok, dv)
    ctx.check_status()
    o = orc.value_loss_fwd_bwd(v.numpy(), ov.numpy(), ret.numpy(), w.cu_seqlens.numpy(), w.inv_role.numpy(),
                               w.role_model.numpy(), None if mask is None else mask.numpy(), clip_v=clip_v, norm=norm,
                               K=w.K)
    assert np.all(np.abs(loss.cpu().numpy() - o["loss"]) <= pu.TOL_LOSS * np.abs(o["loss"]) + 1e-7)
    assert np.abs(frac.cpu().numpy() - o["clip_frac"]).max() <= 1e-4
    assert np.abs(tok.cpu().numpy() - o["tok_loss"]).max() <= 1e-5 * max(1.0, float(o["tok_loss"].max()))
    # the branch is a comparison of two squares: where they agree to rounding either side may win, and the
    # gradient jumps there; such tokens (a handful in a million) are compared against both branches
    vd, ovd, rd = (x.numpy().astype(np.float64) for x in (v, ov, ret))
    d = vd - ovd
    vc = np.where(np.abs(d) <= clip_v, vd, ovd + np.sign(d) * clip_v)
    su, sc = (vd - rd) ** 2, (vc - rd) ** 2
    near = (np.abs(su - sc) <= 1e-5 * np.maximum(su, sc)) & (np.abs(d) > clip_v)
    assert near.sum() <= 1e-4 * w.n_tok + 2
    g = dv.cpu().numpy().astype(np.float64)
    scale = np.abs(o["dvalues"]).max()
    assert np.abs(g - o["dvalues"])[~near].max() <= 1e-5 * scale
    keep = np.ones(w.n_tok, bool) if mask is None else mask.numpy() != 0
    assert np.all(g[~keep] == 0) and np.all(tok.cpu().numpy()[~keep] == 0)
    ctx.close()


def test_gae_unaligned_views_take_the_scalar_path():
    import oracle.unity_oracle as orc
    w = wl.make_structure("rag_qa")
    n = w.n_tok
    r, v = wl.normal(14, 1, n), wl.normal(14, 2, n)
    pad = lambda t: torch.cat([torch.zeros(1, dtype=t.dtype), t]).cuda()[1:]       # data pointer off by one element
    ctx = ub.Context(0, 1 << 20)
    adv = torch.full((n + 1,), 7.0, device="cuda")[1:]
    ret = torch.full((n + 1,), 7.0, device="cuda")[1:]
    ctx.gae(w.cu_seqlens.cuda(), pad(r), pad(v), pad(w.tok_mask), 0.98, 0.9, adv, ret)
    ctx.check_status()
    oa, orr = orc.gae(r.numpy(), v.numpy(), w.cu_seqlens.numpy(), 0.98, 0.9, w.tok_mask.numpy())
    scale = max(1.0, float(np.abs(oa).max()))
    assert np.abs(adv.cpu().numpy() - oa).max() <= 1e-5 * scale and np.abs(ret.cpu().numpy() - orr).max() <= 1e-5 * scale
    ctx.close()


def test_value_loss_unaligned_views_take_the_scalar_path():
    import oracle.unity_oracle as orc
    w = wl.make_structure("rag_qa")
    n = w.n_tok
    v, ov, ret = wl.normal(13, 1, n), wl.normal(13, 2, n), wl.normal(13, 3, n)
    pad = lambda t: torch.cat([torch.zeros(1, dtype=t.dtype), t]).cuda()[1:]       # data pointer off by one element
    ctx = ub.Context(0, 1 << 20)
    loss = torch.empty(w.K, device="cuda")
    dv = torch.full((n + 1,), 7.0, device="cuda")[1:]
    ctx.value_loss_fwd_bwd(w.cu_seqlens.cuda(), w.inv_role.cuda(), w.role_model.tolist(), w.K, pad(w.tok_mask), pad(v),
                           pad(ov), pad(ret), 0.5, None, loss, None, None, dv)
    ctx.check_status()
    o = orc.value_loss_fwd_bwd(v.numpy(), ov.numpy(), ret.numpy(), w.cu_seqlens.numpy(), w.inv_role.numpy(),
                               w.role_model.numpy(), w.tok_mask.numpy(), clip_v=0.5, K=w.K)
    assert np.all(np.abs(loss.cpu().numpy() - o["loss"]) <= pu.TOL_LOSS * np.abs(o["loss"]))
    assert np.abs(dv.cpu().numpy() - o["dvalues"]).max() <= 1e-5 * np.abs(o["dvalues"]).max() + 1e-9
    ctx.close()


# ------------------------------------------------------------------------------------ stages 2 + 3

def test_tiny_full():
    run_all_stages(wl.make("tiny", device="cuda"))


@pytest.mark.parametrize("name", ["rag_qa", "search", "code", "stress"])
def test_config_parity_cut(name):
    # same H, V, K, roles and groups as the full configuration; token batch cut to ~300 rows
    run_all_stages(wl.make(name, device="cuda", cut_rows=300, cut_max_len=64))


def small_workload(H, V, rows, role_model=None, K=None, max_len=48, seed_offset=0):
    w = wl.make_structure("search", cut_rows=rows, cut_max_len=max_len, H=H, V=V, seed_offset=seed_offset)
    if role_model is not None:
        w.role_model = torch.tensor(role_model, dtype=torch.int32)
        w.K = K or int(max(role_model)) + 1
    return wl.materialize(w, device="cuda")


@pytest.mark.parametrize("H,V,rows", [(64, 1000, 150), (128, 4096 + 8, 700), (320, 2048, 129), (256, 520, 40)])
def test_small_shapes_and_ragged_tails(H, V, rows):
    # V not a multiple of the 256-wide vocabulary tile, rows not a multiple of the 128-row tile
    run_all_stages(small_workload(H, V, rows))


@pytest.mark.parametrize("name", ["tiny", "search", "four_models"])
def test_calls_with_host_side_row_counts_match_the_oracle(name):
    # By default the host never learns the row counts: it walks every chunk a model could have and the kernels cut their
    # spans on the device (most launches of a model with few rows return at once) - that is what every other test runs.
    # UNITY_OPT_HOST_COUNTS = 1: the counts are read back once and launches that would be empty are skipped.
    if name == "four_models":      # four models, one of them without rows (the stress configuration's mapping, small sizes)
        w = small_workload(320, 2048 + 264, 1200, role_model=[0, 3, 1], K=4)
    else:
        w = wl.make(name, device="cuda", **({} if name == "tiny" else dict(cut_rows=1200, cut_max_len=64)))
    run_all_stages(w, options=[(ub.OPT_HOST_COUNTS, 1)])
    if name == "tiny":
        run_all_stages(w, options=[(ub.OPT_HOST_COUNTS, 1), (ub.OPT_LOGIT_STASH, 1)])


def test_calls_return_while_the_stream_is_busy():
    """Neither unity_logprob_fwd nor unity_ppo_loss_fwd_bwd waits for the device: behind a kernel that keeps the stream
    busy for about a quarter of a second, both calls return long before it ends.  With UNITY_OPT_HOST_COUNTS = 1 the
    forward call returns only after it (the one synchronisation that reads the row counts)."""
    import time
    w = small_workload(128, 2048, 600)
    d = pu.DeviceInputs(w)
    ctx = pu.make_ctx(w)
    n = w.n_tok
    logp = torch.empty(n, device="cuda")
    old = torch.full((n,), -7.0, device="cuda")
    adv = torch.ones(n, device="cuda")
    loss = torch.empty(w.K, device="cuda")
    dH = torch.empty(n, w.H, device="cuda", dtype=torch.bfloat16)
    dW = [torch.empty(w.V, w.H, device="cuda") for _ in range(w.K)]

    def calls():
        ctx.logprob_fwd(d.hidden, d.W, d.cu_seqlens, d.inv_role, w.role_model.tolist(), d.target, d.tok_mask, 1.0, logp)
        ctx.ppo_loss_fwd_bwd(d.hidden, d.W, d.cu_seqlens, d.inv_role, w.role_model.tolist(), d.target, d.tok_mask, 1.0, 0.2,
                             0.2, 0.01, 3, 0.0, None, False, old, old, adv, loss, None, None, None, None, dH, dW)

    calls()                                        # warm-up
    torch.cuda.synchronize()
    spin = 500_000_000                             # SM clocks: about 0.25 s at 1.9 GHz
    seen = {}
    for mode in (0, 1):
        ctx.set_option(ub.OPT_HOST_COUNTS, mode)
        torch.cuda._sleep(spin)
        t0 = time.perf_counter()
        calls()
        seen[mode] = time.perf_counter() - t0
        busy_after = not torch.cuda.current_stream().query()
        torch.cuda.synchronize()
        if mode == 0:
            assert busy_after
    ctx.check_status()
    assert seen[0] < 0.1 and seen[1] > 0.15, seen
    ctx.close()


@pytest.mark.parametrize("rows,valid,ctas", [(7700, 6289, 2), (7700, 6289, 1), (15400, 12326, 2)])
def test_forward_rounds_with_a_short_last_round(rows, valid, ctas):
    # 6289 valid rows = 25 row tiles of 256 (or 50 of 128): one full round of 24 (48) row tiles x 3 splits and a last
    # round of ONE row tile (two), which the planner cuts into 32 vocabulary splits; 12326 valid rows = 49 row tiles:
    # two full rounds and a last one of one tile
    w = small_workload(128, 8192 + 264, rows, max_len=200, role_model=[0, 0, 0], K=1)
    assert (w.tok_mask != 0).sum().item() == valid
    run_all_stages(w, ctas=(ctas,) * 4, options=[(8, 48)])      # rounds of 48 tiles of 128 rows whatever the hidden size


@pytest.mark.parametrize("ctas,gmax,block", [(2, 16, 1), (1, 16, 1), (2, 48, 2), (2, 148, 1)])
def test_recompute_gemm_on_the_forward_schedule(ctas, gmax, block):
    # the recompute GEMM in rounds of row tiles x vocabulary splits (a worker sweeps its split with one row tile, odd
    # rounds backwards): 25 row tiles of 256 give full rounds and a short last one that is cut into more splits
    w = small_workload(128, 8192 + 264, 7700, max_len=200, role_model=[0, 0, 0], K=1)
    run_all_stages(w, ctas=(ctas,) * 4, options=[(ub.OPT_GRAD_ROUNDS, gmax), (ub.OPT_GRAD_BLOCK, block)], ent_coef=0.01)
    if gmax == 48:       # and once at a full-size hidden width and vocabulary (two models, H = 1536, V = 151936)
        run_all_stages(wl.make("search", device="cuda", cut_rows=300, cut_max_len=64),
                       options=[(ub.OPT_GRAD_ROUNDS, gmax), (ub.OPT_GRAD_BLOCK, block)])


@pytest.mark.parametrize("ctas,in_flight", [(2, 0), (2, 12), (1, 12), (2, 148)])
def test_recompute_gemm_in_runs_of_column_tiles(ctas, in_flight):
    # outside rounds a unit of the recompute GEMM is one output tile (0) or a run of column tiles that the kernel sizes
    # from the rows it finds (25 row tiles of 256, 34 column tiles, the last one ragged)
    w = small_workload(128, 8192 + 264, 7700, max_len=200, role_model=[0, 0, 0], K=1)
    options = [(ub.OPT_GRAD_ROUNDS, 0), (ub.OPT_GRAD_RUNS, in_flight)]
    run_all_stages(w, ctas=(ctas,) * 4, options=options, ent_coef=0.01)


def test_dw_gemm_runs_its_last_vocabulary_tiles_as_a_narrow_launch():
    # 77 vocabulary tiles (the last one ragged) on 74 CTA pairs: the dW GEMM runs tiles 74..76 as a second launch with
    # 64-column tiles; same bits as the single launch (a tile's sum over the rows does not depend on its width), and
    # both match the oracle
    w = small_workload(320, 76 * 256 + 8, 300)
    run_all_stages(w)
    d = pu.DeviceInputs(w)
    ol = pu.oracle_logprob(w)
    cur = torch.from_numpy(ol["logp"].astype(np.float32))
    old, ref = (cur + w.noise_old).cuda(), (cur + w.noise_ref).cuda()
    adv = wl.normal(6, 96, w.n_tok).cuda()
    outs = []
    for tail in (0, 1):
        ctx = pu.make_ctx(w)
        ctx.set_option(29, tail)
        outs.append(pu.gpu_ppo(ctx, w, d, old, ref, adv))
        ctx.close()
    assert all(torch.equal(a, b) for a, b in zip(outs[0]["dW"], outs[1]["dW"]))
    assert torch.equal(outs[0]["dHidden"], outs[1]["dHidden"])


@pytest.mark.parametrize("ctas", [(1, 1, 1, 1), (2, 2, 2, 2), (2, 1, 1, 2)])
def test_single_cta_and_cta_pair_kernels(ctas):
    # every GEMM class exists as a one-CTA kernel (128-row tiles) and as a CTA-pair kernel (256-row tiles)
    run_all_stages(small_workload(320, 2048 + 264, 700), ctas=ctas)
    run_all_stages(wl.make("tiny", device="cuda"), ctas=ctas)


def test_scheduling_options_do_not_change_results():
    """Raster groups, rendezvous switches and periods, L2 hints, tensor-map promotion and the schedule of the recompute
    GEMM (tile by tile or in rounds, per block or per chunk) only move work in time or space: every output must be bitwise what the defaults give.  The forward round size changes the number of
    vocabulary splits and with it the order of a four-term merge: equal within rounding."""
    w = small_workload(320, 4096 + 264, 900)
    d = pu.DeviceInputs(w)
    ol = pu.oracle_logprob(w)
    cur = torch.from_numpy(ol["logp"].astype(np.float32))
    old, ref = (cur + w.noise_old).cuda(), (cur + w.noise_ref).cuda()
    adv = wl.normal(3, 97, w.n_tok).cuda()

    def run(options):
        ctx = pu.make_ctx(w)
        for option, value in options:
            ctx.set_option(option, value)
        out = pu.gpu_ppo(ctx, w, d, old, ref, adv, ent_coef=0.01)
        ctx.close()
        return out

    base = run([])
    same = [[(4, 0)], [(5, 8)], [(9, 0)], [(10, 0)], [(10, 5)], [(12, 4), (13, 6), (14, 2)], [(16, 0), (17, 0)],
            [(17, 41), (18, 9), (19, 38)], [(22, 3), (23, 2), (24, 5)], [(26, 4)], [(26, 48), (27, 2)], [(26, 2), (10, 0)], [(26, 0), (28, 0)], [(26, 0), (28, 8)],
            [(26, 0), (28, 40), (27, 1)]]
    for options in same:
        out = run(options)
        for key in ("loss", "logp", "entropy", "tok_loss", "dHidden", "metrics"):
            assert torch.equal(out[key], base[key]), (options, key)
        assert all(torch.equal(a, b) for a, b in zip(out["dW"], base["dW"])), options
    out = run([(8, 16)])
    assert (out["logp"] - base["logp"]).abs().max().item() <= 1e-5
    assert pu.rel_fro(out["dHidden"].float().cpu().numpy(), base["dHidden"].float().cpu().numpy()) <= 1e-3
    for a, b in zip(out["dW"], base["dW"]):
        assert pu.rel_fro(a.cpu().numpy(), b.cpu().numpy()) <= 1e-4


@pytest.mark.parametrize("wide", [0, 1])
def test_accumulate_gemms_with_256_and_512_column_tiles(wide):
    # the dHidden / dW chunk GEMMs of CTA pairs exist with 256 x 256 tiles (two accumulator stages) and with
    # 256 x 512 tiles (one stage, reductions into C); H = 320 and 832 leave ragged column tails in both
    for H, V, rows in [(320, 2048 + 264, 700), (832, 1536, 300)]:
        run_all_stages(small_workload(H, V, rows), ctas=(2, 2, 2, 2), options=[(11, wide)])


@pytest.mark.parametrize("name", ["tiny", "rag_qa", "code"])
def test_logit_stash_instead_of_recompute(name):
    # the loss call keeps the scaled logits of a row block in bf16 and turns them into dL/dz in place; same outputs
    # within the same tolerances (V = 151936 ends in a half tile; the cuts span all eight vocabulary chunks); the stress
    # configuration runs with the stash at full size in test_gpu_fullsize.py
    w = wl.make(name, device="cuda") if name == "tiny" else wl.make(name, device="cuda", cut_rows=300, cut_max_len=64)
    run_all_stages(w, options=[(ub.OPT_LOGIT_STASH, 1)])


def test_logit_stash_small_shapes_and_entropy_bonus():
    for H, V, rows in [(320, 2048 + 264, 700), (64, 1000, 150)]:
        run_all_stages(small_workload(H, V, rows), options=[(ub.OPT_LOGIT_STASH, 1)], ent_coef=0.02, kl_mode=2)


@pytest.mark.parametrize("kl_mode,ent_coef,clip", [(1, 0.0, (0.2, 0.2)), (2, 0.01, (0.1, 0.3)), (3, 0.02, (0.2, 0.28))])
def test_kl_modes_entropy_bonus_and_temperature(kl_mode, ent_coef, clip):
    w = small_workload(256, 3000, 400, seed_offset=kl_mode)
    w.inv_temperature = 0.7
    w.noise_old = w.noise_old * 6.0            # log-ratio noise 0.3: many tokens on the clipped branch
    run_all_stages(w, kl_mode=kl_mode, kl_coef=0.1, ent_coef=ent_coef, clip=clip)


def test_on_policy_shortcut_reuses_an_earlier_forward():
    # logp / entropy / lse from unity_logprob_fwd on the same weights replace the forward sweep of the loss call
    w = small_workload(256, 3000, 500)
    d = pu.DeviceInputs(w)
    ctx = pu.make_ctx(w)
    fwd = pu.gpu_logprob(ctx, w, d)
    old = fwd["logp"] + w.noise_old.cuda()
    ref = fwd["logp"] + w.noise_ref.cuda()
    adv = wl.normal(9, 3, w.n_tok).cuda()
    full = pu.gpu_ppo(ctx, w, d, old, ref, adv, ent_coef=0.01)
    launches = ctx.launch_count
    short = pu.gpu_ppo(ctx, w, d, old, ref, adv, ent_coef=0.01, fwd=fwd)
    assert ctx.launch_count - launches < launches                         # fewer kernels: no forward GEMM
    for key in ("loss", "logp", "entropy", "tok_loss", "dHidden"):
        assert torch.equal(short[key], full[key]), key                    # same statistics in, same bits out
    assert all(torch.equal(a, b) for a, b in zip(short["dW"], full["dW"]))
    op = pu.oracle_ppo(w, old.cpu().numpy(), ref.cpu().numpy(), adv.cpu().numpy(), ent_coef=0.01)
    check_ppo(short, op, w)
    with pytest.raises(ub.UnityError) as e:                               # all three or none
        ctx.ppo_loss_fwd_bwd(d.hidden, d.W, d.cu_seqlens, d.inv_role, w.role_model.tolist(), d.target, d.tok_mask, 1.0,
                             0.2, 0.2, 0.0, 3, 0.0, None, False, old, ref, adv, full["loss"], None, None, None, None,
                             full["dHidden"], full["dW"], logp_in=fwd["logp"])
    assert e.value.code == -1
    ctx.close()


def test_model_without_rows_and_three_models():
    # roles map to models 0 and 1; model 2 is never used: its dW must come back as zeros
    run_all_stages(small_workload(128, 1024, 300, role_model=[0, 1, 0], K=3))


def test_sixteen_models_and_sixty_four_roles():
    # the limits of the interface: UNITY_MAX_MODELS models, UNITY_MAX_ROLES roles (most groups x role segments are tiny)
    w = wl.make_structure("search", cut_rows=1500, cut_max_len=32, H=128, V=1024 + 72)
    R, K = ub.UNITY_MAX_ROLES, ub.UNITY_MAX_MODELS
    s = torch.arange(w.n_inv)
    w.inv_role = ((w.inv_role.long() + 3 * (s % 22)) % R).to(torch.int32)
    w.n_roles, w.K = R, K
    w.role_model = (torch.arange(R) % K).to(torch.int32)
    w.lam = torch.ones(R, 3)
    run_all_stages(wl.materialize(w, device="cuda"))


def test_all_rows_masked_and_single_row():
    w = small_workload(128, 1024, 200)
    w.tok_mask.zero_()
    d = pu.DeviceInputs(w)
    ctx = pu.make_ctx(w)
    z = torch.zeros(w.n_tok, device="cuda")
    g = pu.gpu_ppo(ctx, w, d, z, z, z)
    assert torch.all(g["loss"] == 0) and torch.all(g["dHidden"] == 0) and all(torch.all(x == 0) for x in g["dW"])
    assert torch.all(g["logp"] == 0) and torch.all(g["tok_loss"] == 0)
    gl = pu.gpu_logprob(ctx, w, d)
    assert torch.all(gl["logp"] == 0)
    ctx.close()
    w.tok_mask[17] = 1
    run_all_stages(w)


def test_gradient_accumulation_is_additive_and_runs_are_bitwise_reproducible():
    w = small_workload(256, 2048, 600)
    d = pu.DeviceInputs(w)
    ctx = pu.make_ctx(w)
    ol = pu.oracle_logprob(w)
    cur = torch.from_numpy(ol["logp"].astype(np.float32))
    old, ref = (cur + w.noise_old).cuda(), (cur + w.noise_ref).cuda()
    adv = wl.normal(3, 99, w.n_tok).cuda()
    full = pu.gpu_ppo(ctx, w, d, old, ref, adv)
    again = pu.gpu_ppo(ctx, w, d, old, ref, adv)
    assert torch.equal(full["dHidden"], again["dHidden"]) and torch.equal(full["loss"], again["loss"])
    assert all(torch.equal(a, b) for a, b in zip(full["dW"], again["dW"]))
    # two micro-batches (mask halves) with the full-batch norm, accumulated into one dW
    norm = [max(float(full["metrics"][k, 0].item()), 1.0) for k in range(w.K)]
    half = w.n_tok // 2
    mask_a, mask_b = w.tok_mask.clone(), w.tok_mask.clone()
    mask_a[half:] = 0
    mask_b[:half] = 0
    dW = [torch.zeros(w.V, w.H, device="cuda") for _ in range(w.K)]
    d.tok_mask = mask_a.cuda()
    ga = pu.gpu_ppo(ctx, w, d, old, ref, adv, norm=norm, accumulate=True, dW=dW)
    d.tok_mask = mask_b.cuda()
    gb = pu.gpu_ppo(ctx, w, d, old, ref, adv, norm=norm, accumulate=True, dW=dW)
    assert torch.allclose(ga["loss"] + gb["loss"], full["loss"], rtol=1e-4, atol=1e-7)
    for k in range(w.K):
        assert pu.rel_fro(dW[k].cpu().numpy(), full["dW"][k].cpu().numpy()) <= 1e-3
    dH_sum = (ga["dHidden"].float() + gb["dHidden"].float()).cpu().numpy()
    assert pu.rel_fro(dH_sum, full["dHidden"].float().cpu().numpy()) <= 1e-3
    # column sums of dW over the vocabulary vanish (sum_v dL/dz_v = 0 for every row)
    for k in range(w.K):
        col = full["dW"][k].double().sum(0).abs().max().item()
        assert col <= 1e-2 * full["dW"][k].double().abs().sum(0).max().item() + 1e-9
    ctx.close()


def test_small_workspace_uses_smaller_chunks_and_too_small_is_an_error():
    w = small_workload(256, 4096, 1500, max_len=200)
    d = pu.DeviceInputs(w)
    need = ub.unity_workspace_bytes(w.n_tok, w.H, w.V, w.K, w.n_inv)
    least = ub.unity_workspace_min_bytes(w.n_tok, w.H, w.V, w.K, w.n_inv)
    assert least < need
    ol = pu.oracle_logprob(w)
    cur = torch.from_numpy(ol["logp"].astype(np.float32))
    old, ref = cur + w.noise_old, cur + w.noise_ref
    adv = wl.normal(4, 98, w.n_tok)
    ctx = ub.Context(0, least)                 # several row chunks and vocabulary chunks
    gp = pu.gpu_ppo(ctx, w, d, old.cuda(), ref.cuda(), adv.cuda())
    op = pu.oracle_ppo(w, old.numpy(), ref.numpy(), adv.numpy())
    check_ppo(gp, op, w)
    ctx.close()
    ctx = ub.Context(0, 1 << 16)
    with pytest.raises(ub.UnityError) as e:
        pu.gpu_logprob(ctx, w, d)
    assert e.value.code == -4
    ctx.close()


@pytest.mark.parametrize("case", range(10))
def test_seeded_random_shapes_schedules_and_workspaces(case):
    """Shapes, model mappings, scheduling options and workspace sizes drawn from a seeded generator: every combination
    must match the oracle within the stated tolerances (the planners that cut launches into rounds, runs, chunks and
    tail launches see extents here that no hand-picked case covers)."""
    rng = np.random.default_rng(20260528 + case)
    H = int(rng.choice([64, 128, 192, 320, 448, 512]))
    V = 8 * int(rng.integers(16, 450))
    rows = int(rng.integers(40, 1400))
    K = int(rng.integers(1, 4))
    role_model = [int(x) for x in rng.integers(0, K, 3)]
    role_model[int(rng.integers(0, 3))] = K - 1                    # the last model is used; others may stay empty
    w = small_workload(H, V, rows, role_model=role_model, K=K, max_len=int(rng.choice([16, 48, 200])), seed_offset=case)
    options = [(ub.OPT_GRAD_ROUNDS, int(rng.choice([-1, 0, 4, 16, 148]))), (ub.OPT_GRAD_RUNS, int(rng.choice([-1, 0, 8, 40]))),
               (ub.OPT_GRAD_BLOCK, int(rng.choice([0, 1, 2]))), (8, int(rng.choice([-1, 0, 16, 48]))),
               (11, int(rng.integers(0, 2))), (29, int(rng.integers(0, 2))), (ub.OPT_HOST_COUNTS, int(rng.integers(0, 2)))]
    ctas = [int(x) for x in rng.integers(1, 3, 4)]
    ent_coef = float(rng.choice([0.0, 0.01]))
    need = ub.unity_workspace_bytes(w.n_tok, w.H, w.V, w.K, w.n_inv)
    least = ub.unity_workspace_min_bytes(w.n_tok, w.H, w.V, w.K, w.n_inv)
    size = [need, least, (need + least) // 2][int(rng.integers(0, 3))]
    d = pu.DeviceInputs(w)
    ctx = ub.Context(0, size)
    try:
        for option, value in list(enumerate(ctas)) + options:
            ctx.set_option(option, value)
        gl, ol = pu.gpu_logprob(ctx, w, d), pu.oracle_logprob(w)
        check_forward(gl, ol, w.tok_mask.numpy() != 0)
        cur = torch.from_numpy(ol["logp"].astype(np.float32))
        old, ref = cur + w.noise_old, cur + w.noise_ref
        adv = wl.normal(5, 99 + case, w.n_tok)
        gp = pu.gpu_ppo(ctx, w, d, old.cuda(), ref.cuda(), adv.cuda(), ent_coef=ent_coef)
        op = pu.oracle_ppo(w, old.numpy(), ref.numpy(), adv.numpy(), ent_coef=ent_coef)
        check_ppo(gp, op, w)
    finally:
        ctx.close()


def test_argument_errors_return_codes():
    w = small_workload(128, 1024, 100)
    d = pu.DeviceInputs(w)
    ctx = pu.make_ctx(w)
    logp = torch.empty(w.n_tok, device="cuda")
    args = [d.hidden, d.W, d.cu_seqlens, d.inv_role, w.role_model.tolist(), d.target, d.tok_mask, 1.0, logp]
    bad_h = torch.empty(w.n_tok, 96, device="cuda", dtype=torch.bfloat16)        # H not a multiple of 64
    with pytest.raises(ub.UnityError) as e:
        ctx.logprob_fwd(bad_h, [torch.empty(w.V, 96, device="cuda", dtype=torch.bfloat16)] * w.K, *args[2:])
    assert e.value.code == -2
    with pytest.raises(ub.UnityError) as e:                                       # model id outside [0, K)
        ctx.logprob_fwd(d.hidden, d.W, d.cu_seqlens, d.inv_role, [0, 0, 5], d.target, d.tok_mask, 1.0, logp)
    assert e.value.code == -1
    with pytest.raises(ub.UnityError) as e:                                       # non-positive temperature
        ctx.logprob_fwd(d.hidden, d.W, d.cu_seqlens, d.inv_role, w.role_model.tolist(), d.target, d.tok_mask, 0.0, logp)
    assert e.value.code == -1
    odd = torch.empty(w.n_tok * w.H + 8, device="cuda", dtype=torch.bfloat16)[1:1 + w.n_tok * w.H].view(w.n_tok, w.H)
    with pytest.raises(ub.UnityError) as e:                                       # hidden not 16-byte aligned
        ctx.logprob_fwd(odd, *args[1:])
    assert e.value.code == -3
    # a target outside the vocabulary: flagged, row treated as masked, nothing else disturbed
    tgt = w.target.clone()
    row = int(torch.nonzero(w.tok_mask)[5])
    tgt[row] = w.V + 3
    ctx.logprob_fwd(d.hidden, d.W, d.cu_seqlens, d.inv_role, w.role_model.tolist(), tgt.cuda(), d.tok_mask, 1.0, logp)
    with pytest.raises(ub.UnityError) as e:
        ctx.check_status()
    assert e.value.code == -7
    o = pu.oracle_logprob(w)
    got = logp.cpu().numpy()
    assert got[row] == 0
    keep = np.arange(w.n_tok) != row
    assert np.abs(got[keep] - o["logp"][keep]).max() <= pu.TOL_LOGP
    ctx.close()
