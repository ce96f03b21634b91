"""Pins for the fp64 oracle: closed forms, invariants, library special cases, finite differences,
an autograd third opinion and brute force.  No GPU, no CUDA library."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import unity_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def tiny_problem(seed=0, n_inv=6, H=8, V=16, K=2, R=3, max_len=5, mask_p=0.8):
    rng = np.random.default_rng(seed)
    role_model = np.array([v % K for v in range(R)])
    inv_role = rng.integers(0, R, n_inv)
    inv_role[:R] = np.arange(R)[:n_inv] if n_inv >= R else inv_role[:R]
    lens = rng.integers(1, max_len + 1, n_inv)
    cu = np.concatenate([[0], np.cumsum(lens)])
    N = int(cu[-1])
    hidden = rng.normal(size=(N, H))
    W = [rng.normal(size=(V, H)) * 0.3 for _ in range(K)]
    target = rng.integers(0, V, N)
    mask = (rng.random(N) < mask_p).astype(np.uint8)
    mask[0] = 1
    return dict(hidden=hidden, W=W, cu_seqlens=cu, inv_role=inv_role, role_model=role_model,
                target=target, tok_mask=mask)


def fwd(p, **kw):
    return orc.logprob_fwd(p["hidden"], p["W"], p["cu_seqlens"], p["inv_role"], p["role_model"],
                           p["target"], p["tok_mask"], **kw)


def ppo(p, old, ref, adv, **kw):
    return orc.ppo_loss_fwd_bwd(p["hidden"], p["W"], p["cu_seqlens"], p["inv_role"], p["role_model"],
                                p["target"], p["tok_mask"], old, ref, adv, **kw)


# ---------------------------------------------------------------------------- stage 2 pins

def test_probabilities_sum_to_one_over_vocab():
    p = tiny_problem(seed=1, V=16)
    N = p["hidden"].shape[0]
    p["tok_mask"] = np.ones(N, np.uint8)
    total = np.zeros(N)
    for y in range(16):
        p["target"] = np.full(N, y)
        total += np.exp(fwd(p)["logp"])
    assert np.abs(total - 1.0).max() < 1e-12


def test_zero_weights_give_uniform_distribution():
    p = tiny_problem(seed=2, V=16)
    p["W"] = [np.zeros_like(w) for w in p["W"]]
    out = fwd(p)
    valid = p["tok_mask"] != 0
    assert np.allclose(out["logp"][valid], -math.log(16), atol=1e-14)
    assert np.allclose(out["entropy"][valid], math.log(16), atol=1e-14)
    assert np.allclose(out["lse"][valid], math.log(16), atol=1e-14)
    assert np.all(out["logp"][~valid] == 0) and np.all(out["entropy"][~valid] == 0)


def test_two_way_vocab_is_logistic():
    p = tiny_problem(seed=3, V=2, K=1, R=1)
    out = fwd(p)
    z = p["hidden"] @ p["W"][0].T
    y = p["target"]
    n = np.arange(len(y))
    diff = z[n, 1 - y] - z[n, y]
    softplus = np.log1p(np.exp(-np.abs(diff))) + np.maximum(diff, 0)
    q = 1.0 / (1.0 + np.exp(-(z[:, 1] - z[:, 0])))
    bin_ent = -(q * np.log(q) + (1 - q) * np.log(1 - q))
    valid = p["tok_mask"] != 0
    assert np.allclose(out["logp"][valid], -softplus[valid], atol=1e-13)
    assert np.allclose(out["entropy"][valid], bin_ent[valid], atol=1e-13)


def test_matches_torch_cross_entropy_and_categorical_entropy():
    p = tiny_problem(seed=4, n_inv=10, H=12, V=40, K=2, R=3)
    out = fwd(p, inv_temperature=0.7)
    tok_role, tok_model = orc.token_role_model(p["cu_seqlens"], p["inv_role"], p["role_model"])
    h = torch.tensor(p["hidden"])
    for k in range(2):
        idx = np.nonzero((p["tok_mask"] != 0) & (tok_model == k))[0]
        z = 0.7 * h[idx] @ torch.tensor(p["W"][k]).T
        ce = torch.nn.functional.cross_entropy(z, torch.tensor(p["target"][idx]), reduction="none")
        ent = torch.distributions.Categorical(logits=z).entropy()
        assert np.allclose(out["logp"][idx], -ce.numpy(), atol=1e-12)
        assert np.allclose(out["entropy"][idx], ent.numpy(), atol=1e-12)
        assert np.allclose(out["lse"][idx], torch.logsumexp(z, 1).numpy(), atol=1e-12)


def test_routing_uses_role_model_table_not_role_id():
    # two roles sharing one model must give the same numbers as a single role
    p = tiny_problem(seed=5, K=1, R=2)
    a = fwd(p)
    q = dict(p)
    q["inv_role"] = np.zeros_like(p["inv_role"])
    q["role_model"] = np.array([0])
    b = fwd(q)
    assert np.array_equal(a["logp"], b["logp"])
    # swapping the mapping swaps which matrix a token sees
    p2 = tiny_problem(seed=5, K=2, R=2)
    s = dict(p2)
    s["role_model"] = p2["role_model"][::-1].copy()
    s["W"] = p2["W"][::-1]
    assert np.allclose(fwd(p2)["logp"], fwd(s)["logp"], atol=1e-15)


# ---------------------------------------------------------------------------- stage 3 pins

def test_loss_is_minus_mean_advantage_at_ratio_one_without_kl():
    p = tiny_problem(seed=6, n_inv=12)
    cur = fwd(p)["logp"]
    N = cur.size
    adv = np.random.default_rng(0).normal(size=N)
    out = ppo(p, cur, cur, adv, kl_coef=0.0, ent_coef=0.0)
    _, tok_model = orc.token_role_model(p["cu_seqlens"], p["inv_role"], p["role_model"])
    for k in range(2):
        sel = (p["tok_mask"] != 0) & (tok_model == k)
        assert abs(out["loss"][k] - (-adv[sel].mean())) < 1e-13
    # with ref == logp the k3/k2/k1 penalties vanish too
    for mode in (1, 2, 3):
        o2 = ppo(p, cur, cur, adv, kl_coef=0.7, kl_mode=mode)
        assert np.allclose(o2["loss"], out["loss"], atol=1e-13)


def test_kl_estimators_hand_values():
    d = np.array([0.0, 0.5, -0.25])
    k1, g1 = orc.kl_term(d, 1)
    k2, g2 = orc.kl_term(d, 2)
    k3, g3 = orc.kl_term(d, 3)
    assert np.allclose(k1, [0.0, -0.5, 0.25]) and np.allclose(g1, 1.0)
    assert np.allclose(k2, [0.0, 0.125, 0.03125]) and np.allclose(g2, [0.0, -0.5, 0.25])
    assert np.allclose(k3, [0.0, math.e ** 0.5 - 1.5, math.e ** -0.25 - 0.75])
    assert np.allclose(g3, [0.0, 1 - math.e ** 0.5, 1 - math.e ** -0.25])
    dd = np.linspace(-2, 2, 401)
    assert np.all(orc.kl_term(dd, 3)[0] >= 0) and orc.kl_term(np.zeros(1), 3)[0][0] == 0


def test_clipped_tokens_have_zero_gradient():
    p = tiny_problem(seed=7, n_inv=10, K=1, R=2)
    cur = fwd(p)["logp"]
    N = cur.size
    adv = np.where(np.arange(N) % 2 == 0, 1.0, -1.0)
    # even rows: A>0 and ratio = e^0.5 > 1.2 ; odd rows: A<0 and ratio = e^-0.5 < 0.8 -> all clipped
    old = cur - np.where(adv > 0, 0.5, -0.5)
    out = ppo(p, old, cur, adv, kl_coef=0.0, ent_coef=0.0)
    assert np.all(out["a"] == 0)
    assert np.all(out["dHidden"] == 0) and np.all(out["dW"][0] == 0)
    valid = p["tok_mask"] != 0
    expect = np.where(adv > 0, -1.2, 0.8)            # -clip(rho) * A
    assert np.allclose(out["tok_loss"][valid], expect[valid], atol=1e-14)
    assert out["metrics_model"][0, 4] == 1.0           # clip fraction
    # opposite signs: the unclipped branch is the maximum -> gradient -A*rho
    out2 = ppo(p, old, cur, -adv, kl_coef=0.0, ent_coef=0.0)
    M = valid.sum()
    rho = np.exp(cur - old)
    assert np.allclose(out2["a"][valid], (adv * rho)[valid] / M, atol=1e-15)
    assert out2["metrics_model"][0, 4] == 0.0


def test_logit_gradient_sums_to_zero():
    p = tiny_problem(seed=8, n_inv=12, V=24)
    cur = fwd(p)["logp"]
    rng = np.random.default_rng(1)
    N = cur.size
    out = ppo(p, cur + 0.1 * rng.normal(size=N), cur + 0.1 * rng.normal(size=N), rng.normal(size=N),
              kl_coef=0.3, ent_coef=0.05)
    for k in range(2):
        assert np.abs(out["dW"][k].sum(axis=0)).max() < 1e-13     # column sums over the vocabulary
    # all rows of W equal -> every row of dHidden vanishes
    q = dict(p)
    q["W"] = [np.tile(w[:1], (w.shape[0], 1)) for w in p["W"]]
    cur_q = fwd(q)["logp"]
    out_q = ppo(q, cur_q + 0.1, cur_q - 0.1, rng.normal(size=N), kl_coef=0.3, ent_coef=0.05)
    assert np.abs(out_q["dHidden"]).max() < 1e-13


@pytest.mark.parametrize("kl_mode", [1, 2, 3])
def test_backward_matches_central_finite_differences(kl_mode):
    p = tiny_problem(seed=9, n_inv=5, H=6, V=10, K=2, R=2, max_len=3)
    cur = fwd(p)["logp"]
    rng = np.random.default_rng(2)
    N = cur.size
    old = cur + 0.05 * rng.normal(size=N)       # ratios well inside the clip interval
    ref = cur + 0.2 * rng.normal(size=N)
    adv = rng.normal(size=N)
    kw = dict(kl_coef=0.2, kl_mode=kl_mode, ent_coef=0.03, inv_temperature=0.8)
    out = ppo(p, old, ref, adv, **kw)
    step = 1e-6

    def loss_sum(q):
        return orc.ppo_loss_value(q["hidden"], q["W"], q["cu_seqlens"], q["inv_role"], q["role_model"],
                                  q["target"], q["tok_mask"], old, ref, adv, **kw).sum()

    for _ in range(12):
        i, j = rng.integers(0, N), rng.integers(0, 6)
        qp, qm = dict(p), dict(p)
        qp["hidden"] = p["hidden"].copy(); qp["hidden"][i, j] += step
        qm["hidden"] = p["hidden"].copy(); qm["hidden"][i, j] -= step
        fd = (loss_sum(qp) - loss_sum(qm)) / (2 * step)
        assert abs(fd - out["dHidden"][i, j]) <= 1e-6 * max(1.0, abs(fd)) + 1e-9
    for _ in range(12):
        k, v, j = rng.integers(0, 2), rng.integers(0, 10), rng.integers(0, 6)
        qp, qm = dict(p), dict(p)
        qp["W"] = [w.copy() for w in p["W"]]; qp["W"][k][v, j] += step
        qm["W"] = [w.copy() for w in p["W"]]; qm["W"][k][v, j] -= step
        fd = (loss_sum(qp) - loss_sum(qm)) / (2 * step)
        assert abs(fd - out["dW"][k][v, j]) <= 1e-6 * max(1.0, abs(fd)) + 1e-9


@pytest.mark.parametrize("kl_mode,noise", [(3, 0.05), (2, 0.4), (1, 0.4)])
def test_matches_torch_autograd_of_plain_composite_loss(kl_mode, noise):
    p = tiny_problem(seed=10, n_inv=14, H=10, V=30, K=2, R=3)
    cur = fwd(p)["logp"]
    rng = np.random.default_rng(3)
    N = cur.size
    old = cur + noise * rng.normal(size=N)      # noise 0.4 puts many tokens on the clipped branch
    ref = cur + 0.2 * rng.normal(size=N)
    adv = rng.normal(size=N)
    lo, hi, beta, cent, tau = 0.2, 0.3, 0.15, 0.02, 1.3
    out = ppo(p, old, ref, adv, clip_lo=lo, clip_hi=hi, kl_coef=beta, kl_mode=kl_mode, ent_coef=cent,
              inv_temperature=tau)
    _, tok_model = orc.token_role_model(p["cu_seqlens"], p["inv_role"], p["role_model"])
    h = torch.tensor(p["hidden"], requires_grad=True)
    Ws = [torch.tensor(w, requires_grad=True) for w in p["W"]]
    total = 0
    for k in range(2):
        idx = torch.tensor(np.nonzero((p["tok_mask"] != 0) & (tok_model == k))[0])
        z = tau * h[idx] @ Ws[k].T
        logq = torch.log_softmax(z, 1)
        lp = logq.gather(1, torch.tensor(p["target"])[idx][:, None])[:, 0]
        ent = -(logq.exp() * logq).sum(1)
        ratio = torch.exp(lp - torch.tensor(old)[idx])
        A = torch.tensor(adv)[idx]
        pg = torch.maximum(-ratio * A, -torch.clamp(ratio, 1 - lo, 1 + hi) * A)
        d = torch.tensor(ref)[idx] - lp
        kl = {1: -d, 2: 0.5 * d * d, 3: torch.exp(d) - d - 1}[kl_mode]
        Lk = (pg + beta * kl - cent * ent).mean()
        assert abs(Lk.item() - out["loss"][k]) < 1e-12
        total = total + Lk
    total.backward()
    assert np.abs(h.grad.numpy() - out["dHidden"]).max() < 1e-12
    for k in range(2):
        assert np.abs(Ws[k].grad.numpy() - out["dW"][k]).max() < 1e-12
    if noise > 0.2:
        assert 0.05 < out["metrics_model"][:, 4].mean() < 0.95      # both branches exercised


def test_permutation_and_model_copies():
    p = tiny_problem(seed=11, n_inv=9, K=2, R=2)
    cur = fwd(p)["logp"]
    rng = np.random.default_rng(4)
    N = cur.size
    old, ref, adv = cur + 0.1 * rng.normal(size=N), cur + 0.1 * rng.normal(size=N), rng.normal(size=N)
    base = ppo(p, old, ref, adv, kl_coef=0.1)
    # permute invocations (whole token spans move with them)
    perm = rng.permutation(9)
    cu = p["cu_seqlens"]
    tok_perm = np.concatenate([np.arange(cu[s], cu[s + 1]) for s in perm])
    q = dict(p)
    q["inv_role"] = p["inv_role"][perm]
    q["cu_seqlens"] = np.concatenate([[0], np.cumsum(np.diff(cu)[perm])])
    for key in ("hidden", "target", "tok_mask"):
        q[key] = p[key][tok_perm]
    outp = ppo(q, old[tok_perm], ref[tok_perm], adv[tok_perm], kl_coef=0.1)
    assert np.allclose(outp["logp"], base["logp"][tok_perm], atol=1e-14)
    assert np.allclose(outp["dHidden"], base["dHidden"][tok_perm], atol=1e-14)
    assert np.allclose(outp["loss"], base["loss"], atol=1e-14)
    for k in range(2):
        assert np.allclose(outp["dW"][k], base["dW"][k], atol=1e-14)
    # K copies of one matrix with norm = total count reproduce the single-model result
    one = dict(p)
    one["W"] = [p["W"][0]]
    one["role_model"] = np.zeros_like(p["role_model"])
    single = ppo(one, old, ref, adv, kl_coef=0.1)
    two = dict(p)
    two["W"] = [p["W"][0], p["W"][0].copy()]
    M = float((p["tok_mask"] != 0).sum())
    both = ppo(two, old, ref, adv, kl_coef=0.1, norm=[M, M])
    assert np.allclose(both["dW"][0] + both["dW"][1], single["dW"][0], atol=1e-14)
    assert np.allclose(both["dHidden"], single["dHidden"], atol=1e-14)
    assert abs(both["loss"].sum() - single["loss"][0]) < 1e-14


def test_additivity_over_row_chunks_with_fixed_norm():
    p = tiny_problem(seed=12, n_inv=10, K=2, R=2)
    cur = fwd(p)["logp"]
    rng = np.random.default_rng(5)
    N = cur.size
    old, ref, adv = cur + 0.1 * rng.normal(size=N), cur + 0.1 * rng.normal(size=N), rng.normal(size=N)
    full = ppo(p, old, ref, adv, kl_coef=0.1, ent_coef=0.01)
    rows_a = np.arange(0, N // 2)
    rows_b = np.arange(N // 2, N)
    pa = ppo(p, old, ref, adv, kl_coef=0.1, ent_coef=0.01, rows=rows_a)
    pb = ppo(p, old, ref, adv, kl_coef=0.1, ent_coef=0.01, rows=rows_b)
    assert np.allclose(pa["loss"] + pb["loss"], full["loss"], atol=1e-14)
    for k in range(2):
        assert np.allclose(pa["dW"][k] + pb["dW"][k], full["dW"][k], atol=1e-14)
    assert np.allclose(pa["dHidden"], full["dHidden"][pa["dh_index"]], atol=1e-15)
    assert np.array_equal(pa["M"], full["M"])


def test_brute_force_single_row_loops():
    """One row, every sum written as a python loop."""
    p = tiny_problem(seed=13, n_inv=1, H=4, V=5, K=1, R=1, max_len=1)
    p["tok_mask"] = np.ones(1, np.uint8)
    h, W, y = p["hidden"][0], p["W"][0], int(p["target"][0])
    z = [sum(W[v][j] * h[j] for j in range(4)) for v in range(5)]
    mx = max(z)
    s = sum(math.exp(zv - mx) for zv in z)
    lse = mx + math.log(s)
    prob = [math.exp(zv - lse) for zv in z]
    logp = z[y] - lse
    ent = -sum(pv * (zv - lse) for pv, zv in zip(prob, z))
    old, ref, A, beta, cent = logp - 0.05, logp + 0.1, 0.7, 0.2, 0.03
    rho = math.exp(logp - old)
    dd = ref - logp
    loss = -rho * A + beta * (math.exp(dd) - dd - 1) - cent * ent
    a = -A * rho + beta * (1 - math.exp(dd))
    G = [a * ((1.0 if v == y else 0.0) - prob[v]) + cent * prob[v] * (z[v] - lse + ent) for v in range(5)]
    dh = [sum(G[v] * W[v][j] for v in range(5)) for j in range(4)]
    out = ppo(p, np.array([old]), np.array([ref]), np.array([A]), kl_coef=beta, ent_coef=cent)
    assert abs(out["logp"][0] - logp) < 1e-14 and abs(out["entropy"][0] - ent) < 1e-14
    assert abs(out["loss"][0] - loss) < 1e-14
    assert np.allclose(out["dHidden"][0], dh, atol=1e-14)
    assert np.allclose(out["dW"][0], np.outer(G, h), atol=1e-14)


def test_bf16_bit_patterns_are_widened_exactly():
    x = torch.randn(64, dtype=torch.float32).to(torch.bfloat16)
    bits = x.view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.to_f64(bits), x.to(torch.float64).numpy())


# ---------------------------------------------------------------------------- stage 1 pins

def seg_problem(seed=0, G=5, R=3, per=6):
    rng = np.random.default_rng(seed)
    S = G * R * per
    inv_group = rng.permutation(np.repeat(np.arange(G), R * per))
    inv_role = rng.integers(0, R, S)
    n_traj = S // 2
    inv_traj = rng.integers(0, n_traj, S)
    lens = rng.integers(0, 4, S)
    cu = np.concatenate([[0], np.cumsum(lens)])
    return dict(inv_role=inv_role, inv_group=inv_group, inv_traj=inv_traj,
                r_node=rng.normal(size=S), r_turn=rng.normal(size=S), r_traj=rng.normal(size=n_traj),
                lam=rng.uniform(0.5, 1.5, size=(R, 3)), n_roles=R, n_groups=G, cu_seqlens=cu,
                tok_mask=(rng.random(int(cu[-1])) < 0.7).astype(np.uint8))


def test_advantage_segment_invariants():
    p = seg_problem(seed=1)
    out = orc.role_advantage(**p, eps=1e-6, ddof=0)
    seg = p["inv_group"] * p["n_roles"] + p["inv_role"]
    for q in range(p["n_groups"] * p["n_roles"]):
        m = seg == q
        if m.sum() < 2:
            continue
        A = out["adv_inv"][m]
        sigma = out["seg_std"][q]
        assert abs(A.mean()) < 1e-12
        assert abs(A.std() - sigma / (sigma + 1e-6)) < 1e-12
    # shift invariance
    p2 = dict(p)
    p2["r_node"] = p["r_node"] + 3.25 / p["lam"][p["inv_role"], 0]
    assert np.allclose(orc.role_advantage(**p2)["adv_inv"], out["adv_inv"], atol=1e-10)
    # scale invariance up to eps
    p3 = dict(p)
    for key in ("r_node", "r_turn", "r_traj"):
        p3[key] = p[key] * 7.0
    assert np.allclose(orc.role_advantage(**p3)["adv_inv"], out["adv_inv"], atol=1e-5)
    # token broadcast
    tok_inv = orc.token_invocation(p["cu_seqlens"])
    assert np.array_equal(out["adv_tok"], out["adv_inv"][tok_inv] * (p["tok_mask"] != 0))


def test_advantage_combination_and_degenerate_segments():
    # role 0 in group 0: constant rewards -> 0 ; role 1 in group 0: single member -> 0
    inv_role = np.array([0, 0, 0, 1, 0, 0])
    inv_group = np.array([0, 0, 0, 0, 1, 1])
    inv_traj = np.array([0, 1, 2, 0, 3, 4])
    r_node = np.array([1.0, 1.0, 1.0, 5.0, 1.0, 3.0])
    r_turn = np.array([0.5, 0.5, 0.5, 0.0, 0.0, 0.0])
    r_traj = np.array([2.0, 2.0, 2.0, 0.0, 4.0])
    lam = np.array([[1.0, 2.0, 0.5], [1.0, 1.0, 1.0]])
    cu = np.array([0, 2, 2, 3, 4, 6, 7])
    out = orc.role_advantage(inv_role, inv_group, inv_traj, r_node, r_turn, r_traj, lam, 2, 2, cu, eps=0.0)
    assert np.allclose(out["r"], [3.0, 3.0, 3.0, 7.0, 1.0, 5.0])      # 1 + 2*0.5 + 0.5*2 ; 5+0+2 ; 1+0+0 ; 3+0+2
    assert np.all(out["adv_inv"][:4] == 0)
    assert np.allclose(out["adv_inv"][4:], [-1.0, 1.0])
    assert np.array_equal(out["seg_n"], [3, 1, 2, 0])
    assert np.allclose(out["adv_tok"], [0, 0, 0, 0, -1, -1, 1])
    # sample standard deviation
    out1 = orc.role_advantage(inv_role, inv_group, inv_traj, r_node, r_turn, r_traj, lam, 2, 2, cu, eps=0.0, ddof=1)
    assert np.allclose(out1["adv_inv"][4:], [-1 / math.sqrt(2), 1 / math.sqrt(2)])
    assert np.all(out1["adv_inv"][:4] == 0)      # n - ddof = 0 for the single-member segment


def test_role_wise_statistics_under_full_sharing_and_single_group():
    # one rollout group: role-wise batch whitening; roles stay separate although the model is shared
    rng = np.random.default_rng(7)
    S = 40
    inv_role = rng.integers(0, 2, S)
    r = rng.normal(size=S) + 10.0 * inv_role
    out = orc.role_advantage(inv_role, np.zeros(S, int), np.arange(S), r, None, None, None, 2, 1,
                             np.arange(S + 1), eps=0.0)
    for v in range(2):
        A = out["adv_inv"][inv_role == v]
        assert abs(A.mean()) < 1e-12 and abs(A.std() - 1) < 1e-12


def test_workflow_d_hand_fixture():
    rows, adv = [], None
    for line in open(os.path.join(GOLDEN, "workflow_d_rewards.txt")):
        if line.startswith("#") or not line.strip():
            continue
        if line.startswith("adv"):
            adv = np.array([float(x) for x in line.split()[1:]])
        else:
            rows.append([float(x) for x in line.split()])
    rows = np.array(rows)
    scores, rewards = rows[:, 1:4], rows[:, 4:7]
    # the rule itself: first round credits s_0, later rounds credit the improvement
    assert np.allclose(rewards, np.diff(np.concatenate([np.zeros((2, 1)), scores], 1), axis=1))
    # coder invoked once per round in both trajectories -> one segment of six members
    r_turn = rewards.reshape(-1)
    out = orc.role_advantage(np.zeros(6, int), np.zeros(6, int), np.repeat([0, 1], 3), None, r_turn, None,
                             None, 1, 1, np.arange(7), eps=0.0)
    assert np.allclose(out["adv_inv"], adv, atol=1e-12)


# ---------------------------------------------------------------------------- GAE pins

def test_gae_special_cases_and_recursion():
    rng = np.random.default_rng(8)
    cu = np.array([0, 5, 5, 9, 10])
    r, v = rng.normal(size=10), rng.normal(size=10)
    gamma = 0.9
    # lambda = 0: one-step TD error
    A0, _ = orc.gae(r, v, cu, gamma, 0.0)
    # lambda = 1: discounted return minus value
    A1, ret1 = orc.gae(r, v, cu, gamma, 1.0)
    for s in range(4):
        lo, hi = cu[s], cu[s + 1]
        for t in range(lo, hi):
            nxt = v[t + 1] if t + 1 < hi else 0.0
            assert abs(A0[t] - (r[t] + gamma * nxt - v[t])) < 1e-13
            disc = sum(gamma ** (u - t) * r[u] for u in range(t, hi))
            assert abs(A1[t] - (disc - v[t])) < 1e-12 and abs(ret1[t] - disc) < 1e-12
    # general lambda: backward recursion A_t = delta_t + gamma*lambda*A_{t+1}
    lam = 0.95
    A, _ = orc.gae(r, v, cu, gamma, lam)
    for s in range(4):
        lo, hi = cu[s], cu[s + 1]
        nxtA = 0.0
        for t in range(hi - 1, lo - 1, -1):
            nxt = v[t + 1] if t + 1 < hi else 0.0
            nxtA = r[t] + gamma * nxt - v[t] + gamma * lam * nxtA
            assert abs(A[t] - nxtA) < 1e-12


def test_gae_masked_tokens_are_transparent():
    rng = np.random.default_rng(9)
    cu = np.array([0, 7, 12, 12, 20])
    n = 20
    r, v = rng.normal(size=n), rng.normal(size=n)
    mask = (rng.random(n) < 0.6).astype(np.uint8)
    mask[7:12] = 0                                      # a sequence with no valid token
    A, ret = orc.gae(r, v, cu, 0.97, 0.9, mask)
    # removing the masked tokens and running the unmasked formula gives the same numbers
    keep = mask != 0
    lens = [int(keep[cu[s]:cu[s + 1]].sum()) for s in range(4)]
    cu2 = np.concatenate([[0], np.cumsum(lens)])
    A2, ret2 = orc.gae(r[keep], v[keep], cu2, 0.97, 0.9)
    assert np.allclose(A[keep], A2, atol=1e-14) and np.allclose(ret[keep], ret2, atol=1e-14)
    assert np.all(A[~keep] == 0) and np.all(ret[~keep] == 0)


def test_reward_assembly_follows_the_workflow_rules():
    # Workflow D (reflective verification loop), scores and expected rewards from the hand fixture
    rows = np.array([[float(x) for x in line.split()] for line in open(os.path.join(GOLDEN, "workflow_d_rewards.txt"))
                     if line[0].isdigit()])
    scores, expect = rows[:, 1:4], rows[:, 4:7]
    # roles: 0 planner, 1 coder (paid the improvement of their own round), 2 reflector (paid the improvement of the
    # NEXT round; there is no reflector after the last round)
    rules = [(orc.RULE_MARGINAL, 0), (orc.RULE_MARGINAL, 0), (orc.RULE_MARGINAL, 1)]
    inv = [(j, t, v) for j in range(2) for t in range(3) for v in (0, 1, 2) if not (v == 2 and t == 2)]
    traj, turn, role = (np.array(x) for x in zip(*inv))
    r = orc.reward_assembly(role, traj, turn, scores, [3, 3], rules)
    for s, (j, t, v) in enumerate(inv):
        want = expect[j, t] if v < 2 else expect[j, t + 1]      # r(Reflector_i) = s_{i+1} - s_i
        assert abs(r[s] - want) < 1e-12
    # Workflow C (iterative search): planner F1(a_0); answer agent F1(a_t); loop agents F1(a_t) - F1(a_{t-1});
    # a search agent that outputs <end> gets 0
    f1 = np.array([[0.25, 0.5, 0.4, 0.9]])
    rules = [(orc.RULE_ABSOLUTE, 0), (orc.RULE_MARGINAL, 0), (orc.RULE_ABSOLUTE, 0)]      # planner, searcher, answerer
    role = np.array([0, 1, 2, 1, 2, 1, 2])
    turn = np.array([0, 1, 1, 2, 2, 3, 3])
    end = np.array([0, 0, 0, 0, 0, 1, 0])
    r = orc.reward_assembly(role, np.zeros(7, int), turn, f1, [4], rules, end)
    assert np.allclose(r, [0.25, 0.25, 0.5, -0.1, 0.4, 0.0, 0.9])
    # a turn without a score pays nothing, and so does a role without a turn-level rule (Workflows A / B)
    r = orc.reward_assembly(np.array([1, 0]), np.zeros(2, int), np.array([2, 0]), f1, [2], [(orc.RULE_NONE, 0), (orc.RULE_ABSOLUTE, 0)])
    assert np.all(r == 0)


# ---------------------------------------------------------------------------- value-loss pins

def value_problem(seed=11, n_inv=7, R=3, K=2, max_len=6):
    rng = np.random.default_rng(seed)
    role_model = np.array([v % K for v in range(R)])
    inv_role = rng.integers(0, R, n_inv)
    inv_role[:R] = np.arange(R)
    lens = rng.integers(0, max_len + 1, n_inv)
    cu = np.concatenate([[0], np.cumsum(lens)])
    n = int(cu[-1])
    mask = (rng.random(n) < 0.75).astype(np.uint8)
    return dict(cu=cu, inv_role=inv_role, role_model=role_model, mask=mask, v=rng.normal(size=n),
                ov=rng.normal(size=n), R=rng.normal(size=n), K=K)


def test_value_loss_without_clipping_is_half_mse_per_model():
    p = value_problem()
    out = orc.value_loss_fwd_bwd(p["v"], p["ov"], p["R"], p["cu"], p["inv_role"], p["role_model"], p["mask"],
                                 clip_v=1e30, K=p["K"])
    tok_model = p["role_model"][p["inv_role"]][np.repeat(np.arange(len(p["cu"]) - 1), np.diff(p["cu"]))]
    for k in range(p["K"]):
        sel = (p["mask"] != 0) & (tok_model == k)
        assert sel.sum() > 0
        # numpy's mean of squared errors is the library special case
        assert abs(out["loss"][k] - 0.5 * np.mean((p["v"][sel] - p["R"][sel]) ** 2)) < 1e-14
        assert np.allclose(out["dvalues"][sel], (p["v"][sel] - p["R"][sel]) / sel.sum(), atol=1e-15)
        assert out["clip_frac"][k] == 0
    assert np.all(out["dvalues"][p["mask"] == 0] == 0) and np.all(out["tok_loss"][p["mask"] == 0] == 0)


def test_value_loss_clip_branches_hand_values():
    # one token per case, old value 0, clip 0.2, a single model:
    #   v      R      v_clip  (v-R)^2  (v_clip-R)^2   branch      loss     dl/dv
    #   0.1    1.0    0.1     0.81     0.81           unclipped   0.405    -0.9     (inside the range: tie)
    #   0.5    1.0    0.2     0.25     0.64           clipped     0.32      0       (moved towards R too far)
    #   0.5    0.0    0.2     0.25     0.04           unclipped   0.125     0.5     (moved away from R)
    #  -0.6   -0.1   -0.2     0.25     0.01           unclipped   0.125    -0.5
    #  -0.6   -1.0   -0.2     0.16     0.64           clipped     0.32      0
    v = np.array([0.1, 0.5, 0.5, -0.6, -0.6])
    R = np.array([1.0, 1.0, 0.0, -0.1, -1.0])
    out = orc.value_loss_fwd_bwd(v, np.zeros(5), R, np.array([0, 5]), np.array([0]), np.array([0]), None, clip_v=0.2)
    assert np.allclose(out["tok_loss"], [0.405, 0.32, 0.125, 0.125, 0.32], atol=1e-15)
    assert np.allclose(out["dvalues"] * 5, [-0.9, 0.0, 0.5, -0.5, 0.0], atol=1e-15)
    assert abs(out["loss"][0] - (0.405 + 0.32 + 0.125 + 0.125 + 0.32) / 5) < 1e-15
    assert abs(out["clip_frac"][0] - 0.4) < 1e-15
    # the clipped loss is never below the plain one (pessimistic bound)
    plain = orc.value_loss_fwd_bwd(v, np.zeros(5), R, np.array([0, 5]), np.array([0]), np.array([0]), None, clip_v=1e30)
    assert np.all(out["tok_loss"] >= plain["tok_loss"] - 1e-15)


def test_value_loss_gradient_matches_autograd_and_finite_differences():
    p = value_problem(seed=12)
    norm = [5.0, 3.0]
    out = orc.value_loss_fwd_bwd(p["v"], p["ov"], p["R"], p["cu"], p["inv_role"], p["role_model"], p["mask"],
                                 clip_v=0.3, norm=norm)
    tok_model = torch.from_numpy(p["role_model"][p["inv_role"]][np.repeat(np.arange(len(p["cu"]) - 1), np.diff(p["cu"]))])
    v = torch.tensor(p["v"], dtype=torch.float64, requires_grad=True)
    ov, R = torch.from_numpy(p["ov"]), torch.from_numpy(p["R"])
    vc = ov + torch.clamp(v - ov, -0.3, 0.3)
    tok = 0.5 * torch.maximum((v - R) ** 2, (vc - R) ** 2) * torch.from_numpy((p["mask"] != 0).astype(np.float64))
    total = sum(tok[tok_model == k].sum() / norm[k] for k in range(2))
    total.backward()
    # inside the clip range the two branches coincide and autograd splits the gradient between them; the sum is the
    # same number, so the comparison holds everywhere
    assert np.allclose(out["dvalues"], v.grad.numpy(), atol=1e-14)
    assert abs(float(total) - out["loss"].sum()) < 1e-14
    h = 1e-6
    for i in np.nonzero(p["mask"])[0][:8]:
        vp, vm = p["v"].copy(), p["v"].copy()
        vp[i] += h
        vm[i] -= h
        f = lambda x: orc.value_loss_fwd_bwd(x, p["ov"], p["R"], p["cu"], p["inv_role"], p["role_model"], p["mask"],
                                             clip_v=0.3, norm=norm)["loss"].sum()
        assert abs((f(vp) - f(vm)) / (2 * h) - out["dvalues"][i]) < 1e-8


# ---------------------------------------------------------------------------- ready-batch pins

def test_fmix32_published_values_and_permutation_is_a_bijection():
    # MurmurHash3's finaliser: 0 is its fixed point and 1 maps to 0x514E28B7 (the value quoted with the algorithm)
    assert orc.fmix32(0) == 0 and orc.fmix32(1) == 0x514E28B7
    # it is a bijection of 32-bit words (each step is invertible); spot check: no collision among 2^16 inputs
    assert len({orc.fmix32(x) for x in range(1 << 16)}) == 1 << 16
    for n in [1, 2, 3, 4, 5, 16, 17, 100, 255, 256, 257, 1000, 4097]:
        for seed in (0, 1, 20260528, (1 << 63) + 12345):
            perm = orc.seeded_permutation(n, seed)
            assert np.array_equal(np.sort(perm), np.arange(n))
    assert orc.seeded_permutation(0, 3).size == 0
    # different seeds give different orders, the same seed the same order
    a, b = orc.seeded_permutation(1000, 1), orc.seeded_permutation(1000, 2)
    assert not np.array_equal(a, b) and np.array_equal(a, orc.seeded_permutation(1000, 1))
    # it shuffles: over many seeds, element 0 lands in every quarter of the range about equally often
    pos = np.array([int(np.nonzero(orc.seeded_permutation(64, s) == 0)[0][0]) for s in range(400)])
    hist = np.bincount(pos // 16, minlength=4)
    assert hist.min() > 60 and hist.max() < 140
    # and neighbours do not stay neighbours
    assert np.mean(np.abs(np.diff(a)) == 1) < 0.05


def batch_problem(seed=3, n_traj=40, R=3, K=2, max_len=9):
    rng = np.random.default_rng(seed)
    role_model = np.array([0, 1, 0])
    inv_traj = np.repeat(np.arange(n_traj), rng.integers(1, 5, n_traj))
    n_inv = inv_traj.size
    inv_role = rng.integers(0, R, n_inv)
    lens = rng.integers(0, max_len + 1, n_inv)
    cu = np.concatenate([[0], np.cumsum(lens)])
    done = (rng.random(n_traj) < 0.7).astype(np.uint8)
    return dict(cu=cu, inv_role=inv_role, inv_traj=inv_traj, done=done, role_model=role_model, K=K, n_inv=n_inv)


@pytest.mark.parametrize("n_parts,pad_to", [(1, 1), (4, 1), (3, 8)])
def test_ready_batch_plan_properties(n_parts, pad_to):
    p = batch_problem()
    out = orc.ready_batch_plan(p["cu"], p["inv_role"], p["inv_traj"], p["done"], p["role_model"], p["K"], seed=77,
                               n_parts=n_parts, pad_to=pad_to)
    order, out_cu = out["order"], out["out_cu"]
    # kept set = brute-force filter: complete trajectory (and a role that maps to a model)
    want = {s for s in range(p["n_inv"]) if p["done"][p["inv_traj"][s]]}
    assert set(order.tolist()) == want and len(order) == len(want) == out["n_kept"]
    # model-major: the models of the listed invocations are non-decreasing and match model_offsets
    models = p["role_model"][p["inv_role"][order]]
    assert np.all(np.diff(models) >= 0)
    for k in range(p["K"]):
        lo, hi = out["model_offsets"][k], out["model_offsets"][k + 1]
        assert np.all(models[lo:hi] == k) and hi - lo == int((models == k).sum())
    # inside a model the order is the shuffled order (increasing position in the permutation)
    position = np.argsort(orc.seeded_permutation(p["n_inv"], 77))
    for k in range(p["K"]):
        lo, hi = out["model_offsets"][k], out["model_offsets"][k + 1]
        assert np.all(np.diff(position[order[lo:hi]]) > 0)
    # padded slots: each holds its invocation, is a multiple of pad_to, and wastes less than pad_to
    lens = np.diff(p["cu"])[order]
    slots = np.diff(out_cu)
    assert np.all(slots % pad_to == 0) and np.all(slots >= lens) and np.all(slots - lens < pad_to)
    assert out["n_tok"] == out_cu[-1] == slots.sum()
    # partitions: contiguous, cover each model's range, and balanced in tokens up to one slot
    po = out["part_offsets"]
    assert po.size == p["K"] * n_parts + 1 and np.all(np.diff(po) >= 0) and po[-1] == out["n_kept"]
    for k in range(p["K"]):
        assert po[k * n_parts] == out["model_offsets"][k]
        T = out_cu[out["model_offsets"][k + 1]] - out_cu[out["model_offsets"][k]]
        for q in range(n_parts):
            lo, hi = po[k * n_parts + q], po[k * n_parts + q + 1]
            tokens = out_cu[hi] - out_cu[lo]
            assert abs(tokens - T / n_parts) <= slots.max()


def test_ready_batch_plan_hand_case_gather_and_reward_alignment():
    # four invocations of lengths 3, 2, 4, 1; trajectory 1 (invocation 2) is incomplete; one model; pad to 4
    cu = np.array([0, 3, 5, 9, 10])
    out = orc.ready_batch_plan(cu, [0, 0, 0, 0], [0, 0, 1, 2], [1, 0, 1], [0], 1, seed=5, n_parts=1, pad_to=4)
    perm = orc.seeded_permutation(4, 5)
    assert out["order"].tolist() == [s for s in perm.tolist() if s != 2]
    assert out["out_cu"].tolist() == [0, 4, 8, 12] and out["n_tok"] == 12
    tok = np.arange(10) + 100
    g = orc.ready_batch_gather(tok, cu, out["order"], out["out_cu"], -1)
    for j, s in enumerate(out["order"]):
        L = cu[s + 1] - cu[s]
        assert g[4 * j:4 * j + L].tolist() == tok[cu[s]:cu[s + 1]].tolist() and np.all(g[4 * j + L:4 * j + 4] == -1)
    # delayed rewards: on the last unmasked token of each invocation
    mask = np.array([1, 1, 0, 1, 1, 0, 0, 0, 0, 1], np.uint8)
    r = orc.align_rewards([0.5, -1.0, 2.0, 3.0], cu, mask)
    assert r.tolist() == [0, 0.5, 0, 0, -1.0, 0, 0, 0, 0, 3.0]           # invocation 2 has no unmasked token
    assert orc.align_rewards([0.5, -1.0, 2.0, 3.0], cu).tolist() == [0, 0, 0.5, 0, -1.0, 0, 0, 0, 2.0, 3.0]
    # with gamma = lambda = 1 and zero values, GAE of the aligned reward gives every unmasked token its
    # invocation's reward: the delayed reward reaches the whole response
    A, _ = orc.gae(r, np.zeros(10), cu, 1.0, 1.0, mask)
    assert A.tolist() == [0.5, 0.5, 0, -1.0, -1.0, 0, 0, 0, 0, 3.0]


# ---------------------------------------------------------------------------- metric records (per model / per role)
# Section "Parameter Sharing in the System": role identity and agent-level metrics are kept even when roles share
# parameters; paragraph "Batch construction": role identifiers are preserved for role-specific analysis.

METRIC_NAMES = ["n", "pg", "kl", "entropy", "clip_frac", "ratio", "logp", "adv"]


def brute_force_records(p, cur_logp, cur_ent, old, ref, adv, lo, hi, kl_mode, keys, n_classes):
    """The eight numbers of every class, token by token with python scalars; `keys[i]` is the class of token i.
    Independent of the oracle's own per-token intermediates: it starts from the (separately pinned) log-probs and
    entropies and restates each quantity's definition."""
    acc = [[0.0] * 8 for _ in range(n_classes)]
    for i in range(len(cur_logp)):
        if not p["tok_mask"][i]:
            continue
        c = int(keys[i])
        ratio = math.exp(cur_logp[i] - old[i])
        un = -ratio * adv[i]
        cl = -min(max(ratio, 1.0 - lo), 1.0 + hi) * adv[i]
        d = ref[i] - cur_logp[i]
        kl = {1: -d, 2: 0.5 * d * d, 3: math.exp(d) - d - 1.0}[kl_mode]
        row = [1.0, max(un, cl), kl, cur_ent[i], 1.0 if cl > un else 0.0, ratio, cur_logp[i], adv[i]]
        for j in range(8):
            acc[c][j] += row[j]
    out = np.zeros((n_classes, 8))
    for c in range(n_classes):
        n = acc[c][0]
        out[c, 0] = n
        for j in range(1, 8):
            out[c, j] = acc[c][j] / max(n, 1.0)
    return out


@pytest.mark.parametrize("K,R,role_model,kl_mode", [(1, 2, [0, 0], 3), (2, 3, [0, 0, 1], 3), (2, 3, [0, 0, 1], 2),
                                                   (2, 4, [1, 0, 1, 0], 1)])
def test_metric_records_match_brute_force_per_model_and_per_role(K, R, role_model, kl_mode):
    p = tiny_problem(seed=40 + R, n_inv=16, H=8, V=12, K=K, R=R, max_len=6, mask_p=0.7)
    p["role_model"] = np.array(role_model)
    f = fwd(p)
    rng = np.random.default_rng(5)
    N = f["logp"].size
    old = f["logp"] + 0.3 * rng.normal(size=N)           # wide ratios: both clip branches occur
    ref = f["logp"] + 0.2 * rng.normal(size=N)
    adv = rng.normal(size=N) + 0.3
    lo, hi = 0.2, 0.3
    out = ppo(p, old, ref, adv, clip_lo=lo, clip_hi=hi, kl_coef=0.1, kl_mode=kl_mode, ent_coef=0.01, n_roles=R)
    tok_inv = np.repeat(np.arange(len(p["inv_role"])), np.diff(p["cu_seqlens"]))
    tok_role = p["inv_role"][tok_inv]
    tok_model = p["role_model"][tok_role]
    bm = brute_force_records(p, f["logp"], f["entropy"], old, ref, adv, lo, hi, kl_mode, tok_model, K)
    br = brute_force_records(p, f["logp"], f["entropy"], old, ref, adv, lo, hi, kl_mode, tok_role, R)
    assert out["metrics_model"].shape == (K, 8) and out["metrics_role"].shape == (R, 8)
    assert np.abs(out["metrics_model"] - bm).max() < 1e-12
    assert np.abs(out["metrics_role"] - br).max() < 1e-12
    # the fixture must be able to tell columns and classes apart: no two columns and no two roles coincide, both
    # clip branches occur, and roles that share a model still have different records
    assert 0.0 < br[:, 4].max() and br[:, 4].min() < 1.0
    for a in range(8):
        for b in range(a + 1, 8):
            assert np.abs(br[:, a] - br[:, b]).max() > 1e-3, (METRIC_NAMES[a], METRIC_NAMES[b])
    shared = [v for v in range(R) if role_model.count(role_model[v]) > 1]
    assert len(shared) >= 2 and np.abs(br[shared[0], 1:] - br[shared[1], 1:]).max() > 1e-3
    # per-model counts are the sums of their roles' counts; per-model means are the count-weighted role means
    for k in range(K):
        roles_k = [v for v in range(R) if role_model[v] == k]
        n_k = sum(br[v, 0] for v in roles_k)
        assert out["metrics_model"][k, 0] == n_k
        for j in range(1, 8):
            assert abs(out["metrics_model"][k, j] - sum(br[v, 0] * br[v, j] for v in roles_k) / max(n_k, 1.0)) < 1e-12


def test_metric_records_closed_form_columns():
    """Every column gets a different known value: W = 0 makes logp = -ln V and entropy = ln V on every row; old =
    logp - delta makes the ratio e^delta (inside the clip range, so nothing is clipped); ref = logp + d0 makes
    the k3 term e^d0 - d0 - 1; a constant advantage c makes the surrogate -c e^delta."""
    V, c, delta, d0 = 16, 0.75, 0.1, 0.3
    p = tiny_problem(seed=50, n_inv=10, V=V, K=2, R=3)
    p["role_model"] = np.array([0, 0, 1])
    p["W"] = [np.zeros_like(w) for w in p["W"]]
    N = p["hidden"].shape[0]
    lp = np.full(N, -math.log(V))
    out = ppo(p, lp - delta, lp + d0, np.full(N, c), kl_coef=0.1, kl_mode=3, ent_coef=0.0, n_roles=3)
    valid = p["tok_mask"] != 0
    tok_inv = np.repeat(np.arange(10), np.diff(p["cu_seqlens"]))
    tok_role = p["inv_role"][tok_inv]
    expect = [None, -c * math.exp(delta), math.exp(d0) - d0 - 1.0, math.log(V), 0.0, math.exp(delta), -math.log(V), c]
    for v in range(3):
        rec = out["metrics_role"][v]
        assert rec[0] == float((valid & (tok_role == v)).sum()) and rec[0] > 0
        for j in range(1, 8):
            assert abs(rec[j] - expect[j]) < 1e-13, METRIC_NAMES[j]
    for k, roles_k in enumerate([(0, 1), (2,)]):
        rec = out["metrics_model"][k]
        assert rec[0] == float((valid & np.isin(tok_role, roles_k)).sum())
        for j in range(1, 8):
            assert abs(rec[j] - expect[j]) < 1e-13, METRIC_NAMES[j]


def test_metric_record_of_a_role_without_valid_tokens_is_zero():
    p = tiny_problem(seed=51, n_inv=9, K=1, R=3)
    p["role_model"] = np.array([0, 0, 0])
    tok_inv = np.repeat(np.arange(9), np.diff(p["cu_seqlens"]))
    p["tok_mask"][p["inv_role"][tok_inv] == 1] = 0            # role 1 present but fully masked
    p["inv_role"][p["inv_role"] == 2] = 0                     # role 2 never invoked
    cur = fwd(p)["logp"]
    out = ppo(p, cur, cur, np.ones(cur.size), n_roles=3)
    assert np.all(out["metrics_role"][1] == 0) and np.all(out["metrics_role"][2] == 0)
    assert out["metrics_role"][0, 0] == out["metrics_model"][0, 0] == float((p["tok_mask"] != 0).sum())
    assert np.abs(out["metrics_role"][0] - out["metrics_model"][0]).max() == 0
