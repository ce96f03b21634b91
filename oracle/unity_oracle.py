"""fp64 CPU oracle for the multi-agent PPO hot path.  TEST INFRASTRUCTURE ONLY.

This file is the reference the CUDA library is judged against.  It is plain numpy in float64,
slow and direct: every quantity is its definition written out, one block of rows at a time,
with the full logit vector of each row materialised.  It shares no code with the CUDA path and
imports nothing from it.  Only tests, the smoke check and the benchmark's CPU-baseline leg may
call it; the product never does.

What each function follows:

* ``role_advantage``  - the additive role reward r_v = lam_node r_node + lam_turn r_turn +
  lam_traj r_traj (Section "Agent-Specific Reward Interface", the lambda-weighted equation) with
  rewards committed per role invocation (Section "Optimization Objective and System Interface");
  role identity is kept even when parameters are shared (Section "Parameter Sharing in the
  System"), so statistics are per (rollout group, role), never per model.  The normalisation
  itself (mean / std per segment, epsilon added to std) is not printed in the paper; it is the
  reading fixed for this path.
* ``logprob_fwd``     - "old log probabilities, reference-policy log probabilities" of the
  paragraph "Advantage computation and policy evaluation": log-softmax of the LM-head logits
  of the model that phi assigns to the token's role, gathered at the target token, and the
  Shannon entropy of that softmax.
* ``ppo_loss_fwd_bwd``- the "PPO-style" update of Section "PPO-Style Training Loop" with the
  standard clipped surrogate, a KL-to-reference penalty (k1/k2/k3 estimators) and an entropy
  bonus, averaged over valid tokens per model (paragraph "Model-specific updates and
  synchronization": each worker group updates its own actor), and its exact gradient with
  respect to the hidden states and each LM-head matrix.
* ``reward_assembly`` - the turn-level reward rules of Section "Workflows and Rewards": a role is paid either the
  score of a turn (Workflow C: planner F1(a_0), answer agent F1(a_t)) or the improvement of the score over the
  previous turn (Workflow C: F1(a_t) - F1(a_{t-1}) for the loop agents; Workflow D: s_0, s_1 - s_0, s_2 - s_1, the
  reflector of round i being paid the improvement of round i+1); an agent that ended the loop gets 0.
* ``gae``             - the generalized-advantage equation printed in the same section
  (A_t = sum_l (gamma lambda)^l delta_{t+l}), evaluated as the literal double sum.

Pins: tests/test_oracle_pins.py (closed forms, invariants, library special cases, finite
differences, autograd third opinion, brute force).  No function here is unpinned.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def to_f64(x) -> np.ndarray:
    """Exact widening.  uint16 arrays are bf16 bit patterns; anything else is cast."""
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(F64)
    return x.astype(F64)


# ----------------------------------------------------------------------------------------------
# stage 1: role-level advantage
# ----------------------------------------------------------------------------------------------

def role_advantage(inv_role, inv_group, inv_traj, r_node, r_turn, r_traj, lam,
                   n_roles, n_groups, cu_seqlens, tok_mask=None, eps=1e-6, ddof=0):
    """Combine rewards per invocation, normalise per (group, role), broadcast to tokens.

    Returns dict(r, adv_inv, adv_tok, seg_n, seg_mean, seg_std); segment index = g*n_roles+v.
    """
    inv_role = np.asarray(inv_role, dtype=np.int64)
    inv_group = np.asarray(inv_group, dtype=np.int64)
    inv_traj = np.asarray(inv_traj, dtype=np.int64)
    S = inv_role.shape[0]
    lam = np.ones((n_roles, 3), F64) if lam is None else to_f64(lam).reshape(n_roles, 3)
    rn = np.zeros(S, F64) if r_node is None else to_f64(r_node)
    rt = np.zeros(S, F64) if r_turn is None else to_f64(r_turn)
    rj = np.zeros(S, F64) if r_traj is None else to_f64(r_traj)[inv_traj]
    r = lam[inv_role, 0] * rn + lam[inv_role, 1] * rt + lam[inv_role, 2] * rj

    n_seg = n_groups * n_roles
    seg = inv_group * n_roles + inv_role
    seg_n = np.zeros(n_seg, np.int64)
    seg_mean = np.zeros(n_seg, F64)
    seg_std = np.zeros(n_seg, F64)
    adv_inv = np.zeros(S, F64)
    for q in range(n_seg):
        members = np.nonzero(seg == q)[0]
        n = members.size
        seg_n[q] = n
        if n == 0:
            continue
        mu = r[members].sum() / n
        seg_mean[q] = mu
        if n - ddof <= 0:
            continue                                    # A = 0, std reported as 0
        sigma = np.sqrt(((r[members] - mu) ** 2).sum() / (n - ddof))
        seg_std[q] = sigma
        if sigma + eps == 0.0:
            continue                                    # all rewards equal and eps = 0: A = 0
        adv_inv[members] = (r[members] - mu) / (sigma + eps)

    cu = np.asarray(cu_seqlens, dtype=np.int64)
    n_tok = int(cu[-1])
    mask = np.ones(n_tok, F64) if tok_mask is None else (np.asarray(tok_mask) != 0).astype(F64)
    adv_tok = np.zeros(n_tok, F64)
    for s in range(S):
        adv_tok[cu[s]:cu[s + 1]] = adv_inv[s]
    adv_tok *= mask
    return dict(r=r, adv_inv=adv_inv, adv_tok=adv_tok, seg_n=seg_n, seg_mean=seg_mean, seg_std=seg_std)


# ----------------------------------------------------------------------------------------------
# turn-level reward assembly (the step before stage 1)
# ----------------------------------------------------------------------------------------------

RULE_NONE, RULE_ABSOLUTE, RULE_MARGINAL = 0, 1, 2


def reward_assembly(inv_role, inv_traj, inv_turn, score, n_scores, rules, inv_end=None):
    """r_turn per invocation from per-trajectory, per-turn scores.

    ``score[j, t]`` is the score after turn t of trajectory j (answer F1, verifier pass rate); ``n_scores[j]`` turns
    have a score.  ``rules[v] = (mode, shift)``: with u = turn + shift, mode ABSOLUTE pays score[j, u], mode MARGINAL
    pays score[j, u] - score[j, u-1] (the score before the first turn counts as 0), mode NONE pays 0.  No score at
    u (u < 0 or u >= n_scores[j]) pays 0; ``inv_end[s] != 0`` pays 0."""
    S = len(inv_role)
    score = to_f64(score)
    out = np.zeros(S, F64)
    for s in range(S):
        mode, shift = rules[int(inv_role[s])]
        j, u = int(inv_traj[s]), int(inv_turn[s]) + shift
        if mode == RULE_NONE or u < 0 or u >= int(n_scores[j]):
            continue
        if inv_end is not None and inv_end[s]:
            continue
        if mode == RULE_ABSOLUTE:
            out[s] = score[j, u]
        else:
            out[s] = score[j, u] - (score[j, u - 1] if u >= 1 else 0.0)
    return out


# ----------------------------------------------------------------------------------------------
# token routing through phi
# ----------------------------------------------------------------------------------------------

def token_invocation(cu_seqlens) -> np.ndarray:
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    return np.repeat(np.arange(cu.size - 1, dtype=np.int64), np.diff(cu))


def token_role_model(cu_seqlens, inv_role, role_model):
    tok_inv = token_invocation(cu_seqlens)
    tok_role = np.asarray(inv_role, dtype=np.int64)[tok_inv]
    tok_model = np.asarray(role_model, dtype=np.int64)[tok_role]
    return tok_role, tok_model


# ----------------------------------------------------------------------------------------------
# stage 2: log-prob, entropy, log-sum-exp
# ----------------------------------------------------------------------------------------------

def _row_stats(Z):
    """lse, entropy and probabilities of each row of a logit block Z [n, V] (float64)."""
    m = Z.max(axis=1, keepdims=True)
    E = np.exp(Z - m)
    s = E.sum(axis=1, keepdims=True)
    lse = (m + np.log(s))[:, 0]
    P = E / s
    logP = Z - lse[:, None]
    ent = -(P * logP).sum(axis=1)
    return lse, ent, P


def logprob_fwd(hidden, W, cu_seqlens, inv_role, role_model, target, tok_mask=None,
                inv_temperature=1.0, rows=None, block=256):
    """logp, entropy, lse per token (zeros where mask == 0).

    ``rows`` restricts the computation to the given token indices (sampled parity at full size);
    other rows are returned as zero.
    """
    n_tok = int(np.asarray(cu_seqlens)[-1])
    _, tok_model = token_role_model(cu_seqlens, inv_role, role_model)
    mask = np.ones(n_tok, bool) if tok_mask is None else (np.asarray(tok_mask) != 0)
    target = np.asarray(target, dtype=np.int64)
    want = mask.copy()
    if rows is not None:
        sel = np.zeros(n_tok, bool)
        sel[np.asarray(rows, dtype=np.int64)] = True
        want &= sel
    logp = np.zeros(n_tok, F64)
    ent = np.zeros(n_tok, F64)
    lse = np.zeros(n_tok, F64)
    for k in range(len(W)):
        idx = np.nonzero(want & (tok_model == k))[0]
        if idx.size == 0:
            continue
        Wk = to_f64(W[k])
        for b0 in range(0, idx.size, block):
            ib = idx[b0:b0 + block]
            Z = inv_temperature * (to_f64(hidden[ib]) @ Wk.T)
            l, e, _ = _row_stats(Z)
            lse[ib] = l
            ent[ib] = e
            logp[ib] = Z[np.arange(ib.size), target[ib]] - l
    return dict(logp=logp, entropy=ent, lse=lse)


# ----------------------------------------------------------------------------------------------
# stage 3: PPO-clip + KL-to-reference (+ entropy bonus): forward and backward
# ----------------------------------------------------------------------------------------------

def kl_term(d, mode):
    """KL-to-reference estimators as functions of d = ref_logp - logp, and d(kl)/d(logp)."""
    if mode == 1:
        return -d, np.ones_like(d)
    if mode == 2:
        return 0.5 * d * d, -d
    if mode == 3:
        return np.exp(d) - d - 1.0, 1.0 - np.exp(d)
    raise ValueError("kl_mode must be 1, 2 or 3")


def ppo_token_terms(logp, entropy, old_logp, ref_logp, adv, clip_lo, clip_hi, kl_coef, kl_mode, ent_coef):
    """Per-token loss pieces and the derivative of the token loss w.r.t. its log-prob."""
    rho = np.exp(logp - old_logp)
    rho_c = np.clip(rho, 1.0 - clip_lo, 1.0 + clip_hi)
    unclipped = -rho * adv
    clipped = -rho_c * adv
    u = (unclipped >= clipped)                      # ties -> unclipped branch
    pg = np.where(u, unclipped, clipped)
    d = ref_logp - logp
    kl, dkl = kl_term(d, kl_mode)
    tok_loss = pg + kl_coef * kl - ent_coef * entropy
    dl_dlogp = np.where(u, -adv * rho, 0.0) + kl_coef * dkl
    return dict(rho=rho, pg=pg, kl=kl, u=u, tok_loss=tok_loss, dl_dlogp=dl_dlogp)


def ppo_loss_fwd_bwd(hidden, W, cu_seqlens, inv_role, role_model, target, tok_mask,
                     old_logp, ref_logp, adv_tok, clip_lo=0.2, clip_hi=0.2, kl_coef=0.0, kl_mode=3,
                     ent_coef=0.0, norm=None, inv_temperature=1.0, n_roles=None,
                     want_dW=True, dW_models=None, rows=None, block=256):
    """Loss per model, metrics, per-token outputs, dHidden [N,H] and dW_k [V,H] (float64).

    ``norm``      : optional per-model denominator M_k (gradient accumulation across calls).
    ``dW_models`` : models whose dW is materialised (default: all); others are returned as None.
    ``rows``      : if given, only these token rows are evaluated (sampled parity at full size).
                    M_k still counts every valid row of the batch, so the per-token outputs and
                    dHidden rows of the selected rows are exact (a row's gradient needs only that
                    row, W_k and M_k); ``loss`` and ``dW`` are then the contribution of the
                    selected rows alone.
    """
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    n_tok = int(cu[-1])
    K = len(W)
    H = hidden.shape[1]
    tok_role, tok_model = token_role_model(cu, inv_role, role_model)
    R = int(n_roles if n_roles is not None else np.asarray(role_model).size)
    mask = np.ones(n_tok, bool) if tok_mask is None else (np.asarray(tok_mask) != 0)
    target = np.asarray(target, dtype=np.int64)
    old_logp = to_f64(old_logp)
    ref_logp = to_f64(ref_logp)
    adv = to_f64(adv_tok)
    tau = float(inv_temperature)

    logp = np.zeros(n_tok, F64)
    ent = np.zeros(n_tok, F64)
    lse = np.zeros(n_tok, F64)
    tok_loss = np.zeros(n_tok, F64)
    pg = np.zeros(n_tok, F64)
    kl = np.zeros(n_tok, F64)
    rho = np.zeros(n_tok, F64)
    clipped_flag = np.zeros(n_tok, F64)
    a = np.zeros(n_tok, F64)
    b = np.zeros(n_tok, F64)
    M = np.zeros(K, F64)
    loss = np.zeros(K, F64)
    dW = [None] * K
    dW_models = range(K) if dW_models is None else dW_models

    # the counts M_k come first: every token's coefficient is scaled by 1/M_k
    for k in range(K):
        cnt = float((mask & (tok_model == k)).sum())
        M[k] = float(norm[k]) if norm is not None else max(cnt, 1.0)

    want = mask.copy()
    if rows is not None:
        sel_rows = np.zeros(n_tok, bool)
        sel_rows[np.asarray(rows, dtype=np.int64)] = True
        want &= sel_rows
    # dHidden: all N rows (zeros where masked), or, with ``rows``, one line per evaluated row
    dh_index = np.arange(n_tok) if rows is None else np.nonzero(want)[0]
    dh_pos = np.full(n_tok, -1, np.int64)
    dh_pos[dh_index] = np.arange(dh_index.size)
    dHidden = np.zeros((dh_index.size, H), F64)

    for k in range(K):
        idx = np.nonzero(want & (tok_model == k))[0]
        Wk = to_f64(W[k]) if idx.size or (want_dW and k in dW_models) else None
        if want_dW and k in dW_models:
            dW[k] = np.zeros((Wk.shape[0], H), F64)
        for b0 in range(0, idx.size, block):
            ib = idx[b0:b0 + block]
            hb = to_f64(hidden[ib])
            Z = tau * (hb @ Wk.T)
            l, e, P = _row_stats(Z)
            lp = Z[np.arange(ib.size), target[ib]] - l
            t = ppo_token_terms(lp, e, old_logp[ib], ref_logp[ib], adv[ib],
                                clip_lo, clip_hi, kl_coef, kl_mode, ent_coef)
            logp[ib], ent[ib], lse[ib] = lp, e, l
            tok_loss[ib], pg[ib], kl[ib], rho[ib] = t["tok_loss"], t["pg"], t["kl"], t["rho"]
            clipped_flag[ib] = (~t["u"]).astype(F64)
            a[ib] = t["dl_dlogp"] / M[k]
            b[ib] = -ent_coef / M[k]
            # dL/dz for every vocabulary entry of every selected row
            Gm = -a[ib][:, None] * P - b[ib][:, None] * P * (Z - l[:, None] + e[:, None])
            Gm[np.arange(ib.size), target[ib]] += a[ib]
            dHidden[dh_pos[ib]] = tau * (Gm @ Wk)
            if dW[k] is not None:
                dW[k] += tau * (Gm.T @ hb)
        loss[k] = tok_loss[idx].sum() / M[k]

    def _metrics(sel):
        n = float(sel.sum())
        dn = max(n, 1.0)
        return np.array([n, pg[sel].sum() / dn, kl[sel].sum() / dn, ent[sel].sum() / dn,
                         clipped_flag[sel].sum() / dn, rho[sel].sum() / dn,
                         logp[sel].sum() / dn, adv[sel].sum() / dn], F64)

    metrics_model = np.stack([_metrics(want & (tok_model == k)) for k in range(K)])
    metrics_role = np.stack([_metrics(want & (tok_role == v)) for v in range(R)])
    return dict(loss=loss, M=M, logp=logp, entropy=ent, lse=lse, tok_loss=tok_loss, a=a, b=b,
                dHidden=dHidden, dh_index=dh_index, dW=dW, metrics_model=metrics_model, metrics_role=metrics_role)


def ppo_loss_value(hidden, W, cu_seqlens, inv_role, role_model, target, tok_mask,
                   old_logp, ref_logp, adv_tok, **kw):
    """Loss per model only (used by the finite-difference pin)."""
    out = ppo_loss_fwd_bwd(hidden, W, cu_seqlens, inv_role, role_model, target, tok_mask,
                           old_logp, ref_logp, adv_tok, want_dW=False, **kw)
    return out["loss"]


# ----------------------------------------------------------------------------------------------
# token-level generalized advantage estimation (the advantage formula the paper prints)
# ----------------------------------------------------------------------------------------------

def gae(rewards, values, cu_seqlens, gamma, lam, tok_mask=None):
    """A_t = sum_{l=0}^{T-t} (gamma*lam)^l delta_{t+l},  delta_t = r_t + gamma V(s_{t+1}) - V(s_t),
    per sequence, with V past the last token taken as 0.  Returns (advantages, returns=A+V).

    Tokens with tok_mask == 0 are not part of the sequence: the formula is applied to the remaining tokens of each
    sequence in order (their "next" token is the next unmasked one) and masked tokens receive 0 in both outputs."""
    r = to_f64(rewards)
    v = to_f64(values)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    keep = np.ones(r.shape[0], bool) if tok_mask is None else (np.asarray(tok_mask) != 0)
    A = np.zeros_like(r)
    for s in range(cu.size - 1):
        idx = np.arange(int(cu[s]), int(cu[s + 1]))
        idx = idx[keep[idx]]
        T = idx.size
        if T == 0:
            continue
        vs = np.concatenate([v[idx], [0.0]])
        delta = r[idx] + gamma * vs[1:] - vs[:-1]
        powers = (gamma * lam) ** np.arange(T)           # (gamma*lam)^l, l = 0 .. T-1
        for t in range(T):
            A[idx[t]] = (powers[:T - t] * delta[t:]).sum()   # the sum over l written out for this t
    return A, np.where(keep, A + v, 0.0)


# ----------------------------------------------------------------------------------------------
# critic side of the update: clipped value loss (paragraph "Model-specific updates and synchronization":
# each worker group updates its own actor AND critic; "value estimates, returns" are the quantities the
# paragraph "Advantage computation and policy evaluation" lists for it)
# ----------------------------------------------------------------------------------------------

def value_loss_fwd_bwd(values, old_values, returns, cu_seqlens, inv_role, role_model, tok_mask=None,
                       clip_v=0.2, norm=None, K=None):
    """PPO's clipped value regression, token-mean per model, and its gradient w.r.t. the value estimates.

    v_clip = old_v + clip(v - old_v, -clip_v, +clip_v);  l = 0.5 * max((v - R)^2, (v_clip - R)^2);
    L_k = (1/M_k) sum over valid tokens of model k of l, M_k = norm[k] if given else max(#valid tokens, 1).
    The paper prints no value loss; this is the reading fixed for the critic update.  Where the two squares are
    equal (in particular whenever v is inside the clip range, where v_clip = v) the unclipped branch is taken, so
    dl/dv = v - R there and 0 where the clipped square is strictly larger (v_clip does not depend on v then).
    Returns dict(loss[K], M[K], tok_loss[N], dvalues[N], clip_frac[K])."""
    v = to_f64(values)
    ov = to_f64(old_values)
    R = to_f64(returns)
    n_tok = v.shape[0]
    if K is None:
        K = int(np.max(np.asarray(role_model))) + 1 if norm is None else len(norm)
    _, tok_model = token_role_model(cu_seqlens, inv_role, role_model)
    mask = np.ones(n_tok, bool) if tok_mask is None else (np.asarray(tok_mask) != 0)
    d = v - ov
    # inside the range v_clip IS v (written so, not as ov + (v - ov), which rounds); outside it is the range's end
    v_clip = np.where(np.abs(d) <= clip_v, v, ov + np.sign(d) * clip_v)
    sq_u = (v - R) ** 2
    sq_c = (v_clip - R) ** 2
    unclipped = sq_u >= sq_c
    tok = 0.5 * np.where(unclipped, sq_u, sq_c)
    loss = np.zeros(K, F64)
    M = np.zeros(K, F64)
    clip_frac = np.zeros(K, F64)
    dv = np.zeros(n_tok, F64)
    for k in range(K):
        sel = mask & (tok_model == k)
        cnt = float(sel.sum())
        M[k] = float(norm[k]) if norm is not None else max(cnt, 1.0)
        loss[k] = tok[sel].sum() / M[k]
        clip_frac[k] = (~unclipped[sel]).sum() / max(cnt, 1.0)
        dv[sel] = np.where(unclipped[sel], v[sel] - R[sel], 0.0) / M[k]
    return dict(loss=loss, M=M, tok_loss=np.where(mask, tok, 0.0), dvalues=dv, clip_frac=clip_frac)


# ----------------------------------------------------------------------------------------------
# ready-batch construction (Section "Model-Local Buffers": B_i -> D_i^ready may include filtering incomplete
# trajectories, aligning delayed rewards with token sequences, padding, shuffling and matching the data-parallel
# configuration of the worker group; batches are built per model instance)
# ----------------------------------------------------------------------------------------------

_M32 = 0xFFFFFFFF


def fmix32(h: int) -> int:
    """The 32-bit finaliser of MurmurHash3 (public domain, A. Appleby): xor-shift 16, multiply 0x85ebca6b,
    xor-shift 13, multiply 0xc2b2ae35, xor-shift 16."""
    h &= _M32
    h ^= h >> 16
    h = (h * 0x85EBCA6B) & _M32
    h ^= h >> 13
    h = (h * 0xC2B2AE35) & _M32
    h ^= h >> 16
    return h


def seeded_permutation(n: int, seed: int):
    """perm[p] for p in [0, n): a seeded bijection of [0, n) built as a 4-round balanced Feistel network on the
    smallest even-width bit domain that holds n, with cycle walking for values that fall outside [0, n)
    (Black and Rogaway's construction of ciphers on arbitrary finite domains).  Round keys: key_i =
    fmix32(seed32 + 0x9E3779B9*(i+1)), seed32 = low word of seed xor high word; round function F(r, i) =
    fmix32(r xor key_i) truncated to the half width."""
    if n <= 0:
        return np.zeros(0, np.int64)
    bits = max(2, int(n - 1).bit_length())
    bits += bits & 1
    half = bits // 2
    hmask = (1 << half) - 1
    seed32 = (seed ^ (seed >> 32)) & _M32
    keys = [fmix32((seed32 + 0x9E3779B9 * (i + 1)) & _M32) for i in range(4)]
    out = np.zeros(n, np.int64)
    for p in range(n):
        x = p
        while True:
            left, right = x >> half, x & hmask
            for i in range(4):
                left, right = right, left ^ (fmix32(right ^ keys[i]) & hmask)
            x = (left << half) | right
            if x < n:
                break
        out[p] = x
    return out


def ready_batch_plan(cu_seqlens, inv_role, inv_traj, traj_done, role_model, K, seed, n_parts=1, pad_to=1):
    """Which invocations of the buffer enter the ready batch, in what order, and where their tokens go.

    Steps, in the paper's order: (1) filter - an invocation is kept when its trajectory is complete
    (traj_done != 0) and its role maps to a model in [0, K); (2) shuffle - positions p = 0..n_inv-1 are visited
    in order and position p holds buffer invocation seeded_permutation(n_inv, seed)[p]; (3) per model - kept
    invocations are listed model by model (each model builds its own batch), in shuffled order inside a model;
    (4) padding - each kept invocation occupies its length rounded up to a multiple of pad_to; (5) data-parallel
    split - inside model k, with P_j the padded tokens before invocation j and T_k the model's padded total,
    invocation j belongs to partition floor(P_j * n_parts / T_k): partitions are contiguous and equal in tokens
    up to one invocation.

    Returns dict(order[n_kept] buffer indices, out_cu[n_kept+1], model_offsets[K+1] (into order),
    part_offsets[K*n_parts+1] (into order), n_kept, n_tok)."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    n_inv = cu.size - 1
    perm = seeded_permutation(n_inv, seed)
    role_model = np.asarray(role_model, dtype=np.int64)
    per_model = [[] for _ in range(K)]
    for p in range(n_inv):
        s = int(perm[p])
        role, traj = int(inv_role[s]), int(inv_traj[s])
        if role < 0 or role >= role_model.size or traj < 0 or traj >= len(traj_done):
            continue
        k = int(role_model[role])
        if k < 0 or k >= K or not traj_done[traj]:
            continue
        per_model[k].append(s)
    order, out_cu, model_offsets, part_offsets = [], [0], [0], []
    for k in range(K):
        padded = [-(-int(cu[s + 1] - cu[s]) // pad_to) * pad_to for s in per_model[k]]
        T = sum(padded)
        P = 0
        parts = []
        for s, L in zip(per_model[k], padded):
            parts.append(min(n_parts - 1, (P * n_parts) // T) if T > 0 else 0)
            P += L
            order.append(s)
            out_cu.append(out_cu[-1] + L)
        base = model_offsets[-1]
        for q in range(n_parts):
            part_offsets.append(base + sum(1 for x in parts if x < q))
        model_offsets.append(base + len(per_model[k]))
    part_offsets.append(model_offsets[-1])
    return dict(order=np.asarray(order, np.int64), out_cu=np.asarray(out_cu, np.int64),
                model_offsets=np.asarray(model_offsets, np.int64), part_offsets=np.asarray(part_offsets, np.int64),
                n_kept=len(order), n_tok=out_cu[-1])


def ready_batch_gather(src, src_cu, order, out_cu, pad_value):
    """Token-level tensor of the ready batch: the rows of each kept invocation, then pad rows up to its slot."""
    src = np.asarray(src)
    out = np.empty((int(out_cu[-1]),) + src.shape[1:], src.dtype)
    out[...] = pad_value
    for j, s in enumerate(order):
        L = int(src_cu[s + 1] - src_cu[s])
        out[int(out_cu[j]):int(out_cu[j]) + L] = src[int(src_cu[s]):int(src_cu[s + 1])]
    return out


def align_rewards(r_inv, cu_seqlens, tok_mask=None):
    """Token-level reward sequence of a delayed (invocation-level) reward: the invocation's reward sits on its last
    unmasked response token, every other token gets 0 (paragraph "Batch construction": delayed rewards are aligned
    with the token sequences).  An invocation without an unmasked token has nowhere to put its reward."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    r = to_f64(r_inv)
    out = np.zeros(int(cu[-1]), F64)
    for s in range(cu.size - 1):
        for t in range(int(cu[s + 1]) - 1, int(cu[s]) - 1, -1):
            if tok_mask is None or tok_mask[t]:
                out[t] = r[s]
                break
    return out
