"""Parity harness - TEST INFRASTRUCTURE, not part of the library: runs one workload through libunity (C ABI) and
through the fp64 oracle and holds the tolerances of the parity contract.  Used by the tests, by the smoke check and by
the benchmark's CPU-baseline leg; the product (paper_2605_26646_b200) never imports it."""
from __future__ import annotations

import numpy as np
import torch

from oracle import unity_oracle as orc
from paper_2605_26646_b200 import binding as ub
from paper_2605_26646_b200 import workloads as wl

# tolerances of the parity contract
TOL_ADV = 1e-5        # advantages, absolute (fp32)
TOL_LOGP = 1e-2       # per-token log-prob and entropy, absolute
TOL_LOSS = 1e-3       # loss, relative
TOL_GRAD = 2e-2       # dHidden / dW, relative Frobenius


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def rel_fro(a: np.ndarray, b: np.ndarray) -> float:
    den = float(np.linalg.norm(b.astype(np.float64).ravel()))
    num = float(np.linalg.norm((a.astype(np.float64) - b.astype(np.float64)).ravel()))
    return num / den if den > 0 else num


def worst_row_rel(a: np.ndarray, b: np.ndarray, allowance=None) -> float:
    """Largest relative error of a row of `a` against the same row of `b` (2-norms), after taking off a per-row
    absolute `allowance` (see dh_row_allowance); a row that is zero in `b` must be zero in `a` up to its allowance
    (it counts as an infinite error otherwise)."""
    a, b = a.astype(np.float64), b.astype(np.float64)
    num = np.linalg.norm(a - b, axis=1)
    if allowance is not None:
        num = np.maximum(num - np.asarray(allowance, np.float64), 0.0)
    den = np.linalg.norm(b, axis=1)
    if np.any((den == 0) & (num > 0)):
        return float("inf")
    return float((num[den > 0] / den[den > 0]).max()) if np.any(den > 0) else 0.0


def dh_row_allowance(w, o, logp_gpu, old, ref, adv, clip=None, kl_coef=None, kl_mode=None, ent_coef=None, mask=None):
    """Per-row slack for comparing dHidden row by row.  A row's gradient is a_i * (W_y - sum_v p_v W_v) + (entropy
    term), and a_i = dL/dlogp_i depends on the row's log-prob: the contract lets the library's log-prob differ from
    the oracle's by up to TOL_LOGP, and for a row whose a_i nearly vanishes (zero advantage, reference log-prob
    equal to the current one) that admissible difference moves a_i by as much as a_i itself.  The slack is that
    effect and nothing else: |a_i evaluated at the library's log-prob - a_i of the oracle| times a bound on
    ||tau (W_y - sum_v p_v W_v)||, namely 2 tau max_v ||W_k[v]||.  Rows are those of o["dh_index"]; `mask` is the token
    mask the oracle was given (default: the workload's)."""
    idx = o["dh_index"]
    lo, hi = (w.clip_lo, w.clip_hi) if clip is None else clip
    t = orc.ppo_token_terms(np.asarray(logp_gpu, np.float64)[idx], o["entropy"][idx], orc.to_f64(np.asarray(old))[idx],
                            orc.to_f64(np.asarray(ref))[idx], orc.to_f64(np.asarray(adv))[idx], lo, hi,
                            w.kl_coef if kl_coef is None else kl_coef, w.kl_mode if kl_mode is None else kl_mode,
                            w.ent_coef if ent_coef is None else ent_coef)
    _, tok_model = orc.token_role_model(w.cu_seqlens.numpy(), w.inv_role.numpy(), w.role_model.numpy())
    km = tok_model[idx]
    valid = (w.tok_mask.numpy() if mask is None else np.asarray(mask))[idx] != 0
    a_alt = np.where(valid, t["dl_dlogp"] / o["M"][km], 0.0)
    reach = np.array([2.0 * w.inv_temperature * float(x.float().norm(dim=1).max().item()) for x in w.W])
    return np.abs(a_alt - o["a"][idx]) * reach[km]


def worst_block_rel_fro(a: np.ndarray, b: np.ndarray, block: int = 256) -> float:
    """Largest relative Frobenius error over blocks of `block` consecutive rows (the last one may be ragged)."""
    worst = 0.0
    for r0 in range(0, b.shape[0], block):
        bb = b[r0:r0 + block].astype(np.float64)
        err = np.linalg.norm(a[r0:r0 + block].astype(np.float64) - bb)
        den = np.linalg.norm(bb)
        if den == 0:
            if err > 0:
                return float("inf")
            continue
        worst = max(worst, err / den)
    return worst


def make_ctx(w: wl.Workload, extra: int = 0, stash: bool = False) -> ub.Context:
    size = ub.unity_workspace_bytes_stash if stash else ub.unity_workspace_bytes
    return ub.Context(0, size(w.n_tok, w.H, w.V, w.K, w.n_inv) + extra)


def dev(t, device="cuda"):
    return None if t is None else t.to(device)


class DeviceInputs:
    def __init__(self, w: wl.Workload, device="cuda"):
        self.inv_role = dev(w.inv_role)
        self.inv_group = dev(w.inv_group)
        self.inv_traj = dev(w.inv_traj)
        self.r_node, self.r_turn, self.r_traj = dev(w.r_node), dev(w.r_turn), dev(w.r_traj)
        self.cu_seqlens = dev(w.cu_seqlens)
        self.tok_mask = dev(w.tok_mask)
        self.target = dev(w.target)
        self.hidden = dev(w.hidden)
        self.W = [dev(x) for x in w.W]


def gpu_advantage(ctx: ub.Context, w: wl.Workload, d: DeviceInputs, lam=None, eps=None, ddof=None):
    adv_inv = torch.full((w.n_inv,), 7.0, device="cuda")
    adv_tok = torch.full((w.n_tok,), 7.0, device="cuda")
    seg_mean = torch.full((w.n_groups * w.n_roles,), 7.0, device="cuda")
    seg_std = torch.full((w.n_groups * w.n_roles,), 7.0, device="cuda")
    ctx.role_advantage(w.n_traj, w.n_roles, w.n_groups, d.inv_role, d.inv_group, d.inv_traj, d.r_node, d.r_turn,
                       d.r_traj, lam if lam is not None else w.lam.tolist(), w.adv_eps if eps is None else eps,
                       w.adv_ddof if ddof is None else ddof, d.cu_seqlens, d.tok_mask, adv_inv, adv_tok, seg_mean,
                       seg_std)
    ctx.check_status()
    return dict(adv_inv=adv_inv, adv_tok=adv_tok, seg_mean=seg_mean, seg_std=seg_std)


def oracle_advantage(w: wl.Workload, lam=None, eps=None, ddof=None):
    return orc.role_advantage(w.inv_role.numpy(), w.inv_group.numpy(), w.inv_traj.numpy(), w.r_node.numpy(),
                              w.r_turn.numpy(), w.r_traj.numpy(), w.lam.numpy() if lam is None else np.asarray(lam),
                              w.n_roles, w.n_groups, w.cu_seqlens.numpy(), w.tok_mask.numpy(),
                              eps=w.adv_eps if eps is None else eps, ddof=w.adv_ddof if ddof is None else ddof)


def gpu_logprob(ctx: ub.Context, w: wl.Workload, d: DeviceInputs):
    logp = torch.full((w.n_tok,), 7.0, device="cuda")
    ent = torch.full((w.n_tok,), 7.0, device="cuda")
    lse = torch.full((w.n_tok,), 7.0, device="cuda")
    ctx.logprob_fwd(d.hidden, d.W, d.cu_seqlens, d.inv_role, w.role_model.tolist(), d.target, d.tok_mask,
                    w.inv_temperature, logp, ent, lse)
    ctx.check_status()
    return dict(logp=logp, entropy=ent, lse=lse)


def oracle_logprob(w: wl.Workload, rows=None):
    return orc.logprob_fwd(bf16_bits(w.hidden), [bf16_bits(x) for x in w.W], w.cu_seqlens.numpy(),
                           w.inv_role.numpy(), w.role_model.numpy(), w.target.numpy(), w.tok_mask.numpy(),
                           inv_temperature=w.inv_temperature, rows=rows)


def gpu_ppo(ctx: ub.Context, w: wl.Workload, d: DeviceInputs, old, ref, adv, norm=None, accumulate=False, dW=None,
            kl_mode=None, kl_coef=None, ent_coef=None, clip=None, fwd=None):
    K = w.K
    loss = torch.full((K,), 7.0, device="cuda")
    metrics = torch.full(((K + w.n_roles) * ub.UNITY_N_METRICS,), 7.0, device="cuda")
    logp = torch.full((w.n_tok,), 7.0, device="cuda")
    ent = torch.full((w.n_tok,), 7.0, device="cuda")
    tok_loss = torch.full((w.n_tok,), 7.0, device="cuda")
    dH = torch.full((w.n_tok, w.H), 7.0, device="cuda", dtype=torch.bfloat16)
    if dW is None:
        dW = [torch.full((w.V, w.H), 7.0, device="cuda") for _ in range(K)]
    lo, hi = (w.clip_lo, w.clip_hi) if clip is None else clip
    ctx.ppo_loss_fwd_bwd(d.hidden, d.W, d.cu_seqlens, d.inv_role, w.role_model.tolist(), d.target, d.tok_mask,
                         w.inv_temperature, lo, hi, w.kl_coef if kl_coef is None else kl_coef,
                         w.kl_mode if kl_mode is None else kl_mode, w.ent_coef if ent_coef is None else ent_coef,
                         norm, accumulate, old, ref, adv, loss, metrics, logp, ent, tok_loss, dH, dW,
                         **({} if fwd is None else dict(logp_in=fwd["logp"], entropy_in=fwd["entropy"], lse_in=fwd["lse"])))
    ctx.check_status()
    return dict(loss=loss, metrics=metrics.view(K + w.n_roles, ub.UNITY_N_METRICS), logp=logp, entropy=ent,
                tok_loss=tok_loss, dHidden=dH, dW=dW)


def oracle_ppo(w: wl.Workload, old, ref, adv, norm=None, rows=None, dW_models=None, kl_mode=None, kl_coef=None,
               ent_coef=None, clip=None, want_dW=True):
    lo, hi = (w.clip_lo, w.clip_hi) if clip is None else clip
    out = _oracle_ppo(w, old, ref, adv, norm, rows, dW_models, kl_mode, kl_coef, ent_coef, lo, hi, want_dW)
    # what a conditioning-aware comparison of dHidden needs later (see dh_row_allowance)
    out["inputs"] = dict(old=np.asarray(old), ref=np.asarray(ref), adv=np.asarray(adv), clip=(lo, hi), kl_coef=kl_coef,
                         kl_mode=kl_mode, ent_coef=ent_coef)
    return out


def _oracle_ppo(w, old, ref, adv, norm, rows, dW_models, kl_mode, kl_coef, ent_coef, lo, hi, want_dW):
    return orc.ppo_loss_fwd_bwd(bf16_bits(w.hidden), [bf16_bits(x) for x in w.W], w.cu_seqlens.numpy(),
                                w.inv_role.numpy(), w.role_model.numpy(), w.target.numpy(), w.tok_mask.numpy(),
                                np.asarray(old), np.asarray(ref), np.asarray(adv), clip_lo=lo, clip_hi=hi,
                                kl_coef=w.kl_coef if kl_coef is None else kl_coef,
                                kl_mode=w.kl_mode if kl_mode is None else kl_mode,
                                ent_coef=w.ent_coef if ent_coef is None else ent_coef, norm=norm,
                                inv_temperature=w.inv_temperature, n_roles=w.n_roles, rows=rows,
                                dW_models=dW_models, want_dW=want_dW)
