"""ctypes binding of libunity.so: argument marshalling only.

Every function mirrors the C entry point of the same name in ``include/unity.h``; tensors are
torch CUDA tensors whose ``data_ptr()`` is passed through, small host tables are python
sequences.  No arithmetic of the path happens here, and there is no fallback: if the shared
library cannot be loaded the import of a symbol raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

from . import build as _build

UNITY_OK = 0
ERR_NAMES = {0: "UNITY_OK", -1: "UNITY_ERR_INVALID_ARG", -2: "UNITY_ERR_SHAPE", -3: "UNITY_ERR_ALIGNMENT",
             -4: "UNITY_ERR_WORKSPACE", -5: "UNITY_ERR_CUDA", -6: "UNITY_ERR_UNSUPPORTED_ARCH",
             -7: "UNITY_ERR_BAD_INDEX", -8: "UNITY_ERR_TIMEOUT"}
UNITY_MAX_MODELS = 16
UNITY_MAX_ROLES = 64
UNITY_N_METRICS = 8

EXPORTS = ["unity_create", "unity_destroy", "unity_workspace_hint", "unity_workspace_bytes", "unity_workspace_min_bytes",
           "unity_workspace_bytes_stash",
           "unity_check_status", "unity_last_error", "unity_launch_count", "unity_set_profiling",
           "unity_get_profile", "unity_set_option", "unity_advantage_workspace_bytes", "unity_role_advantage", "unity_reward_assembly", "unity_gae", "unity_value_loss_fwd_bwd",
           "unity_ready_batch_plan", "unity_ready_batch_gather", "unity_align_rewards",
           "unity_role_advantage_noalloc",
           "unity_logprob_fwd", "unity_ppo_loss_fwd_bwd"]


class UnityError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{ERR_NAMES.get(code, code)}: {msg}")
        self.code = code


class unity_adv_params(C.Structure):
    _fields_ = [("eps", C.c_float), ("ddof", C.c_int)]


class unity_reward_rule(C.Structure):
    _fields_ = [("mode", C.c_int), ("shift", C.c_int)]


class unity_batch_params(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("n_parts", C.c_int32), ("pad_to", C.c_int32)]


class unity_rows(C.Structure):
    _fields_ = [("n_tok", C.c_int64), ("H", C.c_int32), ("V", C.c_int32), ("K", C.c_int32),
                ("n_inv", C.c_int32), ("n_roles", C.c_int32),
                ("hidden", C.c_void_p), ("W", C.POINTER(C.c_void_p)), ("cu_seqlens", C.c_void_p),
                ("inv_role", C.c_void_p), ("role_model", C.POINTER(C.c_int32)), ("target", C.c_void_p),
                ("tok_mask", C.c_void_p), ("inv_temperature", C.c_float)]


class unity_ppo_params(C.Structure):
    _fields_ = [("clip_lo", C.c_float), ("clip_hi", C.c_float), ("kl_coef", C.c_float), ("kl_mode", C.c_int),
                ("ent_coef", C.c_float), ("norm", C.POINTER(C.c_float)), ("accumulate_dW", C.c_int),
                ("logp_in", C.c_void_p), ("entropy_in", C.c_void_p), ("lse_in", C.c_void_p)]


_LIB = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Load (building first if the sources are newer) libunity.so.  Raises if that is impossible."""
    global _LIB
    if _LIB is not None and path is None:
        return _LIB
    if path is None:
        path = _build.LIB_PATH
        if _build.needs_build():
            _build.build()
    if not os.path.exists(path):
        raise RuntimeError(f"libunity.so not found at {path}: build it with python -m paper_2605_26646_b200.build")
    lib = C.CDLL(path)
    vp, i32, i64, f32p = C.c_void_p, C.c_int32, C.c_int64, C.POINTER(C.c_float)
    lib.unity_create.argtypes = [C.POINTER(vp), C.c_int, vp, vp, C.c_size_t]
    lib.unity_create.restype = C.c_int
    lib.unity_destroy.argtypes = [vp]
    lib.unity_destroy.restype = C.c_int
    for fn in (lib.unity_workspace_bytes, lib.unity_workspace_min_bytes, lib.unity_workspace_bytes_stash):
        fn.argtypes = [i64, i32, i32, i32, i32]
        fn.restype = C.c_size_t
    lib.unity_workspace_hint.argtypes = [i64, i32, i32, i32]
    lib.unity_workspace_hint.restype = C.c_size_t
    lib.unity_check_status.argtypes = [vp]
    lib.unity_check_status.restype = C.c_int
    lib.unity_last_error.argtypes = [vp]
    lib.unity_last_error.restype = C.c_char_p
    lib.unity_launch_count.argtypes = [vp]
    lib.unity_launch_count.restype = i64
    lib.unity_set_profiling.argtypes = [vp, C.c_int]
    lib.unity_set_profiling.restype = C.c_int
    lib.unity_set_option.argtypes = [vp, C.c_int, C.c_int]
    lib.unity_set_option.restype = C.c_int
    lib.unity_get_profile.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i64)]
    lib.unity_get_profile.restype = C.c_int
    lib.unity_advantage_workspace_bytes.argtypes = [i32, i32, i32]
    lib.unity_advantage_workspace_bytes.restype = C.c_size_t
    lib.unity_role_advantage.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, f32p,
                                         C.POINTER(unity_adv_params), i64, vp, vp, vp, vp, vp, vp]
    lib.unity_role_advantage.restype = C.c_int
    lib.unity_role_advantage_noalloc.argtypes = [C.c_int, vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, f32p,
                                                 C.POINTER(unity_adv_params), i64, vp, vp, vp, vp, vp, vp, vp,
                                                 C.c_char_p, C.c_size_t]
    lib.unity_role_advantage_noalloc.restype = C.c_int
    lib.unity_reward_assembly.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp,
                                          C.POINTER(unity_reward_rule), vp]
    lib.unity_reward_assembly.restype = C.c_int
    lib.unity_gae.argtypes = [vp, i32, i64, vp, vp, vp, vp, C.c_float, C.c_float, vp, vp]
    lib.unity_gae.restype = C.c_int
    lib.unity_value_loss_fwd_bwd.argtypes = [vp, i32, i32, i32, i64, vp, vp, C.POINTER(i32), vp, vp, vp, vp, C.c_float,
                                             f32p, vp, vp, vp, vp]
    lib.unity_value_loss_fwd_bwd.restype = C.c_int
    lib.unity_ready_batch_plan.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, C.POINTER(i32),
                                           C.POINTER(unity_batch_params), vp, vp, vp, vp, vp]
    lib.unity_ready_batch_plan.restype = C.c_int
    lib.unity_ready_batch_gather.argtypes = [vp, i32, i64, vp, vp, vp, vp, i64, vp, vp, vp, i32]
    lib.unity_ready_batch_gather.restype = C.c_int
    lib.unity_align_rewards.argtypes = [vp, i32, i64, vp, vp, vp, vp]
    lib.unity_align_rewards.restype = C.c_int
    lib.unity_logprob_fwd.argtypes = [vp, C.POINTER(unity_rows), vp, vp, vp]
    lib.unity_logprob_fwd.restype = C.c_int
    lib.unity_ppo_loss_fwd_bwd.argtypes = [vp, C.POINTER(unity_rows), C.POINTER(unity_ppo_params), vp, vp, vp,
                                           vp, vp, vp, vp, vp, vp, C.POINTER(vp)]
    lib.unity_ppo_loss_fwd_bwd.restype = C.c_int
    if path == _build.LIB_PATH:
        _LIB = lib
    return lib


def _ptr(t: Optional[torch.Tensor], dtype=None, name="tensor", host=False) -> Optional[int]:
    if t is None:
        return None
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if not host and not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    return t.data_ptr()


def _raise(ctx, code: int):
    if code != UNITY_OK:
        raise UnityError(code, load_library().unity_last_error(ctx).decode())


# ------------------------------------------------------------------------------------------------
# functions with the names of the C entry points
# ------------------------------------------------------------------------------------------------
def unity_workspace_hint(n_tok: int, H: int, V: int, K: int) -> int:
    return int(load_library().unity_workspace_hint(n_tok, H, V, K))


def unity_workspace_bytes(n_tok: int, H: int, V: int, K: int, n_inv: int) -> int:
    return int(load_library().unity_workspace_bytes(n_tok, H, V, K, n_inv))


def unity_workspace_min_bytes(n_tok: int, H: int, V: int, K: int, n_inv: int) -> int:
    return int(load_library().unity_workspace_min_bytes(n_tok, H, V, K, n_inv))


def unity_advantage_workspace_bytes(n_inv: int, n_groups: int, n_roles: int) -> int:
    return int(load_library().unity_advantage_workspace_bytes(n_inv, n_groups, n_roles))


def unity_workspace_bytes_stash(n_tok: int, H: int, V: int, K: int, n_inv: int) -> int:
    return int(load_library().unity_workspace_bytes_stash(n_tok, H, V, K, n_inv))


OPT_LOGIT_STASH = 15
OPT_WAIT_KCYCLES = 20
OPT_HOST_COUNTS = 25
OPT_TEST_DROP_SLAB = 21
OPT_GRAD_ROUNDS = 26
OPT_GRAD_BLOCK = 27
OPT_GRAD_RUNS = 28


def unity_create(device: int, stream_ptr: int, workspace: torch.Tensor) -> C.c_void_p:
    ctx = C.c_void_p()
    code = load_library().unity_create(C.byref(ctx), device, stream_ptr, workspace.data_ptr(),
                                       workspace.numel() * workspace.element_size())
    if code != UNITY_OK:
        raise UnityError(code, "unity_create failed")
    return ctx


def unity_destroy(ctx) -> None:
    load_library().unity_destroy(ctx)


def unity_check_status(ctx) -> None:
    _raise(ctx, load_library().unity_check_status(ctx))


def unity_launch_count(ctx) -> int:
    return int(load_library().unity_launch_count(ctx))


PROF_CLASSES = ["fwd_gemm", "grad_gemm", "dh_gemm", "dw_gemm"]


def unity_set_profiling(ctx, enable: bool) -> None:
    _raise(ctx, load_library().unity_set_profiling(ctx, 1 if enable else 0))


OPT_CTAS = {"fwd_gemm": 0, "grad_gemm": 1, "dh_gemm": 2, "dw_gemm": 3}


def unity_set_option(ctx, option: int, value: int) -> None:
    _raise(ctx, load_library().unity_set_option(ctx, option, value))


def unity_get_profile(ctx) -> dict:
    n = len(PROF_CLASSES)
    ms = (C.c_double * n)()
    cnt = (C.c_int64 * n)()
    _raise(ctx, load_library().unity_get_profile(ctx, ms, cnt))
    return {name: {"ms": float(ms[i]), "launches": int(cnt[i])} for i, name in enumerate(PROF_CLASSES)}


def unity_role_advantage(ctx, n_traj: int, n_roles: int, n_groups: int, inv_role, inv_group, inv_traj,
                         r_node, r_turn, r_traj, lam: Optional[Sequence[float]], eps: float, ddof: int,
                         cu_seqlens, tok_mask, adv_inv, adv_tok, seg_mean=None, seg_std=None) -> None:
    n_inv = int(inv_role.numel())
    n_tok = int(adv_tok.numel()) if adv_tok is not None else 0
    lam_arr = None
    if lam is not None:
        flat = [float(x) for row in lam for x in (row if hasattr(row, "__iter__") else [row])]
        lam_arr = (C.c_float * len(flat))(*flat)
    p = unity_adv_params(eps, ddof)
    i32, f32 = torch.int32, torch.float32
    code = load_library().unity_role_advantage(
        ctx, n_inv, n_traj, n_roles, n_groups, _ptr(inv_role, i32, "inv_role"), _ptr(inv_group, i32, "inv_group"),
        _ptr(inv_traj, i32, "inv_traj"), _ptr(r_node, f32, "r_node"), _ptr(r_turn, f32, "r_turn"),
        _ptr(r_traj, f32, "r_traj"), lam_arr, C.byref(p), n_tok, _ptr(cu_seqlens, torch.int64, "cu_seqlens"),
        _ptr(tok_mask, torch.uint8, "tok_mask"), _ptr(adv_inv, f32, "adv_inv"), _ptr(adv_tok, f32, "adv_tok"),
        _ptr(seg_mean, f32, "seg_mean"), _ptr(seg_std, f32, "seg_std"))
    _raise(ctx, code)


RULE_NONE, RULE_ABSOLUTE, RULE_MARGINAL = 0, 1, 2


def unity_reward_assembly(ctx, inv_role, inv_traj, inv_turn, score, n_scores, inv_end, rules, r_turn) -> None:
    """score: f32 CUDA tensor [n_traj, max_turns]; rules: sequence of (mode, shift) per role."""
    n_traj, max_turns = int(score.shape[0]), int(score.shape[1])
    arr = (unity_reward_rule * len(rules))(*[unity_reward_rule(int(m), int(sh)) for m, sh in rules])
    i32 = torch.int32
    code = load_library().unity_reward_assembly(
        ctx, int(inv_role.numel()), n_traj, len(rules), max_turns, _ptr(inv_role, i32, "inv_role"),
        _ptr(inv_traj, i32, "inv_traj"), _ptr(inv_turn, i32, "inv_turn"), _ptr(score, torch.float32, "score"),
        _ptr(n_scores, i32, "n_scores"), _ptr(inv_end, torch.uint8, "inv_end"), arr,
        _ptr(r_turn, torch.float32, "r_turn"))
    _raise(ctx, code)


def unity_gae(ctx, cu_seqlens, rewards, values, tok_mask, gamma: float, lam: float, advantages, returns) -> None:
    f32 = torch.float32
    code = load_library().unity_gae(ctx, int(cu_seqlens.numel()) - 1, int(rewards.numel()),
                                    _ptr(cu_seqlens, torch.int64, "cu_seqlens"), _ptr(rewards, f32, "rewards"),
                                    _ptr(values, f32, "values"), _ptr(tok_mask, torch.uint8, "tok_mask"), gamma, lam,
                                    _ptr(advantages, f32, "advantages"), _ptr(returns, f32, "returns"))
    _raise(ctx, code)


def unity_value_loss_fwd_bwd(ctx, cu_seqlens, inv_role, role_model: Sequence[int], K: int, tok_mask, values,
                             old_values, returns, clip_v: float, norm: Optional[Sequence[float]], loss,
                             clip_frac=None, tok_loss=None, dvalues=None) -> None:
    f32 = torch.float32
    rm = (C.c_int32 * len(role_model))(*[int(x) for x in role_model])
    norm_arr = None if norm is None else (C.c_float * len(norm))(*[float(x) for x in norm])
    code = load_library().unity_value_loss_fwd_bwd(
        ctx, int(inv_role.numel()), len(role_model), K, int(values.numel()),
        _ptr(cu_seqlens, torch.int64, "cu_seqlens"), _ptr(inv_role, torch.int32, "inv_role"), rm,
        _ptr(tok_mask, torch.uint8, "tok_mask"), _ptr(values, f32, "values"), _ptr(old_values, f32, "old_values"),
        _ptr(returns, f32, "returns"), float(clip_v), norm_arr, _ptr(loss, f32, "loss"),
        _ptr(clip_frac, f32, "clip_frac"), _ptr(tok_loss, f32, "tok_loss"), _ptr(dvalues, f32, "dvalues"))
    _raise(ctx, code)


def unity_ready_batch_plan(ctx, cu_seqlens, inv_role, inv_traj, traj_done, role_model: Sequence[int], K: int,
                           seed: int, n_parts: int, pad_to: int, order, out_cu_seqlens, model_offsets, part_offsets,
                           totals) -> None:
    """order: int32 [n_inv]; out_cu_seqlens: int64 [n_inv+1]; model_offsets: int32 [K+1]; part_offsets: int32
    [K*n_parts+1]; totals: int64 [2] - all CUDA tensors written by the call."""
    i32, i64 = torch.int32, torch.int64
    rm = (C.c_int32 * len(role_model))(*[int(x) for x in role_model])
    p = unity_batch_params(int(seed) & 0xFFFFFFFFFFFFFFFF, int(n_parts), int(pad_to))
    code = load_library().unity_ready_batch_plan(
        ctx, int(inv_role.numel()), int(traj_done.numel()), len(role_model), K, _ptr(cu_seqlens, i64, "cu_seqlens"),
        _ptr(inv_role, i32, "inv_role"), _ptr(inv_traj, i32, "inv_traj"), _ptr(traj_done, torch.uint8, "traj_done"),
        rm, C.byref(p), _ptr(order, i32, "order"), _ptr(out_cu_seqlens, i64, "out_cu_seqlens"),
        _ptr(model_offsets, i32, "model_offsets"), _ptr(part_offsets, i32, "part_offsets"), _ptr(totals, i64, "totals"))
    _raise(ctx, code)


def unity_ready_batch_gather(ctx, order, src_cu_seqlens, out_cu_seqlens, totals, src, dst, pad_value=0) -> None:
    """src: CUDA tensor [n_tok_src, ...] in buffer order; dst: CUDA tensor [>= totals[1], ...] of the same dtype and
    trailing shape; pad rows are filled with pad_value."""
    if src.dtype != dst.dtype or tuple(src.shape[1:]) != tuple(dst.shape[1:]):
        raise TypeError("src and dst must agree in dtype and trailing shape")
    row_bytes = src.element_size()
    for d in src.shape[1:]:
        row_bytes *= int(d)
    pad = bytes(torch.tensor([pad_value], dtype=src.dtype).view(torch.uint8).tolist())
    code = load_library().unity_ready_batch_gather(
        ctx, int(order.numel()), int(src.shape[0]), _ptr(order, torch.int32, "order"),
        _ptr(src_cu_seqlens, torch.int64, "src_cu_seqlens"), _ptr(out_cu_seqlens, torch.int64, "out_cu_seqlens"),
        _ptr(totals, torch.int64, "totals"), row_bytes, _ptr(src, None, "src"), _ptr(dst, None, "dst"), pad, len(pad))
    _raise(ctx, code)


def unity_align_rewards(ctx, cu_seqlens, tok_mask, r_inv, tok_reward) -> None:
    code = load_library().unity_align_rewards(
        ctx, int(r_inv.numel()), int(tok_reward.numel()), _ptr(cu_seqlens, torch.int64, "cu_seqlens"),
        _ptr(tok_mask, torch.uint8, "tok_mask"), _ptr(r_inv, torch.float32, "r_inv"),
        _ptr(tok_reward, torch.float32, "tok_reward"))
    _raise(ctx, code)


UNITY_NOALLOC_MAX_INV = 65536
UNITY_NOALLOC_MAX_SEG = 65536


def unity_role_advantage_noalloc(device: int, stream_ptr: int, n_traj: int, n_roles: int, n_groups: int, inv_role,
                                 inv_group, inv_traj, r_node, r_turn, r_traj, lam: Optional[Sequence[float]],
                                 eps: float, ddof: int, cu_seqlens, tok_mask, adv_inv, adv_tok, seg_mean=None,
                                 seg_std=None, bad_index_out=None) -> None:
    """Context-free, allocation-free form of unity_role_advantage (scratch is a fixed array inside the library;
    at most UNITY_NOALLOC_MAX_INV invocations).  Same arguments otherwise; `bad_index_out` is an optional int32
    CUDA tensor of one element."""
    n_inv = int(inv_role.numel())
    n_tok = int(adv_tok.numel()) if adv_tok is not None else 0
    lam_arr = None
    if lam is not None:
        flat = [float(x) for row in lam for x in (row if hasattr(row, "__iter__") else [row])]
        lam_arr = (C.c_float * len(flat))(*flat)
    p = unity_adv_params(eps, ddof)
    i32, f32 = torch.int32, torch.float32
    msg = C.create_string_buffer(256)
    code = load_library().unity_role_advantage_noalloc(
        device, stream_ptr, n_inv, n_traj, n_roles, n_groups, _ptr(inv_role, i32, "inv_role"),
        _ptr(inv_group, i32, "inv_group"), _ptr(inv_traj, i32, "inv_traj"), _ptr(r_node, f32, "r_node"),
        _ptr(r_turn, f32, "r_turn"), _ptr(r_traj, f32, "r_traj"), lam_arr, C.byref(p), n_tok,
        _ptr(cu_seqlens, torch.int64, "cu_seqlens"), _ptr(tok_mask, torch.uint8, "tok_mask"),
        _ptr(adv_inv, f32, "adv_inv"), _ptr(adv_tok, f32, "adv_tok"), _ptr(seg_mean, f32, "seg_mean"),
        _ptr(seg_std, f32, "seg_std"), _ptr(bad_index_out, i32, "bad_index_out"), msg, 256)
    if code != UNITY_OK:
        raise UnityError(code, msg.value.decode())


def _make_rows(hidden, W, cu_seqlens, inv_role, role_model, target, tok_mask, inv_temperature, keep):
    K = len(W)
    n_tok, H = int(hidden.shape[0]), int(hidden.shape[1])
    V = int(W[0].shape[0])
    for k, w in enumerate(W):
        if tuple(w.shape) != (V, H):
            raise ValueError(f"W[{k}] has shape {tuple(w.shape)}, expected {(V, H)}")
    Wp = (C.c_void_p * K)(*[_ptr(w, torch.bfloat16, "W") for w in W])
    rm = (C.c_int32 * len(role_model))(*[int(x) for x in role_model])
    keep.extend([Wp, rm])
    rows = unity_rows(n_tok, H, V, K, int(inv_role.numel()), len(role_model),
                      _ptr(hidden, torch.bfloat16, "hidden"), Wp, _ptr(cu_seqlens, torch.int64, "cu_seqlens"),
                      _ptr(inv_role, torch.int32, "inv_role"), rm, _ptr(target, torch.int32, "target"),
                      _ptr(tok_mask, torch.uint8, "tok_mask"), float(inv_temperature))
    return rows


def unity_logprob_fwd(ctx, hidden, W, cu_seqlens, inv_role, role_model, target, tok_mask, inv_temperature,
                      logp, entropy=None, lse=None) -> None:
    keep = []
    rows = _make_rows(hidden, W, cu_seqlens, inv_role, role_model, target, tok_mask, inv_temperature, keep)
    f32 = torch.float32
    code = load_library().unity_logprob_fwd(ctx, C.byref(rows), _ptr(logp, f32, "logp"),
                                            _ptr(entropy, f32, "entropy"), _ptr(lse, f32, "lse"))
    _raise(ctx, code)


def unity_ppo_loss_fwd_bwd(ctx, hidden, W, cu_seqlens, inv_role, role_model, target, tok_mask, inv_temperature,
                           clip_lo, clip_hi, kl_coef, kl_mode, ent_coef, norm: Optional[Sequence[float]],
                           accumulate_dW: bool, old_logp, ref_logp, adv_tok, loss, metrics, logp, entropy,
                           tok_loss, dHidden, dW, logp_in=None, entropy_in=None, lse_in=None) -> None:
    keep = []
    rows = _make_rows(hidden, W, cu_seqlens, inv_role, role_model, target, tok_mask, inv_temperature, keep)
    norm_arr = None
    if norm is not None:
        norm_arr = (C.c_float * len(norm))(*[float(x) for x in norm])
    f32_ = torch.float32
    p = unity_ppo_params(clip_lo, clip_hi, kl_coef, kl_mode, ent_coef, norm_arr, 1 if accumulate_dW else 0,
                         _ptr(logp_in, f32_, "logp_in"), _ptr(entropy_in, f32_, "entropy_in"), _ptr(lse_in, f32_, "lse_in"))
    dWp = (C.c_void_p * len(dW))(*[_ptr(g, torch.float32, "dW") for g in dW])
    f32 = torch.float32
    code = load_library().unity_ppo_loss_fwd_bwd(
        ctx, C.byref(rows), C.byref(p), _ptr(old_logp, f32, "old_logp"), _ptr(ref_logp, f32, "ref_logp"),
        _ptr(adv_tok, f32, "adv_tok"), _ptr(loss, f32, "loss"), _ptr(metrics, f32, "metrics"),
        _ptr(logp, f32, "logp"), _ptr(entropy, f32, "entropy"), _ptr(tok_loss, f32, "tok_loss"),
        _ptr(dHidden, torch.bfloat16, "dHidden"), dWp)
    _raise(ctx, code)


# ------------------------------------------------------------------------------------------------
class Context:
    """Owns a workspace tensor and a unity_ctx bound to a torch stream."""

    def __init__(self, device: int = 0, workspace_bytes: int = 1 << 28, stream: Optional[torch.cuda.Stream] = None):
        self.device = int(device)
        with torch.cuda.device(self.device):
            self.stream = stream or torch.cuda.current_stream()
            self.workspace = torch.empty(int(workspace_bytes), dtype=torch.uint8, device=f"cuda:{self.device}")
        self.ctx = unity_create(self.device, self.stream.cuda_stream, self.workspace)

    def close(self):
        if self.ctx is not None:
            unity_destroy(self.ctx)
            self.ctx = None
            self.workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def check_status(self):
        unity_check_status(self.ctx)

    @property
    def launch_count(self) -> int:
        return unity_launch_count(self.ctx)

    def set_profiling(self, enable: bool):
        unity_set_profiling(self.ctx, enable)

    def set_option(self, option: int, value: int):
        unity_set_option(self.ctx, option, value)

    def get_profile(self) -> dict:
        return unity_get_profile(self.ctx)

    def role_advantage(self, *a, **kw):
        return unity_role_advantage(self.ctx, *a, **kw)

    def reward_assembly(self, *a, **kw):
        return unity_reward_assembly(self.ctx, *a, **kw)

    def gae(self, *a, **kw):
        return unity_gae(self.ctx, *a, **kw)

    def value_loss_fwd_bwd(self, *a, **kw):
        return unity_value_loss_fwd_bwd(self.ctx, *a, **kw)

    def ready_batch_plan(self, *a, **kw):
        return unity_ready_batch_plan(self.ctx, *a, **kw)

    def ready_batch_gather(self, *a, **kw):
        return unity_ready_batch_gather(self.ctx, *a, **kw)

    def align_rewards(self, *a, **kw):
        return unity_align_rewards(self.ctx, *a, **kw)

    def logprob_fwd(self, *a, **kw):
        return unity_logprob_fwd(self.ctx, *a, **kw)

    def ppo_loss_fwd_bwd(self, *a, **kw):
        return unity_ppo_loss_fwd_bwd(self.ctx, *a, **kw)
