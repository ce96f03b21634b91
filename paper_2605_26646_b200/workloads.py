"""Seeded synthetic workloads shaped like the paper's QA, search and code workflows.

This module only *draws inputs*: role/turn/trajectory structure, rewards, token masks,
targets, hidden states and LM-head weights.  It contains none of the method's arithmetic
(no advantage, soft-max, loss or gradient code) and is the one module that both the CUDA
path's callers and the CPU oracle's callers may share.

Randomness is a stateless counter generator: ``value = f(seed, tag, index)`` built from a
32-bit integer mixer (the "lowbias32" finaliser: xor-shift 16, multiply 0x7feb352d,
xor-shift 15, multiply 0x846ca68b, xor-shift 16) evaluated with int64 tensor ops, so any
slice of any tensor can be regenerated on any device without state.  Normal variates use
Box-Muller on two such uniforms.  Callers always hand *the same generated tensor* (copied
between devices) to both implementations, so equality of inputs never rests on CPU and GPU
transcendental functions agreeing.

Shapes follow the five benchmark configurations (tiny, RAG QA, iterative search,
reflective code generation, stress); the workflow structure of each follows the reward
rules of Section "Workflows and Rewards" (shared final score plus node-level format term;
turn-level rewards; verifier-score deltas per reflection round) and the three sharing
regimes of the agent-to-model mapping (full sharing, partial sharing, full separation).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional

import torch

_M32 = 0xFFFFFFFF

# tensor tags (one per generated quantity)
TAG_HIDDEN, TAG_W, TAG_TARGET, TAG_MASK, TAG_NOISE_OLD, TAG_NOISE_REF = 1, 2, 3, 4, 5, 6
TAG_LEN, TAG_TURNS, TAG_RNODE, TAG_RTURN, TAG_RTRAJ, TAG_P, TAG_CONST, TAG_PERM = 10, 11, 12, 13, 14, 15, 16, 17
TAG_ADV = 18


def _mul32(x: torch.Tensor, c: int) -> torch.Tensor:
    """(x * c) mod 2^32 for 0 <= x < 2^32 held in int64, without signed overflow."""
    lo = (x * (c & 0x7FFFFFFF)) & _M32
    if c & 0x80000000:
        lo = (lo + ((x & 1) << 31)) & _M32
    return lo


def _mix32(x: torch.Tensor) -> torch.Tensor:
    x = x ^ (x >> 16)
    x = _mul32(x, 0x7FEB352D)
    x = x ^ (x >> 15)
    x = _mul32(x, 0x846CA68B)
    x = x ^ (x >> 16)
    return x


def hash_u32(seed: int, tag: int, idx: torch.Tensor) -> torch.Tensor:
    """32-bit hash of (seed, tag, idx); idx is an int64 tensor of non-negative counters."""
    key = (int(seed) * 0x9E3779B1 + int(tag) * 0x85EBCA77 + 0x165667B1) & _M32
    x = _mix32((idx & _M32) ^ key)
    x = _mix32((x + ((idx >> 32) & _M32) * 0x27D4EB2F + int(tag)) & _M32)
    return x


def _counter(n: int, device, offset: int = 0) -> torch.Tensor:
    return torch.arange(offset, offset + n, dtype=torch.int64, device=device)


def uniform(seed: int, tag: int, n: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """float64 uniforms in (0, 1)."""
    h = hash_u32(seed, tag, _counter(n, device, offset))
    return (h.to(torch.float64) + 0.5) * (1.0 / 4294967296.0)


def normal(seed: int, tag: int, n: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """float32 standard normals (Box-Muller on counters 2i and 2i+1)."""
    c = _counter(n, device, offset) * 2
    u1 = (hash_u32(seed, tag, c).to(torch.float32) + 1.0) * (1.0 / 4294967296.0)
    u2 = hash_u32(seed, tag, c + 1).to(torch.float32) * (1.0 / 4294967296.0)
    u1 = u1.clamp_min(2.0 ** -33)
    return torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)


def randint(seed: int, tag: int, n: int, lo: int, hi: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """int64 integers uniform in [lo, hi)."""
    h = hash_u32(seed, tag, _counter(n, device, offset))
    return lo + (h * (hi - lo) >> 32)


def bernoulli(seed: int, tag: int, n: int, p: float, device="cpu", offset: int = 0) -> torch.Tensor:
    return uniform(seed, tag, n, device, offset) < p


def normal_bf16(seed: int, tag: int, rows: int, cols: int, std: float, device="cpu",
                chunk_elems: int = 1 << 25) -> torch.Tensor:
    """[rows, cols] bf16 tensor: N(0, std) drawn in f32 then rounded to nearest-even bf16."""
    out = torch.empty((rows, cols), dtype=torch.bfloat16, device=device)
    flat = out.view(-1)
    total = rows * cols
    for start in range(0, total, chunk_elems):
        n = min(chunk_elems, total - start)
        flat[start:start + n] = (normal(seed, tag, n, device, start) * std).to(torch.bfloat16)
    return out


# ----------------------------------------------------------------------------------------------
# configurations
# ----------------------------------------------------------------------------------------------

CONFIGS: Dict[str, dict] = {
    "tiny": dict(index=0, H=256, V=4096, n_groups=8, samples=4, roles=["answerer", "critic"],
                 role_model=[0, 0], kl_coef=0.01, ent_coef=0.0),
    "rag_qa": dict(index=1, H=896, V=151936, n_groups=64, samples=8, roles=["rewriter", "answerer"],
                   role_model=[0, 0], kl_coef=0.01, ent_coef=0.0),
    "search": dict(index=2, H=1536, V=151936, n_groups=128, samples=8,
                   roles=["planner", "searcher", "answerer"], role_model=[0, 0, 1],
                   kl_coef=0.01, ent_coef=0.0),
    "code": dict(index=3, H=3584, V=152064, n_groups=64, samples=8, roles=["coder", "reflector"],
                 role_model=[0, 1], kl_coef=0.01, ent_coef=0.0),
    "stress": dict(index=4, H=5120, V=152064, n_groups=256, samples=8,
                   roles=["r0", "r1", "r2", "r3"], role_model=[0, 1, 2, 3],
                   kl_coef=0.05, ent_coef=0.001),
}
BASE_SEED = 20260528


@dataclass
class Workload:
    """All inputs of one batch.  Small tables are CPU tensors; ``hidden`` / ``W`` live on
    ``device`` once :func:`materialize` has run."""
    name: str
    seed: int
    H: int
    V: int
    K: int
    n_roles: int
    n_groups: int
    n_traj: int
    n_inv: int
    n_tok: int
    role_model: torch.Tensor          # int32 [R]  (the mapping phi)
    inv_role: torch.Tensor            # int32 [S]
    inv_group: torch.Tensor           # int32 [S]
    inv_traj: torch.Tensor            # int32 [S]
    inv_turn: torch.Tensor            # int32 [S]
    r_node: torch.Tensor              # f32 [S]
    r_turn: torch.Tensor              # f32 [S]
    r_traj: torch.Tensor              # f32 [n_traj]
    lam: torch.Tensor                 # f32 [R, 3]
    cu_seqlens: torch.Tensor          # int64 [S+1]
    tok_mask: torch.Tensor            # uint8 [N]
    target: torch.Tensor              # int32 [N]
    noise_old: torch.Tensor           # f32 [N]  N(0, 0.05): old_logp = current logp + noise_old
    noise_ref: torch.Tensor           # f32 [N]
    adv_eps: float = 1e-6
    adv_ddof: int = 0
    clip_lo: float = 0.2
    clip_hi: float = 0.2
    kl_coef: float = 0.01
    kl_mode: int = 3
    ent_coef: float = 0.0
    inv_temperature: float = 1.0
    hidden: Optional[torch.Tensor] = None       # bf16 [N, H]
    W: List[torch.Tensor] = field(default_factory=list)   # K x bf16 [V, H]

    @property
    def n_valid(self) -> int:
        return int(self.tok_mask.sum().item())


def _log_uniform_int(seed, tag, n, lo, hi):
    u = uniform(seed, tag, n)
    v = torch.floor(torch.exp(u * (math.log(hi + 1) - math.log(lo)) + math.log(lo))).to(torch.int64)
    return v.clamp(lo, hi)


def make_structure(name: str, cut_rows: Optional[int] = None, cut_max_len: Optional[int] = None,
                   H: Optional[int] = None, V: Optional[int] = None, seed_offset: int = 0) -> Workload:
    """Draw the trajectory structure, rewards and token-level integer inputs of a configuration.

    ``cut_rows`` / ``cut_max_len`` produce a *parity cut*: the same invocations, groups, roles
    and rewards, but only a seeded subset of invocations keeps response tokens (each truncated
    to ``cut_max_len`` rows) until about ``cut_rows`` rows are kept, every model represented.
    Invocations without tokens have zero length in ``cu_seqlens``.  ``H`` / ``V`` override the
    sizes (used by small CPU tests).
    """
    cfg = CONFIGS[name]
    seed = BASE_SEED + cfg["index"] + seed_offset
    Hh = H or cfg["H"]
    Vv = V or cfg["V"]
    G, samples = cfg["n_groups"], cfg["samples"]
    R = len(cfg["roles"])
    role_model = torch.tensor(cfg["role_model"], dtype=torch.int32)
    K = int(role_model.max().item()) + 1
    n_traj = G * samples
    traj_group = torch.arange(n_traj, dtype=torch.int64) // samples

    # ---- invocations: (trajectory, turn, role) in execution order -------------------------
    if name in ("tiny", "rag_qa", "stress"):
        turns = torch.ones(n_traj, dtype=torch.int64)
    elif name == "search":
        turns = randint(seed, TAG_TURNS, n_traj, 1, 5)
    else:  # code
        turns = randint(seed, TAG_TURNS, n_traj, 2, 4)
    inv_traj = torch.repeat_interleave(torch.arange(n_traj, dtype=torch.int64), turns * R)
    S = int(inv_traj.numel())
    first = torch.cumsum(turns * R, 0) - turns * R
    within = torch.arange(S, dtype=torch.int64) - first[inv_traj]
    inv_turn = within // R
    inv_role = within % R
    inv_group = traj_group[inv_traj]

    # ---- rewards ---------------------------------------------------------------------------
    r_node = torch.zeros(S, dtype=torch.float32)
    r_turn = torch.zeros(S, dtype=torch.float32)
    r_traj = torch.zeros(n_traj, dtype=torch.float32)
    if name == "tiny":
        r_node = bernoulli(seed, TAG_RNODE, S, 0.5).to(torch.float32)
    elif name == "rag_qa":
        # shared final 0/1 answer score + node-level format term in {0, 0.1}
        r_traj = bernoulli(seed, TAG_RTRAJ, n_traj, 0.5).to(torch.float32)
        r_node = bernoulli(seed, TAG_RNODE, S, 0.5).to(torch.float32) * 0.1
    elif name == "search":
        r_turn = normal(seed, TAG_RTURN, S)
        r_traj = bernoulli(seed, TAG_RTRAJ, n_traj, 0.5).to(torch.float32)
    elif name == "code":
        # verifier score per round: fraction of 10 tests passed; round 0 credits the score,
        # later rounds credit the improvement over the previous round.
        p = uniform(seed, TAG_P, n_traj)
        max_turns = 3
        draws = uniform(seed, TAG_RTURN, n_traj * max_turns * 10).view(n_traj, max_turns, 10)
        score = (draws < p.view(-1, 1, 1)).sum(-1).to(torch.float64) / 10.0      # [n_traj, 3]
        prev = torch.cat([torch.zeros(n_traj, 1, dtype=torch.float64), score[:, :-1]], 1)
        delta = score - prev
        r_turn = delta[inv_traj, inv_turn].to(torch.float32)
    else:  # stress
        r_node = normal(seed, TAG_RNODE, S)
        seg = inv_group * R + inv_role
        const_seg = bernoulli(seed, TAG_CONST, G * R, 0.10)
        seg_value = normal(seed, TAG_CONST + 100, G * R)
        r_node = torch.where(const_seg[seg], seg_value[seg], r_node)

    # ---- response lengths --------------------------------------------------------------------
    pad_to = 1
    if name == "tiny":
        real_len = torch.full((S,), 16, dtype=torch.int64)
    elif name == "rag_qa":
        real_len = randint(seed, TAG_LEN, S, 16, 65)
    elif name == "search":
        real_len = randint(seed, TAG_LEN, S, 32, 257)
    elif name == "code":
        real_len = _log_uniform_int(seed, TAG_LEN, S, 64, 2048)
        pad_to = 128
    else:
        real_len = _log_uniform_int(seed, TAG_LEN, S, 32, 1024)

    keep = torch.ones(S, dtype=torch.bool)
    if name == "stress" and cut_rows is None:
        # token stages run on a mini-batch: invocations in a seeded order until 131072 rows
        order = torch.argsort(hash_u32(seed, TAG_PERM, torch.arange(S, dtype=torch.int64)), stable=True)
        csum = torch.cumsum(real_len[order], 0)
        budget = 131072
        n_full = int((csum <= budget).sum().item())
        keep[:] = False
        keep[order[:n_full]] = True
        if n_full < S and (n_full == 0 or int(csum[n_full - 1]) < budget):
            last = order[n_full]
            used = int(csum[n_full - 1]) if n_full > 0 else 0
            real_len[last] = budget - used
            keep[last] = True
    if cut_rows is not None:
        order = torch.argsort(hash_u32(seed, TAG_PERM + 50, torch.arange(S, dtype=torch.int64)), stable=True)
        if cut_max_len is not None:
            real_len = real_len.clamp_max(cut_max_len)
        keep[:] = False
        total = 0
        models_seen = set()
        for s in order.tolist():
            m = int(role_model[inv_role[s]])
            if total >= cut_rows and len(models_seen) == K:
                break
            if total >= cut_rows and m in models_seen:
                continue
            keep[s] = True
            models_seen.add(m)
            total += int(real_len[s])
    real_len = torch.where(keep, real_len, torch.zeros_like(real_len))
    padded_len = (real_len + pad_to - 1) // pad_to * pad_to
    cu = torch.zeros(S + 1, dtype=torch.int64)
    cu[1:] = torch.cumsum(padded_len, 0)
    N = int(cu[-1].item())

    # ---- token-level inputs -------------------------------------------------------------------
    tok_inv = torch.repeat_interleave(torch.arange(S, dtype=torch.int64), padded_len)
    pos = torch.arange(N, dtype=torch.int64) - cu[:-1][tok_inv]
    is_real = pos < real_len[tok_inv]
    tok_mask = (bernoulli(seed, TAG_MASK, N, 0.8) & is_real).to(torch.uint8)
    target = randint(seed, TAG_TARGET, N, 0, Vv).to(torch.int32)
    noise_old = normal(seed, TAG_NOISE_OLD, N) * 0.05
    noise_ref = normal(seed, TAG_NOISE_REF, N) * 0.05

    return Workload(
        name=name, seed=seed, H=Hh, V=Vv, K=K, n_roles=R, n_groups=G, n_traj=n_traj, n_inv=S, n_tok=N,
        role_model=role_model, inv_role=inv_role.to(torch.int32), inv_group=inv_group.to(torch.int32),
        inv_traj=inv_traj.to(torch.int32), inv_turn=inv_turn.to(torch.int32),
        r_node=r_node.to(torch.float32), r_turn=r_turn.to(torch.float32), r_traj=r_traj,
        lam=torch.ones(R, 3, dtype=torch.float32), cu_seqlens=cu, tok_mask=tok_mask, target=target,
        noise_old=noise_old, noise_ref=noise_ref, kl_coef=cfg["kl_coef"], ent_coef=cfg["ent_coef"])


def materialize(w: Workload, device="cpu", with_hidden: bool = True, with_W: bool = True) -> Workload:
    """Draw the large tensors: hidden ~ N(0,1) and K LM heads ~ N(0, 0.02), both bf16."""
    if with_hidden:
        w.hidden = normal_bf16(w.seed, TAG_HIDDEN, w.n_tok, w.H, 1.0, device)
    if with_W:
        w.W = [normal_bf16(w.seed, TAG_W + 1000 * (k + 1), w.V, w.H, 0.02, device) for k in range(w.K)]
    return w


def make(name: str, device="cpu", **kw) -> Workload:
    return materialize(make_structure(name, **kw), device)
